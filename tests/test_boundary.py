"""The C-ABI library loads and exports every symbol include/pearl_prb.h declares (no GPU needed),
and the host-side argument checks that need no device answer as documented."""
import ctypes as C
import os
import re

import pytest

from conftest import ROOT


@pytest.fixture(scope="module")
def built():
    from paper_2311_09445_b200 import build
    return build.build()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "pearl_prb.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pearl_prb_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported(built):
    lib = C.CDLL(built)
    names = declared_symbols()
    assert len(names) >= 17
    for name in names:
        assert hasattr(lib, name), name


def test_binding_covers_header(built):
    from paper_2311_09445_b200 import binding
    assert sorted(binding.SIGNATURES) == declared_symbols()


def test_slab_bytes_and_argument_checks(built):
    from paper_2311_09445_b200 import binding
    lib = binding.load_library()
    lay = binding._Layout(28224, 4)
    need = lib.pearl_prb_slab_bytes(1 << 19, 32, C.byref(lay), 512)
    store = (1 << 19) * (2 * 28224 + 4 + 4 + 1)
    assert store < need < store + (1 << 28)
    assert lib.pearl_prb_slab_bytes(1 << 19, 3, C.byref(lay), 512) == 0        # bad fanout
    assert lib.pearl_prb_slab_bytes(0, 16, C.byref(lay), 512) == 0             # bad capacity
    assert lib.pearl_prb_slab_bytes(1 << 19, 16, C.byref(lay), 0) == 0         # bad max_batch
    h = C.c_void_p()
    assert lib.pearl_prb_create(C.byref(h), 1024, 5, C.byref(lay), 32, 0, None, None, 0) == -2
    assert lib.pearl_prb_create(None, 1024, 4, C.byref(lay), 32, 0, None, None, 0) == -1
    assert lib.pearl_prb_insert(None, 1, None, None, None, None, None, None) == -1
    assert lib.pearl_prb_error_string(-5).decode().startswith("a pointer is misaligned")
    assert lib.pearl_prb_kernel_launches(None) == 0


def test_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2311_09445_b200 import PrioritizedReplay
    with pytest.raises(RuntimeError):
        PrioritizedReplay(1024, 4, 16, 4, 32)
