"""ctypes binding of libpearl_prb.so: argument marshalling only.

Method names and arguments mirror the C ABI in include/pearl_prb.h.  torch supplies device
memory and the stream; every step of the replay path runs in the library's CUDA kernels.
There is no CPU fallback: if the library is missing or no CUDA device is present the
constructor raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

from . import build as _build

ST_BAD_INDEX, ST_BAD_PRIORITY, ST_EMPTY, ST_CLAMPED, ST_INTERNAL, ST_STALE = 1, 2, 4, 8, 16, 32


class PearlError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__("%s failed: %s (%d)" % (what, _lib_error_string(code), code))
        self.code = code


class _Layout(C.Structure):
    _fields_ = [("obs_bytes", C.c_uint32), ("act_bytes", C.c_uint32)]


_lib = None

# name -> (restype, argtypes); every symbol include/pearl_prb.h declares
_vp, _u32, _u64, _f32, _i = C.c_void_p, C.c_uint32, C.c_uint64, C.c_float, C.c_int
SIGNATURES = {
    "pearl_prb_slab_bytes": (_u64, [_u64, _u32, C.POINTER(_Layout), _u32]),
    "pearl_prb_create": (_i, [C.POINTER(_vp), _u64, _u32, C.POINTER(_Layout), _u32, _i, _vp, _vp, _u64]),
    "pearl_prb_slab_bytes_frames": (_u64, [_u64, _u32, _u32, _u32, _u32, _u32]),
    "pearl_prb_create_frames": (_i, [C.POINTER(_vp), _u64, _u32, _u32, _u32, _u32, _u32, _i, _vp, _vp, _u64]),
    "pearl_prb_slab_bytes_opts": (_u64, [_u64, _u32, C.POINTER(_Layout), _u32, _u32, _u32]),
    "pearl_prb_create_opts": (_i, [C.POINTER(_vp), _u64, _u32, C.POINTER(_Layout), _u32, _u32, _u32, _i, _vp, _vp, _u64]),
    "pearl_prb_destroy": (_i, [_vp]),
    "pearl_prb_insert": (_i, [_vp, _u32, _vp, _vp, _vp, _vp, _vp, _vp]),
    "pearl_prb_sample": (_i, [_vp, _u32, _f32, _u64, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "pearl_prb_sample_buffer_norm": (_i, [_vp, _u32, _f32, _u64, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "pearl_prb_sample_streamed": (_i, [_vp, _u32, _f32, _u64, _u32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "pearl_prb_wait_sub_batch": (_i, [_vp, _u32, _vp]),
    "pearl_prb_sample_uniform": (_i, [_vp, _u32, _u64, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "pearl_prb_sample_static_scratch": (_i, [_vp, _u32, _f32, _u64, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "pearl_prb_update": (_i, [_vp, _u32, _vp, _vp, _f32, _f32]),
    "pearl_prb_update_priorities": (_i, [_vp, _u32, _vp, _vp]),
    "pearl_prb_update_delta": (_i, [_vp, _u32, _vp, _vp]),
    "pearl_prb_update_after_insert": (_i, [_vp, _u32, _vp, _vp, _f32, _f32, _u32]),
    "pearl_prb_get_priorities": (_i, [_vp, _u32, _vp, _vp]),
    "pearl_prb_update_insert": (_i, [_vp, _u32, _vp, _vp, _f32, _f32, _u32, _vp, _vp, _vp, _vp, _vp, _vp]),
    "pearl_prb_step": (_i, [_vp, _u32, _vp, _vp, _f32, _f32, _u32, _vp, _vp, _vp, _vp, _vp, _vp,
                            _u32, _f32, _u64, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "pearl_prb_step_host": (_i, [_vp, _u32, _vp, _vp, _f32, _f32, _u32, _vp, _vp, _vp, _vp, _vp, _vp,
                                 _u32, _f32, _u64, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "pearl_prb_insert_host": (_i, [_vp, _u32, _vp, _vp, _vp, _vp, _vp, _vp]),
    "pearl_prb_sample_host": (_i, [_vp, _u32, _f32, _u64, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "pearl_prb_update_host": (_i, [_vp, _u32, _vp, _vp, _f32, _f32]),
    "pearl_prb_sync": (_i, [_vp, C.POINTER(_u32)]),
    "pearl_prb_info": (_i, [_vp, C.POINTER(_u64), C.POINTER(_u64), C.POINTER(_u64), C.POINTER(_u32)]),
    "pearl_prb_max_priority": (_i, [_vp, C.POINTER(_f32)]),
    "pearl_prb_read_level": (_i, [_vp, _u32, _vp, _u64]),
    "pearl_prb_read_min_level": (_i, [_vp, _u32, _vp, _u64]),
    "pearl_prb_image_bytes": (_u64, [_vp]),
    "pearl_prb_export": (_i, [_vp, _u64, _vp, _u64]),
    "pearl_prb_import": (_i, [_vp, _u64, _vp, _u64]),
    "pearl_prb_level_alloc": (_u64, [_vp, _u32]),
    "pearl_prb_read_rows": (_i, [_vp, _vp, _u32, _vp, _vp, _vp, _vp, _vp]),
    "pearl_prb_kernel_launches": (_u64, [_vp]),
    "pearl_prb_error_string": (C.c_char_p, [_i]),
}


def load_library(path: Optional[str] = None):
    """Loads libpearl_prb.so (built in-tree by build.py) and declares its signatures."""
    global _lib
    if _lib is None:
        path = path or os.environ.get("PEARL_PRB_LIB") or _build.LIB      # PEARL_PRB_LIB: an alternate build of the library
        if not os.path.exists(path):
            raise ImportError("libpearl_prb.so is not built (%s); run paper_2311_09445_b200/build.py" % path)
        lib = C.CDLL(path)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _lib_error_string(code: int) -> str:
    try:
        return load_library().pearl_prb_error_string(code).decode()
    except Exception:
        return "error"


# (addresses are handed to ctypes as plain integers: every pointer parameter is declared c_void_p, which takes
# an int or None, and a step makes fifteen of these conversions)
def _dptr(t: Optional[torch.Tensor], what: str):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("%s must be a contiguous CUDA tensor" % what)
    return t.data_ptr()


def _hptr(t, what: str):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("%s must be a contiguous host tensor" % what)
        return t.data_ptr()
    return t.ctypes.data      # numpy array


def _row_bytes(t: torch.Tensor, n: int) -> int:
    return t.numel() * t.element_size() // n


class PrioritizedReplay:
    """One prioritized replay buffer on one GPU.

    capacity / fanout / obs_bytes / act_bytes / max_batch are pearl_prb_create's arguments.
    Device memory is one torch uint8 slab; the handle enqueues on `stream` (default: the
    current torch stream at construction).
    """

    def __init__(self, capacity: int, fanout: int, obs_bytes: int, act_bytes: int, max_batch: int,
                 device: Optional[torch.device] = None, stream: Optional[torch.cuda.Stream] = None, frame_stack: int = 0,
                 min_tree: bool = False):
        self._h = None
        lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("PrioritizedReplay needs a CUDA device; there is no CPU path")
        self.device = torch.device(device if device is not None else "cuda:%d" % torch.cuda.current_device())
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        self.capacity, self.fanout, self.max_batch = capacity, fanout, max_batch
        self.obs_bytes, self.act_bytes = obs_bytes, act_bytes
        self.frame_stack = frame_stack          # > 0: pearl_prb_create_frames; obs_bytes is then a whole stack
        self.min_tree = bool(min_tree)          # PEARL_OPT_MIN_TREE (pearl_prb_create_opts)
        lay = _Layout(obs_bytes, act_bytes)
        if frame_stack and obs_bytes % frame_stack:
            raise ValueError("obs_bytes must be frame_stack frames")
        if min_tree:
            lay = _Layout(obs_bytes // frame_stack if frame_stack else obs_bytes, act_bytes)
            need = lib.pearl_prb_slab_bytes_opts(capacity, fanout, C.byref(lay), frame_stack, 1, max_batch)
        elif frame_stack:
            need = lib.pearl_prb_slab_bytes_frames(capacity, fanout, obs_bytes // frame_stack, frame_stack, act_bytes, max_batch)
        else:
            need = lib.pearl_prb_slab_bytes(capacity, fanout, C.byref(lay), max_batch)
        if need == 0:
            raise PearlError(-7, "pearl_prb_slab_bytes")
        self.slab_bytes = int(need)
        self._slab = torch.empty(self.slab_bytes, dtype=torch.uint8, device=self.device)
        h = C.c_void_p()
        if min_tree:
            rc = lib.pearl_prb_create_opts(C.byref(h), capacity, fanout, C.byref(lay), frame_stack, 1, max_batch,
                                           self.device.index or 0, C.c_void_p(self.stream.cuda_stream),
                                           C.c_void_p(self._slab.data_ptr()), self.slab_bytes)
        elif frame_stack:
            rc = lib.pearl_prb_create_frames(C.byref(h), capacity, fanout, obs_bytes // frame_stack, frame_stack, act_bytes, max_batch,
                                             self.device.index or 0, C.c_void_p(self.stream.cuda_stream),
                                             C.c_void_p(self._slab.data_ptr()), self.slab_bytes)
        else:
            rc = lib.pearl_prb_create(C.byref(h), capacity, fanout, C.byref(lay), max_batch, self.device.index or 0,
                                      C.c_void_p(self.stream.cuda_stream), C.c_void_p(self._slab.data_ptr()),
                                      self.slab_bytes)
        if rc != 0:
            raise PearlError(rc, "pearl_prb_create")
        self._h = h
        self.depth = self.info()[3]

    # ---- the four calls, device buffers ------------------------------------------------
    def insert(self, obs, act, rew, next_obs, done, prio, n: Optional[int] = None) -> None:
        """prio=None (with n given): the new transitions take the largest priority written so far."""
        n = prio.numel() if prio is not None else int(n)
        rc = load_library().pearl_prb_insert(self._h, n, _dptr(obs, "obs"), _dptr(act, "act"), _dptr(rew, "rew"),
                                             _dptr(next_obs, "next_obs"), _dptr(done, "done"), _dptr(prio, "prio"))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_insert")

    def sample(self, B: int, beta: float, seed: int, idx, w=None, obs=None, act=None, rew=None, next_obs=None,
               done=None) -> None:
        rc = load_library().pearl_prb_sample(self._h, B, beta, seed, _dptr(idx, "idx"), _dptr(w, "w"),
                                             _dptr(obs, "obs"), _dptr(act, "act"), _dptr(rew, "rew"),
                                             _dptr(next_obs, "next_obs"), _dptr(done, "done"))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_sample")

    def sample_buffer_norm(self, B: int, beta: float, seed: int, idx, w=None, obs=None, act=None, rew=None, next_obs=None,
                           done=None) -> None:
        rc = load_library().pearl_prb_sample_buffer_norm(self._h, B, beta, seed, _dptr(idx, "idx"), _dptr(w, "w"),
                                                         _dptr(obs, "obs"), _dptr(act, "act"), _dptr(rew, "rew"),
                                                         _dptr(next_obs, "next_obs"), _dptr(done, "done"))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_sample_buffer_norm")

    def sample_streamed(self, B: int, beta: float, seed: int, n_sub: int, idx, w=None, obs=None, act=None, rew=None,
                        next_obs=None, done=None) -> None:
        rc = load_library().pearl_prb_sample_streamed(self._h, B, beta, seed, n_sub, _dptr(idx, "idx"), _dptr(w, "w"),
                                                      _dptr(obs, "obs"), _dptr(act, "act"), _dptr(rew, "rew"),
                                                      _dptr(next_obs, "next_obs"), _dptr(done, "done"))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_sample_streamed")

    def wait_sub_batch(self, sub_batch: int, stream: torch.cuda.Stream) -> None:
        """Makes `stream` wait for sub-batch `sub_batch` of the last sample_streamed call."""
        rc = load_library().pearl_prb_wait_sub_batch(self._h, sub_batch, C.c_void_p(stream.cuda_stream))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_wait_sub_batch")

    def sample_uniform(self, B: int, seed: int, idx, w=None, obs=None, act=None, rew=None, next_obs=None, done=None) -> None:
        rc = load_library().pearl_prb_sample_uniform(self._h, B, seed, _dptr(idx, "idx"), _dptr(w, "w"), _dptr(obs, "obs"),
                                                     _dptr(act, "act"), _dptr(rew, "rew"), _dptr(next_obs, "next_obs"),
                                                     _dptr(done, "done"))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_sample_uniform")

    def sample_static_scratch(self, B: int, beta: float, seed: int, idx, w=None, obs=None, act=None, rew=None,
                              next_obs=None, done=None) -> None:
        """pearl_prb_sample_static_scratch: the sample call for callers that cannot allocate device
        memory (B <= 4096); its scratch is a static array inside the library, shared by every
        handle on the device, so overlapping calls on one GPU race."""
        rc = load_library().pearl_prb_sample_static_scratch(self._h, B, beta, seed, _dptr(idx, "idx"), _dptr(w, "w"),
                                                            _dptr(obs, "obs"), _dptr(act, "act"), _dptr(rew, "rew"),
                                                            _dptr(next_obs, "next_obs"), _dptr(done, "done"))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_sample_static_scratch")

    def update(self, idx, td, alpha: float, eps: float) -> None:
        rc = load_library().pearl_prb_update(self._h, idx.numel(), _dptr(idx, "idx"), _dptr(td, "td"), alpha, eps)
        if rc != 0:
            raise PearlError(rc, "pearl_prb_update")

    def update_priorities(self, idx, prio) -> None:
        rc = load_library().pearl_prb_update_priorities(self._h, idx.numel(), _dptr(idx, "idx"), _dptr(prio, "prio"))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_update_priorities")

    def update_delta(self, idx, delta) -> None:
        rc = load_library().pearl_prb_update_delta(self._h, idx.numel(), _dptr(idx, "idx"), _dptr(delta, "delta"))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_update_delta")

    def update_after_insert(self, idx, td, alpha: float, eps: float, inserted: int) -> None:
        rc = load_library().pearl_prb_update_after_insert(self._h, idx.numel(), _dptr(idx, "idx"), _dptr(td, "td"),
                                                          alpha, eps, inserted)
        if rc != 0:
            raise PearlError(rc, "pearl_prb_update_after_insert")

    def get_priorities(self, idx, out) -> None:
        rc = load_library().pearl_prb_get_priorities(self._h, idx.numel(), _dptr(idx, "idx"), _dptr(out, "out"))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_get_priorities")

    def update_insert(self, idx, td, alpha: float, eps: float, obs, act, rew, next_obs, done, prio,
                      n: Optional[int] = None) -> None:
        rc = load_library().pearl_prb_update_insert(self._h, idx.numel(), _dptr(idx, "idx"), _dptr(td, "td"), alpha, eps,
                                                    prio.numel() if prio is not None else int(n), _dptr(obs, "obs"), _dptr(act, "act"),
                                                    _dptr(rew, "rew"), _dptr(next_obs, "next_obs"),
                                                    _dptr(done, "done"), _dptr(prio, "prio"))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_update_insert")

    def step(self, upd_idx, td, alpha: float, eps: float, new_obs, new_act, new_rew, new_next_obs, new_done, new_prio,
             B: int, beta: float, seed: int, idx, w=None, obs=None, act=None, rew=None, next_obs=None, done=None,
             n: Optional[int] = None) -> None:
        """pearl_prb_step: update_insert for the previous batch, then the sample of the next one, as one call."""
        rc = load_library().pearl_prb_step(self._h, upd_idx.numel(), _dptr(upd_idx, "upd_idx"), _dptr(td, "td"), alpha, eps,
                                           new_prio.numel() if new_prio is not None else int(n), _dptr(new_obs, "new_obs"),
                                           _dptr(new_act, "new_act"), _dptr(new_rew, "new_rew"),
                                           _dptr(new_next_obs, "new_next_obs"), _dptr(new_done, "new_done"),
                                           _dptr(new_prio, "new_prio"), B, beta, seed, _dptr(idx, "idx"), _dptr(w, "w"),
                                           _dptr(obs, "obs"), _dptr(act, "act"), _dptr(rew, "rew"),
                                           _dptr(next_obs, "next_obs"), _dptr(done, "done"))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_step")

    # ---- the same calls, host buffers (numpy arrays or host torch tensors) -----------------
    def insert_host(self, obs, act, rew, next_obs, done, prio, n: Optional[int] = None) -> None:
        n = int(prio.shape[0]) if prio is not None else int(n)
        rc = load_library().pearl_prb_insert_host(self._h, n, _hptr(obs, "obs"), _hptr(act, "act"), _hptr(rew, "rew"),
                                                  _hptr(next_obs, "next_obs"), _hptr(done, "done"),
                                                  _hptr(prio, "prio"))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_insert_host")

    def sample_host(self, B: int, beta: float, seed: int, idx, w=None, obs=None, act=None, rew=None, next_obs=None,
                    done=None) -> None:
        rc = load_library().pearl_prb_sample_host(self._h, B, beta, seed, _hptr(idx, "idx"), _hptr(w, "w"),
                                                  _hptr(obs, "obs"), _hptr(act, "act"), _hptr(rew, "rew"),
                                                  _hptr(next_obs, "next_obs"), _hptr(done, "done"))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_sample_host")

    def step_host(self, upd_idx, td, alpha: float, eps: float, new_obs, new_act, new_rew, new_next_obs, new_done, new_prio,
                  B: int, beta: float, seed: int, idx, w=None, obs=None, act=None, rew=None, next_obs=None, done=None,
                  n: Optional[int] = None) -> None:
        """pearl_prb_step_host: one iteration (update, insertion, next sample) with host arrays."""
        rc = load_library().pearl_prb_step_host(self._h, int(upd_idx.shape[0]), _hptr(upd_idx, "upd_idx"), _hptr(td, "td"), alpha,
                                                eps, int(new_prio.shape[0]) if new_prio is not None else int(n or 0),
                                                _hptr(new_obs, "new_obs"), _hptr(new_act, "new_act"), _hptr(new_rew, "new_rew"),
                                                _hptr(new_next_obs, "new_next_obs"), _hptr(new_done, "new_done"),
                                                _hptr(new_prio, "new_prio"), B, beta, seed, _hptr(idx, "idx"), _hptr(w, "w"),
                                                _hptr(obs, "obs"), _hptr(act, "act"), _hptr(rew, "rew"),
                                                _hptr(next_obs, "next_obs"), _hptr(done, "done"))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_step_host")

    def update_host(self, idx, td, alpha: float, eps: float) -> None:
        rc = load_library().pearl_prb_update_host(self._h, int(idx.shape[0]), _hptr(idx, "idx"), _hptr(td, "td"),
                                                  alpha, eps)
        if rc != 0:
            raise PearlError(rc, "pearl_prb_update_host")

    # ---- synchronisation and read-back -----------------------------------------------------
    def sync(self) -> int:
        st = C.c_uint32(0)
        rc = load_library().pearl_prb_sync(self._h, C.byref(st))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_sync")
        return int(st.value)

    def info(self):
        f, c, n, d = C.c_uint64(), C.c_uint64(), C.c_uint64(), C.c_uint32()
        rc = load_library().pearl_prb_info(self._h, C.byref(f), C.byref(c), C.byref(n), C.byref(d))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_info")
        return f.value, c.value, n.value, d.value

    def max_priority(self) -> float:
        out = C.c_float(0.0)
        rc = load_library().pearl_prb_max_priority(self._h, C.byref(out))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_max_priority")
        return float(out.value)

    def level_alloc(self, level: int) -> int:
        return int(load_library().pearl_prb_level_alloc(self._h, level))

    def read_level(self, level: int):
        import numpy as np
        n = self.level_alloc(level)
        out = np.zeros(n, dtype=np.float32)
        rc = load_library().pearl_prb_read_level(self._h, level, C.c_void_p(out.ctypes.data), n)
        if rc != 0:
            raise PearlError(rc, "pearl_prb_read_level")
        return out

    def read_min_level(self, level: int):
        import numpy as np
        n = self.level_alloc(level)
        out = np.zeros(n, dtype=np.float32)
        rc = load_library().pearl_prb_read_min_level(self._h, level, C.c_void_p(out.ctypes.data), n)
        if rc != 0:
            raise PearlError(rc, "pearl_prb_read_min_level")
        return out

    def export_image(self, piece_bytes: int = 1 << 28):
        """The buffer's checkpoint image as a host array of bytes (pearl_prb_export, piece by piece)."""
        import numpy as np
        lib = load_library()
        total = int(lib.pearl_prb_image_bytes(self._h))
        out = np.empty(total, dtype=np.uint8)
        for off in range(0, total, piece_bytes):
            n = min(piece_bytes, total - off)
            rc = lib.pearl_prb_export(self._h, off, C.c_void_p(out.ctypes.data + off), n)
            if rc != 0:
                raise PearlError(rc, "pearl_prb_export")
        return out

    def import_image(self, image, piece_bytes: int = 1 << 28) -> None:
        """Restores the buffer from an image made by export_image (pearl_prb_import; the geometry must match)."""
        import numpy as np
        lib = load_library()
        image = np.ascontiguousarray(image, dtype=np.uint8)
        total = int(lib.pearl_prb_image_bytes(self._h))
        if image.shape[0] != total:
            raise PearlError(-7, "pearl_prb_import")
        for off in range(0, total, piece_bytes):
            n = min(piece_bytes, total - off)
            rc = lib.pearl_prb_import(self._h, off, C.c_void_p(image.ctypes.data + off), n)
            if rc != 0:
                raise PearlError(rc, "pearl_prb_import")

    def read_rows(self, idx):
        import numpy as np
        idx = np.ascontiguousarray(idx, dtype=np.int32)
        n = idx.shape[0]
        out = {"obs": np.zeros((n, self.obs_bytes), np.uint8), "act": np.zeros((n, self.act_bytes), np.uint8),
               "rew": np.zeros(n, np.float32), "next_obs": np.zeros((n, self.obs_bytes), np.uint8),
               "done": np.zeros(n, np.uint8)}
        rc = load_library().pearl_prb_read_rows(self._h, _hptr(idx, "idx"), n, _hptr(out["obs"], "obs"),
                                                _hptr(out["act"], "act"), _hptr(out["rew"], "rew"),
                                                _hptr(out["next_obs"], "next_obs"), _hptr(out["done"], "done"))
        if rc != 0:
            raise PearlError(rc, "pearl_prb_read_rows")
        return out

    def kernel_launches(self) -> int:
        return int(load_library().pearl_prb_kernel_launches(self._h))

    def close(self) -> None:
        if self._h is not None:
            load_library().pearl_prb_destroy(self._h)
            self._h = None
            self._slab = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
