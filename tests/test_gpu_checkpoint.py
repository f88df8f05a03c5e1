"""Checkpoint and resume (pearl_prb_export / pearl_prb_import) through the C ABI.

A buffer is driven beside the oracle, exported, and imported into a NEW buffer of the same geometry; the run
then goes on with the new buffer on the GPU side and the same, uninterrupted oracle on the other: every
later sample, tree level, counter and stored row must still agree -- the image holds everything the results
depend on."""
import numpy as np
import pytest
import torch

from paper_2311_09445_b200 import workloads as wk
from prb_harness import Pair

pytestmark = pytest.mark.gpu


def _drive(pr, wl, rng, steps, first_id, B, n, frames=None):
    for step in range(steps):
        o, g = pr.sample(B, wl.beta, 50 + step)
        idx, td = wk.update_batch(wl, rng, o["idx"])
        if frames is not None:
            b = frames.next(n, stacks=False)
            batch = {"obs": b["frame"], "act": b["act"], "rew": b["rew"], "done": b["done"], "prio": b["prio"]}
        else:
            batch = wk.transitions(wl, rng, n, first_id)
        first_id += n
        if step % 2:
            pr.update_insert(idx, td, wl.alpha, wl.eps, batch)
        else:
            pr.update(idx, td, wl.alpha, wl.eps)
            pr.insert(batch)
        pr.compare_tree()
        pr.compare_state()
    return first_id


@pytest.mark.parametrize("wl,N,B,n,stack,min_tree,piece", [(wk.CARTPOLE, 3000, 64, 500, 0, False, 1 << 28),
                                                          (wk.DDPG, 20_000, 256, 1000, 0, True, 100_000),
                                                          (wk.ATARI, 300, 128, 90, 0, False, 1 << 22),
                                                          (wk.ATARI, 400, 64, 70, 4, True, 1 << 28)])
def test_resumed_buffer_goes_on_like_the_exported_one(oracle_mod, wl, N, B, n, stack, min_tree, piece):
    from paper_2311_09445_b200 import PrioritizedReplay
    wl = wk.scaled(wl, N)
    rng = np.random.default_rng(N + B)
    frames = wk.FrameTrajectory(rng, wl.obs_bytes // stack, stack, episode_steps=(1, 30)) if stack else None
    pr = Pair(oracle_mod, N, wl.fanout, wl.obs_bytes, wl.act_bytes, 1024, frame_stack=stack, min_tree=min_tree)
    first = 0
    for _ in range(2):                                           # something to sample from
        if frames is not None:
            b = frames.next(n, stacks=False)
            pr.insert({"obs": b["frame"], "act": b["act"], "rew": b["rew"], "done": b["done"], "prio": b["prio"]})
        else:
            pr.insert(wk.transitions(wl, rng, n, first))
        first += n
    first = _drive(pr, wl, rng, 5, first, B, n, frames)          # fills and wraps the ring
    image = pr.gpu.export_image(piece)
    assert 256 < image.shape[0] < pr.gpu.slab_bytes              # (scratch and staging areas are not part of it)
    # the exported buffer is untouched by the export
    pr.compare_tree()
    pr.compare_state()
    fresh = PrioritizedReplay(N, wl.fanout, wl.obs_bytes, wl.act_bytes, 1024, frame_stack=stack, min_tree=min_tree)
    fresh.import_image(image, piece)
    old = pr.gpu
    pr.gpu = fresh
    old.close()
    pr.compare_tree()
    if min_tree:
        pr.compare_min_tree()
    pr.compare_state()
    keep = np.nonzero(pr.ora.read_level(pr.ora.depth)[:N] > 0)[0].astype(np.int32)[:300]
    pr.compare_rows(keep)
    _drive(pr, wl, rng, 5, first, B, n, frames)                  # ... and the run goes on
    if min_tree:
        pr.compare_min_tree()
    assert np.array_equal(fresh.export_image(piece)[:256], image[:256])
    pr.compare_status()
    pr.close()


def test_import_checks_the_geometry_and_the_range(oracle_mod):
    from paper_2311_09445_b200 import PearlError, PrioritizedReplay
    from paper_2311_09445_b200.binding import load_library
    import ctypes as C
    a = PrioritizedReplay(1000, 16, 64, 8, 256)
    image = a.export_image()
    for other in (PrioritizedReplay(1000, 8, 64, 8, 256), PrioritizedReplay(1001, 16, 64, 8, 256),
                  PrioritizedReplay(1000, 16, 64, 8, 256, min_tree=True), PrioritizedReplay(1000, 16, 48, 8, 256)):
        fitted = np.zeros(int(load_library().pearl_prb_image_bytes(other._h)), np.uint8)     # the other's size, this header
        m = min(fitted.shape[0], image.shape[0])
        fitted[:m] = image[:m]
        with pytest.raises(PearlError) as e:
            other.import_image(fitted)
        assert e.value.code == -7
        assert other.info()[0] == 0 and other.sync() == 0        # nothing was copied
        other.close()
    lib = load_library()
    total = int(lib.pearl_prb_image_bytes(a._h))
    buf = np.zeros(64, np.uint8)
    assert lib.pearl_prb_export(a._h, total - 10, C.c_void_p(buf.ctypes.data), 64) == -7       # past the end
    assert lib.pearl_prb_import(a._h, 8, C.c_void_p(buf.ctypes.data), 64) == -7               # a part of the header
    assert lib.pearl_prb_export(a._h, total - 10, C.c_void_p(buf.ctypes.data), 10) == 0
    same = PrioritizedReplay(1000, 16, 64, 8, 256)
    same.import_image(image, 777)                                 # odd pieces; the first covers the header
    assert same.info() == a.info()
    same.close()
    a.close()
