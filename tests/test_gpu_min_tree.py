"""The optional min-tree (PEARL_OPT_MIN_TREE) through the C ABI.

The oracle keeps no min-tree: it finds the smallest positive priority by scanning its leaves.  So the
GPU's min-tree is checked against its definition evaluated on the oracle's leaves (every node: the
smallest positive leaf below it), after every kind of call that writes the tree, and the sample whose
weights are normalised over the buffer is checked against the oracle's -- which a buffer with a min-tree
serves from the min-tree's root and one without it from a scan."""
import numpy as np
import pytest
import torch

from paper_2311_09445_b200 import workloads as wk
from prb_harness import Pair

pytestmark = pytest.mark.gpu


def _buffer_norm_sample(pr, B, beta, seed):
    dev = pr.dev
    o = pr.ora.sample(B, beta, seed, buffer_norm=True)
    t = {"idx": torch.full((B,), -1, dtype=torch.int32, device=dev), "w": torch.zeros(B, device=dev),
         "obs": torch.zeros((B, pr.obs_bytes), dtype=torch.uint8, device=dev),
         "next_obs": torch.zeros((B, pr.obs_bytes), dtype=torch.uint8, device=dev)}
    before = pr.gpu.kernel_launches()
    pr.gpu.sample_buffer_norm(B, beta, seed, t["idx"], t["w"], t["obs"], None, None, t["next_obs"], None)
    torch.cuda.synchronize()
    assert np.array_equal(t["idx"].cpu().numpy(), o["idx"])
    np.testing.assert_allclose(t["w"].cpu().numpy(), o["w"], rtol=1e-5, atol=0)
    assert t["w"].max().item() <= 1.0
    assert np.array_equal(t["obs"].cpu().numpy().reshape(-1), np.ascontiguousarray(o["obs"]).view(np.uint8).reshape(-1))
    return o, pr.gpu.kernel_launches() - before


# (workload, capacity, fanout, batch): short rows, rows long enough for the bulk-copy ring (where an update +
# insertion runs its tree kernel beside the row copy), a cluster of eight CTAs per update (32 x 512 >= 8192),
# small fanouts with many levels, a tree of one level, a capacity that is not a power of the fanout
@pytest.mark.parametrize("wl,N,K,B", [(wk.CARTPOLE, 3000, 16, 64), (wk.ATARI, 700, 32, 512), (wk.DDPG, 40_000, 32, 512),
                                      (wk.CARTPOLE, 5000, 2, 128), (wk.CARTPOLE, 777, 4, 100), (wk.TINY, 9, 16, 8),
                                      (wk.DDPG, 20_000, 8, 1000)])
def test_min_tree_follows_every_tree_write(oracle_mod, wl, N, K, B):
    wl = wk.scaled(wl, N, fanout=K)
    rng = np.random.default_rng(N + K)
    pr = Pair(oracle_mod, N, K, wl.obs_bytes, wl.act_bytes, max(B, 512), min_tree=True)
    pr.compare_min_tree()                                       # all zero
    n_ins = max(1, min(400, N // 3))
    first = 0
    for step in range(12):                                      # fills, then wraps the ring
        b = wk.transitions(wl, rng, n_ins, first)
        first += n_ins
        if step % 4 == 1:
            b["prio"][::3] = 0.0                                # zero priorities are never a minimum
        if step % 4 == 2:
            b["prio"] = None                                    # default priority: the running maximum
        if b["prio"] is None:
            assert pr.ora.insert(b["obs"], b.get("act"), b["rew"], b["next_obs"], b["done"], None, n=n_ins) == 0
            d = {k: torch.from_numpy(np.ascontiguousarray(v)).to(pr.dev) for k, v in b.items() if isinstance(v, np.ndarray)}
            pr.gpu.insert(d["obs"], d.get("act"), d["rew"], d["next_obs"], d["done"], None, n=n_ins)
        else:
            pr.insert(b)
        pr.compare_tree()
        pr.compare_min_tree()
        o, launches = _buffer_norm_sample(pr, B, wl.beta, 100 + step)
        assert launches == 1                                    # no scan of the leaves
        idx, td = wk.update_batch(wl, rng, o["idx"])
        kind = step % 5
        if kind == 0:
            pr.update(idx, td, wl.alpha, wl.eps)
        elif kind == 1:
            small = np.abs(td) * np.float32(1e-4)               # new minima
            small[::5] = 0.0                                    # and leaves that stop being positive
            pr.update_priorities(idx, small)
        elif kind == 2:
            nb = wk.transitions(wl, rng, n_ins // 2 + 1, first)
            first += n_ins // 2 + 1
            pr.update_insert(idx, td, wl.alpha, wl.eps, nb)
        elif kind == 3:
            nb = wk.transitions(wl, rng, n_ins // 3 + 1, first)
            first += n_ins // 3 + 1
            pr.step(idx, td, wl.alpha, wl.eps, nb, B, wl.beta, 7)
        else:
            have = pr.ora.get_priorities(idx)
            pr.update_delta(idx, (-0.5 * have / np.maximum(1, np.bincount(idx, minlength=N)[idx])).astype(np.float32))
        pr.compare_tree()
        pr.compare_min_tree()
        pr.compare_state()
    pr.compare_status()
    pr.close()


@pytest.mark.parametrize("N,K,B", [(200_000, 2, 20_000), (200_000, 4, 5000), (100_000, 16, 3000), (70_000, 32, 2048)])
def test_min_tree_after_updates_of_large_batches(oracle_mod, N, K, B):
    # more than 1024 entries: the update is one launch of many thread blocks, level by level
    wl = wk.scaled(wk.DDPG, N, fanout=K)
    rng = np.random.default_rng(N + K + B)
    pr = Pair(oracle_mod, N, K, 0, 0, max(B, 1024), oracle_store=False, min_tree=True)
    for first in range(0, N, pr.gpu.max_batch):
        m = min(pr.gpu.max_batch, N - first)
        pr.insert({"rew": np.zeros(m, np.float32), "done": np.zeros(m, np.uint8), "prio": wk.priorities(wl, rng, m)})
    pr.compare_min_tree()
    for call in range(3):
        idx = rng.integers(0, N, B).astype(np.int32)
        idx[::17] = idx[3]                                       # repeated indices: the last entry wins
        td = wk.td_errors(wl, rng, B)
        if call == 1:
            td[::9] *= np.float32(1e-5)
        pr.update(idx, td, wl.alpha, wl.eps)
        pr.compare_tree()
        pr.compare_min_tree()
    pr.update_priorities(rng.integers(0, N, B).astype(np.int32), np.zeros(B, np.float32))      # clears leaves
    pr.compare_tree()
    pr.compare_min_tree()
    assert pr.compare_status() == 0
    pr.close()


def test_min_tree_with_the_frame_layout(oracle_mod):
    S, F, N, K, B = 4, 7056, 3000, 32, 512
    rng = np.random.default_rng(5)
    traj = wk.FrameTrajectory(rng, F, S, episode_steps=(1, 25))
    pr = Pair(oracle_mod, N, K, S * F, 4, 512, frame_stack=S, min_tree=True)
    for step in range(10):
        b = traj.next(400, stacks=False)
        pr.insert({"obs": b["frame"], "act": b["act"], "rew": b["rew"], "done": b["done"], "prio": b["prio"]})
        pr.compare_tree()
        pr.compare_min_tree()                                   # markers and cleared leaves are 0: never a minimum
        o, launches = _buffer_norm_sample(pr, B, 0.4, step)
        b = traj.next(100, stacks=False)
        pr.update_insert(o["idx"], (rng.standard_normal(B) * 2).astype(np.float32), 0.6, 1e-6,
                         {"obs": b["frame"], "act": b["act"], "rew": b["rew"], "done": b["done"], "prio": b["prio"]})
        pr.compare_tree()
        pr.compare_min_tree()
    pr.compare_status()
    pr.close()


def test_min_tree_is_an_option(oracle_mod):
    from paper_2311_09445_b200 import PearlError, PrioritizedReplay
    plain = PrioritizedReplay(1000, 16, 64, 8, 256)
    with pytest.raises(PearlError) as e:
        plain.read_min_level(0)
    assert e.value.code == -7
    with_min = PrioritizedReplay(1000, 16, 64, 8, 256, min_tree=True)
    assert with_min.slab_bytes > plain.slab_bytes
    assert np.array_equal(with_min.read_min_level(0), np.zeros(1, np.float32))
    with pytest.raises(PearlError) as e:
        with_min.read_min_level(with_min.depth)                 # the leaves belong to the sum tree
    assert e.value.code == -7
    plain.close()
    with_min.close()
