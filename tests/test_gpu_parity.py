"""Parity of the CUDA library (through the C ABI) against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from conftest import golden_lines
from paper_2311_09445_b200 import workloads as wk
from prb_harness import Pair, seed_for_sliver, sliver_leaves

pytestmark = pytest.mark.gpu

P8 = np.array([3, 1, 4, 1, 5, 9, 2, 6], dtype=np.float32)
FANOUTS = [2, 4, 8, 16, 32]


def raw_fields(rng, n, obs_bytes, act_bytes):
    return dict(obs=rng.integers(0, 256, size=(n, obs_bytes), dtype=np.uint8),
                act=rng.integers(0, 256, size=(n, act_bytes), dtype=np.uint8),
                rew=rng.standard_normal(n).astype(np.float32),
                next_obs=rng.integers(0, 256, size=(n, obs_bytes), dtype=np.uint8),
                done=rng.integers(0, 2, size=n, dtype=np.uint8))


@pytest.mark.parametrize("K", [2, 4, 8])
def test_hand_worked_tree(oracle_mod, K):
    rows = golden_lines("eight_leaf_levels.txt")
    pr = Pair(oracle_mod, 8, K, 0, 0, 16)
    pr.insert(dict(prio=P8))
    for case, k, level, *vals in rows:
        if case == "init" and int(k) == K:
            assert pr.gpu.read_level(int(level)).tolist() == [float(v) for v in vals]
    pr.update_priorities(np.array([5, 5], np.int32), np.array([7.0, 2.0], np.float32))
    for case, k, level, *vals in rows:
        if case == "upd" and int(k) == K:
            assert pr.gpu.read_level(int(level)).tolist() == [float(v) for v in vals]
    pr.compare_tree()
    pr.close()


@pytest.mark.parametrize("K", FANOUTS)
@pytest.mark.parametrize("N,obs_bytes,act_bytes", [(1, 16, 4), (7, 3, 1), (100, 68, 24), (1000, 16, 4), (4097, 40, 2)])
def test_small_buffers_all_calls(oracle_mod, K, N, obs_bytes, act_bytes):
    rng = np.random.default_rng(K * 10007 + N)
    maxb = 300
    pr = Pair(oracle_mod, N, K, obs_bytes, act_bytes, maxb)
    # sampling an empty buffer
    o, g = pr.sample(5, 0.4, 1)
    assert g["idx"].tolist() == [-1] * 5
    assert pr.compare_status() == 4
    pr.compare_state()
    inserted = 0
    for step in range(12):
        n = int(rng.integers(1, min(N, maxb) + 1))
        b = raw_fields(rng, n, obs_bytes, act_bytes)
        b["prio"] = (np.abs(rng.standard_normal(n)) + 1e-6).astype(np.float32) ** np.float32(0.6)
        if step == 3:
            b["prio"][0] = np.nan
        pr.insert(b)
        inserted += n
        pr.compare_state()
        pr.compare_tree()
        B = int(rng.integers(1, maxb + 1))
        o, g = pr.sample(B, 0.4, seed=77 + step)
        fill = min(inserted, N)
        idx = o["idx"].copy()
        if B > 4:
            idx[1] = idx[0]                # duplicates with different TD errors
            idx[B // 2] = idx[B - 1]
        if step % 3 == 1 and B > 6:
            idx[2] = -1                    # invalid entries are skipped
            idx[3] = fill
        td = rng.standard_normal(B).astype(np.float32)
        if step % 4 == 2:
            td[B - 1] = np.inf
        pr.update(idx, td, 0.6, 1e-6)
        pr.compare_tree()
        pr.compare_status()
    pr.compare_rows(np.arange(min(inserted, N), dtype=np.int32))
    pr.close()


def test_tiny_workload_100_steps(oracle_mod):
    wl = wk.TINY
    rng = np.random.default_rng(wl.seed)
    pr = Pair(oracle_mod, wl.capacity, wl.fanout, wl.obs_bytes, wl.act_bytes, 4096)
    pr.insert(wk.transitions(wl, rng, wl.capacity))
    pr.compare_tree()
    for step in range(wl.steps):
        o, g = pr.sample(wl.batch, wl.beta, wl.philox_seed)
        idx, td = wk.update_batch(wl, rng, o["idx"])
        pr.update(idx, td, wl.alpha, wl.eps)
        pr.compare_tree()
    pr.compare_state()
    assert pr.compare_status() & ~8 == 0
    pr.close()


@pytest.mark.parametrize("wl,steps,prefill_chunk", [(wk.CARTPOLE, 60, 4096), (wk.DDPG, 40, 4096)])
def test_full_size_mlp_workloads(oracle_mod, wl, steps, prefill_chunk):
    rng = np.random.default_rng(wl.seed)
    pr = Pair(oracle_mod, wl.capacity, wl.fanout, wl.obs_bytes, wl.act_bytes, prefill_chunk)
    for first in range(0, wl.capacity, prefill_chunk):
        pr.insert(wk.transitions(wl, rng, prefill_chunk, first))
    pr.compare_tree()
    pr.compare_state()
    top = range(0, pr.ora.depth)
    for step in range(steps):
        pr.insert(wk.transitions(wl, rng, wl.n_insert))
        o, g = pr.sample(wl.batch, wl.beta, wl.philox_seed)
        idx, td = wk.update_batch(wl, rng, o["idx"])
        if wl.dup_frac:
            assert len(set(idx.tolist())) < len(idx)
        pr.update(idx, td, wl.alpha, wl.eps)
        pr.compare_tree(None if step % 10 == 9 else top)
    pr.compare_state()
    assert pr.compare_status() & ~8 == 0
    pr.compare_rows(rng.integers(0, wl.capacity, size=2000).astype(np.int32))
    pr.close()


def test_atari_shaped_reduced_capacity(oracle_mod):
    # Full oracle mirror (storage included) at a capacity the host can hold; same row shape,
    # fanout and batch as the Atari-shaped workload.
    wl = wk.scaled(wk.ATARI, 2048)
    rng = np.random.default_rng(wl.seed)
    pr = Pair(oracle_mod, wl.capacity, wl.fanout, wl.obs_bytes, wl.act_bytes, 512)
    next_id = 0
    for _ in range(5):                       # 2560 rows: fills and wraps
        pr.insert(wk.transitions(wl, rng, 512, next_id))
        next_id += 512
    pr.compare_tree()
    for step in range(6):
        pr.insert(wk.transitions(wl, rng, wl.n_insert if step % 2 == 0 else 100, next_id))
        next_id += wl.n_insert if step % 2 == 0 else 100
        o, g = pr.sample(wl.batch, wl.beta, wl.philox_seed)
        idx, td = wk.update_batch(wl, rng, o["idx"])
        pr.update(idx, td, wl.alpha, wl.eps)
        pr.compare_tree()
    pr.compare_state()
    pr.compare_rows(np.arange(0, 2048, 7, dtype=np.int32))
    pr.close()


def test_atari_shaped_full_size(oracle_mod):
    # 2^19 slots x 56 457 B cannot be mirrored on the host: the oracle keeps the tree (and the
    # small fields) only, and gathered observations are checked against rows regenerated from the
    # global insert id of the sampled slot.  Launch configuration = the benchmark's.
    wl = wk.ATARI
    free, _ = torch.cuda.mem_get_info()
    need = wl.capacity * wl.transition_bytes + (2 << 30)
    if free < need:
        pytest.skip("not enough free device memory for the full-size store")
    rng = np.random.default_rng(wl.seed)
    pr = Pair(oracle_mod, wl.capacity, wl.fanout, wl.obs_bytes, wl.act_bytes, 512, oracle_store=False)
    dev = pr.dev
    slot_id = np.full(wl.capacity, -1, dtype=np.int64)
    next_id, cursor = 0, 0

    def insert(n):
        nonlocal next_id, cursor
        small = wk.transitions(wl, rng, n, with_obs=False)
        ids = torch.arange(next_id, next_id + n, dtype=torch.int64, device=dev)
        d = {"obs": wk.counter_row_bytes(ids, 0, wl.obs_bytes), "next_obs": wk.counter_row_bytes(ids, 1, wl.obs_bytes)}
        for k in ("act", "rew", "done", "prio"):
            d[k] = torch.from_numpy(small[k]).to(dev)
        pr.insert(dict(rew=small["rew"], done=small["done"], prio=small["prio"]), dev_batch=d)
        slot_id[(cursor + np.arange(n)) % wl.capacity] = np.arange(next_id, next_id + n)
        next_id += n
        cursor = (cursor + n) % wl.capacity

    for _ in range(wl.capacity // 512):
        insert(512)
    pr.compare_tree()
    pr.compare_state()
    for step in range(4):
        insert(wl.n_insert)
        o, g = pr.sample(wl.batch, wl.beta, wl.philox_seed)      # indices, weights checked inside
        ids = torch.from_numpy(slot_id[o["idx"]])
        assert np.array_equal(g["obs"], wk.counter_row_bytes(ids, 0, wl.obs_bytes).numpy())
        assert np.array_equal(g["next_obs"], wk.counter_row_bytes(ids, 1, wl.obs_bytes).numpy())
        rows = pr.ora.read_rows(o["idx"])
        assert np.array_equal(g["rew"], rows["rew"]) and np.array_equal(g["done"], rows["done"])
        idx, td = wk.update_batch(wl, rng, o["idx"])
        pr.update(idx, td, wl.alpha, wl.eps)
        pr.compare_tree()
    pr.compare_state()
    # the benchmark's step: sample, then update and insertion in one call (for rows this long the tree
    # work runs as a kernel of its own beside the row copy)
    for step in range(3):
        o, g = pr.sample(wl.batch, wl.beta, wl.philox_seed)
        ids = torch.from_numpy(slot_id[o["idx"]])
        assert np.array_equal(g["obs"], wk.counter_row_bytes(ids, 0, wl.obs_bytes).numpy())
        idx, td = wk.update_batch(wl, rng, o["idx"])
        n = wl.n_insert
        small = wk.transitions(wl, rng, n, with_obs=False)
        new_ids = torch.arange(next_id, next_id + n, dtype=torch.int64, device=dev)
        assert pr.ora.update(idx, td, wl.alpha, wl.eps) == 0
        assert pr.ora.insert(None, None, small["rew"], None, small["done"], small["prio"]) == 0
        pr.gpu.update_insert(torch.from_numpy(idx).to(dev), torch.from_numpy(td).to(dev), wl.alpha, wl.eps,
                             wk.counter_row_bytes(new_ids, 0, wl.obs_bytes), torch.from_numpy(small["act"]).to(dev),
                             torch.from_numpy(small["rew"]).to(dev), wk.counter_row_bytes(new_ids, 1, wl.obs_bytes),
                             torch.from_numpy(small["done"]).to(dev), torch.from_numpy(small["prio"]).to(dev))
        slot_id[(cursor + np.arange(n)) % wl.capacity] = np.arange(next_id, next_id + n)
        next_id += n
        cursor = (cursor + n) % wl.capacity
        pr.compare_tree()
        pr.compare_state()
    o, g = pr.sample(wl.batch, wl.beta, wl.philox_seed)
    ids = torch.from_numpy(slot_id[o["idx"]])
    assert np.array_equal(g["obs"], wk.counter_row_bytes(ids, 0, wl.obs_bytes).numpy())
    assert np.array_equal(g["next_obs"], wk.counter_row_bytes(ids, 1, wl.obs_bytes).numpy())
    pr.compare_status()
    pr.close()


SWEEP_CAPACITIES = [1 << 16, 1 << 18, 1 << 20, 1 << 22, 1 << 24, 1 << 26]
SWEEP_FANOUTS = [2, 4, 16, 32]
SWEEP_BATCHES = [32, 256, 1024, 4096, 16384, 65536]


def test_sweep_grid_is_the_stated_one():
    # capacity 2^16..2^26 x fanout {2,4,16,32} x batch {32..65536}, batches up to half the capacity: 140 cells
    cells = [(N, K, B) for N in SWEEP_CAPACITIES for K in SWEEP_FANOUTS for B in SWEEP_BATCHES if B <= N // 2]
    assert len(cells) == 140


@pytest.mark.parametrize("K", SWEEP_FANOUTS)
@pytest.mark.parametrize("N", SWEEP_CAPACITIES)
def test_sweep_cells(oracle_mod, N, K):
    # Every cell of the scaling sweep: one buffer per (capacity, fanout), filled once, then for every
    # batch size of the grid two mixed steps (insert 1024, sample B, update B) compared with the oracle
    # call by call -- indices, weights, rows, every tree level, counters, status bits.  Up to 2^22
    # slots the oracle mirrors the whole store; above, the tree and the short fields (the
    # observations then live on the device only and the reward stands in for the row).
    full = N <= (1 << 22)
    if not full:
        free, _ = torch.cuda.mem_get_info()
        if free < N * 165 + (3 << 30):
            pytest.skip("not enough free device memory")
    wl = wk.sweep_cell(N, K, 1024, cell_id=N % 997 + K)
    rng = np.random.default_rng(wl.seed)
    chunk = min(N, 1 << 18)
    batches = [B for B in SWEEP_BATCHES if B <= N // 2]
    pr = Pair(oracle_mod, N, K, wl.obs_bytes, wl.act_bytes, max(chunk, max(batches)), oracle_store=full)
    dev = pr.dev
    zeros = None if full else {"obs": torch.zeros((chunk, wl.obs_bytes), dtype=torch.uint8, device=dev),
                               "act": torch.zeros((chunk, wl.act_bytes), dtype=torch.uint8, device=dev)}

    def insert(n, first):
        if full:
            pr.insert(wk.transitions(wl, rng, n, first))
            return
        prio = wk.priorities(wl, rng, n)
        rew = rng.standard_normal(n).astype(np.float32)
        done = (rng.random(n) < 0.05).astype(np.uint8)
        d = dict(obs=zeros["obs"][:n], next_obs=zeros["obs"][:n], act=zeros["act"][:n], rew=torch.from_numpy(rew).to(dev),
                 done=torch.from_numpy(done).to(dev), prio=torch.from_numpy(prio).to(dev))
        pr.insert(dict(rew=rew, done=done, prio=prio), dev_batch=d)

    for first in range(0, N, chunk):
        insert(chunk, first)
    D = pr.ora.depth
    assert D == pr.gpu.depth
    pr.compare_tree()
    pr.compare_state()
    upper = range(0, D if full else max(1, D - 2))      # (the two widest levels of the largest trees: once per batch size)
    for B in batches:
        for step in range(2):
            insert(wl.n_insert, N)
            o, g = pr.sample(B, wl.beta, wl.philox_seed)
            if not full:
                rows = pr.ora.read_rows(o["idx"])
                assert np.array_equal(g["rew"], rows["rew"]) and np.array_equal(g["done"], rows["done"])
            idx, td = wk.update_batch(wl, rng, o["idx"])
            pr.update(idx, td, wl.alpha, wl.eps)
            pr.compare_tree(upper if step == 0 else None)
        pr.compare_state()
        assert pr.compare_status() & ~8 == 0
    pr.close()


@pytest.mark.parametrize("K,N,B", [(2, 1 << 16, 16384), (2, 5000, 5), (4, 5000, 5), (4, 20_000, 2001), (8, 40_000, 3),
                                   (8, 40_000, 1100), (16, 70_000, 3), (16, 70_000, 777), (4, 20_000, 2049), (8, 40_000, 5000),
                                   (32, 100_000, 3333), (16, 70_000, 2048)])
def test_sample_with_a_ragged_last_warp(oracle_mod, K, N, B):
    # The strata of a CTA need not fill its last warp of lane groups (several groups share a warp
    # below fanout 32) while the leaves are prefetched: every group of the warp walks all the same.
    rng = np.random.default_rng(K + N + B)
    pr = Pair(oracle_mod, N, K, 8, 4, max(B, 4096))
    for first in range(0, N, 4096):
        n = min(4096, N - first)
        b = raw_fields(rng, n, 8, 4)
        b["prio"] = rng.uniform(0.01, 1, n).astype(np.float32)
        pr.insert(b)
    for _ in range(3):
        pr.sample(B, 0.4, 3)
    pr.compare_status()
    pr.close()


@pytest.mark.parametrize("K", FANOUTS)
@pytest.mark.parametrize("B", [2048, 4099, 20_000])
def test_large_batch_sample_cases(oracle_mod, K, B):
    # Large batches of short rows take the one-stratum-per-thread kernel: most leaves zero, the rest
    # spread over many orders of magnitude (prefix sums that round), every beta, weights optional.
    rng = np.random.default_rng(K * 31 + B)
    N = 50_000
    pr = Pair(oracle_mod, N, K, 12, 4, max(B, 4096))
    for first in range(0, N - 3, 4096):
        n = min(4096, N - 3 - first)
        b = raw_fields(rng, n, 12, 4)
        p = np.exp(4.0 * rng.standard_normal(n)).astype(np.float32)
        p[rng.random(n) < 0.9] = 0.0
        b["prio"] = p
        pr.insert(b)
    for beta in (0.0, 0.4, 1.0):
        pr.sample(B, beta, 17)
    pr.compare_status()
    # the same call without weights leaves the state as the oracle's
    t = torch.full((B,), -1, dtype=torch.int32, device=pr.dev)
    pr.gpu.sample(B, 0.4, 17, t)
    o = pr.ora.sample(B, 0.4, 17, gather=False)
    assert np.array_equal(o["idx"], t.cpu().numpy())
    pr.sample(B, 0.4, 17)
    pr.compare_state()
    pr.close()


@pytest.mark.parametrize("K,D,lift,B", [
    # a lane group per stratum (prb_sample_kernel<K>): the group falls off in a staged level, in a level
    # read from global memory, in prefetched leaves, and at an inner level
    (2, 10, 0, 1024), (2, 14, 0, 1024), (2, 9, 2, 1024), (4, 6, 1, 1024), (8, 4, 0, 1024), (16, 3, 0, 1024),
    (16, 5, 0, 1024), (16, 3, 1, 1024), (32, 3, 0, 1024), (32, 4, 0, 1024), (32, 2, 1, 512),
    # a thread per stratum (prb_sample_wide_kernel<K>, from 2048 strata of short rows)
    (2, 14, 0, 4096), (2, 9, 2, 2048), (4, 6, 1, 4096), (8, 4, 0, 4096), (16, 5, 0, 4096), (16, 3, 1, 65536),
    (32, 3, 0, 2048), (32, 2, 1, 4096)])
def test_descent_falls_off_a_child_group(oracle_mod, K, D, lift, B):
    # The rounding sliver: a prefix that rounded up leaves a residual no child group can hold, and the
    # walk takes the last positive child (status CLAMPED).  The tree is built through insert alone and
    # the Philox seed is found on the CPU so that the batch's last stratum draws such a target; the
    # oracle must report the fall-off, and indices, weights, rows and status bits must agree.
    p, leaf = sliver_leaves(K, D, lift)
    N = p.shape[0]
    rng = np.random.default_rng(K * 100 + D)
    pr = Pair(oracle_mod, N, K, 12, 4, max(B, 4096))
    for first in range(0, N, 4096):
        n = min(4096, N - first)
        b = raw_fields(rng, n, 12, 4)
        b["prio"] = p[first:first + n]
        pr.insert(b)
    pr.compare_tree()
    assert pr.ora.total() == np.float32(2 ** 24 + 4)
    for call in range(2):                    # the call counter is part of the Philox counter
        seed = seed_for_sliver(oracle_mod, B, call=call)
        o, g = pr.sample(B, 0.4, seed)
        assert o["idx"][-1] == leaf
        assert pr.compare_status() == 8      # CLAMPED on both sides, nothing else
    pr.compare_state()
    pr.close()


def test_degenerate_sampling_cases(oracle_mod):
    rng = np.random.default_rng(17)
    pr = Pair(oracle_mod, 300, 16, 68, 24, 128)
    b = raw_fields(rng, 100, 68, 24)
    b["prio"] = np.zeros(100, np.float32)
    pr.insert(b)                                         # stored, but the total is zero
    o, g = pr.sample(16, 0.4, 3)
    assert g["idx"].tolist() == [-1] * 16 and pr.compare_status() == 4
    pr.compare_state()
    pr.update_priorities(np.array([7], np.int32), np.array([2.5], np.float32))   # a single positive leaf
    for beta in (0.0, 1.0, 0.4):
        o, g = pr.sample(33, beta, 3)
        assert np.all(g["idx"] == 7) and np.all(g["w"] == 1.0)
    pr.update_priorities(np.arange(100, dtype=np.int32), rng.uniform(0.1, 1, 100).astype(np.float32))
    for beta in (0.0, 1.0):
        o, g = pr.sample(128, beta, 5)
        if beta == 0.0:
            assert np.all(g["w"] == 1.0)
    o, g = pr.sample(1, 0.4, 5)                          # B = 1
    assert g["w"][0] == 1.0
    # outputs are optional: indices only, then indices + weights + one field
    dev = pr.dev
    idx = torch.full((64,), -1, dtype=torch.int32, device=dev)
    o = pr.ora.sample(64, 0.4, 5)
    pr.gpu.sample(64, 0.4, 5, idx)
    assert np.array_equal(idx.cpu().numpy(), o["idx"])
    w = torch.zeros(64, device=dev)
    rew = torch.zeros(64, device=dev)
    o = pr.ora.sample(64, 0.4, 5)
    pr.gpu.sample(64, 0.4, 5, idx, w, rew=rew)
    assert np.array_equal(idx.cpu().numpy(), o["idx"]) and np.array_equal(rew.cpu().numpy(), o["rew"])
    np.testing.assert_allclose(w.cpu().numpy(), o["w"], rtol=1e-5)
    pr.compare_state()
    assert pr.compare_status() == 0
    pr.close()


def test_priority_transform_bits(oracle_mod):
    # The power is compared through the leaves it writes: 4096 TD errors x several exponents.
    rng = np.random.default_rng(21)
    N = 4096
    pr = Pair(oracle_mod, N, 16, 0, 0, 4096)
    pr.insert(dict(prio=np.ones(N, np.float32)))
    idx = np.arange(N, dtype=np.int32)
    for alpha, eps in [(0.6, 1e-6), (1.0, 0.0), (0.5, 1e-3), (0.0, 1e-6), (1.7, 1e-6), (0.123, 0.5)]:
        td = np.concatenate([rng.standard_normal(N // 2), np.exp(2 * rng.standard_normal(N // 4)),
                             rng.uniform(-1e-5, 1e-5, N // 4)]).astype(np.float32)
        td[:4] = [0.0, -0.0, 1e-30, 3e38]
        pr.update(idx, td, alpha, eps)
        pr.compare_tree()
        leaves = pr.gpu.read_level(pr.gpu.depth)[:N]
        for i in (0, 5, 100, 4095):
            assert leaves[i] == oracle_mod.priority_pow(td[i], eps, alpha)
    pr.compare_status()
    pr.close()


def test_host_buffer_calls(oracle_mod):
    wl = wk.scaled(wk.DDPG, 5000)
    rng = np.random.default_rng(5)
    pr = Pair(oracle_mod, wl.capacity, wl.fanout, wl.obs_bytes, wl.act_bytes, 1024)
    for _ in range(7):
        pr.insert(wk.transitions(wl, rng, 1000), host_call=True)
        o, g = pr.sample(256, 0.4, 9, host_call=True)
        idx, td = wk.update_batch(wl, rng, o["idx"])
        pr.update(idx, td, 0.6, 1e-6, host_call=True)
        pr.compare_tree()
    pr.compare_state()
    pr.close()


@pytest.mark.parametrize("wl,N,B,n", [(wk.CARTPOLE, 5000, 64, 64), (wk.DDPG, 70_000, 256, 256), (wk.DDPG, 5000, 3000, 1000),
                                      (wk.ATARI, 600, 16, 8), (wk.ATARI, 700, 512, 512), (wk.ATARI, 1500, 300, 37),
                                      (wk.ATARI, 600, 64, 600), (wk.ATARI, 900, 4096, 100)])
def test_step_through_host_buffers(oracle_mod, wl, N, B, n):
    # pearl_prb_step_host: a small step travels through the handle's mapped pinned buffer (no copy call); a
    # larger one with long rows has its copies in both directions in flight at once, the rows of strata that
    # drew a slot of the very insertion of the step being copied last (here: few of them, most, or all); any
    # other is the three host calls.  Whichever way, the oracle's update, insert, sample
    wl = wk.scaled(wl, N)
    rng = np.random.default_rng(N + B)
    pr = Pair(oracle_mod, N, wl.fanout, wl.obs_bytes, wl.act_bytes, 4096)
    next_id = 0
    for first in range(0, N, 1000):
        m = min(1000, N - first)
        pr.insert(wk.transitions(wl, rng, m, next_id), host_call=True)
        next_id += m
    o, g = pr.sample(B, wl.beta, 1, host_call=True)
    for step in range(6):
        idx, td = wk.update_batch(wl, rng, o["idx"])
        b = wk.transitions(wl, rng, n, next_id)
        next_id += n
        assert pr.ora.update(idx, td, wl.alpha, wl.eps) == 0
        assert pr.ora.insert(b["obs"], b["act"], b["rew"], b["next_obs"], b["done"], b["prio"]) == 0
        o = pr.ora.sample(B, wl.beta, 2 + step)
        g = {"idx": np.full(B, -1, np.int32), "w": np.zeros(B, np.float32), "obs": np.zeros((B, wl.obs_bytes), np.uint8),
             "act": np.zeros((B, wl.act_bytes), np.uint8), "rew": np.zeros(B, np.float32),
             "next_obs": np.zeros((B, wl.obs_bytes), np.uint8), "done": np.zeros(B, np.uint8)}
        c = {k: np.ascontiguousarray(v) for k, v in b.items()}
        pr.gpu.step_host(np.ascontiguousarray(idx, np.int32), np.ascontiguousarray(td, np.float32), wl.alpha, wl.eps, c["obs"], c["act"],
                         c["rew"], c["next_obs"], c["done"], c["prio"], B, wl.beta, 2 + step, g["idx"], g["w"], g["obs"], g["act"],
                         g["rew"], g["next_obs"], g["done"])
        pr.compare_sample(o, g)
        pr.compare_tree()
        pr.compare_state()
    pr.compare_status()
    pr.close()


@pytest.mark.parametrize("wl,N,B,n", [(wk.CARTPOLE, 5000, 64, 64), (wk.DDPG, 70_000, 256, 256), (wk.DDPG, 3000, 1000, 777),
                                      (wk.ATARI, 1500, 512, 512), (wk.ATARI, 700, 37, 1), (wk.ATARI, 700, 4096, 300)])
def test_fused_update_insert(oracle_mod, wl, N, B, n):
    # update + insert in one launch == update, then insert; the inserted slots overlap updated ones
    wl = wk.scaled(wl, N)
    rng = np.random.default_rng(B + n)
    pr = Pair(oracle_mod, N, wl.fanout, wl.obs_bytes, wl.act_bytes, 4096)
    chunk = min(N, 4096)
    next_id = 0
    for first in range(0, N + chunk, chunk):            # fill and wrap
        m = min(chunk, N)
        pr.insert(wk.transitions(wl, rng, m, next_id))
        next_id += m
    for step in range(5):
        o, g = pr.sample(min(B, 4096), wl.beta, wl.philox_seed)
        idx, td = wk.update_batch(wl, rng, o["idx"])
        if step % 2 == 1:
            rng.shuffle(idx)                               # unsorted batch: the sort path
            idx[:3] = [(pr.ora.info()[1] + j) % N for j in range(3)]   # slots the insertion overwrites
        pr.update_insert(idx, td, wl.alpha, wl.eps, wk.transitions(wl, rng, n, next_id))
        next_id += n
        pr.compare_tree()
        pr.compare_state()
    pr.compare_status()
    pr.compare_rows(np.arange(0, N, max(1, N // 500), dtype=np.int32))
    pr.close()


@pytest.mark.parametrize("B,n", [(512, 300), (40, 512)])
def test_fused_long_rows_replayed_as_cuda_graph(oracle_mod, B, n):
    # Long rows: update_insert runs its tree kernel on the handle's side stream beside the row copy.
    # Captured into a CUDA graph with a sample between the calls and replayed, it must leave what the
    # oracle leaves after the same sequence of calls.
    from paper_2311_09445_b200 import PrioritizedReplay
    N = 900
    wl = wk.scaled(wk.ATARI, N)
    rng = np.random.default_rng(B)
    dev = torch.device("cuda:0")
    stream = torch.cuda.Stream(dev)
    ora = oracle_mod.OraclePRB(N, wl.fanout, wl.obs_bytes, wl.act_bytes)
    with torch.cuda.stream(stream):
        gpu = PrioritizedReplay(N, wl.fanout, wl.obs_bytes, wl.act_bytes, 512, device=dev, stream=stream)
        first = wk.transitions(wl, rng, 512, 0)
        assert ora.insert(first["obs"], first["act"], first["rew"], first["next_obs"], first["done"], first["prio"]) == 0
        d = wk.to_device(first, dev)
        gpu.insert(d["obs"], d["act"], d["rew"], d["next_obs"], d["done"], d["prio"])
        calls = []
        for c in range(3):
            b = wk.transitions(wl, rng, n, 512 + c * n)
            idx = rng.integers(0, 512, size=B).astype(np.int32)          # unsorted, with duplicates
            td = rng.standard_normal(B).astype(np.float32)
            calls.append((b, idx, td, wk.to_device(b, dev), torch.from_numpy(idx).to(dev), torch.from_numpy(td).to(dev)))
        out_idx = torch.zeros(64, dtype=torch.int32, device=dev)
        out_w = torch.zeros(64, device=dev)

        def sequence():
            for b, idx, td, db, didx, dtd in calls:
                gpu.update_insert(didx, dtd, wl.alpha, wl.eps, db["obs"], db["act"], db["rew"], db["next_obs"], db["done"], db["prio"])
                gpu.sample(64, wl.beta, 5, out_idx, out_w)

        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            sequence()
        for rep in range(2):
            graph.replay()
            torch.cuda.synchronize()
            for b, idx, td, *_ in calls:
                assert ora.update(idx, td, wl.alpha, wl.eps) == 0
                assert ora.insert(b["obs"], b["act"], b["rew"], b["next_obs"], b["done"], b["prio"]) == 0
                o = ora.sample(64, wl.beta, 5, gather=False)
            assert np.array_equal(out_idx.cpu().numpy(), o["idx"])
            np.testing.assert_allclose(out_w.cpu().numpy(), o["w"], rtol=1e-5, atol=0)
            for l in range(ora.depth + 1):
                assert np.array_equal(ora.read_level(l).view(np.uint32), gpu.read_level(l).view(np.uint32)), "level %d" % l
            assert gpu.info() == ora.info()
        assert gpu.sync() == ora.status()
        rows = np.arange(0, N, 7, dtype=np.int32)
        g_rows, o_rows = gpu.read_rows(rows), ora.read_rows(rows)
        for f in g_rows:
            assert np.array_equal(np.ascontiguousarray(g_rows[f]).view(np.uint8).reshape(-1),
                                  np.ascontiguousarray(o_rows[f]).view(np.uint8).reshape(-1)), f
    gpu.close()
    ora.close()


@pytest.mark.parametrize("B,n,beta_mode", [(512, 512, "batch"), (37, 300, "buffer"), (2500, 64, "batch"), (64, 200, "uniform")])
def test_captured_steps_with_two_kernel_sample(oracle_mod, B, n, beta_mode):
    # Inside a stream capture a sample of long rows is two kernels -- the descents on the handle's second
    # stream, the indexed row copy on the caller's -- so that in a replayed sequence of steps the descents
    # of one call overlap the row copies of the calls before.  A captured sequence of back-to-back
    # samples and of whole steps (sample, update + insertion), replayed, must give every call the
    # outputs the oracle gives it, and leave the oracle's tree and state.
    from paper_2311_09445_b200 import PrioritizedReplay
    N = 3000
    wl = wk.scaled(wk.ATARI, N)
    rng = np.random.default_rng(B + n)
    dev = torch.device("cuda:0")
    stream = torch.cuda.Stream(dev)
    ora = oracle_mod.OraclePRB(N, wl.fanout, wl.obs_bytes, wl.act_bytes)

    def outputs():
        return {"idx": torch.full((B,), -1, dtype=torch.int32, device=dev), "w": torch.full((B,), -1.0, device=dev),
                "obs": torch.zeros((B, wl.obs_bytes), dtype=torch.uint8, device=dev),
                "act": torch.zeros((B, wl.act_bytes), dtype=torch.uint8, device=dev), "rew": torch.zeros(B, device=dev),
                "next_obs": torch.zeros((B, wl.obs_bytes), dtype=torch.uint8, device=dev),
                "done": torch.zeros(B, dtype=torch.uint8, device=dev)}

    def gpu_sample(gpu, o):
        args = (o["idx"], o["w"], o["obs"], o["act"], o["rew"], o["next_obs"], o["done"])
        if beta_mode == "uniform":
            gpu.sample_uniform(B, 5, *args)
        elif beta_mode == "buffer":
            gpu.sample_buffer_norm(B, wl.beta, 5, *args)
        else:
            gpu.sample(B, wl.beta, 5, *args)

    def ora_sample():
        if beta_mode == "uniform":
            return ora.sample_uniform(B, 5)
        return ora.sample(B, wl.beta, 5, buffer_norm=(beta_mode == "buffer"))

    def check(o, t):
        g = {k: v.cpu().numpy() for k, v in t.items()}
        assert np.array_equal(o["idx"], g["idx"])
        np.testing.assert_allclose(g["w"], o["w"], rtol=1e-5, atol=0)
        for f in ("obs", "act", "rew", "next_obs", "done"):
            assert np.array_equal(np.ascontiguousarray(o[f]).view(np.uint8).reshape(-1), g[f].view(np.uint8).reshape(-1)), f

    with torch.cuda.stream(stream):
        gpu = PrioritizedReplay(N, wl.fanout, wl.obs_bytes, wl.act_bytes, 4096, device=dev, stream=stream)
        # a captured sample of an empty buffer writes nothing and raises EMPTY
        t0 = outputs()
        torch.cuda.synchronize()
        g0 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g0, stream=stream):
            gpu_sample(gpu, t0)
        g0.replay()
        torch.cuda.synchronize()
        ora_sample()
        assert t0["idx"].min().item() == -1 and t0["idx"].max().item() == -1 and t0["w"].max().item() == -1.0
        assert gpu.sync() == ora.status() == 4
        next_id = 0
        for _ in range(5):
            b = wk.transitions(wl, rng, 512, next_id)
            next_id += 512
            assert ora.insert(b["obs"], b["act"], b["rew"], b["next_obs"], b["done"], b["prio"]) == 0
            d = wk.to_device(b, dev)
            gpu.insert(d["obs"], d["act"], d["rew"], d["next_obs"], d["done"], d["prio"])
        steps = []
        for c in range(3):
            b = wk.transitions(wl, rng, n, next_id + c * n)
            td = (rng.standard_normal(B) * 2).astype(np.float32)
            steps.append((b, td, wk.to_device(b, dev), torch.from_numpy(td).to(dev)))
        outs = [outputs() for _ in range(3 + 4)]

        def sequence():
            for c, (b, td, db, dtd) in enumerate(steps):          # whole steps: the update names what the step sampled
                gpu_sample(gpu, outs[c])
                gpu.update_insert(outs[c]["idx"], dtd, wl.alpha, wl.eps, db["obs"], db["act"], db["rew"], db["next_obs"],
                                  db["done"], db["prio"])
            for c in range(3, 7):                                    # back-to-back samples: the hand-off areas take turns
                gpu_sample(gpu, outs[c])

        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            sequence()
        for rep in range(3):
            graph.replay()
            torch.cuda.synchronize()
            for c, (b, td, db, dtd) in enumerate(steps):
                o = ora_sample()
                check(o, outs[c])
                assert ora.update(o["idx"], td, wl.alpha, wl.eps) == 0
                assert ora.insert(b["obs"], b["act"], b["rew"], b["next_obs"], b["done"], b["prio"]) == 0
            for c in range(3, 7):
                check(ora_sample(), outs[c])
            for l in range(ora.depth + 1):
                assert np.array_equal(ora.read_level(l).view(np.uint32), gpu.read_level(l).view(np.uint32)), "level %d" % l
            assert gpu.info() == ora.info()
            # an eager call between replays (one kernel, on the caller's stream) sees what the replay left
            t = outputs()
            gpu_sample(gpu, t)
            torch.cuda.synchronize()
            check(ora_sample(), t)
        assert gpu.sync() == ora.status()
        rows = np.arange(0, N, 11, dtype=np.int32)
        g_rows, o_rows = gpu.read_rows(rows), ora.read_rows(rows)
        for f in g_rows:
            assert np.array_equal(np.ascontiguousarray(g_rows[f]).view(np.uint8).reshape(-1),
                                  np.ascontiguousarray(o_rows[f]).view(np.uint8).reshape(-1)), f
    gpu.close()
    ora.close()


@pytest.mark.parametrize("wl,N,B_upd,n,B", [(wk.ATARI, 1500, 512, 512, 512), (wk.ATARI, 700, 37, 1, 64), (wk.ATARI, 3000, 300, 300, 3000),
                                            (wk.ATARI, 700, 4096, 300, 512), (wk.ATARI, 900, 5000, 100, 128),
                                            (wk.CARTPOLE, 5000, 64, 64, 64), (wk.DDPG, 70_000, 256, 256, 2500)])
def test_step_is_update_insert_then_sample(oracle_mod, wl, N, B_upd, n, B):
    # pearl_prb_step == pearl_prb_update_insert followed by pearl_prb_sample.  With long rows the sample's
    # descents and weights come from the tree kernel (sampling ahead), its rows from the indexed copy;
    # with short rows, or an update beyond one tree kernel, the call is the two calls.
    wl = wk.scaled(wl, N)
    rng = np.random.default_rng(B_upd + n + B)
    pr = Pair(oracle_mod, N, wl.fanout, wl.obs_bytes, wl.act_bytes, 8192)
    # a step on an empty buffer whose insertion carries zero priorities only: nothing to sample
    first = wk.transitions(wl, rng, min(n, N), 0)
    first["prio"][:] = 0.0
    o, g = pr.step(np.zeros(3, np.int32), np.ones(3, np.float32), wl.alpha, wl.eps, first, 16, wl.beta, 1)
    assert g["idx"].tolist() == [-1] * 16 and pr.compare_status() == 1 | 4      # BAD_INDEX (nothing stored yet), EMPTY
    pr.compare_state()
    next_id = first["prio"].shape[0]
    chunk = min(N, 4096)
    for _ in range(0, N + chunk, chunk):            # fill and wrap
        m = min(chunk, N)
        pr.insert(wk.transitions(wl, rng, m, next_id))
        next_id += m
    o, g = pr.sample(min(B_upd, 8192), wl.beta, wl.philox_seed)
    for step in range(5):
        idx, td = wk.update_batch(wl, rng, o["idx"])
        if step % 2 == 1:
            rng.shuffle(idx)                               # unsorted batch: the sort path
            idx[:3] = [(pr.ora.info()[1] + j) % N for j in range(3)]   # slots the insertion overwrites
            idx[3] = -1
        o, g = pr.step(idx, td, wl.alpha, wl.eps, wk.transitions(wl, rng, n, next_id), B, wl.beta, wl.philox_seed + step)
        next_id += n
        pr.compare_tree()
        pr.compare_state()
        pr.compare_status()
        if B != B_upd:
            o, g = pr.sample(min(B_upd, 8192), wl.beta, wl.philox_seed)
    pr.compare_rows(np.arange(0, N, max(1, N // 500), dtype=np.int32))
    pr.close()


def test_step_in_place_and_captured(oracle_mod):
    # The loop as a trainer runs it: one set of buffers, the update naming the indices the previous step
    # left in the very buffer the step's sample overwrites; captured once, replayed.
    from paper_2311_09445_b200 import PrioritizedReplay
    N, B, n = 2000, 512, 512
    wl = wk.scaled(wk.ATARI, N)
    rng = np.random.default_rng(77)
    dev = torch.device("cuda:0")
    stream = torch.cuda.Stream(dev)
    ora = oracle_mod.OraclePRB(N, wl.fanout, wl.obs_bytes, wl.act_bytes)
    with torch.cuda.stream(stream):
        gpu = PrioritizedReplay(N, wl.fanout, wl.obs_bytes, wl.act_bytes, 512, device=dev, stream=stream)
        next_id = 0
        for _ in range(4):
            b = wk.transitions(wl, rng, 512, next_id)
            next_id += 512
            assert ora.insert(b["obs"], b["act"], b["rew"], b["next_obs"], b["done"], b["prio"]) == 0
            d = wk.to_device(b, dev)
            gpu.insert(d["obs"], d["act"], d["rew"], d["next_obs"], d["done"], d["prio"])
        t = {"idx": torch.full((B,), -1, dtype=torch.int32, device=dev), "w": torch.zeros(B, device=dev),
             "obs": torch.zeros((B, wl.obs_bytes), dtype=torch.uint8, device=dev),
             "act": torch.zeros((B, wl.act_bytes), dtype=torch.uint8, device=dev), "rew": torch.zeros(B, device=dev),
             "next_obs": torch.zeros((B, wl.obs_bytes), dtype=torch.uint8, device=dev),
             "done": torch.zeros(B, dtype=torch.uint8, device=dev)}
        gpu.sample(B, wl.beta, 3, t["idx"], t["w"], t["obs"], t["act"], t["rew"], t["next_obs"], t["done"])
        last = ora.sample(B, wl.beta, 3)
        new = wk.transitions(wl, rng, n, next_id)
        dnew = wk.to_device(new, dev)
        td = (rng.standard_normal(B) * 2).astype(np.float32)
        dtd = torch.from_numpy(td).to(dev)

        def one_step():
            gpu.step(t["idx"], dtd, wl.alpha, wl.eps, dnew["obs"], dnew["act"], dnew["rew"], dnew["next_obs"], dnew["done"],
                     dnew["prio"], B, wl.beta, 3, t["idx"], t["w"], t["obs"], t["act"], t["rew"], t["next_obs"], t["done"])

        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            one_step()
            one_step()
        for rep in range(4):
            if rep == 2:
                one_step()                       # an eager step between replays
                one_step()
            else:
                graph.replay()
            torch.cuda.synchronize()
            for _ in range(2):
                assert ora.update(last["idx"], td, wl.alpha, wl.eps) == 0
                assert ora.insert(new["obs"], new["act"], new["rew"], new["next_obs"], new["done"], new["prio"]) == 0
                last = ora.sample(B, wl.beta, 3)
            assert np.array_equal(t["idx"].cpu().numpy(), last["idx"])
            np.testing.assert_allclose(t["w"].cpu().numpy(), last["w"], rtol=1e-5, atol=0)
            assert np.array_equal(t["obs"].cpu().numpy().reshape(-1), np.ascontiguousarray(last["obs"]).reshape(-1))
            assert np.array_equal(t["next_obs"].cpu().numpy().reshape(-1), np.ascontiguousarray(last["next_obs"]).reshape(-1))
            assert np.array_equal(t["done"].cpu().numpy(), last["done"])
            for l in range(ora.depth + 1):
                assert np.array_equal(ora.read_level(l).view(np.uint32), gpu.read_level(l).view(np.uint32)), "level %d" % l
            assert gpu.info() == ora.info()
        assert gpu.sync() == ora.status()
    gpu.close()
    ora.close()


def test_step_sample_falls_off_a_child_group(oracle_mod):
    # the rounding sliver met by a tree kernel that samples ahead (long rows), both as a step and as the
    # first kernel of a captured two-kernel sample
    K, D, B = 32, 3, 512
    p, leaf = sliver_leaves(K, D, 0)
    N = p.shape[0]
    rng = np.random.default_rng(5)
    pr = Pair(oracle_mod, N, K, 8192, 4, 4096, oracle_store=False)
    dev = pr.dev
    for first in range(0, N, 4096):
        b = dict(rew=rng.standard_normal(4096).astype(np.float32), done=np.zeros(4096, np.uint8), prio=p[first:first + 4096])
        d = {k: torch.from_numpy(v).to(dev) for k, v in b.items()}
        d["obs"] = torch.zeros((4096, 8192), dtype=torch.uint8, device=dev)
        d["next_obs"], d["act"] = d["obs"], torch.zeros((4096, 4), dtype=torch.uint8, device=dev)
        pr.insert(b, dev_batch=d)
    # the step re-writes two zero leaves with zero (update_priorities form is not part of the step: use a
    # TD error with alpha > 0 and eps = 0, |0|^alpha = 0) and inserts nothing that changes the total
    seed = seed_for_sliver(oracle_mod, B, call=0)
    z = np.zeros(1, np.float32)
    cur = pr.ora.info()[1]
    newb = dict(rew=z, done=np.zeros(1, np.uint8), prio=p[cur:cur + 1].copy())
    dnew = {k: torch.from_numpy(v).to(dev) for k, v in newb.items()}
    dnew["obs"] = torch.zeros((1, 8192), dtype=torch.uint8, device=dev)
    dnew["next_obs"], dnew["act"] = dnew["obs"], torch.zeros((1, 4), dtype=torch.uint8, device=dev)
    assert pr.ora.update(np.array([0, 1], np.int32), np.zeros(2, np.float32), 0.6, 0.0) == 0
    assert pr.ora.insert(None, None, newb["rew"], None, newb["done"], newb["prio"]) == 0
    o = pr.ora.sample(B, 0.4, seed, gather=False)
    t = {"idx": torch.full((B,), -1, dtype=torch.int32, device=dev), "w": torch.zeros(B, device=dev),
         "obs": torch.zeros((B, 8192), dtype=torch.uint8, device=dev)}
    pr.gpu.step(torch.tensor([0, 1], dtype=torch.int32, device=dev), torch.zeros(2, device=dev), 0.6, 0.0, dnew["obs"], dnew["act"],
                dnew["rew"], dnew["next_obs"], dnew["done"], dnew["prio"], B, 0.4, seed, t["idx"], t["w"], t["obs"])
    torch.cuda.synchronize()
    assert o["idx"][-1] == leaf and np.array_equal(t["idx"].cpu().numpy(), o["idx"])
    np.testing.assert_allclose(t["w"].cpu().numpy(), o["w"], rtol=1e-5, atol=0)
    assert pr.compare_status() == 8
    pr.compare_tree()
    pr.compare_state()
    pr.close()


@pytest.mark.parametrize("wl", [wk.CARTPOLE, wk.ATARI])
def test_fused_update_uses_fill_before_insert(oracle_mod, wl):
    # In the fused call the update comes first: an index that only the insertion makes valid is refused.
    wl = wk.scaled(wl, 400)
    rng = np.random.default_rng(3)
    pr = Pair(oracle_mod, 400, wl.fanout, wl.obs_bytes, wl.act_bytes, 256)
    pr.insert(wk.transitions(wl, rng, 100, 0))
    for rep in range(20):
        idx = np.array([5, 99, 100, 120, 149, 7], dtype=np.int32)       # fill is 100 before, 150 after
        td = rng.standard_normal(6).astype(np.float32)
        pr.update_insert(idx, td, 0.6, 1e-6, wk.transitions(wl, rng, 50, 100))
        pr.compare_tree()
        assert pr.compare_status() == 1
        pr.close()
        pr = Pair(oracle_mod, 400, wl.fanout, wl.obs_bytes, wl.act_bytes, 256)
        pr.insert(wk.transitions(wl, rng, 100, 0))
    pr.close()


@pytest.mark.parametrize("K,B", [(2, 4097), (16, 10_000), (32, 65536)])
def test_update_beyond_one_subbatch(oracle_mod, K, B):
    # Sub-batches of 4096 in batch order: duplicates that span sub-batches, unsorted, some invalid.
    rng = np.random.default_rng(K + B)
    N = 30_000
    pr = Pair(oracle_mod, N, K, 0, 0, 65536)
    pr.insert(dict(prio=rng.uniform(0.1, 1, N).astype(np.float32)))
    for _ in range(3):
        idx = rng.integers(0, 2000, size=B).astype(np.int32)       # every index many times over
        idx[::1000] = -1
        td = rng.standard_normal(B).astype(np.float32)
        pr.update(idx, td, 0.6, 1e-6)
        pr.compare_tree()
        pr.update_insert(idx[::-1].copy(), td, 0.6, 1e-6, dict(prio=rng.uniform(0.1, 1, 100).astype(np.float32)))
        pr.compare_tree()
        assert pr.compare_status() == 1
    pr.compare_state()
    pr.close()


@pytest.mark.parametrize("K,N,B", [(2, 1 << 20, 5000), (4, 300_000, 8192), (16, 1 << 20, 20_000), (32, 1 << 19, 65536),
                                   (16, 9000, 4097), (8, 70_000, 30_011)])
def test_many_cta_update(oracle_mod, K, N, B):
    # Batches beyond one CTA's reach go to one launch of many CTAs: values and TD errors, sorted and
    # shuffled, sparse (levels with far more nodes than entries) and dense, with repeated indices,
    # refused priorities, indices out of range and entries made stale by an insertion.
    rng = np.random.default_rng(K * 7 + N + B)
    pr = Pair(oracle_mod, N, K, 0, 0, 65536)
    fill = N - 37
    for first in range(0, fill, 65536):
        pr.insert(dict(prio=rng.uniform(0.1, 1, min(65536, fill - first)).astype(np.float32)))
    pr.compare_tree()
    seen = 0
    for step in range(4):
        idx = rng.integers(0, fill, size=B).astype(np.int32)
        if step % 2 == 0:
            idx.sort()                                   # as a stratified sample returns them
        rep = rng.integers(0, B, size=B // 10)
        idx[rep] = idx[rng.integers(0, B, size=B // 10)]          # repeats anywhere in the batch
        idx[rng.integers(0, B, size=7)] = [-1, N, fill, N - 1, 2 ** 31 - 1, -2 ** 31, fill + 5]
        td = (rng.standard_normal(B) * 3).astype(np.float32)
        td[rng.integers(0, B, size=3)] = [np.nan, np.inf, -np.inf]
        if step == 1:
            prio = np.abs(td)
            prio[rng.integers(0, B, size=2)] = [-1.0, np.nan]
            pr.update_priorities(idx, prio)
        elif step == 3:
            pr.insert(dict(prio=rng.uniform(0.1, 1, 777).astype(np.float32)))
            idx[rng.integers(0, B, size=50)] = (pr.ora.info()[1] - 1 - rng.integers(0, 777, size=50)) % N   # just overwritten
            pr.update_after_insert(idx, td, 0.6, 1e-6, 777)
        else:
            pr.update(idx, td, 0.6, 1e-6)
        pr.compare_tree()
        seen |= pr.compare_status()
        pr.compare_state()
    assert seen & 1 and seen & 2 and seen & 32            # bad index, bad priority, stale
    # and the buffer still samples identically afterwards (only priorities were stored: no rows to compare)
    o, g = pr.sample(256, 0.4, 5, check=False)
    assert np.array_equal(o["idx"], g["idx"])
    np.testing.assert_allclose(g["w"], o["w"], rtol=1e-5, atol=0)
    pr.close()


@pytest.mark.parametrize("K,N,B,n", [(2, 300, 64, 50), (16, 5000, 256, 700), (32, 900, 512, 512)])
def test_update_after_insert_and_retrieval(oracle_mod, K, N, B, n):
    # collision-free scheduling: sample, insert, then the update skips what the insertion overwrote
    rng = np.random.default_rng(K * N)
    pr = Pair(oracle_mod, N, K, 8, 4, 1024)
    b = raw_fields(rng, N - 10, 8, 4)
    b["prio"] = rng.uniform(0.1, 1, N - 10).astype(np.float32)
    for first in range(0, N - 10, 1024):
        pr.insert({k: v[first:first + 1024] for k, v in b.items()})
    stale_seen = 0
    for step in range(12):
        o, g = pr.sample(B, 0.4, 11)
        nb = raw_fields(rng, n, 8, 4)
        nb["prio"] = rng.uniform(0.1, 1, n).astype(np.float32)
        pr.insert(nb)
        td = rng.standard_normal(B).astype(np.float32)
        pr.update_after_insert(o["idx"], td, 0.6, 1e-6, n)
        pr.compare_tree()
        stale_seen |= pr.compare_status()
        pr.compare_priorities(np.concatenate([o["idx"], [-1, N, N - 1, 0]]).astype(np.int32))
        pr.compare_status()
    assert stale_seen & 32
    pr.compare_state()
    pr.close()


@pytest.mark.parametrize("wl,N,B", [(wk.CARTPOLE, 3000, 128), (wk.ATARI, 600, 128), (wk.ATARI, 600, 512)])
def test_default_insert_priority(oracle_mod, wl, N, B):
    # insertion without priorities: the running maximum of everything written so far (1 before any)
    wl = wk.scaled(wl, N)
    rng = np.random.default_rng(N)
    pr = Pair(oracle_mod, N, wl.fanout, wl.obs_bytes, wl.act_bytes, 512)
    dev = pr.dev

    def insert_default(n, first, fused_with=None):
        b = wk.transitions(wl, rng, n, first)
        d = {k: torch.from_numpy(np.ascontiguousarray(v)).to(dev) for k, v in b.items() if k != "prio"}
        if fused_with is None:
            assert pr.ora.insert(b["obs"], b["act"], b["rew"], b["next_obs"], b["done"], None, n=n) == 0
            pr.gpu.insert(d["obs"], d["act"], d["rew"], d["next_obs"], d["done"], None, n=n)
        else:
            idx, td = fused_with
            assert pr.ora.update(idx, td, 0.6, 1e-6) == 0
            assert pr.ora.insert(b["obs"], b["act"], b["rew"], b["next_obs"], b["done"], None, n=n) == 0
            pr.gpu.update_insert(torch.from_numpy(idx).to(dev), torch.from_numpy(td).to(dev), 0.6, 1e-6, d["obs"], d["act"],
                                 d["rew"], d["next_obs"], d["done"], None, n=n)

    insert_default(100, 0)                        # nothing written yet: priority 1
    pr.compare_tree()
    pr.compare_state()
    pr.insert(wk.transitions(wl, rng, 200, 100))  # explicit priorities raise the maximum
    pr.compare_state()
    for step in range(6):
        o, g = pr.sample(B, 0.4, 1)          # (B = 512 at fanout 32: the update's CTAs form a cluster)
        td = (rng.standard_normal(B) * (step + 1) * 3).astype(np.float32)
        if step % 2 == 0:
            pr.update(o["idx"], td, 0.6, 1e-6)
            insert_default(77, 300 + 77 * step)
        else:
            insert_default(77, 300 + 77 * step, fused_with=(o["idx"], td))   # the update's writes count already
        pr.compare_tree()
        pr.compare_state()
    pr.compare_status()
    pr.close()


@pytest.mark.parametrize("wl,N,B", [(wk.CARTPOLE, 3000, 64), (wk.DDPG, 100_000, 4096), (wk.ATARI, 700, 512)])
def test_uniform_replay(oracle_mod, wl, N, B):
    wl = wk.scaled(wl, N)
    rng = np.random.default_rng(B)
    pr = Pair(oracle_mod, N, wl.fanout, wl.obs_bytes, wl.act_bytes, 4096)
    dev = pr.dev
    first = 0
    for _ in range(3):
        m = min(N // 4, 4096)
        pr.insert(wk.transitions(wl, rng, m, first))
        first += m
        for call in range(2):
            o = pr.ora.sample_uniform(B, 9)
            t = {"idx": torch.full((B,), -1, dtype=torch.int32, device=dev), "w": torch.zeros(B, device=dev),
                 "obs": torch.zeros((B, wl.obs_bytes), dtype=torch.uint8, device=dev),
                 "act": torch.zeros((B, wl.act_bytes), dtype=torch.uint8, device=dev), "rew": torch.zeros(B, device=dev),
                 "next_obs": torch.zeros((B, wl.obs_bytes), dtype=torch.uint8, device=dev),
                 "done": torch.zeros(B, dtype=torch.uint8, device=dev)}
            pr.gpu.sample_uniform(B, 9, t["idx"], t["w"], t["obs"], t["act"], t["rew"], t["next_obs"], t["done"])
            torch.cuda.synchronize()
            g = {k: v.cpu().numpy() for k, v in t.items()}
            assert g["idx"].max() < first
            pr.compare_sample(o, g)
        o, g = pr.sample(B, 0.4, 9)            # prioritized and uniform calls share the call counter
    pr.compare_state()
    assert pr.compare_status() == 0
    pr.close()


@pytest.mark.parametrize("wl,N,B", [(wk.ATARI, 2000, 512), (wk.DDPG, 200_000, 256)])
def test_weights_over_many_calls(oracle_mod, wl, N, B):
    # The weights of a call are normalised by the last thread block to have published its raw weights,
    # while the others are still copying rows: 150 calls in a row, every weight checked.
    wl = wk.scaled(wl, N)
    rng = np.random.default_rng(N)
    pr = Pair(oracle_mod, N, wl.fanout, wl.obs_bytes, wl.act_bytes, 512, oracle_store=False)
    dev = pr.dev
    for first in range(0, N, 500):
        m = min(500, N - first)
        b = wk.transitions(wl, rng, m, first)
        pr.insert(dict(rew=b["rew"], done=b["done"], prio=b["prio"]), dev_batch=wk.to_device(b, dev))
    t = {"idx": torch.zeros(B, dtype=torch.int32, device=dev), "w": torch.zeros(B, device=dev),
         "obs": torch.zeros((B, wl.obs_bytes), dtype=torch.uint8, device=dev),
         "act": torch.zeros((B, max(wl.act_bytes, 1)), dtype=torch.uint8, device=dev), "rew": torch.zeros(B, device=dev),
         "next_obs": torch.zeros((B, wl.obs_bytes), dtype=torch.uint8, device=dev),
         "done": torch.zeros(B, dtype=torch.uint8, device=dev)}
    for call in range(150):
        o = pr.ora.sample(B, wl.beta, wl.philox_seed, gather=False)
        t["w"].fill_(-1.0)
        pr.gpu.sample(B, wl.beta, wl.philox_seed, t["idx"], t["w"], t["obs"], t["act"] if wl.act_bytes else None, t["rew"],
                      t["next_obs"], t["done"])
        assert np.array_equal(t["idx"].cpu().numpy(), o["idx"])
        w = t["w"].cpu().numpy()
        np.testing.assert_allclose(w, o["w"], rtol=1e-5, atol=0)
        assert w.max() == np.float32(1.0)
        if call % 10 == 0:
            pr.update(o["idx"], (rng.standard_normal(B) * 2).astype(np.float32), wl.alpha, wl.eps)
    pr.compare_status()
    pr.close()


@pytest.mark.parametrize("wl,N,B", [(wk.CARTPOLE, 3000, 64), (wk.DDPG, 100_000, 1000), (wk.ATARI, 700, 512), (wk.TINY, 9, 32)])
def test_sample_normalised_over_the_buffer(oracle_mod, wl, N, B):
    # Weights divided by the largest weight any stored transition could get (smallest positive priority).
    wl = wk.scaled(wl, N)
    rng = np.random.default_rng(N * 7 + B)
    pr = Pair(oracle_mod, N, wl.fanout, wl.obs_bytes, wl.act_bytes, 1024)
    dev = pr.dev
    filled = 0
    for first in range(0, N - N // 3, 512):                  # a third of the ring stays unwritten
        m = min(512, N - N // 3 - first)
        b = wk.transitions(wl, rng, m, first)
        b["prio"][::7] = 0.0                                    # zero priorities are never the minimum
        pr.insert(b)
        filled += m
    for call in range(4):
        o = pr.ora.sample(B, wl.beta, wl.philox_seed, buffer_norm=True)
        t = {"idx": torch.full((B,), -1, dtype=torch.int32, device=dev), "w": torch.zeros(B, device=dev),
             "obs": torch.zeros((B, wl.obs_bytes), dtype=torch.uint8, device=dev),
             "act": torch.zeros((B, max(wl.act_bytes, 1)), dtype=torch.uint8, device=dev), "rew": torch.zeros(B, device=dev),
             "next_obs": torch.zeros((B, wl.obs_bytes), dtype=torch.uint8, device=dev),
             "done": torch.zeros(B, dtype=torch.uint8, device=dev)}
        pr.gpu.sample_buffer_norm(B, wl.beta, wl.philox_seed, t["idx"], t["w"], t["obs"], t["act"] if wl.act_bytes else None,
                                  t["rew"], t["next_obs"], t["done"])
        torch.cuda.synchronize()
        g = {k: v.cpu().numpy() for k, v in t.items()}
        assert np.array_equal(o["idx"], g["idx"])
        np.testing.assert_allclose(g["w"], o["w"], rtol=1e-5, atol=0)
        assert g["w"].max() <= 1.0
        assert np.array_equal(np.ascontiguousarray(o["obs"]).view(np.uint8).reshape(-1), g["obs"].reshape(-1))
        pr.compare_state()
        idx, td = wk.update_batch(wl, rng, o["idx"])
        pr.update(idx, td, wl.alpha, wl.eps)                    # the minimum moves between calls
        o2, g2 = pr.sample(B, wl.beta, wl.philox_seed)          # and the batch-normalised call still agrees
    pr.compare_status()
    pr.close()


@pytest.mark.parametrize("wl,N,B,n_sub", [(wk.CARTPOLE, 3000, 64, 2), (wk.DDPG, 100_000, 1000, 4), (wk.DDPG, 5000, 3, 3),
                                          (wk.ATARI, 700, 512, 4), (wk.ATARI, 700, 37, 3)])
def test_sample_streamed_as_sub_batches(oracle_mod, wl, N, B, n_sub):
    # Sub-batch streaming (Section IV-C): the same sample, issued as launches on several streams.  A
    # consumer stream that waits for sub-batch i alone must find that sub-batch's indices and rows.
    wl = wk.scaled(wl, N)
    rng = np.random.default_rng(N + B)
    pr = Pair(oracle_mod, N, wl.fanout, wl.obs_bytes, wl.act_bytes, 1024)
    dev = pr.dev
    for first in range(0, N, 512):
        pr.insert(wk.transitions(wl, rng, min(512, N - first), first))
    consumer = torch.cuda.Stream(dev)
    for call in range(3):
        o = pr.ora.sample(B, wl.beta, wl.philox_seed)
        t = {"idx": torch.full((B,), -1, dtype=torch.int32, device=dev), "w": torch.zeros(B, device=dev),
             "obs": torch.zeros((B, wl.obs_bytes), dtype=torch.uint8, device=dev),
             "act": torch.zeros((B, max(wl.act_bytes, 1)), dtype=torch.uint8, device=dev), "rew": torch.zeros(B, device=dev),
             "next_obs": torch.zeros((B, wl.obs_bytes), dtype=torch.uint8, device=dev),
             "done": torch.zeros(B, dtype=torch.uint8, device=dev)}
        torch.cuda.synchronize()
        pr.gpu.sample_streamed(B, wl.beta, wl.philox_seed, n_sub, t["idx"], t["w"], t["obs"],
                               t["act"] if wl.act_bytes else None, t["rew"], t["next_obs"], t["done"])
        early = []
        with torch.cuda.stream(consumer):
            for i in range(n_sub):                  # each sub-batch is copied out as soon as it alone is ready
                pr.gpu.wait_sub_batch(i, consumer)
                k0, k1 = i * B // n_sub, (i + 1) * B // n_sub
                early.append((k0, k1, t["idx"][k0:k1].clone(), t["obs"][k0:k1].clone(), t["done"][k0:k1].clone()))
        torch.cuda.synchronize()
        for k0, k1, idx_i, obs_i, done_i in early:
            assert np.array_equal(idx_i.cpu().numpy(), o["idx"][k0:k1])
            assert np.array_equal(obs_i.cpu().numpy().reshape(-1), np.ascontiguousarray(o["obs"][k0:k1]).view(np.uint8).reshape(-1))
            assert np.array_equal(done_i.cpu().numpy(), o["done"][k0:k1])
        g = {k: v.cpu().numpy() for k, v in t.items()}
        if not wl.act_bytes:
            g["act"] = o["act"]
        pr.compare_sample(o, g)                    # the whole batch, weights included, after the join
        pr.compare_state()
        idx, td = wk.update_batch(wl, rng, o["idx"])
        pr.update(idx, td, wl.alpha, wl.eps)
    with pytest.raises(Exception):
        pr.gpu.wait_sub_batch(n_sub, consumer)
    pr.compare_status()
    pr.close()


@pytest.mark.parametrize("K,N,B", [(2, 300, 64), (4, 5000, 700), (16, 70_000, 256), (32, 900, 512), (8, 20_000, 3000),
                                   (16, 50_000, 9000)])
def test_delta_update(oracle_mod, K, N, B):
    # Section V-A's index + change form: repeats accumulate in batch order, refused sums leave the leaf alone.
    rng = np.random.default_rng(K * 1000 + B)
    pr = Pair(oracle_mod, N, K, 8, 4, max(B, 1024))
    for first in range(0, N, 1024):
        m = min(1024, N - first)
        b = raw_fields(rng, m, 8, 4)
        b["prio"] = np.exp(rng.standard_normal(m)).astype(np.float32)
        pr.insert(b)
    for step in range(4):
        idx = rng.integers(0, N, size=B).astype(np.int32)
        idx[: B // 4] = idx[B // 4: 2 * (B // 4)]                      # many repeats, far apart in the batch
        delta = (rng.standard_normal(B) * (0.3 if step < 3 else 3.0)).astype(np.float32)    # last step: many sums go negative
        if step == 1:
            idx[3], idx[5] = -1, N
            delta[7], delta[9] = np.nan, np.inf
            big = np.float32(2 ** 24)
            idx[11], idx[12], delta[11], delta[12] = 17, 17, big, -big   # rounding-order probe
        if step == 2:
            idx = np.sort(idx)                                            # already in order: no sort in the kernel
        pr.update_delta(idx, delta)
        pr.compare_tree()
        pr.compare_state()
        pr.compare_status()
    pr.close()


@pytest.mark.parametrize("seed", range(12))
def test_random_call_sequences(oracle_mod, seed):
    # Random geometry and a random sequence of every call, compared with the oracle after each one.
    rng = np.random.default_rng(9000 + seed)
    K = int(rng.choice([2, 4, 8, 16, 32]))
    N = int(rng.choice([1, 3, 17, 256, 1000, 4099, 20_000]))
    obs_bytes = int(rng.choice([0, 1, 6, 16, 68, 100, 8192, 8208]))
    act_bytes = int(rng.choice([0, 4, 24]))
    maxb = 700
    pr = Pair(oracle_mod, N, K, obs_bytes, act_bytes, maxb)
    dev = pr.dev
    inserted_since, last_idx = 0, None

    def new_batch(n, with_prio=True):
        b = raw_fields(rng, n, obs_bytes, act_bytes)
        b["prio"] = np.exp(rng.standard_normal(n)).astype(np.float32) if with_prio else None
        return b

    for step in range(40):
        op = rng.choice(["insert", "insert_default", "sample", "uniform", "update", "raw", "after", "fused", "get"],
                        p=[0.2, 0.05, 0.2, 0.05, 0.15, 0.05, 0.1, 0.15, 0.05])
        fill = pr.ora.info()[0]
        n = int(rng.integers(1, min(N, maxb) + 1))
        B = int(rng.integers(1, maxb + 1))
        some_idx = (rng.integers(-1, max(fill, 1) + 1, size=B)).astype(np.int32)     # a few out of range
        td = (rng.standard_normal(B) * 3).astype(np.float32)
        if op == "insert":
            pr.insert(new_batch(n))
            inserted_since += n
        elif op == "insert_default":
            b = new_batch(n, with_prio=False)
            assert pr.ora.insert(b["obs"], b["act"], b["rew"], b["next_obs"], b["done"], None, n=n) == 0
            d = {k: torch.from_numpy(v).to(dev) for k, v in b.items() if v is not None}
            pr.gpu.insert(d["obs"], d["act"], d["rew"], d["next_obs"], d["done"], None, n=n)
            inserted_since += n
        elif op == "sample":
            o, g = pr.sample(B, float(rng.choice([0.0, 0.4, 1.0])), seed)
            if o["idx"][0] >= 0:
                last_idx, inserted_since = o["idx"].copy(), 0
        elif op == "uniform":
            o = pr.ora.sample_uniform(B, seed)
            t = {"idx": torch.full((B,), -1, dtype=torch.int32, device=dev), "w": torch.zeros(B, device=dev),
                 "obs": torch.zeros((B, obs_bytes), dtype=torch.uint8, device=dev),
                 "act": torch.zeros((B, act_bytes), dtype=torch.uint8, device=dev), "rew": torch.zeros(B, device=dev),
                 "next_obs": torch.zeros((B, obs_bytes), dtype=torch.uint8, device=dev),
                 "done": torch.zeros(B, dtype=torch.uint8, device=dev)}
            pr.gpu.sample_uniform(B, seed, t["idx"], t["w"], t["obs"], t["act"], t["rew"], t["next_obs"], t["done"])
            torch.cuda.synchronize()
            pr.compare_sample(o, {k: v.cpu().numpy() for k, v in t.items()})
        elif op == "update":
            pr.update(some_idx, td, 0.6, 1e-6)
        elif op == "raw":
            pr.update_priorities(some_idx, np.abs(td))
        elif op == "after" and last_idx is not None:
            m = min(inserted_since, N)
            pr.update_after_insert(last_idx, td[:len(last_idx)] if len(last_idx) <= B else np.resize(td, len(last_idx)),
                                   0.6, 1e-6, m)
        elif op == "fused":
            pr.update_insert(some_idx, td, 0.6, 1e-6, new_batch(n))
            inserted_since += n
        elif op == "get":
            pr.compare_priorities(some_idx)
        pr.compare_tree()
        pr.compare_state()
        pr.compare_status()
    pr.compare_rows(np.arange(min(pr.ora.info()[0], N), dtype=np.int32)[:2000])
    pr.close()


def test_update_is_deterministic(oracle_mod):
    # The same batch with many duplicates, replayed: identical tree bytes every time.
    rng = np.random.default_rng(13)
    N = 50_000
    pr = Pair(oracle_mod, N, 8, 0, 0, 4096)
    pr.insert(dict(prio=rng.uniform(0.1, 1, 4096).astype(np.float32)))
    for _ in range(12):
        pr.insert(dict(prio=rng.uniform(0.1, 1, 4096).astype(np.float32)))
    idx = rng.integers(0, 300, size=4096).astype(np.int32)
    td = rng.standard_normal(4096).astype(np.float32)
    pr.update(idx, td, 0.6, 1e-6)
    ref = [pr.gpu.read_level(l).copy() for l in range(pr.gpu.depth + 1)]
    pr.compare_tree()
    for _ in range(20):
        pr.gpu.update(torch.from_numpy(idx).to(pr.dev), torch.from_numpy(td).to(pr.dev), 0.6, 1e-6)
        for l, r in enumerate(ref):
            assert np.array_equal(pr.gpu.read_level(l).view(np.uint32), r.view(np.uint32))
    pr.close()


def test_argument_errors_leave_state_untouched(oracle_mod):
    from paper_2311_09445_b200 import PearlError
    pr = Pair(oracle_mod, 64, 4, 16, 4, 32)
    rng = np.random.default_rng(1)
    b = raw_fields(rng, 32, 16, 4)
    b["prio"] = rng.uniform(0.5, 1, 32).astype(np.float32)
    pr.insert(b)
    dev = pr.dev
    idx = torch.zeros(64, dtype=torch.int32, device=dev)
    td = torch.zeros(64, dtype=torch.float32, device=dev)
    before = [pr.gpu.read_level(l).copy() for l in range(pr.gpu.depth + 1)]
    with pytest.raises(PearlError) as e:
        pr.gpu.sample(33, 0.4, 0, idx)                       # B > max_batch
    assert e.value.code == -3
    with pytest.raises(PearlError) as e:
        pr.gpu.sample(0, 0.4, 0, idx)
    assert e.value.code == -3
    with pytest.raises(PearlError) as e:
        pr.gpu.sample(8, float("nan"), 0, idx)
    assert e.value.code == -7
    with pytest.raises(PearlError) as e:
        pr.gpu.update(idx[:8], td[:8], -0.5, 1e-6)
    assert e.value.code == -7
    with pytest.raises(PearlError) as e:
        pr.gpu.sample(8, 0.4, 0, idx, obs=torch.zeros(8 * 16 + 16, dtype=torch.uint8, device=dev)[4:4 + 8 * 16])
    assert e.value.code == -5                                # misaligned 16-byte rows
    with pytest.raises(PearlError) as e:
        pr.gpu.wait_sub_batch(0, torch.cuda.current_stream(dev))      # no streamed call yet
    assert e.value.code == -7
    for bad_subs in (0, 5, 9):                                        # 1..4 sub-batches, and not more than B
        with pytest.raises(PearlError) as e:
            pr.gpu.sample_streamed(8 if bad_subs != 9 else 3, 0.4, 0, bad_subs if bad_subs != 9 else 4, idx)
        assert e.value.code == -7
    with pytest.raises(PearlError) as e:
        pr.gpu.sample_buffer_norm(8, -1.0, 0, idx)
    assert e.value.code == -7
    with pytest.raises(PearlError) as e:
        pr.gpu.update_delta(idx[:40], td[:40])                        # B > max_batch
    assert e.value.code == -3
    big = Pair(oracle_mod, 16, 2, 0, 0, 32)
    with pytest.raises(PearlError) as e:
        big.gpu.insert(None, None, None, None, None, torch.ones(17, device=dev))
    assert e.value.code == -4                                # n > capacity
    big.close()
    for l, r in enumerate(before):
        assert np.array_equal(pr.gpu.read_level(l), r)
    pr.compare_state()
    assert pr.gpu.kernel_launches() == 1
    pr.close()
