"""Pins for the oracle's frame-deduplicated layout: what it rebuilds is what the plain layout stores."""
import numpy as np
import pytest

from paper_2311_09445_b200 import workloads as wk


def feed(o_frames, o_plain, b):
    assert o_frames.insert(b["frame"], b["act"], b["rew"], None, b["done"], b["prio"]) == 0
    if o_plain is not None:
        assert o_plain.insert(b["obs"], b["act"], b["rew"], b["next_obs"], b["done"], b["prio"]) == 0


@pytest.mark.parametrize("S,F,N,K", [(4, 48, 300, 4), (1, 16, 64, 2), (2, 100, 1000, 16), (4, 7056, 200, 32), (3, 5, 50, 8)])
def test_rebuilt_stacks_equal_the_stored_ones(oracle_mod, S, F, N, K):
    # The same single-actor trajectory goes into a buffer that stores whole stacks and into one that stores one
    # frame per slot.  Before the ring wraps the two hold the same tree (a marker's priority is 0 in both), so
    # they sample the same indices -- and every gathered stack must be byte-equal.  After it has wrapped,
    # every slot that keeps a priority in the frame layout must still rebuild to the plain layout's row.
    rng = np.random.default_rng(S * 1000 + F)
    traj = wk.FrameTrajectory(rng, F, S, episode_steps=(1, 12))
    fr = oracle_mod.OraclePRB(N, K, S * F, 4, frame_stack=S)
    pl = oracle_mod.OraclePRB(N, K, S * F, 4)
    inserted = 0
    while inserted + 40 <= N - S:
        feed(fr, pl, traj.next(40))
        inserted += 40
        for l in range(fr.depth + 1):
            assert np.array_equal(fr.read_level(l).view(np.uint32), pl.read_level(l).view(np.uint32))
        a, b = fr.sample(32, 0.4, 7), pl.sample(32, 0.4, 7)
        assert np.array_equal(a["idx"], b["idx"]) and np.array_equal(a["w"], b["w"])
        for f in ("obs", "next_obs", "act", "rew", "done"):
            assert np.array_equal(a[f], b[f]), f
        assert not (a["done"] & 2).any()                        # a marker is never sampled
    for _ in range(3 * N // 40):                                # wrap the ring a few times
        feed(fr, pl, traj.next(40))
    leaves = fr.read_level(fr.depth)[:N]
    plain_leaves = pl.read_level(pl.depth)[:N]
    cursor = fr.info()[1]
    behind = (np.arange(N) - cursor) % N < S                    # the slots that follow the cursor lost their history
    assert np.all(leaves[behind] == 0) and np.array_equal(leaves[~behind], plain_leaves[~behind])
    keep = np.nonzero(leaves > 0)[0].astype(np.int32)
    ra, rb = fr.read_rows(keep), pl.read_rows(keep)
    for f in ("obs", "next_obs", "act", "rew", "done"):
        assert np.array_equal(ra[f], rb[f]), f
    fr.rebuild()                                                # and the tree is the sum tree of those leaves
    before = [fr.read_level(l).copy() for l in range(fr.depth + 1)]
    fr.rebuild()
    for l, x in enumerate(before):
        assert np.array_equal(x, fr.read_level(l))
    a = fr.sample(64, 0.4, 1)
    assert np.all(leaves[a["idx"]] > 0) and not (a["done"] & 2).any()


def test_hand_worked_stacks(oracle_mod):
    # stack 3, one-byte frames: marker A, steps b c d (d ends the episode), marker E, step f
    o = oracle_mod.OraclePRB(16, 2, 3, 0, frame_stack=3)
    frames = np.array([[10], [11], [12], [13], [20], [21]], np.uint8)
    done = np.array([2, 0, 0, 1, 2, 0], np.uint8)
    prio = np.ones(6, np.float32)
    assert o.insert(frames, None, np.zeros(6, np.float32), None, done, prio) == 0
    assert o.read_level(o.depth)[:7].tolist() == [0, 1, 1, 1, 0, 1, 0]
    r = o.read_rows(np.array([1, 2, 3, 5], np.int32))
    assert r["obs"].tolist() == [[10, 10, 10], [10, 10, 11], [10, 11, 12], [20, 20, 20]]
    assert r["next_obs"].tolist() == [[10, 10, 11], [10, 11, 12], [11, 12, 13], [20, 20, 21]]


def test_updates_skip_slots_without_history(oracle_mod):
    S, F, N = 4, 8, 64
    rng = np.random.default_rng(3)
    traj = wk.FrameTrajectory(rng, F, S)
    o = oracle_mod.OraclePRB(N, 4, S * F, 4, frame_stack=S)
    for _ in range(3):
        feed(o, None, traj.next(32))
    cursor = o.info()[1]
    idx = np.array([(cursor + 1) % N, (cursor + S) % N], np.int32)
    before = o.read_level(o.depth).copy()
    assert o.update_priorities(idx, np.array([5.0, 6.0], np.float32)) == 0
    after = o.read_level(o.depth)
    assert o.status() == oracle_mod.ST_STALE
    assert after[idx[0]] == before[idx[0]] == 0 and after[idx[1]] == 6.0
    assert o.sample_uniform(4, 0)["rc"] != 0                    # uniform replay is not offered on this layout
    with pytest.raises(ValueError):
        oracle_mod.OraclePRB(4, 2, 16, 0, frame_stack=4)        # capacity must exceed the stack
