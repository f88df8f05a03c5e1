"""Pins for the oracle's sum tree: hand-worked cases, the plain definitions, invariants."""
import numpy as np
import pytest

from conftest import golden_lines

P8 = np.array([3, 1, 4, 1, 5, 9, 2, 6], dtype=np.float32)
FANOUTS = [2, 4, 8, 16, 32]


def make(oracle_mod, prio, K, capacity=None):
    prio = np.asarray(prio, dtype=np.float32)
    o = oracle_mod.OraclePRB(capacity or len(prio), K, 0, 0)
    assert o.insert(None, None, None, None, None, prio) == 0
    return o


def flat_scan(prio, x):
    """Eq. 1 read with half-open intervals: the first i with x < p_0 + ... + p_i."""
    s = 0.0
    for i, p in enumerate(prio):
        s += float(p)
        if x < s:
            return i
    return None


def check_invariant(o):
    """Every internal node is the left-to-right binary32 sum of its children; padding is zero."""
    K = o.fanout
    for l in range(o.depth):
        parent = o.read_level(l)
        child = o.read_level(l + 1).reshape(-1, K)
        acc = child[:, 0].copy()
        for j in range(1, K):
            acc = (acc + child[:, j]).astype(np.float32)
        n = o.level_nodes(l)
        assert np.array_equal(parent[:n].view(np.uint32), acc[:n].view(np.uint32)), "level %d" % l
        assert np.all(parent[n:] == 0)
    assert np.all(o.read_level(o.depth)[o.capacity:] == 0)


def test_hand_worked_levels(oracle_mod):
    rows = golden_lines("eight_leaf_levels.txt")
    for K in (2, 4, 8):
        o = make(oracle_mod, P8, K)
        for case, k, level, *vals in rows:
            if case == "init" and int(k) == K:
                assert o.read_level(int(level)).tolist() == [float(v) for v in vals]
        assert o.update_priorities([5], [2.0]) == 0
        for case, k, level, *vals in rows:
            if case == "upd" and int(k) == K:
                assert o.read_level(int(level)).tolist() == [float(v) for v in vals]


def test_hand_worked_descents(oracle_mod):
    trees = {K: make(oracle_mod, P8, K) for K in (2, 4, 8)}
    for k, x, leaf in golden_lines("eight_leaf_descents.txt"):
        i, p = trees[int(k)].descend(float(x))
        assert i == int(leaf), (k, x)
        assert p == P8[int(leaf)]
    for o in trees.values():
        assert o.status() == 0


def test_paper_literal_reading_differs_only_on_boundaries(oracle_mod):
    # Eq. 1 as printed (prefix sum >= x) picks leaf 5 at x = 23; the half-open reading picks 6.
    o = make(oracle_mod, P8, 2)
    assert o.descend(23.0)[0] == 6
    prefix = np.cumsum(P8.astype(np.float64))
    literal = int(np.argmax(prefix >= 23.0))
    assert literal == 5
    for x in np.linspace(0.01, 30.99, 777):
        if x not in prefix:
            assert o.descend(x)[0] == int(np.argmax(prefix >= x))


@pytest.mark.parametrize("K", FANOUTS)
@pytest.mark.parametrize("N", [1, 2, 7, 8, 33, 100, 257, 1000])
def test_flat_scan_equivalence_on_exact_sums(oracle_mod, K, N):
    # Integer priorities (with zeros) sum exactly in binary32, so the tree descent must
    # agree with the linear scan of Eq. 1 for every fanout and for ragged capacities.
    rng = np.random.default_rng(100 * K + N)
    prio = rng.integers(0, 9, size=N).astype(np.float32)
    prio[rng.integers(0, N)] = 5.0
    o = make(oracle_mod, prio, K)
    check_invariant(o)
    total = float(prio.sum())
    assert float(o.total()) == total
    prefix = np.cumsum(prio.astype(np.float64))
    xs = set(np.linspace(0, total, 97, endpoint=False).tolist())
    for s in prefix[:-1]:
        if s < total:
            xs.update([s, np.nextafter(s, 0.0), np.nextafter(s, np.inf)])
    xs.add(0.0)
    xs.add(np.nextafter(total, 0.0))
    for x in xs:
        if 0 <= x < total:
            i, p = o.descend(x)
            assert i == flat_scan(prio, x), (K, N, x)
            assert p == prio[i] and p > 0
    assert o.status() == 0


def test_leaf_does_not_depend_on_fanout(oracle_mod):
    rng = np.random.default_rng(5)
    prio = (rng.integers(1, 64, size=600) / 8.0).astype(np.float32)     # dyadic: exact sums
    trees = [make(oracle_mod, prio, K) for K in FANOUTS]
    total = float(prio.astype(np.float64).sum())
    for x in rng.uniform(0, total, size=400):
        leaves = {o.descend(x)[0] for o in trees}
        assert len(leaves) == 1


def test_exact_measure_on_integer_grid(oracle_mod):
    # With integer priorities, targets x = 0.5, 1.5, ... hit leaf i exactly p_i times:
    # P(i) = p_i / sum_k p_k by construction.
    prio = np.array([2, 0, 3, 1, 0, 0, 4, 1, 1, 5, 0, 2, 7], dtype=np.float32)
    for K in FANOUTS:
        o = make(oracle_mod, prio, K)
        counts = np.zeros(len(prio), dtype=np.int64)
        for t in range(int(prio.sum())):
            counts[o.descend(t + 0.5)[0]] += 1
        assert counts.tolist() == prio.astype(np.int64).tolist()


@pytest.mark.parametrize("K", FANOUTS)
def test_incremental_update_equals_rebuild(oracle_mod, K):
    rng = np.random.default_rng(K)
    N = 777
    prio = np.abs(rng.normal(size=N)).astype(np.float32) ** np.float32(0.6)
    o = make(oracle_mod, prio, K)
    leaves = prio.copy()
    for step in range(25):
        B = int(rng.integers(1, 80))
        idx = rng.integers(0, N, size=B).astype(np.int32)
        idx[B // 2:] = idx[: B - B // 2]            # plenty of duplicates
        newp = np.abs(rng.normal(size=B)).astype(np.float32)
        assert o.update_priorities(idx, newp) == 0
        for i, p in zip(idx, newp):                 # batch order: last writer wins
            leaves[i] = p
        assert np.array_equal(o.read_level(o.depth)[:N], leaves)
        check_invariant(o)
        fresh = make(oracle_mod, leaves, K)         # built from scratch by one insert
        for l in range(o.depth + 1):
            assert np.array_equal(o.read_level(l).view(np.uint32), fresh.read_level(l).view(np.uint32))
        o.rebuild()                                  # the definition applied to every node
        for l in range(o.depth + 1):
            assert np.array_equal(o.read_level(l).view(np.uint32), fresh.read_level(l).view(np.uint32))


def test_root_close_to_binary64_sum(oracle_mod):
    rng = np.random.default_rng(9)
    prio = np.exp(2 * rng.normal(size=5000)).astype(np.float32)
    for K in FANOUTS:
        o = make(oracle_mod, prio, K)
        exact = prio.astype(np.float64).sum()
        assert abs(float(o.total()) - exact) <= (o.depth * K) * 2.0**-24 * exact


def test_last_writer_wins_and_invalid_entries(oracle_mod):
    o = make(oracle_mod, P8, 2)
    assert o.update_priorities([5, 5], [7.0, 2.0]) == 0
    assert o.read_level(3)[5] == 2.0 and o.total() == 24.0
    before = [o.read_level(l).copy() for l in range(4)]
    assert o.update_priorities([-1, 8, 3, 2, 1], [1.0, 1.0, np.nan, -1.0, np.inf]) == 0
    assert o.status() == (oracle_mod.ST_BAD_INDEX | oracle_mod.ST_BAD_PRIORITY)
    for l in range(4):
        assert np.array_equal(o.read_level(l), before[l])
    assert o.update([0], [np.nan], 0.6, 1e-6) == 0
    assert o.status() == oracle_mod.ST_BAD_PRIORITY
    assert o.update([0], [1.0], -1.0, 1e-6) != 0       # bad alpha is a host error


def test_update_applies_transform(oracle_mod):
    o = make(oracle_mod, P8, 4)
    td = np.array([0.5, -2.0, 3.0], dtype=np.float32)
    assert o.update([1, 2, 7], td, 0.6, 1e-6) == 0
    leaves = o.read_level(o.depth)
    for i, d in zip([1, 2, 7], td):
        assert leaves[i] == oracle_mod.priority_pow(d, 1e-6, 0.6)
    check_invariant(o)


def test_ring_insert(oracle_mod):
    o = oracle_mod.OraclePRB(8, 2, 4, 2)

    def batch(first, n):
        ids = np.arange(first, first + n)
        return dict(obs=(ids[:, None] * 4 + np.arange(4)).astype(np.uint8),
                    act=(ids[:, None] * 2 + np.arange(2)).astype(np.uint8),
                    rew=ids.astype(np.float32), next_obs=(200 - ids[:, None] - np.arange(4)).astype(np.uint8),
                    done=(ids % 2).astype(np.uint8), prio=(ids + 1).astype(np.float32))

    assert o.insert(**batch(0, 6)) == 0
    assert o.info()[:2] == (6, 6)
    assert o.total() == 21.0
    assert o.insert(**batch(6, 5)) == 0                 # wraps: slots 6 7 0 1 2
    assert o.info()[:2] == (8, 3)
    assert o.read_level(3).tolist() == [9, 10, 11, 4, 5, 6, 7, 8]
    rows = o.read_rows(np.arange(8))
    assert rows["rew"].tolist() == [8, 9, 10, 3, 4, 5, 6, 7]
    assert rows["obs"][0].tolist() == [32, 33, 34, 35]
    assert rows["next_obs"][3].tolist() == [197, 196, 195, 194]
    assert rows["act"][7].tolist() == [14, 15]
    assert rows["done"].tolist() == [0, 1, 0, 1, 0, 1, 0, 1]
    check_invariant(o)
    big = batch(0, 9)
    assert o.insert(**big) != 0                          # n > capacity
    bad = batch(20, 2)
    bad["prio"] = np.array([np.nan, 3.0], dtype=np.float32)
    assert o.insert(**bad) == 0                          # stored, but never sampled
    assert o.status() == oracle_mod.ST_BAD_PRIORITY
    assert o.read_level(3)[3] == 0.0 and o.read_level(3)[4] == 3.0


def test_planted_mistake_is_caught(oracle_mod):
    # A wrong internal node (as a dropped term would leave) must trip the invariant check
    # and the rebuild comparison: the pins above are sensitive to it.
    o = make(oracle_mod, P8, 2)
    o.poke_level(2, 2, [13.0])
    with pytest.raises(AssertionError):
        check_invariant(o)
    assert o.descend(9.0 + 13.5)[0] != flat_scan(P8, 9.0 + 13.5)
    o.rebuild()
    check_invariant(o)


def test_update_after_insert_equals_update_then_insert(oracle_mod):
    # Collision-free scheduling (Section IV-C): sample, insert, then an update that skips the slots
    # written since the sample must leave the same tree as update-then-insert on the same inputs.
    rng = np.random.default_rng(31)
    N, n, B = 200, 37, 64
    for K in (2, 16):
        a = oracle_mod.OraclePRB(N, K, 0, 0)
        b = oracle_mod.OraclePRB(N, K, 0, 0)
        first = rng.uniform(0.1, 1, 150).astype(np.float32)
        for o in (a, b):
            o.insert(None, None, None, None, None, first)
        saw_stale = False
        for step in range(30):
            idx = a.sample(B, 0.4, 7, gather=False)["idx"]
            assert np.array_equal(idx, b.sample(B, 0.4, 7, gather=False)["idx"])
            td = rng.standard_normal(B).astype(np.float32)
            newp = rng.uniform(0.1, 1, n).astype(np.float32)
            a.insert(None, None, None, None, None, newp)
            assert a.update_after_insert(idx, td, 0.6, 1e-6, n) == 0
            assert b.update(idx, td, 0.6, 1e-6) == 0
            b.insert(None, None, None, None, None, newp)
            sa, sb = a.status(), b.status()
            saw_stale |= bool(sa & oracle_mod.ST_STALE)
            assert (sa & ~oracle_mod.ST_STALE) == sb
            for l in range(a.depth + 1):
                assert np.array_equal(a.read_level(l).view(np.uint32), b.read_level(l).view(np.uint32))
            check_invariant(a)
        assert saw_stale                       # the ring wrapped over sampled slots at least once
    # inserted = 0 is the plain update; a stale index is exactly one of the last `inserted` slots
    o = make(oracle_mod, P8, 2)
    o.insert(None, None, None, None, None, np.array([7, 7, 7], np.float32))       # slots 0 1 2, cursor 3
    assert o.update_after_insert([2, 3, 0, 7], [1.0, 1.0, 1.0, 1.0], 1.0, 0.0, 2) == 0
    assert o.status() == oracle_mod.ST_STALE
    assert o.read_level(3).tolist() == [1, 7, 7, 1, 5, 9, 2, 1]                      # 1 and 2 were skipped
    assert o.get_priorities([0, 2, 7, 8, -1]).tolist() == [1, 7, 1, 0, 0]
    assert o.status() == oracle_mod.ST_BAD_INDEX


def test_default_insert_priority_is_running_maximum(oracle_mod):
    # Schaul et al.: a new transition enters with the largest priority seen so far (1 before any).
    o = oracle_mod.OraclePRB(16, 4, 0, 0)
    assert o.max_priority() == 0
    assert o.insert(None, None, None, None, None, None, n=2) == 0
    assert o.read_level(2)[:2].tolist() == [1.0, 1.0] and o.max_priority() == 1.0
    o.insert(None, None, None, None, None, np.array([3, 0.5, 4], np.float32))
    assert o.max_priority() == 4.0
    o.insert(None, None, None, None, None, None, n=2)
    assert o.read_level(2)[:7].tolist() == [1, 1, 3, 0.5, 4, 4, 4]
    o.update([0, 0], [100.0, 2.0], 0.5, 0.0)                 # 10 loses the duplicate race but was written
    assert o.max_priority() == 10.0 and o.read_level(2)[0] == np.float32(2.0) ** np.float32(0.5)
    o.update_priorities([1, 99], [50.0, 70.0])               # an invalid index does not count
    assert o.max_priority() == 50.0
    o.update([2], [np.nan], 0.5, 0.0)
    o.insert(None, None, None, None, None, np.array([np.inf], np.float32))
    assert o.max_priority() == 50.0 and o.status() == (oracle_mod.ST_BAD_INDEX | oracle_mod.ST_BAD_PRIORITY)
    o.insert(None, None, None, None, None, None, n=1)
    assert o.read_level(2)[8] == 50.0
    check_invariant(o)


@pytest.mark.parametrize("K", FANOUTS)
def test_delta_update_with_exact_arithmetic_equals_setting_the_priority(oracle_mod, K):
    # Section V-A gives the update as index + change.  On small integers every binary32 operation is
    # exact, so adding new - old must leave the tree that writing `new` leaves, whatever the order.
    rng = np.random.default_rng(K)
    N = 777
    old = rng.integers(0, 50, size=N).astype(np.float32)
    a, b = make(oracle_mod, old, K), make(oracle_mod, old, K)
    idx = rng.permutation(N)[:300].astype(np.int32)
    new = rng.integers(0, 50, size=300).astype(np.float32)
    assert a.update_delta(idx, new - old[idx]) == 0
    assert b.update_priorities(idx, new) == 0
    for l in range(a.depth + 1):
        assert np.array_equal(a.read_level(l).view(np.uint32), b.read_level(l).view(np.uint32))
    check_invariant(a)
    assert a.status() == 0


def test_delta_update_accumulates_repeats_in_batch_order(oracle_mod):
    # 2^24 + 1 + 1 in binary32: each addition of 1 is lost to rounding, one addition of 2 is not --
    # so the result tells whether the repeats were added one by one in batch order.
    big = np.float32(2 ** 24)
    o = make(oracle_mod, [big, 1, 1, 1], 2)
    assert o.update_delta([0, 0], [1.0, 1.0]) == 0
    assert o.read_level(2)[0] == big
    assert o.update_delta([0], [2.0]) == 0
    assert o.read_level(2)[0] == big + np.float32(2)
    # order matters: (1 + 2^24) - 2^24 = 0 but (1 - 2^24) is refused (negative), then 1 + 2^24 = 2^24
    o2 = make(oracle_mod, [1, 1, 1, 1], 2)
    assert o2.update_delta([1, 1], [big, -big]) == 0
    assert o2.read_level(2)[1] == 0.0 and o2.status() == 0
    o3 = make(oracle_mod, [1, 1, 1, 1], 2)
    assert o3.update_delta([1, 1], [-big, big]) == 0
    assert o3.read_level(2)[1] == big and o3.status() == oracle_mod.ST_BAD_PRIORITY
    check_invariant(o3)
    assert o3.max_priority() == big


def test_delta_update_skips_invalid_entries(oracle_mod):
    o = make(oracle_mod, P8, 4)
    before = [o.read_level(l).copy() for l in range(o.depth + 1)]
    assert o.update_delta([-1, 8, 0, 1, 2], [1.0, 1.0, np.nan, np.inf, -5.0]) == 0
    assert o.status() == (oracle_mod.ST_BAD_INDEX | oracle_mod.ST_BAD_PRIORITY)
    for l in range(o.depth + 1):
        assert np.array_equal(o.read_level(l), before[l])
    assert o.update_delta([2], [-4.0]) == 0             # exactly to zero is allowed
    assert o.read_level(o.depth)[2] == 0.0 and o.total() == 27.0
