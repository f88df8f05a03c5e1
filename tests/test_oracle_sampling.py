"""Pins for the oracle's stratified sampling, importance-sampling weights and gather."""
import numpy as np
import pytest
from scipy import stats

from conftest import golden_lines

P8 = np.array([3, 1, 4, 1, 5, 9, 2, 6], dtype=np.float32)


def make(oracle_mod, prio, K, obs_bytes=0, act_bytes=0, **fields):
    prio = np.asarray(prio, dtype=np.float32)
    o = oracle_mod.OraclePRB(len(prio), K, obs_bytes, act_bytes)
    assert o.insert(fields.get("obs"), fields.get("act"), fields.get("rew"), fields.get("next_obs"),
                    fields.get("done"), prio) == 0
    return o


def test_hand_worked_stratified_example(oracle_mod):
    g = {row[0]: [float(v) for v in row[1:]] for row in golden_lines("stratified_example.txt")}
    for K in (2, 4, 8):
        o = make(oracle_mod, P8, K)
        leaves = [o.descend(x)[0] for x in g["targets"]]
        assert leaves == [int(v) for v in g["leaves"]]
    # the same batch through sample(): find a draw and check the closed form instead of u = 0.5
    o = make(oracle_mod, P8, 2)
    out = o.sample(4, 0.4, 0)
    p = P8[out["idx"]].astype(np.float64)
    assert np.allclose(out["w"], (p.min() / p) ** 0.4, rtol=1e-6)
    # weights of the worked batch
    p = P8[[int(v) for v in g["leaves"]]].astype(np.float64)
    w = (8 * p / 31.0) ** -0.4
    assert np.allclose(w / w.max(), g["weights"], rtol=1e-9)


def test_targets_are_stratified(oracle_mod):
    o = make(oracle_mod, P8, 2)
    for B in (1, 3, 4, 7, 64):
        for call in (0, 1, 17):
            x = o.targets(B, 5, call)
            seg = 31.0 / B
            u = np.array([oracle_mod.stratum_uniform(5, call, k) for k in range(B)])
            assert np.all(x >= np.arange(B) * seg) and np.all(x < 31.0)
            assert np.all(x <= (np.arange(B) + 1) * seg)
            assert np.allclose(x, (np.arange(B) + u) * seg, rtol=1e-15)
    assert not np.array_equal(o.targets(4, 5, 0), o.targets(4, 5, 1))     # fresh draws per call
    assert not np.array_equal(o.targets(4, 5, 0), o.targets(4, 6, 0))     # and per seed


def test_sample_uses_call_counter_and_targets(oracle_mod):
    rng = np.random.default_rng(1)
    prio = rng.integers(1, 50, size=300).astype(np.float32)
    o = make(oracle_mod, prio, 16)
    prefix = np.cumsum(prio.astype(np.float64))
    for call in range(5):
        assert o.info()[2] == call
        x = o.targets(32, 9, call)
        out = o.sample(32, 0.4, 9, gather=False)
        assert out["rc"] == 0
        assert out["idx"].tolist() == [int(np.searchsorted(prefix, xi, side="right")) for xi in x]


@pytest.mark.parametrize("K,N", [(2, 8), (4, 13), (16, 40), (32, 64)])
def test_chi_square_b1(oracle_mod, K, N):
    # B = 1: independent draws from P(i) = p_i / sum_k p_k.
    rng = np.random.default_rng(K * 1000 + N)
    prio = (np.abs(rng.normal(size=N)) + 1e-6).astype(np.float32) ** np.float32(0.6)
    o = make(oracle_mod, prio, K)
    draws = 60_000
    counts = np.zeros(N, dtype=np.int64)
    for _ in range(draws):
        counts[o.sample(1, 0.4, 123, gather=False)["idx"][0]] += 1
    expect = draws * prio.astype(np.float64) / prio.astype(np.float64).sum()
    chi2 = ((counts - expect) ** 2 / expect).sum()
    assert stats.chi2.sf(chi2, N - 1) > 1e-4


def test_chi_square_detects_wrong_distribution(oracle_mod):
    # Sensitivity of the test above: counts drawn from p^2 instead of p are rejected.
    rng = np.random.default_rng(4)
    prio = (np.abs(rng.normal(size=13)) + 1e-6) ** 0.6
    wrong = rng.multinomial(60_000, prio**2 / (prio**2).sum())
    expect = 60_000 * prio / prio.sum()
    assert stats.chi2.sf(((wrong - expect) ** 2 / expect).sum(), 12) < 1e-4


@pytest.mark.parametrize("K", [2, 16])
def test_stratified_counts_bound_and_mean(oracle_mod, K):
    # In one call leaf i is hit between floor(B P(i)) - 1 and ceil(B P(i)) + 1 times; over many
    # calls the mean count is B P(i).
    rng = np.random.default_rng(K)
    N, B, calls = 48, 24, 3000
    prio = np.exp(rng.normal(size=N)).astype(np.float32)
    o = make(oracle_mod, prio, K)
    P = prio.astype(np.float64) / float(o.total())
    acc = np.zeros(N)
    for _ in range(calls):
        c = np.bincount(o.sample(B, 0.4, 77, gather=False)["idx"], minlength=N)
        assert np.all(c >= np.floor(B * P) - 1) and np.all(c <= np.ceil(B * P) + 1)
        acc += c
    assert np.allclose(acc / calls, B * P, atol=4 * np.sqrt(B * P / calls) + 1e-3)


def test_is_weights_closed_form(oracle_mod):
    rng = np.random.default_rng(2)
    prio = np.exp(2 * rng.normal(size=500)).astype(np.float32)
    o = make(oracle_mod, prio, 16)
    total = np.float64(o.total())
    for beta in (0.0, 0.4, 1.0):
        out = o.sample(64, beta, 3, gather=False)
        p = prio[out["idx"]].astype(np.float64)
        w = (500 * p / total) ** (-np.float64(np.float32(beta)))
        assert np.allclose(out["w"], w / w.max(), rtol=1e-6)
        assert out["w"].max() == np.float32(1.0)
        if beta == 0.0:
            assert np.all(out["w"] == 1.0)
    flat = make(oracle_mod, np.full(64, 0.25, dtype=np.float32), 4)
    assert np.all(flat.sample(16, 0.7, 0, gather=False)["w"] == 1.0)     # uniform priorities


def test_size_is_number_stored_not_capacity(oracle_mod):
    # Half-filled buffer: indices stay below size, weights use size (cancels under batch-max).
    o = oracle_mod.OraclePRB(64, 4, 0, 0)
    prio = np.arange(1, 21, dtype=np.float32)
    o.insert(None, None, None, None, None, prio)
    out = o.sample(16, 0.5, 1, gather=False)
    assert out["idx"].max() < 20 and out["idx"].min() >= 0
    p = prio[out["idx"]].astype(np.float64)
    assert np.allclose(out["w"], (p.min() / p) ** 0.5, rtol=1e-6)


def test_never_returns_zero_priority_or_unfilled(oracle_mod):
    rng = np.random.default_rng(8)
    prio = rng.integers(0, 3, size=200).astype(np.float32)
    prio[0] = 0
    prio[-1] = 0
    o = make(oracle_mod, prio, 8)
    for _ in range(200):
        idx = o.sample(50, 0.4, 5, gather=False)["idx"]
        assert np.all(prio[idx] > 0)


def test_empty_and_zero_total(oracle_mod):
    o = oracle_mod.OraclePRB(16, 2, 0, 0)
    out = o.sample(4, 0.4, 0, gather=False)
    assert out["rc"] == 0 and o.status() == oracle_mod.ST_EMPTY
    assert out["idx"].tolist() == [-1] * 4 and o.info()[2] == 0
    o.insert(None, None, None, None, None, np.zeros(5, dtype=np.float32))
    o.sample(4, 0.4, 0, gather=False)
    assert o.status() == oracle_mod.ST_EMPTY


def test_rounding_sliver_rule(oracle_mod):
    # Force x >= s_{K-1} one level down by making a parent larger than its children's sum:
    # the last positive child is taken and CLAMPED is raised.
    o = make(oracle_mod, P8, 2)
    o.poke_level(2, 3, [9.0])          # children 2 + 6 = 8 < 9
    i, p = o.descend(9.0 + 14.0 + 8.5)
    assert (i, p) == (7, 6.0)
    assert o.status() == oracle_mod.ST_CLAMPED
    o.poke_level(3, 6, [2.0, 0.0])
    assert o.descend(9.0 + 14.0 + 8.5)[0] == 6     # skips the zero child
    o.status()


@pytest.mark.parametrize("K,D,lift", [(2, 2, 0), (2, 10, 0), (4, 3, 1), (16, 3, 0), (32, 2, 0), (32, 2, 1)])
def test_rounding_sliver_reached_without_planting(oracle_mod, K, D, lift):
    # The fall-off is reachable through the public calls alone: a level prefix fl(2^24 + 3) that
    # rounds up to 2^24 + 4 leaves a residual of at least 3 under a node that holds 3.  Every other
    # target of the batch behaves: the flat scan over the exact binary64 prefixes names its leaf.
    from prb_harness import seed_for_sliver, sliver_leaves
    p, leaf = sliver_leaves(K, D, lift)
    o = make(oracle_mod, p, K)
    assert float(o.total()) == 2.0 ** 24 + 4
    i, pl = o.descend(2.0 ** 24 + 3.5)
    assert (i, pl) == (leaf, 2.0) and o.status() == oracle_mod.ST_CLAMPED
    assert o.descend(2.0 ** 24 + 2.5)[0] == leaf and o.status() == 0          # just below the sliver: no fall-off
    B = 1024
    seed = seed_for_sliver(oracle_mod, B)
    x = o.targets(B, seed, 0)
    out = o.sample(B, 0.4, seed, gather=False)
    assert o.status() == oracle_mod.ST_CLAMPED
    flat = np.cumsum(p.astype(np.float64))
    expect = np.searchsorted(flat, x[:-1], side="right")
    assert np.array_equal(out["idx"][:-1], expect) and out["idx"][-1] == leaf


def test_gather_bytes(oracle_mod):
    rng = np.random.default_rng(6)
    N = 100
    f = dict(obs=rng.integers(0, 256, size=(N, 24), dtype=np.uint8), act=rng.integers(0, 256, size=(N, 5), dtype=np.uint8),
             rew=rng.normal(size=N).astype(np.float32), next_obs=rng.integers(0, 256, size=(N, 24), dtype=np.uint8),
             done=rng.integers(0, 2, size=N, dtype=np.uint8))
    prio = rng.uniform(0.1, 1, size=N).astype(np.float32)
    o = make(oracle_mod, prio, 4, 24, 5, **f)
    out = o.sample(37, 0.4, 2)
    i = out["idx"]
    for name in ("obs", "act", "rew", "next_obs", "done"):
        assert np.array_equal(out[name], f[name][i])


def test_uniform_replay(oracle_mod):
    # i_k = floor(u_k * size): in range, uniform (chi-square), independent of the priorities, rows gathered
    rng = np.random.default_rng(12)
    N = 50
    f = dict(obs=rng.integers(0, 256, size=(N, 8), dtype=np.uint8), act=rng.integers(0, 256, size=(N, 2), dtype=np.uint8),
             rew=rng.normal(size=N).astype(np.float32), next_obs=rng.integers(0, 256, size=(N, 8), dtype=np.uint8),
             done=rng.integers(0, 2, size=N, dtype=np.uint8))
    o = oracle_mod.OraclePRB(64, 4, 8, 2)
    assert o.sample_uniform(4, 0)["idx"].tolist() == [-1] * 4 and o.status() == oracle_mod.ST_EMPTY
    o.insert(f["obs"], f["act"], f["rew"], f["next_obs"], f["done"], np.exp(3 * rng.normal(size=N)).astype(np.float32))
    counts = np.zeros(N, dtype=np.int64)
    for call in range(400):
        assert o.info()[2] == call
        out = o.sample_uniform(100, 5)
        i = out["idx"]
        u = np.array([oracle_mod.stratum_uniform(5, call, k) for k in range(100)])
        assert i.tolist() == np.floor(u * N).astype(np.int64).tolist()
        assert np.all(out["w"] == 1.0)
        for name in ("obs", "act", "rew", "next_obs", "done"):
            assert np.array_equal(out[name], f[name][i])
        counts += np.bincount(i, minlength=N)
    chi2 = ((counts - 800.0) ** 2 / 800.0).sum()
    assert stats.chi2.sf(chi2, N - 1) > 1e-4


def test_buffer_wide_weight_normalisation(oracle_mod):
    # Schaul et al., Algorithm 1: the weights are divided by the largest weight over the whole memory,
    # i.e. that of the smallest positive priority.  Closed form: w_k = (p_min / p_k)^beta.
    prio = np.array([3, 1, 4, 0, 5, 9, 0.5, 6], dtype=np.float32)
    for K in (2, 4, 8):
        a, b = make(oracle_mod, prio, K), make(oracle_mod, prio, K)
        for beta in (0.0, 0.4, 1.0):
            out = a.sample(4, beta, 7, buffer_norm=True)
            ref = b.sample(4, beta, 7)
            assert np.array_equal(out["idx"], ref["idx"])               # same draw, same counter
            p = prio[out["idx"]].astype(np.float64)
            assert np.allclose(out["w"], (0.5 / p) ** beta, rtol=1e-6)
            assert np.all(out["w"] <= 1.0 + 1e-6)
            # against the batch-normalised weights: one common factor, the batch's own largest weight
            factor = (0.5 / p.min()) ** beta
            assert np.allclose(out["w"], ref["w"].astype(np.float64) * factor, rtol=1e-6)
        assert a.info() == b.info()
    # uniform priorities: every weight is exactly 1 in either form
    o = make(oracle_mod, np.full(64, 2.5, dtype=np.float32), 4)
    assert np.all(o.sample(16, 0.7, 1, buffer_norm=True)["w"] == 1.0)
    # zero priorities do not count as the minimum; slots not yet written neither
    o = oracle_mod.OraclePRB(16, 2, 0, 0)
    assert o.insert(None, None, None, None, None, np.array([0, 2, 8], dtype=np.float32)) == 0
    out = o.sample(8, 1.0, 3, buffer_norm=True)
    assert np.allclose(out["w"], 2.0 / np.array([0, 2, 8], dtype=np.float64)[out["idx"]], rtol=1e-6)
