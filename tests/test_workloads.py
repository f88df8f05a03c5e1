"""The seeded input generators: shapes, dtypes, determinism, and the counter-based row bytes."""
import numpy as np
import torch

from paper_2311_09445_b200 import workloads as wk


def test_named_workloads_have_the_configured_shapes():
    assert wk.TINY.transition_bytes == 41 and wk.CARTPOLE.transition_bytes == 41
    assert wk.DDPG.obs_bytes == 68 and wk.DDPG.act_bytes == 24 and wk.DDPG.transition_bytes == 165
    assert wk.ATARI.obs_bytes == 4 * 84 * 84 == 28224 and wk.ATARI.transition_bytes == 56457
    assert (wk.CARTPOLE.capacity, wk.CARTPOLE.fanout, wk.CARTPOLE.batch, wk.CARTPOLE.n_insert) == (1 << 20, 16, 64, 64)
    assert (wk.ATARI.capacity, wk.ATARI.fanout, wk.ATARI.batch, wk.ATARI.n_insert) == (1 << 19, 32, 512, 512)
    c = wk.sweep_cell(1 << 22, 4, 1024, 3)
    assert c.obs_bytes == 68 and c.n_insert == 1024 and c.seed == 2003


def test_transitions_are_seeded_and_typed():
    for wl in (wk.TINY, wk.DDPG, wk.scaled(wk.ATARI, 1024)):
        a = wk.transitions(wl, np.random.default_rng(wl.seed), 37, 5)
        b = wk.transitions(wl, np.random.default_rng(wl.seed), 37, 5)
        for k in ("obs", "act", "rew", "next_obs", "done", "prio"):
            assert a[k].shape[0] == 37 and np.array_equal(a[k], b[k]), k
        assert a["obs"].dtype == np.dtype(wl.obs_dtype) and a["obs"].shape[1:] == wl.obs_shape
        assert a["act"].dtype == np.dtype(wl.act_dtype) and a["rew"].dtype == np.float32 and a["done"].dtype == np.uint8
        assert a["prio"].dtype == np.float32 and np.all(a["prio"] > 0) and np.all(np.isfinite(a["prio"]))
    at = wk.transitions(wk.scaled(wk.ATARI, 1024), np.random.default_rng(1), 500)
    assert set(np.unique(at["rew"])) <= {-1.0, 0.0, 1.0} and at["act"].min() >= 0 and at["act"].max() < 18
    d = wk.transitions(wk.DDPG, np.random.default_rng(1), 500)
    assert d["act"].min() >= -1 and d["act"].max() <= 1


def test_counter_rows_depend_only_on_id_field_and_offset():
    ids = torch.tensor([0, 1, 7, 123456789, 2**40 + 5])
    a = wk.counter_row_bytes(ids, 0, 64)
    assert a.dtype == torch.uint8 and a.shape == (5, 64)
    assert torch.equal(a, wk.counter_row_bytes(ids, 0, 64))
    assert torch.equal(a[2], wk.counter_row_bytes(torch.tensor([7]), 0, 64)[0])          # a row can be regenerated alone
    assert torch.equal(a[:, :32], wk.counter_row_bytes(ids, 0, 32))                        # and so can a prefix
    assert not torch.equal(a, wk.counter_row_bytes(ids, 1, 64))                            # fields differ
    big = wk.counter_row_bytes(torch.arange(64), 0, 28224).numpy()
    counts = np.bincount(big.reshape(-1), minlength=256)
    assert counts.min() > 0.9 * big.size / 256 and counts.max() < 1.1 * big.size / 256     # bytes look uniform


def test_update_batch_injects_the_configured_duplicates():
    rng = np.random.default_rng(2)
    idx = np.arange(256, dtype=np.int32) * 3
    out, td = wk.update_batch(wk.DDPG, rng, idx)
    assert td.shape == (256,) and out.shape == (256,)
    assert 0 < 256 - len(set(out.tolist())) <= 13 and set(out.tolist()) <= set(idx.tolist())
    out2, _ = wk.update_batch(wk.CARTPOLE, rng, idx[:64])
    assert np.array_equal(out2, idx[:64])
