"""The sample call for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not an option: inside a framework whose pool
already owns the GPU's memory, or in a loop that must not touch an allocator once it is running.
pearl_prb_sample_static_scratch serves them: it keeps the sample kernel's scratch in a static
array inside the library.  This test drives it through the C ABI on a buffer that the CPU oracle
mirrors, next to the ordinary pearl_prb_sample on a second buffer with identical contents, and
requires identical indices and gathered bytes, and weights within the suite's tolerance, against
both, on two calls in a row (the second call finds the array as the first left it).  The cases
cover the three shapes the call can take: a lane group per stratum with short rows, with long
rows (the bulk-copy ring), and the largest batch it accepts, which runs as a thread per stratum
with a second launch that reads the static array.  It is collected last so that a
stop-at-first-failure run has already run every other test.
"""
import numpy as np
import pytest
import torch

from prb_harness import FIELDS, W_RTOL, Pair

pytestmark = pytest.mark.gpu


def _outputs(dev, B, obs_bytes, act_bytes):
    return {"idx": torch.full((B,), -1, dtype=torch.int32, device=dev), "w": torch.zeros(B, device=dev),
            "obs": torch.zeros((B, obs_bytes), dtype=torch.uint8, device=dev),
            "act": torch.zeros((B, act_bytes), dtype=torch.uint8, device=dev), "rew": torch.zeros(B, device=dev),
            "next_obs": torch.zeros((B, obs_bytes), dtype=torch.uint8, device=dev),
            "done": torch.zeros(B, dtype=torch.uint8, device=dev)}


@pytest.mark.parametrize("fanout,obs_bytes,B", [(16, 68, 256), (32, 8192, 64), (16, 68, 4096), (2, 12, 2048)])
def test_static_scratch_sample_matches_oracle_and_ordinary_sample(oracle_mod, fanout, obs_bytes, B):
    from paper_2311_09445_b200 import PearlError, PrioritizedReplay
    N, act_bytes = 3000, 24
    rng = np.random.default_rng(fanout)
    pr = Pair(oracle_mod, N, fanout, obs_bytes, act_bytes, 8192)        # static scratch + oracle
    dev = pr.dev
    twin = PrioritizedReplay(N, fanout, obs_bytes, act_bytes, 8192)     # the ordinary call
    batch = {"obs": rng.integers(0, 256, (N, obs_bytes), dtype=np.uint8),
             "act": rng.integers(0, 256, (N, act_bytes), dtype=np.uint8),
             "rew": rng.standard_normal(N).astype(np.float32),
             "next_obs": rng.integers(0, 256, (N, obs_bytes), dtype=np.uint8),
             "done": rng.integers(0, 2, N, dtype=np.uint8),
             "prio": np.exp(rng.standard_normal(N)).astype(np.float32)}
    d = {k: torch.from_numpy(v).to(dev) for k, v in batch.items()}
    pr.insert(batch, dev_batch=d)
    twin.insert(d["obs"], d["act"], d["rew"], d["next_obs"], d["done"], d["prio"])
    for call in range(2):                      # two calls in a row share the static array
        o = pr.ora.sample(B, 0.4, 5)
        ot, os_ = _outputs(dev, B, obs_bytes, act_bytes), _outputs(dev, B, obs_bytes, act_bytes)
        twin.sample(B, 0.4, 5, ot["idx"], ot["w"], ot["obs"], ot["act"], ot["rew"], ot["next_obs"], ot["done"])
        pr.gpu.sample_static_scratch(B, 0.4, 5, os_["idx"], os_["w"], os_["obs"], os_["act"], os_["rew"],
                                     os_["next_obs"], os_["done"])
        torch.cuda.synchronize()
        g = {k: v.cpu().numpy() for k, v in os_.items()}
        assert g["idx"].min() >= 0
        pr.compare_sample(o, g)                # the oracle: indices, weights (1e-5 relative, maximum 1), bytes
        assert torch.equal(ot["idx"], os_["idx"])
        np.testing.assert_allclose(g["w"], ot["w"].cpu().numpy(), rtol=W_RTOL, atol=0)
        for f in FIELDS:
            assert torch.equal(ot[f].view(torch.uint8), os_[f].view(torch.uint8)), f
    pr.compare_state()
    assert twin.info() == pr.gpu.info() and twin.sync() == 0 and pr.compare_status() == 0
    big = torch.zeros(4097, dtype=torch.int32, device=dev)
    with pytest.raises(PearlError) as e:       # beyond the static array: a clear error, nothing enqueued
        pr.gpu.sample_static_scratch(4097, 0.4, 5, big)
    assert e.value.code == -3 and "exceeds the maximum" in str(e.value)
    pr.compare_state()
    twin.close()
    pr.close()
