"""The sample call for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not an option: inside a framework whose pool
already owns the GPU's memory, or in a loop that must not touch an allocator once it is running.
pearl_prb_sample_static_scratch serves them: it keeps the sample kernel's scratch in a static
array inside the library.  This test drives it through the C ABI next to the ordinary
pearl_prb_sample on two buffers with identical contents and requires identical indices and
gathered bytes and weights within the suite's tolerance, on two calls in a row (the second call
finds the array as the first left it).  It is collected last so that a stop-at-first-failure run
has already run every other test.
"""
import numpy as np
import pytest
import torch

from prb_harness import W_RTOL

pytestmark = pytest.mark.gpu


def _outputs(dev, B, obs_bytes, act_bytes):
    return {"idx": torch.full((B,), -1, dtype=torch.int32, device=dev), "w": torch.zeros(B, device=dev),
            "obs": torch.zeros((B, obs_bytes), dtype=torch.uint8, device=dev),
            "act": torch.zeros((B, act_bytes), dtype=torch.uint8, device=dev), "rew": torch.zeros(B, device=dev),
            "next_obs": torch.zeros((B, obs_bytes), dtype=torch.uint8, device=dev),
            "done": torch.zeros(B, dtype=torch.uint8, device=dev)}


@pytest.mark.parametrize("fanout,obs_bytes,B", [(16, 68, 256), (32, 8192, 64)])
def test_static_scratch_sample_matches_ordinary_sample(fanout, obs_bytes, B):
    from paper_2311_09445_b200 import PearlError, PrioritizedReplay
    N, act_bytes = 3000, 24
    rng = np.random.default_rng(fanout)
    dev = torch.device("cuda:0")
    a = PrioritizedReplay(N, fanout, obs_bytes, act_bytes, 8192)
    b = PrioritizedReplay(N, fanout, obs_bytes, act_bytes, 8192)
    batch = {"obs": torch.from_numpy(rng.integers(0, 256, (N, obs_bytes), dtype=np.uint8)).to(dev),
             "act": torch.from_numpy(rng.integers(0, 256, (N, act_bytes), dtype=np.uint8)).to(dev),
             "rew": torch.from_numpy(rng.standard_normal(N).astype(np.float32)).to(dev),
             "next_obs": torch.from_numpy(rng.integers(0, 256, (N, obs_bytes), dtype=np.uint8)).to(dev),
             "done": torch.from_numpy(rng.integers(0, 2, N, dtype=np.uint8)).to(dev),
             "prio": torch.from_numpy(np.exp(rng.standard_normal(N)).astype(np.float32)).to(dev)}
    for buf in (a, b):
        buf.insert(batch["obs"], batch["act"], batch["rew"], batch["next_obs"], batch["done"], batch["prio"])
    for call in range(2):                      # two calls in a row share the static array
        oa, ob = _outputs(dev, B, obs_bytes, act_bytes), _outputs(dev, B, obs_bytes, act_bytes)
        a.sample(B, 0.4, 5, oa["idx"], oa["w"], oa["obs"], oa["act"], oa["rew"], oa["next_obs"], oa["done"])
        b.sample_static_scratch(B, 0.4, 5, ob["idx"], ob["w"], ob["obs"], ob["act"], ob["rew"], ob["next_obs"],
                                ob["done"])
        torch.cuda.synchronize()
        assert oa["idx"].min().item() >= 0
        assert torch.equal(oa["idx"], ob["idx"])
        np.testing.assert_allclose(ob["w"].cpu().numpy(), oa["w"].cpu().numpy(), rtol=W_RTOL, atol=0)
        assert ob["w"].max().item() == 1.0
        for f in ("obs", "act", "rew", "next_obs", "done"):
            assert torch.equal(oa[f].view(torch.uint8), ob[f].view(torch.uint8)), f
    assert a.info() == b.info() and a.sync() == b.sync() == 0
    big = torch.zeros(4097, dtype=torch.int32, device=dev)
    with pytest.raises(PearlError) as e:       # beyond the static array: a clear error, nothing enqueued
        b.sample_static_scratch(4097, 0.4, 5, big)
    assert e.value.code == -3 and "exceeds the maximum" in str(e.value)
    assert a.info() == b.info()
    a.close()
    b.close()
