"""Parity of the frame-deduplicated layout (pearl_prb_create_frames) against the oracle's, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2311_09445_b200 import workloads as wk
from prb_harness import Pair

pytestmark = pytest.mark.gpu


def slots(b):
    """An insertion batch of the frame layout from a trajectory chunk: one frame per slot, markers in done."""
    return {"obs": b["frame"], "act": b["act"], "rew": b["rew"], "done": b["done"], "prio": b["prio"]}


@pytest.mark.parametrize("S,F,N,K,B", [(4, 48, 300, 4, 64), (4, 7056, 3000, 32, 512), (2, 1024, 1000, 16, 256), (1, 16, 64, 2, 16),
                                       (3, 5, 50, 8, 8), (4, 2048, 2000, 32, 2500), (4, 1040, 700, 2, 37), (16, 64, 500, 16, 100)])
def test_frame_layout_all_calls(oracle_mod, S, F, N, K, B):
    rng = np.random.default_rng(S * 100 + F + N)
    traj = wk.FrameTrajectory(rng, F, S, episode_steps=(1, 25))
    pr = Pair(oracle_mod, N, K, S * F, 4, max(B, 512), frame_stack=S)
    dev = pr.dev
    n_ins = min(200, N // 3)
    # a sample before anything is stored, and one when only a marker is
    o, g = pr.sample(4, 0.4, 1)
    pr.insert(slots(traj.next(1, stacks=False)))
    o, g = pr.sample(4, 0.4, 1)
    assert g["idx"].tolist() == [-1] * 4 and pr.compare_status() == 4
    stale_seen = 0
    for step in range(14):                        # fills, then wraps the ring several times
        pr.insert(slots(traj.next(n_ins, stacks=False)))
        pr.compare_tree()
        pr.compare_state()
        o, g = pr.sample(B, 0.4, 11 + step)
        assert not (g["done"] & 2).any()
        idx = o["idx"].copy()
        td = (rng.standard_normal(B) * 2).astype(np.float32)
        cursor = pr.ora.info()[1]
        if B >= 8:
            idx[1] = (cursor + 1) % N             # slots behind the cursor: no history once the ring has wrapped
            idx[2] = (cursor + S - 1) % N
            idx[3] = (cursor + S) % N
        if step % 3 == 0:
            pr.update(idx, td, 0.6, 1e-6)
        elif step % 3 == 1:
            pr.update_insert(idx, td, 0.6, 1e-6, slots(traj.next(n_ins // 2 + 1, stacks=False)))
        else:
            o2, g2 = pr.step(idx, td, 0.6, 1e-6, slots(traj.next(n_ins // 3 + 1, stacks=False)), B, 0.4, 5)
        pr.compare_tree()
        pr.compare_state()
        stale_seen |= pr.compare_status()
    if B >= 8:
        assert stale_seen & 32
    # the other sample calls rebuild the same way
    o = pr.ora.sample(B, 0.4, 3, buffer_norm=True)
    t = {"idx": torch.full((B,), -1, dtype=torch.int32, device=dev), "w": torch.zeros(B, device=dev),
         "obs": torch.zeros((B, S * F), dtype=torch.uint8, device=dev), "next_obs": torch.zeros((B, S * F), dtype=torch.uint8, device=dev)}
    pr.gpu.sample_buffer_norm(B, 0.4, 3, t["idx"], t["w"], t["obs"], None, None, t["next_obs"], None)
    torch.cuda.synchronize()
    assert np.array_equal(t["idx"].cpu().numpy(), o["idx"])
    np.testing.assert_allclose(t["w"].cpu().numpy(), o["w"], rtol=1e-5, atol=0)
    assert np.array_equal(t["obs"].cpu().numpy(), o["obs"]) and np.array_equal(t["next_obs"].cpu().numpy(), o["next_obs"])
    if B >= 4:
        o = pr.ora.sample(B, 0.4, 3)
        for k in t:
            t[k].zero_()
        pr.gpu.sample_streamed(B, 0.4, 3, 3, t["idx"], t["w"], None, None, None, t["next_obs"], None)      # next_obs alone
        torch.cuda.synchronize()
        assert np.array_equal(t["idx"].cpu().numpy(), o["idx"]) and np.array_equal(t["next_obs"].cpu().numpy(), o["next_obs"])
        assert t["obs"].max().item() == 0
    pr.compare_state()
    keep = np.nonzero(pr.ora.read_level(pr.ora.depth)[:N] > 0)[0].astype(np.int32)[:400]
    pr.compare_rows(keep)
    from paper_2311_09445_b200 import PearlError
    with pytest.raises(PearlError) as e:
        pr.gpu.sample_uniform(4, 0, t["idx"][:4])
    assert e.value.code == -7
    with pytest.raises(PearlError) as e:          # a next_obs batch has no place in this layout
        pr.gpu.insert(t["obs"][:1, :F].contiguous(), None, None, t["obs"][:1, :F].contiguous(), t["idx"][:1].view(torch.uint8)[:1], None, n=1)
    assert e.value.code == -7
    pr.close()


def test_frame_layout_against_plain_layout_on_the_gpu(oracle_mod):
    # the same trajectory in both layouts on the GPU: before the ring wraps, identical indices, weights and gathered bytes
    from paper_2311_09445_b200 import PrioritizedReplay
    S, F, N, K, B = 4, 7056, 4000, 32, 512
    rng = np.random.default_rng(9)
    traj = wk.FrameTrajectory(rng, F, S, episode_steps=(2, 40))
    dev = torch.device("cuda:0")
    fr = PrioritizedReplay(N, K, S * F, 4, 512, frame_stack=S)
    pl = PrioritizedReplay(N, K, S * F, 4, 512)
    for step in range(7):
        b = traj.next(500)
        d = {k: torch.from_numpy(np.ascontiguousarray(v)).to(dev) for k, v in b.items()}
        act = d["act"].view(torch.uint8).reshape(500, 4)
        fr.insert(d["frame"], act, d["rew"], None, d["done"], d["prio"])
        pl.insert(d["obs"], act, d["rew"], d["next_obs"], d["done"], d["prio"])
        out = []
        for buf in (fr, pl):
            t = {"idx": torch.zeros(B, dtype=torch.int32, device=dev), "w": torch.zeros(B, device=dev),
                 "obs": torch.zeros((B, S * F), dtype=torch.uint8, device=dev), "next_obs": torch.zeros((B, S * F), dtype=torch.uint8, device=dev)}
            buf.sample(B, 0.4, 2, t["idx"], t["w"], t["obs"], None, None, t["next_obs"], None)
            out.append(t)
        torch.cuda.synchronize()
        for k in out[0]:
            assert torch.equal(out[0][k], out[1][k]), k
    fr.close()
    pl.close()


def test_frame_layout_atari_size(oracle_mod):
    # 2^19 slots of 84 x 84 frames, stack 4, fanout 32, batches of 512: the Atari-shaped workload in this layout
    # (3.7 GB of frames instead of 29.6 GB of stacks); the oracle mirrors the whole store.
    S, F, N, K, B = 4, 84 * 84, 1 << 19, 32, 512
    free, _ = torch.cuda.mem_get_info()
    if free < N * (F + 16) + (3 << 30):
        pytest.skip("not enough free device memory")
    rng = np.random.default_rng(4)
    traj = wk.FrameTrajectory(rng, F, S, episode_steps=(20, 400))
    pr = Pair(oracle_mod, N, K, S * F, 4, 8192, frame_stack=S)
    for first in range(0, N + 8192, 8192):        # fills and wraps
        pr.insert(slots(traj.next(8192, stacks=False)))
    pr.compare_tree()
    pr.compare_state()
    o, g = pr.sample(B, 0.4, 0)
    for step in range(4):
        td = rng.standard_normal(B).astype(np.float32)
        o, g = pr.step(o["idx"], td, 0.6, 1e-6, slots(traj.next(512, stacks=False)), B, 0.4, 0)
        pr.compare_tree(range(0, pr.ora.depth))
    pr.compare_tree()
    pr.compare_state()
    assert pr.compare_status() & ~8 == 0
    pr.close()
