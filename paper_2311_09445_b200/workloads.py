"""Seeded synthetic inputs shaped like the paper's DRL workloads (PEARL Table III: CartPole /
MountainCar-like / Pong observations) for the replay buffer's tests and benchmark.

Input generation only: nothing here computes any step of the replay path.  The CPU oracle
and the CUDA library are both fed from these arrays.  Gym environments and recorded
transitions are not available; these stand in for them with the same shapes and dtypes.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Tuple

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    capacity: int
    fanout: int
    obs_shape: Tuple[int, ...]
    obs_dtype: str            # numpy dtype name
    act_shape: Tuple[int, ...]
    act_dtype: str
    batch: int                # B of sample and update
    n_insert: int             # transitions inserted per step (0 = none)
    steps: int
    seed: int
    prio_dist: str            # "normal" or "lognormal" TD errors
    dup_frac: float = 0.0     # fraction of update positions overwritten by another position's index
    alpha: float = 0.6
    beta: float = 0.4
    eps: float = 1e-6
    philox_seed: int = 0
    counter_rows: bool = False   # observations are a function of the global insert id (too large to mirror)
    frame_stack: int = 0         # > 0: the frame-deduplicated layout, obs_shape[0] == frame_stack frames per observation

    @property
    def obs_bytes(self) -> int:
        return int(np.prod(self.obs_shape)) * np.dtype(self.obs_dtype).itemsize

    @property
    def act_bytes(self) -> int:
        return int(np.prod(self.act_shape)) * np.dtype(self.act_dtype).itemsize

    @property
    def transition_bytes(self) -> int:
        """Bytes one transition takes in the Data Storage (and in an insertion's batch)."""
        if self.frame_stack:
            return self.obs_bytes // self.frame_stack + self.act_bytes + 4 + 1
        return 2 * self.obs_bytes + self.act_bytes + 4 + 1

    @property
    def sample_bytes(self) -> int:
        """Bytes a sampled transition makes the gather read and write (both observations whole on the way out;
        with frames, frame_stack + 1 frames on the way in)."""
        small = self.act_bytes + 4 + 1
        if self.frame_stack:
            return (self.frame_stack + 1) * (self.obs_bytes // self.frame_stack) + 2 * self.obs_bytes + 2 * small
        return 2 * (2 * self.obs_bytes + small)


TINY = Workload("tiny", 4096, 2, (4,), "float32", (), "int32", 32, 0, 100, 1001, "normal")
CARTPOLE = Workload("cartpole_dqn", 1 << 20, 16, (4,), "float32", (), "int32", 64, 64, 10_000, 1002, "normal")
DDPG = Workload("mujoco_ddpg", 1 << 20, 16, (17,), "float32", (6,), "float32", 256, 256, 2_000, 1003, "lognormal",
                dup_frac=0.05)
ATARI = Workload("atari_dqn", 1 << 19, 32, (4, 84, 84), "uint8", (), "int32", 512, 512, 1_000, 1004, "normal",
                 counter_rows=True)
# the Atari-shaped workload with one 84 x 84 frame stored per transition (a single actor's trajectory)
ATARI_FRAMES = Workload("atari_dqn_frames", 1 << 19, 32, (4, 84, 84), "uint8", (), "int32", 512, 512, 1_000, 1005, "normal",
                        counter_rows=True, frame_stack=4)
WORKLOADS: Dict[str, Workload] = {w.name: w for w in (TINY, CARTPOLE, DDPG, ATARI, ATARI_FRAMES)}


def sweep_cell(capacity: int, fanout: int, batch: int, cell_id: int = 0) -> Workload:
    """One cell of the scaling sweep: obs fp32[17], action fp32[6], insert 1024 + sample B + update B."""
    return Workload("sweep_N%d_K%d_B%d" % (capacity, fanout, batch), capacity, fanout, (17,), "float32", (6,),
                    "float32", batch, 1024, 20, 2000 + cell_id, "lognormal")


def scaled(wl: Workload, capacity: int, **kw) -> Workload:
    """The same workload at another capacity (used where the CPU oracle cannot hold the full store)."""
    d = dict(wl.__dict__)
    d.update(capacity=capacity, name="%s_N%d" % (wl.name, capacity))
    d.update(kw)
    return Workload(**d)


def td_errors(wl: Workload, rng: np.random.Generator, n: int) -> np.ndarray:
    z = rng.standard_normal(n)
    d = z if wl.prio_dist == "normal" else np.exp(2.0 * z)      # N(0,1) or LogNormal(0, 2)
    return d.astype(np.float32)


def priorities(wl: Workload, rng: np.random.Generator, n: int) -> np.ndarray:
    """Initial priorities handed to insert: (|d| + 1e-6)^0.6 in binary64, rounded to binary32."""
    d = td_errors(wl, rng, n).astype(np.float64)
    return ((np.abs(d) + 1e-6) ** 0.6).astype(np.float32)


_MASK32 = 0xFFFFFFFF


def counter_row_bytes(ids: torch.Tensor, field_id: int, nbytes: int) -> torch.Tensor:
    """Pseudo-random bytes of rows `ids` (int64 global insert ids) of field `field_id`: word j of row g
    is an integer hash of (g, field_id, j).  Runs on whatever device `ids` lives on, so the device
    store can be filled in place and any row regenerated on the host later.  nbytes % 4 == 0."""
    assert nbytes % 4 == 0
    words = nbytes // 4
    j = torch.arange(words, dtype=torch.int64, device=ids.device)
    x = (ids.to(torch.int64)[:, None] * 2654435761 + j[None, :] * 40503 + (field_id + 1) * 97531) & _MASK32
    x = x ^ (x >> 15)
    x = (x * 0x2C1B3C6D) & _MASK32
    x = x ^ (x >> 12)
    x = (x * 0x297A2D39) & _MASK32
    x = x ^ (x >> 15)
    x = torch.where(x >= (1 << 31), x - (1 << 32), x).to(torch.int32)
    return x.contiguous().view(torch.uint8).reshape(ids.shape[0], nbytes)


def transitions(wl: Workload, rng: np.random.Generator, n: int, first_id: int = 0,
                with_obs: bool = True) -> Dict[str, np.ndarray]:
    """n synthetic transitions as host arrays: obs, act, rew, next_obs, done, prio.
    With wl.counter_rows the observations depend on the global insert ids first_id .. first_id+n-1;
    with_obs=False leaves obs/next_obs out (the caller generates them on the device)."""
    obs_dt, act_dt = np.dtype(wl.obs_dtype), np.dtype(wl.act_dtype)
    out: Dict[str, np.ndarray] = {}
    if not with_obs:
        pass
    elif wl.counter_rows:
        ids = torch.arange(first_id, first_id + n, dtype=torch.int64)
        out["obs"] = counter_row_bytes(ids, 0, wl.obs_bytes).numpy().view(obs_dt).reshape((n,) + wl.obs_shape)
        out["next_obs"] = counter_row_bytes(ids, 1, wl.obs_bytes).numpy().view(obs_dt).reshape((n,) + wl.obs_shape)
    elif obs_dt.kind == "f":
        out["obs"] = rng.standard_normal((n,) + wl.obs_shape).astype(obs_dt)
        out["next_obs"] = rng.standard_normal((n,) + wl.obs_shape).astype(obs_dt)
    else:
        out["obs"] = rng.integers(0, 256, size=(n,) + wl.obs_shape, dtype=np.uint8)
        out["next_obs"] = rng.integers(0, 256, size=(n,) + wl.obs_shape, dtype=np.uint8)
    if act_dt.kind == "f":
        out["act"] = rng.uniform(-1.0, 1.0, size=(n,) + wl.act_shape).astype(act_dt)
    else:
        n_actions = 18 if wl.counter_rows else 2
        out["act"] = rng.integers(0, n_actions, size=(n,) + wl.act_shape).astype(act_dt)
    if wl.counter_rows:
        out["rew"] = rng.integers(-1, 2, size=n).astype(np.float32)
        out["done"] = (rng.random(n) < 0.01).astype(np.uint8)
    else:
        out["rew"] = rng.standard_normal(n).astype(np.float32)
        out["done"] = (rng.random(n) < 0.05).astype(np.uint8)
    out["prio"] = priorities(wl, rng, n)
    return out


class FrameTrajectory:
    """A single actor's stream of transitions whose observations are stacks of the last `stack` frames
    (an Atari-style environment behind a frame-stacking wrapper: at reset the stack is filled with the
    first frame, every step pushes one new frame), handed out both ways at once:

      * one frame per ring slot -- the newest frame of the transition's next observation -- with an extra
        slot at every episode start that carries the episode's first frame and has bit 1 of `done` set
        (the frame-deduplicated layout of the replay buffer);
      * the same slots with whole stacks `obs` / `next_obs` (the plain layout); the rows of the extra
        slots are zero and their priority is 0.

    This is the environment side: it knows nothing of how the buffer stores or rebuilds anything."""

    def __init__(self, rng: np.random.Generator, frame_bytes: int, stack: int, episode_steps=(3, 30), n_actions: int = 18):
        self.rng, self.F, self.S = rng, frame_bytes, stack
        self.episode_steps, self.n_actions = episode_steps, n_actions
        self.window = None          # the current observation: `stack` frames, oldest first
        self.left = 0               # steps left in the running episode

    def _frame(self) -> np.ndarray:
        return self.rng.integers(0, 256, size=self.F, dtype=np.uint8)

    def next(self, n: int, stacks: bool = True) -> Dict[str, np.ndarray]:
        """n more slots.  stacks=False leaves "obs" / "next_obs" (the plain layout's rows) out."""
        F, S = self.F, self.S
        out = {"frame": np.zeros((n, F), np.uint8), "obs": np.zeros((n if stacks else 0, S * F), np.uint8),
               "next_obs": np.zeros((n if stacks else 0, S * F), np.uint8),
               "act": self.rng.integers(0, self.n_actions, size=n).astype(np.int32), "rew": self.rng.integers(-1, 2, size=n).astype(np.float32),
               "done": np.zeros(n, np.uint8), "prio": np.exp(self.rng.standard_normal(n)).astype(np.float32)}
        for t in range(n):
            if self.left == 0:                       # reset: the slot carries the first frame only
                first = self._frame()
                self.window = [first] * S
                self.left = int(self.rng.integers(self.episode_steps[0], self.episode_steps[1] + 1))
                out["frame"][t] = first
                out["done"][t] = 2
                out["prio"][t] = 0.0
                out["act"][t], out["rew"][t] = 0, 0.0
                continue
            new = self._frame()
            nxt = self.window[1:] + [new]
            out["frame"][t] = new
            if stacks:
                out["obs"][t] = np.concatenate(self.window)
                out["next_obs"][t] = np.concatenate(nxt)
            self.window = nxt
            self.left -= 1
            out["done"][t] = 1 if self.left == 0 else 0
        return out


def update_batch(wl: Workload, rng: np.random.Generator, sampled_idx: np.ndarray):
    """The update that follows a sample: the sampled indices (with wl.dup_frac of the positions
    overwritten by a copy of another position's index) and fresh TD errors, one per position."""
    idx = np.array(sampled_idx, dtype=np.int32, copy=True)
    B = idx.shape[0]
    n_dup = int(round(wl.dup_frac * B))
    if n_dup:
        pos = rng.choice(B, size=n_dup, replace=False)
        src = rng.integers(0, B, size=n_dup)
        idx[pos] = idx[src]
    return idx, td_errors(wl, rng, B)


def to_device(batch: Dict[str, np.ndarray], device) -> Dict[str, torch.Tensor]:
    return {k: torch.from_numpy(np.ascontiguousarray(v)).to(device) for k, v in batch.items()}
