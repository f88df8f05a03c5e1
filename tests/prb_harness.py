"""Drives the CPU oracle and the CUDA library with the same inputs and compares them.
Integer/byte results and tree contents must match bit for bit; IS weights within 1e-5 relative."""
import numpy as np
import torch

W_RTOL = 1e-5      # importance-sampling weights: relative tolerance (binary64 pow, two libraries)
FIELDS = ("obs", "act", "rew", "next_obs", "done")


def bits(a):
    return np.ascontiguousarray(a).view(np.uint32)


def sliver_leaves(K, D, lift=0):
    """Leaves of a K^D-leaf tree that make one root-to-leaf walk fall off the end of a child group.

    Two sibling nodes of level D-1 hold 2^24 (K leaves of 2^24/K each) and 3 (leaves 1, 2, 0, ...);
    every other leaf is zero.  Their left-to-right binary32 prefix is fl(2^24 + 3) = 2^24 + 4 (a
    tie, rounded to even), and so is every ancestor up to the root.  A target in
    [2^24 + 3, 2^24 + 4) therefore enters the second node with a residual in [3, 4), which has
    passed every prefix of (1, 3, 3, ...): the walk takes the last positive child, the leaf
    holding 2.  With lift > 0 every leaf is pushed down `lift` more levels (leaf i of the small
    tree becomes leaf i * K^lift of a tree of depth D + lift), so the walk falls off at an inner
    level as well.  Returns (leaves, index of the leaf the walk ends in)."""
    p = np.zeros(K ** D, np.float32)
    a = (K ** (D - 1)) // 2
    a -= a % K                               # a and a + 1 are children of one parent
    p[a * K:(a + 1) * K] = np.float32(2 ** 24 / K)
    p[(a + 1) * K], p[(a + 1) * K + 1] = 1.0, 2.0
    leaf = (a + 1) * K + 1
    if lift:
        big = np.zeros(K ** (D + lift), np.float32)
        big[::K ** lift] = p
        p, leaf = big, leaf * K ** lift
    return p, leaf


def seed_for_sliver(oracle_mod, B, call=0, limit=1 << 22):
    """The first Philox seed whose last stratum (of B, sample call `call`) draws a target in the last
    unit of a total of 2^24 + 4, i.e. in [2^24 + 3, 2^24 + 4): found by scanning on the CPU."""
    total = 2.0 ** 24 + 4
    for seed in range(limit):
        x = (B - 1 + oracle_mod.stratum_uniform(seed, call, B - 1)) * (total / B)
        if 2.0 ** 24 + 3 <= x < total:
            return seed
    raise AssertionError("no seed found")


class Pair:
    def __init__(self, oracle_mod, capacity, fanout, obs_bytes, act_bytes, max_batch, oracle_store=True, frame_stack=0,
                 min_tree=False):
        """frame_stack > 0: both sides use the frame-deduplicated layout (obs_bytes = a whole stack; an insertion's
        batch carries one frame per transition under "obs" and no "next_obs").  min_tree: the GPU buffer keeps a
        min-tree (the oracle has none: it scans its leaves)."""
        from paper_2311_09445_b200 import PrioritizedReplay
        self.gpu = PrioritizedReplay(capacity, fanout, obs_bytes, act_bytes, max_batch, frame_stack=frame_stack,
                                     min_tree=min_tree)
        self.oracle_store = oracle_store
        self.ora = oracle_mod.OraclePRB(capacity, fanout, obs_bytes if oracle_store else 0,
                                        act_bytes if oracle_store else 0, frame_stack=frame_stack)
        self.capacity, self.fanout = capacity, fanout
        self.obs_bytes, self.act_bytes = obs_bytes, act_bytes
        self.dev = self.gpu.device
        assert self.gpu.depth == self.ora.depth

    def close(self):
        self.gpu.close()
        self.ora.close()

    # ---- calls on both sides ----------------------------------------------------------
    def insert(self, batch, dev_batch=None, host_call=False):
        """batch: host arrays (obs, act, rew, next_obs, done, prio).  dev_batch: optional device tensors
        to use on the GPU side instead of uploading `batch`."""
        if self.oracle_store:
            rc = self.ora.insert(batch.get("obs"), batch.get("act"), batch.get("rew"), batch.get("next_obs"),
                                 batch.get("done"), batch["prio"])
        else:
            rc = self.ora.insert(None, None, batch.get("rew"), None, batch.get("done"), batch["prio"])
        assert rc == 0
        if host_call:
            c = {k: (np.ascontiguousarray(v) if v is not None else None) for k, v in batch.items()}
            self.gpu.insert_host(c.get("obs"), c.get("act"), c.get("rew"), c.get("next_obs"), c.get("done"), c["prio"])
            return
        if dev_batch is None:
            dev_batch = {k: torch.from_numpy(np.ascontiguousarray(v)).to(self.dev) for k, v in batch.items()
                         if v is not None}
        self.gpu.insert(dev_batch.get("obs"), dev_batch.get("act"), dev_batch.get("rew"), dev_batch.get("next_obs"),
                        dev_batch.get("done"), dev_batch["prio"])

    def sample(self, B, beta, seed, check=True, host_call=False):
        o = self.ora.sample(B, beta, seed, gather=self.oracle_store)
        if host_call:
            g = {"idx": np.full(B, -1, np.int32), "w": np.zeros(B, np.float32),
                 "obs": np.zeros((B, self.obs_bytes), np.uint8), "act": np.zeros((B, self.act_bytes), np.uint8),
                 "rew": np.zeros(B, np.float32), "next_obs": np.zeros((B, self.obs_bytes), np.uint8),
                 "done": np.zeros(B, np.uint8)}
            self.gpu.sample_host(B, beta, seed, g["idx"], g["w"], g["obs"], g["act"], g["rew"], g["next_obs"], g["done"])
        else:
            t = {"idx": torch.full((B,), -1, dtype=torch.int32, device=self.dev),
                 "w": torch.zeros(B, dtype=torch.float32, device=self.dev),
                 "obs": torch.zeros((B, self.obs_bytes), dtype=torch.uint8, device=self.dev),
                 "act": torch.zeros((B, self.act_bytes), dtype=torch.uint8, device=self.dev),
                 "rew": torch.zeros(B, dtype=torch.float32, device=self.dev),
                 "next_obs": torch.zeros((B, self.obs_bytes), dtype=torch.uint8, device=self.dev),
                 "done": torch.zeros(B, dtype=torch.uint8, device=self.dev)}
            self.gpu.sample(B, beta, seed, t["idx"], t["w"], t["obs"], t["act"], t["rew"], t["next_obs"], t["done"])
            torch.cuda.synchronize()
            g = {k: v.cpu().numpy() for k, v in t.items()}
        if check:
            self.compare_sample(o, g)
        return o, g

    def compare_sample(self, o, g):
        assert np.array_equal(o["idx"], g["idx"]), "sampled indices differ"
        np.testing.assert_allclose(g["w"], o["w"], rtol=W_RTOL, atol=0)
        if o["idx"][0] >= 0:
            assert g["w"].max() == np.float32(1.0)
        if self.oracle_store:
            for f in FIELDS:
                a, b = np.ascontiguousarray(o[f]).view(np.uint8), np.ascontiguousarray(g[f]).view(np.uint8)
                assert np.array_equal(a.reshape(-1), b.reshape(-1)), "gathered %s differs" % f

    def update(self, idx, td, alpha, eps, host_call=False):
        assert self.ora.update(idx, td, alpha, eps) == 0
        if host_call:
            self.gpu.update_host(np.ascontiguousarray(idx, np.int32), np.ascontiguousarray(td, np.float32), alpha, eps)
        else:
            self.gpu.update(torch.from_numpy(np.ascontiguousarray(idx, np.int32)).to(self.dev),
                            torch.from_numpy(np.ascontiguousarray(td, np.float32)).to(self.dev), alpha, eps)

    def update_insert(self, idx, td, alpha, eps, batch):
        """One fused launch on the GPU; update then insert on the oracle."""
        assert self.ora.update(idx, td, alpha, eps) == 0
        assert self.ora.insert(batch.get("obs"), batch.get("act"), batch.get("rew"), batch.get("next_obs"),
                               batch.get("done"), batch["prio"]) == 0
        d = {k: torch.from_numpy(np.ascontiguousarray(v)).to(self.dev) for k, v in batch.items() if v is not None}
        self.gpu.update_insert(torch.from_numpy(np.ascontiguousarray(idx, np.int32)).to(self.dev),
                               torch.from_numpy(np.ascontiguousarray(td, np.float32)).to(self.dev), alpha, eps,
                               d.get("obs"), d.get("act"), d.get("rew"), d.get("next_obs"), d.get("done"), d["prio"])

    def step(self, idx, td, alpha, eps, batch, B, beta, seed, check=True):
        """pearl_prb_step on the GPU; update, insert, sample on the oracle.  Returns both sides' samples."""
        assert self.ora.update(idx, td, alpha, eps) == 0
        assert self.ora.insert(batch.get("obs"), batch.get("act"), batch.get("rew"), batch.get("next_obs"),
                               batch.get("done"), batch["prio"]) == 0
        o = self.ora.sample(B, beta, seed, gather=self.oracle_store)
        d = {k: torch.from_numpy(np.ascontiguousarray(v)).to(self.dev) for k, v in batch.items() if v is not None}
        t = {"idx": torch.full((B,), -1, dtype=torch.int32, device=self.dev),
             "w": torch.zeros(B, dtype=torch.float32, device=self.dev),
             "obs": torch.zeros((B, self.obs_bytes), dtype=torch.uint8, device=self.dev),
             "act": torch.zeros((B, self.act_bytes), dtype=torch.uint8, device=self.dev),
             "rew": torch.zeros(B, dtype=torch.float32, device=self.dev),
             "next_obs": torch.zeros((B, self.obs_bytes), dtype=torch.uint8, device=self.dev),
             "done": torch.zeros(B, dtype=torch.uint8, device=self.dev)}
        self.gpu.step(torch.from_numpy(np.ascontiguousarray(idx, np.int32)).to(self.dev),
                      torch.from_numpy(np.ascontiguousarray(td, np.float32)).to(self.dev), alpha, eps,
                      d.get("obs"), d.get("act"), d.get("rew"), d.get("next_obs"), d.get("done"), d["prio"],
                      B, beta, seed, t["idx"], t["w"], t["obs"], t["act"], t["rew"], t["next_obs"], t["done"])
        torch.cuda.synchronize()
        g = {k: v.cpu().numpy() for k, v in t.items()}
        if check:
            self.compare_sample(o, g)
        return o, g

    def update_after_insert(self, idx, td, alpha, eps, inserted):
        assert self.ora.update_after_insert(idx, td, alpha, eps, inserted) == 0
        self.gpu.update_after_insert(torch.from_numpy(np.ascontiguousarray(idx, np.int32)).to(self.dev),
                                     torch.from_numpy(np.ascontiguousarray(td, np.float32)).to(self.dev), alpha, eps,
                                     inserted)

    def compare_priorities(self, idx):
        idx = np.ascontiguousarray(idx, np.int32)
        out = torch.full((idx.shape[0],), -1.0, dtype=torch.float32, device=self.dev)
        self.gpu.get_priorities(torch.from_numpy(idx).to(self.dev), out)
        assert np.array_equal(out.cpu().numpy().view(np.uint32), self.ora.get_priorities(idx).view(np.uint32))

    def update_priorities(self, idx, prio):
        assert self.ora.update_priorities(idx, prio) == 0
        self.gpu.update_priorities(torch.from_numpy(np.ascontiguousarray(idx, np.int32)).to(self.dev),
                                   torch.from_numpy(np.ascontiguousarray(prio, np.float32)).to(self.dev))

    def update_delta(self, idx, delta):
        assert self.ora.update_delta(idx, delta) == 0
        self.gpu.update_delta(torch.from_numpy(np.ascontiguousarray(idx, np.int32)).to(self.dev),
                              torch.from_numpy(np.ascontiguousarray(delta, np.float32)).to(self.dev))

    # ---- comparisons ------------------------------------------------------------------
    def compare_tree(self, levels=None):
        D = self.ora.depth
        for l in (range(D + 1) if levels is None else levels):
            a, b = self.ora.read_level(l), self.gpu.read_level(l)
            assert a.shape == b.shape
            if not np.array_equal(bits(a), bits(b)):
                bad = np.nonzero(bits(a) != bits(b))[0]
                raise AssertionError("tree level %d differs at %d entries, first %d: oracle %r gpu %r"
                                     % (l, bad.size, bad[0], a[bad[0]], b[bad[0]]))

    def compare_min_tree(self):
        """Every node of the GPU's min-tree against its definition, written out on the ORACLE's leaves: the
        smallest positive leaf among the fanout^(depth-l) leaves below node (l, a), 0 if none is positive."""
        D, K = self.ora.depth, self.fanout
        leaves = self.ora.read_level(D)
        for l in range(D):
            span = K ** (D - l)
            n = self.gpu.level_alloc(l)
            padded = np.zeros(n * span, np.float32)
            m = min(leaves.size, padded.size)
            padded[:m] = leaves[:m]
            grouped = np.where(padded > 0, padded, np.float32(np.inf)).reshape(n, span).min(axis=1)
            want = np.where(np.isinf(grouped), np.float32(0), grouped).astype(np.float32)
            got = self.gpu.read_min_level(l)
            if not np.array_equal(bits(want), bits(got)):
                bad = np.nonzero(bits(want) != bits(got))[0]
                raise AssertionError("min-tree level %d differs at %d nodes, first %d: expected %r gpu %r"
                                     % (l, bad.size, bad[0], want[bad[0]], got[bad[0]]))

    def compare_state(self):
        assert self.gpu.info() == self.ora.info()
        assert np.float32(self.gpu.max_priority()) == self.ora.max_priority()

    def compare_status(self):
        s_g, s_o = self.gpu.sync(), self.ora.status()
        assert s_g == s_o, "status bits differ: gpu %d oracle %d" % (s_g, s_o)
        return s_g

    def compare_rows(self, idx):
        a, b = self.ora.read_rows(idx), self.gpu.read_rows(idx)
        for f in FIELDS:
            assert np.array_equal(np.ascontiguousarray(a[f]).view(np.uint8).reshape(-1),
                                  np.ascontiguousarray(b[f]).view(np.uint8).reshape(-1)), f
