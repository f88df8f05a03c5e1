"""CPU oracle for the Prioritized Replay Buffer -- TEST INFRASTRUCTURE.

A ctypes wrapper around ``prb_oracle.c`` (plain single-threaded C, built with
``gcc -O2 -ffp-contract=off``).  Only the tests, the smoke check and the
benchmark's CPU-baseline leg use it; the CUDA library never does and the two
share no code.  All pointers handed to the C side are host numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "prb_oracle.c")
_LIB = os.path.join(_HERE, "libprb_oracle.so")

ST_BAD_INDEX, ST_BAD_PRIORITY, ST_EMPTY, ST_CLAMPED, ST_INTERNAL, ST_STALE = 1, 2, 4, 8, 16, 32


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
             "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, u32, u64, f32 = C.c_void_p, C.c_uint32, C.c_uint64, C.c_float
        L.oracle_prb_create.argtypes = [C.POINTER(vp), u64, u32, u32, u32]
        L.oracle_prb_create_frames.argtypes = [C.POINTER(vp), u64, u32, u32, u32, u32]
        L.oracle_prb_destroy.argtypes = [vp]
        L.oracle_prb_destroy.restype = None
        L.oracle_prb_rebuild.argtypes = [vp]
        L.oracle_prb_rebuild.restype = None
        L.oracle_prb_insert.argtypes = [vp, u32, vp, vp, vp, vp, vp, vp]
        L.oracle_prb_update_priorities.argtypes = [vp, u32, vp, vp]
        L.oracle_prb_update_delta.restype = C.c_int
        L.oracle_prb_update_delta.argtypes = [vp, u32, vp, vp]
        L.oracle_prb_update.argtypes = [vp, u32, vp, vp, f32, f32]
        L.oracle_prb_update_after_insert.argtypes = [vp, u32, vp, vp, f32, f32, u32]
        L.oracle_prb_get_priorities.argtypes = [vp, u32, vp, vp]
        L.oracle_prb_descend.argtypes = [vp, C.c_double, C.POINTER(f32)]
        L.oracle_prb_descend.restype = C.c_int64
        L.oracle_prb_targets.argtypes = [vp, u32, u64, u64, vp]
        L.oracle_prb_targets.restype = None
        L.oracle_prb_sample.argtypes = [vp, u32, f32, u64, vp, vp, vp, vp, vp, vp, vp]
        L.oracle_prb_sample_buffer_norm.restype = C.c_int
        L.oracle_prb_sample_buffer_norm.argtypes = [vp, u32, f32, u64, vp, vp, vp, vp, vp, vp, vp]
        L.oracle_prb_sample_uniform.argtypes = [vp, u32, u64, vp, vp, vp, vp, vp, vp, vp]
        L.oracle_prb_info.argtypes = [vp, C.POINTER(u64), C.POINTER(u64), C.POINTER(u64), C.POINTER(u32)]
        L.oracle_prb_level_nodes.argtypes = [vp, u32]
        L.oracle_prb_level_nodes.restype = u64
        L.oracle_prb_level_alloc.argtypes = [vp, u32]
        L.oracle_prb_level_alloc.restype = u64
        L.oracle_prb_read_level.argtypes = [vp, u32, vp, u64]
        L.oracle_prb_poke_level.argtypes = [vp, u32, u64, vp, u64]
        L.oracle_prb_read_rows.argtypes = [vp, vp, u32, vp, vp, vp, vp, vp]
        L.oracle_prb_max_priority.argtypes = [vp]
        L.oracle_prb_max_priority.restype = f32
        L.oracle_prb_status.argtypes = [vp]
        L.oracle_prb_status.restype = u32
        L.oracle_philox4x32_10.argtypes = [vp, vp, vp]
        L.oracle_philox4x32_10.restype = None
        L.oracle_stratum_uniform.argtypes = [u64, u64, u32]
        L.oracle_stratum_uniform.restype = C.c_double
        L.oracle_priority_pow.argtypes = [f32, f32, f32, C.POINTER(f32)]
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _host(a, dtype=None):
    if a is None:
        return None
    a = np.ascontiguousarray(a) if dtype is None else np.ascontiguousarray(a, dtype=dtype)
    return a


def philox4x32_10(counter, key) -> np.ndarray:
    c = np.ascontiguousarray(counter, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def stratum_uniform(seed: int, call: int, k: int) -> float:
    return float(lib().oracle_stratum_uniform(seed, call, k))


def priority_pow(delta: float, eps: float, alpha: float):
    """Returns the binary32 priority as a numpy float32, or None for an invalid entry."""
    p = C.c_float(0.0)
    bad = lib().oracle_priority_pow(float(np.float32(delta)), float(np.float32(eps)),
                                    float(np.float32(alpha)), C.byref(p))
    return None if bad else np.float32(p.value)


class OraclePRB:
    """The oracle buffer.  Methods mirror the product's C-ABI calls, with host arrays."""

    def __init__(self, capacity: int, fanout: int, obs_bytes: int, act_bytes: int, frame_stack: int = 0):
        """frame_stack > 0: the frame-deduplicated layout; obs_bytes is then the size of a whole stack
        (frame_stack frames) and insert takes one frame per transition in `obs`."""
        self._h = C.c_void_p()
        if frame_stack:
            assert obs_bytes % frame_stack == 0
            rc = lib().oracle_prb_create_frames(C.byref(self._h), capacity, fanout, obs_bytes // frame_stack, frame_stack, act_bytes)
        else:
            rc = lib().oracle_prb_create(C.byref(self._h), capacity, fanout, obs_bytes, act_bytes)
        if rc != 0:
            raise ValueError("oracle_prb_create failed: %d" % rc)
        self.capacity, self.fanout = capacity, fanout
        self.obs_bytes, self.act_bytes = obs_bytes, act_bytes
        self.frame_stack = frame_stack
        _, _, _, self.depth = self.info()

    def close(self):
        if self._h:
            lib().oracle_prb_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- mutation -----------------------------------------------------------
    def insert(self, obs, act, rew, next_obs, done, prio, n=None) -> int:
        """prio=None (with n given): every new transition gets the largest priority written so far."""
        prio = _host(prio, np.float32)
        n = prio.shape[0] if prio is not None else int(n)
        obs, act, next_obs = _host(obs), _host(act), _host(next_obs)
        rew, done = _host(rew, np.float32), _host(done, np.uint8)
        return lib().oracle_prb_insert(self._h, n, _ptr(obs), _ptr(act), _ptr(rew), _ptr(next_obs),
                                       _ptr(done), _ptr(prio))

    def update(self, idx, td, alpha: float, eps: float) -> int:
        idx, td = _host(idx, np.int32), _host(td, np.float32)
        return lib().oracle_prb_update(self._h, idx.shape[0], _ptr(idx), _ptr(td), alpha, eps)

    def update_after_insert(self, idx, td, alpha: float, eps: float, inserted: int) -> int:
        idx, td = _host(idx, np.int32), _host(td, np.float32)
        return lib().oracle_prb_update_after_insert(self._h, idx.shape[0], _ptr(idx), _ptr(td), alpha, eps, inserted)

    def get_priorities(self, idx) -> np.ndarray:
        idx = _host(idx, np.int32)
        out = np.zeros(idx.shape[0], dtype=np.float32)
        rc = lib().oracle_prb_get_priorities(self._h, idx.shape[0], _ptr(idx), _ptr(out))
        assert rc == 0
        return out

    def update_priorities(self, idx, prio) -> int:
        idx, prio = _host(idx, np.int32), _host(prio, np.float32)
        return lib().oracle_prb_update_priorities(self._h, idx.shape[0], _ptr(idx), _ptr(prio))

    def update_delta(self, idx, delta) -> int:
        idx, delta = _host(idx, np.int32), _host(delta, np.float32)
        return lib().oracle_prb_update_delta(self._h, idx.shape[0], _ptr(idx), _ptr(delta))

    def max_priority(self) -> np.float32:
        return np.float32(lib().oracle_prb_max_priority(self._h))

    def rebuild(self):
        lib().oracle_prb_rebuild(self._h)

    # -- sampling -----------------------------------------------------------
    def descend(self, x: float):
        p = C.c_float(0.0)
        i = lib().oracle_prb_descend(self._h, float(x), C.byref(p))
        return int(i), np.float32(p.value)

    def targets(self, B: int, seed: int, call: int) -> np.ndarray:
        x = np.zeros(B, dtype=np.float64)
        lib().oracle_prb_targets(self._h, B, seed, call, _ptr(x))
        return x

    def sample_uniform(self, B: int, seed: int):
        out = {"idx": np.full(B, -1, dtype=np.int32), "w": np.zeros(B, dtype=np.float32),
               "obs": np.zeros((B, self.obs_bytes), dtype=np.uint8), "act": np.zeros((B, self.act_bytes), dtype=np.uint8),
               "rew": np.zeros(B, dtype=np.float32), "next_obs": np.zeros((B, self.obs_bytes), dtype=np.uint8),
               "done": np.zeros(B, dtype=np.uint8)}
        out["rc"] = lib().oracle_prb_sample_uniform(self._h, B, seed, _ptr(out["idx"]), _ptr(out["w"]), _ptr(out["obs"]),
                                                    _ptr(out["act"]), _ptr(out["rew"]), _ptr(out["next_obs"]),
                                                    _ptr(out["done"]))
        return out

    def sample(self, B: int, beta: float, seed: int, gather: bool = True, buffer_norm: bool = False):
        """Returns a dict with idx, w and (if ``gather``) the gathered fields as raw bytes / f32.
        buffer_norm: weights divided by the largest weight in the whole buffer instead of the batch."""
        out = {
            "idx": np.full(B, -1, dtype=np.int32),
            "w": np.zeros(B, dtype=np.float32),
        }
        if gather:
            out["obs"] = np.zeros((B, self.obs_bytes), dtype=np.uint8)
            out["act"] = np.zeros((B, self.act_bytes), dtype=np.uint8)
            out["rew"] = np.zeros(B, dtype=np.float32)
            out["next_obs"] = np.zeros((B, self.obs_bytes), dtype=np.uint8)
            out["done"] = np.zeros(B, dtype=np.uint8)
        fn = lib().oracle_prb_sample_buffer_norm if buffer_norm else lib().oracle_prb_sample
        rc = fn(self._h, B, beta, seed, _ptr(out["idx"]), _ptr(out["w"]),
                _ptr(out.get("obs")), _ptr(out.get("act")), _ptr(out.get("rew")),
                _ptr(out.get("next_obs")), _ptr(out.get("done")))
        out["rc"] = rc
        return out

    # -- read-back ----------------------------------------------------------
    def info(self):
        s, c, n, d = C.c_uint64(), C.c_uint64(), C.c_uint64(), C.c_uint32()
        lib().oracle_prb_info(self._h, C.byref(s), C.byref(c), C.byref(n), C.byref(d))
        return s.value, c.value, n.value, d.value

    def level_nodes(self, level: int) -> int:
        return int(lib().oracle_prb_level_nodes(self._h, level))

    def level_alloc(self, level: int) -> int:
        return int(lib().oracle_prb_level_alloc(self._h, level))

    def read_level(self, level: int, padded: bool = True) -> np.ndarray:
        n = self.level_alloc(level) if padded else self.level_nodes(level)
        a = np.zeros(n, dtype=np.float32)
        rc = lib().oracle_prb_read_level(self._h, level, _ptr(a), n)
        assert rc == 0
        return a

    def poke_level(self, level: int, first: int, values) -> int:
        v = _host(values, np.float32)
        return lib().oracle_prb_poke_level(self._h, level, first, _ptr(v), v.shape[0])

    def total(self) -> np.float32:
        return self.read_level(0)[0]

    def read_rows(self, idx):
        idx = _host(idx, np.int32)
        n = idx.shape[0]
        out = {
            "obs": np.zeros((n, self.obs_bytes), dtype=np.uint8),
            "act": np.zeros((n, self.act_bytes), dtype=np.uint8),
            "rew": np.zeros(n, dtype=np.float32),
            "next_obs": np.zeros((n, self.obs_bytes), dtype=np.uint8),
            "done": np.zeros(n, dtype=np.uint8),
        }
        rc = lib().oracle_prb_read_rows(self._h, _ptr(idx), n, _ptr(out["obs"]), _ptr(out["act"]),
                                        _ptr(out["rew"]), _ptr(out["next_obs"]), _ptr(out["done"]))
        assert rc == 0
        return out

    def status(self) -> int:
        return int(lib().oracle_prb_status(self._h))
