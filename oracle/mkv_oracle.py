"""ctypes front-end of the fp64 Moment-KV oracle (``mkv_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the test-suite, by the smoke check and by
the benchmark's CPU-baseline leg.  The CUDA library never loads this module and
this module never loads the CUDA library.

The arithmetic lives in the C file, which follows Algorithm 1 of the Moment-KV
paper step by step; this file only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mkv_oracle.c")
_LIB = os.path.join(_HERE, "libmkv_oracle.so")

GROUP_MEAN = 0
LAYER_MEAN = 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math: fp64 IEEE arithmetic as written)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fPIC", "-shared", "-std=c99", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        dp, ip, lp = C.POINTER(C.c_double), C.POINTER(C.c_int), C.POINTER(C.c_int64)
        L.mko_create.restype = C.c_void_p
        L.mko_create.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_double, C.c_int, C.c_int]
        L.mko_destroy.argtypes = [C.c_void_p]
        L.mko_prefill.argtypes = [C.c_void_p, dp, dp]
        L.mko_set_budget.argtypes = [C.c_void_p, C.c_int]
        L.mko_load_decode_state.argtypes = [C.c_void_p, C.c_int, C.c_int, dp, dp, dp, lp, C.c_int64]
        L.mko_attend_update.argtypes = [C.c_void_p, dp, dp, dp, dp]
        L.mko_evict.argtypes = [C.c_void_p, lp, ip, C.c_int]
        L.mko_step.argtypes = [C.c_void_p, dp, dp, dp, dp]
        L.mko_select.argtypes = [dp, lp, C.c_int, C.c_int, ip]
        L.mko_update.argtypes = [dp, dp, C.c_int, C.c_double]
        L.mko_choose.argtypes = [C.c_void_p, C.c_int, lp, C.c_int]
        L.mko_decode_count.argtypes = [C.c_void_p, C.c_int]
        L.mko_steps_done.argtypes = [C.c_void_p]
        L.mko_steps_done.restype = C.c_int64
        L.mko_get_decode_state.argtypes = [C.c_void_p, C.c_int, lp, dp, dp, C.c_int]
        L.mko_get_last_evicted.argtypes = [C.c_void_p, C.c_int, lp, dp, C.c_int]
        L.mko_read_decode_kv.argtypes = [C.c_void_p, C.c_int, dp, dp, C.c_int]
        _lib = L
    return _lib


def _d(a):
    return a.ctypes.data_as(C.POINTER(C.c_double))


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def select(score, pos, k):
    """Indices of the k lowest scores, ties to the smaller position id (Eq. 8 as a sort)."""
    score = _f64(score)
    n = score.shape[0]
    pos_a = np.arange(n, dtype=np.int64) if pos is None else np.ascontiguousarray(pos, dtype=np.int64)
    out = np.zeros(max(k, 1), dtype=np.int32)
    rc = lib().mko_select(_d(score), pos_a.ctypes.data_as(C.POINTER(C.c_int64)), n, k,
                          out.ctypes.data_as(C.POINTER(C.c_int)))
    if rc:
        raise ValueError("mko_select: bad k")
    return out[:k].copy()


def update(I, abar, beta):
    """Eq. 5 elementwise; returns the new importance vector."""
    I = _f64(I).copy()
    abar = _f64(abar)
    lib().mko_update(_d(I), _d(abar), I.shape[0], float(beta))
    return I


class OracleSequence:
    """Decode state of ONE sequence in ONE layer (sequences and layers are independent)."""

    def __init__(self, q_heads, kv_heads, head_dim, budget, beta, prefill_len, mode=GROUP_MEAN):
        self.Hq, self.Hkv, self.d, self.Lp = q_heads, kv_heads, head_dim, prefill_len
        self._h = lib().mko_create(q_heads, kv_heads, head_dim, budget, float(beta), prefill_len, mode)
        if not self._h:
            raise ValueError("mko_create: invalid arguments")

    def __del__(self):
        if getattr(self, "_h", None):
            lib().mko_destroy(self._h)
            self._h = None

    def prefill(self, K, V):
        K, V = _f64(K), _f64(V)
        assert K.shape == (self.Hkv, self.Lp, self.d) and V.shape == K.shape
        lib().mko_prefill(self._h, _d(K), _d(V))

    def set_budget(self, budget):
        lib().mko_set_budget(self._h, int(budget))

    def load_decode_state(self, g, K, V, score, pos, steps_done):
        """Puts KV head g's decode pool into the given state (a loader: no arithmetic)."""
        K, V, score = _f64(K), _f64(V), _f64(score)
        pos = np.ascontiguousarray(pos, dtype=np.int64)
        n = score.shape[0]
        assert K.shape == (n, self.d) and V.shape == (n, self.d) and pos.shape == (n,)
        rc = lib().mko_load_decode_state(self._h, g, n, _d(K), _d(V), _d(score),
                                         pos.ctypes.data_as(C.POINTER(C.c_int64)), int(steps_done))
        if rc:
            raise RuntimeError(f"mko_load_decode_state rc={rc}")

    def attend_update(self, q, k_new, v_new):
        q, k_new, v_new = _f64(q), _f64(k_new), _f64(v_new)
        assert q.shape == (self.Hq, self.d) and k_new.shape == (self.Hkv, self.d) and v_new.shape == k_new.shape
        out = np.empty((self.Hq, self.d), dtype=np.float64)
        rc = lib().mko_attend_update(self._h, _d(q), _d(k_new), _d(v_new), _d(out))
        if rc:
            raise RuntimeError(f"mko_attend_update rc={rc}")
        return out

    def choose(self, g):
        n = lib().mko_decode_count(self._h, g)
        buf = np.zeros(max(n, 1), dtype=np.int64)
        k = lib().mko_choose(self._h, g, buf.ctypes.data_as(C.POINTER(C.c_int64)), n)
        return buf[:k].copy()

    def evict(self, force=None):
        """force: None, or a list (one entry per KV head) of position-id arrays to evict."""
        if force is None:
            rc = lib().mko_evict(self._h, None, None, 0)
        else:
            stride = max(1, max(len(f) for f in force))
            fp = np.zeros((self.Hkv, stride), dtype=np.int64)
            fc = np.zeros(self.Hkv, dtype=np.int32)
            for g, f in enumerate(force):
                fp[g, :len(f)] = f
                fc[g] = len(f)
            rc = lib().mko_evict(self._h, fp.ctypes.data_as(C.POINTER(C.c_int64)),
                                 fc.ctypes.data_as(C.POINTER(C.c_int)), stride)
        if rc:
            raise RuntimeError(f"mko_evict rc={rc}")

    def step(self, q, k_new, v_new):
        out = self.attend_update(q, k_new, v_new)
        self.evict()
        return out

    def count(self, g):
        return lib().mko_decode_count(self._h, g)

    def steps_done(self):
        return lib().mko_steps_done(self._h)

    def decode_state(self, g):
        n = self.count(g)
        pos = np.zeros(max(n, 1), dtype=np.int64)
        sc = np.zeros(max(n, 1), dtype=np.float64)
        ab = np.zeros(max(n, 1), dtype=np.float64)
        lib().mko_get_decode_state(self._h, g, pos.ctypes.data_as(C.POINTER(C.c_int64)), _d(sc), _d(ab), n)
        return pos[:n].copy(), sc[:n].copy(), ab[:n].copy()

    def last_evicted(self, g):
        cap = self.count(g) + 4096
        pos = np.zeros(cap, dtype=np.int64)
        sc = np.zeros(cap, dtype=np.float64)
        k = lib().mko_get_last_evicted(self._h, g, pos.ctypes.data_as(C.POINTER(C.c_int64)), _d(sc), cap)
        if k < 0:
            raise RuntimeError("eviction record larger than buffer")
        return pos[:k].copy(), sc[:k].copy()

    def decode_kv(self, g):
        n = self.count(g)
        K = np.zeros((max(n, 1), self.d), dtype=np.float64)
        V = np.zeros_like(K)
        lib().mko_read_decode_kv(self._h, g, _d(K), _d(V), n)
        return K[:n].copy(), V[:n].copy()


class OracleBatch:
    """A batch of independent sequences; ``threads`` > 1 steps them concurrently
    (the C calls release the GIL), which changes no arithmetic."""

    def __init__(self, q_heads, kv_heads, head_dim, budget, beta, prefill_lens, mode=GROUP_MEAN, threads=1):
        self.seqs = [OracleSequence(q_heads, kv_heads, head_dim, budget, beta, int(lp), mode) for lp in prefill_lens]
        self.threads = max(1, int(threads))
        self._pool = ThreadPoolExecutor(self.threads) if self.threads > 1 else None

    def prefill(self, Ks, Vs):
        for s, K, V in zip(self.seqs, Ks, Vs):
            s.prefill(K, V)

    def step(self, q, k_new, v_new):
        """q [B,Hq,d], k_new/v_new [B,Hkv,d] -> out [B,Hq,d] (fp64)."""
        if self._pool is None:
            outs = [s.step(q[b], k_new[b], v_new[b]) for b, s in enumerate(self.seqs)]
        else:
            outs = list(self._pool.map(lambda b: self.seqs[b].step(q[b], k_new[b], v_new[b]), range(len(self.seqs))))
        return np.stack(outs)
