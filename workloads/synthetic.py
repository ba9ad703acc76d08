"""Seeded synthetic inputs shaped like Llama-3.1-8B / Qwen2.5-7B decode attention.

This module serves BOTH the CUDA path's tests/benchmark and the CPU oracle, and
therefore holds none of the method's arithmetic: it only draws tensors.  The
inputs stand in for the long-generation benchmarks the Moment-KV paper measures
on (Sec. 5.1); no item of any benchmark is reproduced.  They imitate the two
phenomena of Sec. 3: persistent heavy hitters with temporary attention dips, and
attention concentrated on few tokens.

Recipe (per layer, per sequence b; every constant is a field of ``Workload``):
  * K, V of prefill and ordinary decode tokens: i.i.d. N(0,1)/sqrt(d).
  * queries: per query head an AR(1) process z_t = rho z_{t-1} + sqrt(1-rho^2) eps_t.
  * heavy hitters: per KV head ``n_heavy`` unit directions u_j (orthonormal; a
    single shared direction when ``shared_direction``).  Heavy hitter j is the
    decode token of step t_j = floor((j+1)(T/2)/(n_heavy+1)) and has key
    ``hh_scale * u_j``; the query of every head of that KV group gets
    ``c * sum_j on_j(t) u_j`` added, c = 2 sqrt(d).  ``on_j`` is always 1, or,
    when ``intermittent``, 1 for 50 steps and 0 for 20 starting at t_j.
  * variant "hot" (parity stress): queries scaled by tau = 2 sqrt(d) with a
    weaker heavy-hitter push (0.1 sqrt(d)), and each new key gets
    0.5 * qbar/|qbar| added (qbar = mean query of its group), so evictions are
    spread over all ages instead of always hitting the newest token.
  * values are drawn in fp64 and rounded ONCE to the workload dtype (bf16
    round-to-nearest-even, or fp32); both sides receive the same bits.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Tuple, Union

import numpy as np
from scipy.signal import lfilter


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round to the bf16 grid (nearest even); result returned as float64."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(np.float64)


def round_to(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return round_bf16(x)
    if dtype == "f32":
        return np.asarray(x, dtype=np.float32).astype(np.float64)
    raise ValueError(dtype)


@dataclass(frozen=True)
class Workload:
    name: str
    layers: int
    batch: int
    q_heads: int
    kv_heads: int
    head_dim: int
    dtype: str                      # "bf16" | "f32"
    prefill: Union[int, Tuple[int, int]]   # fixed length, or (lo, hi) uniform per sequence
    steps: int
    budget: int
    beta: float
    n_heavy: int
    intermittent: bool = True
    shared_direction: bool = False
    variant: str = "literal"        # "literal" | "hot"
    seed: int = 0
    rho: float = 0.95
    hh_scale: float = 3.0
    on_len: int = 50
    off_len: int = 20

    @property
    def group(self) -> int:
        return self.q_heads // self.kv_heads

    def prefill_lens(self) -> np.ndarray:
        if isinstance(self.prefill, int):
            return np.full(self.batch, self.prefill, dtype=np.int32)
        lo, hi = self.prefill
        rng = np.random.default_rng([self.seed, 9001])
        return rng.integers(lo, hi + 1, size=self.batch).astype(np.int32)

    def heavy_steps(self) -> np.ndarray:
        j = np.arange(self.n_heavy)
        return np.floor((j + 1) * (self.steps / 2.0) / (self.n_heavy + 1)).astype(np.int64)

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five configurations the build is measured and checked on.
CONFIGS = {
    "tiny": Workload("tiny", 1, 1, 4, 1, 64, "f32", 64, 512, 64, 0.9, 4,
                     intermittent=False, shared_direction=True, seed=0),
    "llama_b1": Workload("llama_b1", 1, 1, 32, 8, 128, "bf16", 1024, 4096, 512, 0.9, 16, seed=0),
    "llama_b16": Workload("llama_b16", 1, 16, 32, 8, 128, "bf16", (512, 4096), 8192, 1024, 0.9, 16, seed=0),
    "llama_stack": Workload("llama_stack", 32, 4, 32, 8, 128, "bf16", 2048, 32768, 2048, 0.9, 16, seed=0),
    "qwen_b64": Workload("qwen_b64", 1, 64, 28, 4, 128, "bf16", 512, 2048, 1024, 0.9, 16, seed=0),
}
QWEN_SWEEP_BUDGETS = (128, 256, 512, 1024, 2048)
QWEN_SWEEP_BETAS = (0.8, 0.9, 0.99)


class SequenceStream:
    """Inputs of one (layer, sequence): the prefill K/V once, then decode steps in order."""

    def __init__(self, w: Workload, layer: int, b: int, prefill_len: int | None = None):
        self.w, self.layer, self.b = w, layer, b
        self.Lp = int(w.prefill_lens()[b] if prefill_len is None else prefill_len)
        d = w.head_dim
        self._rng_p = np.random.default_rng([w.seed, layer, b, 0])
        # one generator per drawn tensor, so that the stream does not depend on how the
        # steps are split into next() calls
        self._rng_t = np.random.default_rng([w.seed, layer, b, 1])
        self._rng_k = np.random.default_rng([w.seed, layer, b, 3])
        self._rng_v = np.random.default_rng([w.seed, layer, b, 4])
        rng_u = np.random.default_rng([w.seed, layer, b, 2])
        # heavy-hitter directions u[g][j][d]
        if w.n_heavy > 0:
            if w.shared_direction:
                u0 = rng_u.standard_normal(d)
                u0 /= np.linalg.norm(u0)
                self.u = np.broadcast_to(u0, (w.kv_heads, w.n_heavy, d)).copy()
            else:
                self.u = np.empty((w.kv_heads, w.n_heavy, d))
                for g in range(w.kv_heads):
                    qm, _ = np.linalg.qr(rng_u.standard_normal((d, w.n_heavy)))
                    self.u[g] = qm.T
        else:
            self.u = np.zeros((w.kv_heads, 0, d))
        self.t_heavy = w.heavy_steps()
        self._z = self._rng_t.standard_normal((w.q_heads, d))
        self.t = 0

    def prefill(self):
        w = self.w
        shape = (w.kv_heads, self.Lp, w.head_dim)
        K = self._rng_p.standard_normal(shape) / np.sqrt(w.head_dim)
        V = self._rng_p.standard_normal(shape) / np.sqrt(w.head_dim)
        return round_to(K, w.dtype), round_to(V, w.dtype)

    def _on(self, t: np.ndarray) -> np.ndarray:
        """on[n_steps][n_heavy] in {0,1}."""
        w = self.w
        if w.n_heavy == 0:
            return np.zeros((t.shape[0], 0))
        if not w.intermittent:
            return np.ones((t.shape[0], w.n_heavy))
        dt = t[:, None] - self.t_heavy[None, :]
        period = w.on_len + w.off_len
        return ((dt >= 0) & ((dt % period) < w.on_len)).astype(np.float64)

    def next(self, n: int):
        """The next n decode steps: q [n,Hq,d], k_new [n,Hkv,d], v_new [n,Hkv,d]."""
        w = self.w
        d, G = w.head_dim, w.group
        sig = np.sqrt(1.0 - w.rho ** 2)
        eps = self._rng_t.standard_normal((n, w.q_heads, d))
        kk = self._rng_k.standard_normal((n, w.kv_heads, d)) / np.sqrt(d)
        vv = self._rng_v.standard_normal((n, w.kv_heads, d)) / np.sqrt(d)
        z, _ = lfilter([sig], [1.0, -w.rho], eps, axis=0, zi=(w.rho * self._z)[None])
        self._z = z[-1].copy()
        ts = np.arange(self.t, self.t + n)
        on = self._on(ts)                                  # [n, J]
        push = np.einsum("nj,gjd->ngd", on, self.u)        # [n, Hkv, d]
        push_q = np.repeat(push, G, axis=1)                # [n, Hq, d]
        if w.variant == "literal":
            q = z + 2.0 * np.sqrt(d) * push_q
        elif w.variant == "hot":
            q = 2.0 * np.sqrt(d) * (z + 0.1 * np.sqrt(d) * push_q)
            qbar = q.reshape(n, w.kv_heads, G, d).mean(axis=2)
            kk = kk + 0.5 * qbar / np.linalg.norm(qbar, axis=-1, keepdims=True)
        else:
            raise ValueError(w.variant)
        for j, tj in enumerate(self.t_heavy):
            if self.t <= tj < self.t + n:
                kk[tj - self.t] = w.hh_scale * self.u[:, j, :]
        self.t += n
        return round_to(q, w.dtype), round_to(kk, w.dtype), round_to(vv, w.dtype)


class BatchStream:
    """All sequences of one layer, stepped together; arrays are stacked over the batch."""

    def __init__(self, w: Workload, layer: int = 0, sequences=None):
        self.w = w
        self.ids = list(range(w.batch)) if sequences is None else list(sequences)
        self.streams = [SequenceStream(w, layer, b) for b in self.ids]
        self.lens = np.array([s.Lp for s in self.streams], dtype=np.int32)

    def prefill(self):
        """Returns lists (one entry per sequence) of K, V arrays [Hkv, Lp_b, d]."""
        ks, vs = zip(*(s.prefill() for s in self.streams))
        return list(ks), list(vs)

    def next(self, n: int):
        """q [n,B,Hq,d], k_new [n,B,Hkv,d], v_new [n,B,Hkv,d]."""
        qs, ks, vs = zip(*(s.next(n) for s in self.streams))
        return np.stack(qs, 1), np.stack(ks, 1), np.stack(vs, 1)
