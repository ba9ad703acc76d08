"""ctypes binding of libmkv.so.  Same names as the C ABI (``include/mkv.h``); this file
only marshals arguments -- torch provides device memory and streams, every step of the
method runs in the library's CUDA kernels.  If the library is missing or has no usable
GPU the calls raise: there is no fallback of any kind."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

MKV_BF16, MKV_F32 = 0, 1
MKV_SCORE_GROUP_MEAN, MKV_SCORE_LAYER_MEAN = 0, 1
MKV_KERNEL_AUTO, MKV_KERNEL_SIMT, MKV_KERNEL_MMA = 0, 1, 2
MKV_FLAG_RECORD_PROBS, MKV_FLAG_INPUTS_READY, MKV_FLAG_REPRODUCIBLE = 1, 2, 4
MKV_OPT_RING_STAGES, MKV_OPT_HEAD_TILES, MKV_OPT_WAIT_LIMIT_US, MKV_OPT_OVERLAP, MKV_OPT_GRID_SHARE = 1, 2, 3, 4, 5
MKV_INJECT_LOST_TILE = 0

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmkv.so")

EXPORTED_SYMBOLS = [
    "mkv_workspace_bytes", "mkv_kv_bytes_per_token", "mkv_create", "mkv_destroy", "mkv_prefill",
    "mkv_decode_step", "mkv_decode_step_host", "mkv_attend_only", "mkv_set_budget", "mkv_reset",
    "mkv_status_sync", "mkv_launch_count", "mkv_get_decode_state", "mkv_get_last_evicted",
    "mkv_get_last_probs", "mkv_read_kv", "mkv_get_step", "mkv_status_string", "mkv_attend_noalloc", "mkv_plan_starts", "mkv_prefill_units",
    "mkv_recency_diagnostics", "mkv_set_option", "mkv_plan_ranges", "mkv_grid_limit", "mkv_decode_step_layers",
    "mkv_attend_only_layers", "mkv_get_grid", "mkv_debug_inject",
]


class MkvError(RuntimeError):
    def __init__(self, code, where):
        self.code = int(code)
        super().__init__(f"{where}: {status_string(code)} (mkv_status {int(code)})")


_lib = None


def load_library(path: str | None = None):
    """Loads libmkv.so (built in-tree by ``build.py``).  Raises if it is not there."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(f"{p} not found: build it with `python -m paper_2605_29873_b200.build`")
    L = C.CDLL(p)
    vp, i32p, f32p = C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_float)
    L.mkv_workspace_bytes.restype = C.c_size_t
    L.mkv_workspace_bytes.argtypes = [C.c_int] * 9
    L.mkv_kv_bytes_per_token.restype = C.c_size_t
    L.mkv_kv_bytes_per_token.argtypes = [C.c_int] * 4
    L.mkv_create.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, C.c_int, C.c_int, C.c_int,
                             C.c_int, C.c_int, C.c_int, C.c_uint, vp, C.c_size_t, C.c_int, C.POINTER(vp)]
    L.mkv_destroy.restype = None
    L.mkv_destroy.argtypes = [vp]
    L.mkv_prefill.argtypes = [vp, C.c_int, vp, vp, i32p, C.c_int, vp]
    L.mkv_prefill_units.argtypes = [vp, C.c_int, vp, vp, i32p, C.c_int, vp]
    L.mkv_decode_step.argtypes = [vp, C.c_int, vp, vp, vp, vp, vp]
    L.mkv_decode_step_host.argtypes = [vp, C.c_int, vp, vp, vp, vp, vp]
    L.mkv_attend_only.argtypes = [vp, C.c_int, vp, vp, vp]
    L.mkv_set_budget.argtypes = [vp, C.c_int]
    L.mkv_reset.argtypes = [vp]
    L.mkv_status_sync.argtypes = [vp, vp]
    L.mkv_launch_count.restype = C.c_int64
    L.mkv_launch_count.argtypes = [vp]
    L.mkv_get_decode_state.argtypes = [vp, C.c_int, C.c_int, C.c_int, i32p, i32p, f32p, C.c_int]
    L.mkv_get_last_evicted.argtypes = [vp, C.c_int, C.c_int, C.c_int, i32p, i32p, f32p, C.c_int]
    L.mkv_get_last_probs.argtypes = [vp, C.c_int, C.c_int, C.c_int, i32p, f32p, i32p, C.c_int]
    L.mkv_recency_diagnostics.argtypes = [vp, C.c_int, C.c_int, vp, vp, vp, vp]
    L.mkv_read_kv.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int, i32p, vp, vp, C.c_int]
    L.mkv_get_step.argtypes = [vp, C.c_int, C.POINTER(C.c_int64)]
    L.mkv_attend_noalloc.argtypes = [vp, vp, vp, vp] + [C.c_int] * 9 + [vp]
    L.mkv_plan_starts.argtypes = [C.c_int, C.c_int, C.c_int, i32p, C.c_int, C.c_int, i32p, i32p, i32p, i32p, i32p, i32p]
    L.mkv_plan_ranges.argtypes = [C.c_int, C.c_int, C.c_int, i32p, C.c_int, i32p, i32p, i32p, i32p]
    L.mkv_grid_limit.restype = C.c_int
    L.mkv_grid_limit.argtypes = [C.c_int, C.c_int, C.c_int]
    L.mkv_set_option.argtypes = [vp, C.c_int, C.c_longlong]
    L.mkv_decode_step_layers.argtypes = [vp, C.c_int, C.c_int, vp, vp, vp, vp, vp]
    L.mkv_attend_only_layers.argtypes = [vp, C.c_int, C.c_int, vp, vp, vp]
    L.mkv_get_grid.argtypes = [vp, C.c_int, i32p, i32p]
    L.mkv_debug_inject.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int]
    L.mkv_status_string.restype = C.c_char_p
    L.mkv_status_string.argtypes = [C.c_int]
    if path is None:
        _lib = L
    return L


def status_string(code) -> str:
    return load_library().mkv_status_string(int(code)).decode()


def workspace_bytes(layers, batch, q_heads, kv_heads, head_dim, budget, max_prefill, kv_dtype=MKV_BF16,
                    score_mode=MKV_SCORE_GROUP_MEAN) -> int:
    return int(load_library().mkv_workspace_bytes(layers, batch, q_heads, kv_heads, head_dim, budget, max_prefill,
                                                  kv_dtype, score_mode))


def kv_bytes_per_token(layers, kv_heads, head_dim, kv_dtype=MKV_BF16) -> int:
    return int(load_library().mkv_kv_bytes_per_token(layers, kv_heads, head_dim, kv_dtype))


def attend_noalloc(q, K, V, out, n_tokens, stream=None):
    """Plain decode attention without context or workspace (``mkv_attend_noalloc``): for
    callers that may not allocate device memory.  q [B,Hq,d], K/V [B,Hkv,rows,d], out
    [B,Hq,d] are device tensors; every sequence attends rows [0, n_tokens).  Calls share a
    scratch array built into the library, so calls on different streams must not overlap."""
    import torch
    B, Hq, d = q.shape
    Hkv, rows = K.shape[1], K.shape[2]
    assert q.is_contiguous() and K.is_contiguous() and V.is_contiguous() and out.is_contiguous()
    assert tuple(K.shape) == (B, Hkv, rows, d) == tuple(V.shape) and tuple(out.shape) == (B, Hq, d)
    assert q.dtype == K.dtype == V.dtype
    kv = MKV_BF16 if q.dtype == torch.bfloat16 else MKV_F32
    od = MKV_BF16 if out.dtype == torch.bfloat16 else MKV_F32
    st = stream if stream is not None else torch.cuda.current_stream(q.device)
    _check(load_library().mkv_attend_noalloc(_ptr(q), _ptr(K), _ptr(V), _ptr(out), B, Hq, Hkv, d, int(n_tokens),
                                             rows, kv, od, q.device.index or 0, C.c_void_p(st.cuda_stream)),
           "mkv_attend_noalloc")


def grid_limit(sm_count, resident_per_sm, wanted_per_sm) -> int:
    return int(load_library().mkv_grid_limit(sm_count, resident_per_sm, wanted_per_sm))


def plan_ranges(batch, kv_heads, budget, prefill_lens, n_ctas_max):
    """The table of the reproducible mode (``mkv_plan_ranges``; host arithmetic only).
    Returns (cta_t0 [n_ctas+1], tile_begin [units+1], unit_cta0 [units]) as int32 arrays."""
    lens = np.ascontiguousarray(prefill_lens, dtype=np.int32)
    assert lens.shape == (batch,)
    n = C.c_int32(0)
    t0 = np.zeros(n_ctas_max + 1, dtype=np.int32)
    tb = np.zeros(batch * kv_heads + 1, dtype=np.int32)
    uc = np.zeros(batch * kv_heads, dtype=np.int32)
    p = lambda a: a.ctypes.data_as(C.POINTER(C.c_int32))
    _check(load_library().mkv_plan_ranges(batch, kv_heads, budget, p(lens), n_ctas_max, C.byref(n), p(t0), p(tb), p(uc)),
           "mkv_plan_ranges")
    return t0[: n.value + 1].copy(), tb, uc


def plan_starts(batch, kv_heads, budget, prefill_lens, n_ctas_max, head_tiles=3):
    """The kernels' start table for these lengths (``mkv_plan_starts``; host arithmetic only).
    Returns (cta_unit0, cta_head0, cta_headn, unit_next0, unit_chunk) as int32 arrays."""
    lens = np.ascontiguousarray(prefill_lens, dtype=np.int32)
    assert lens.shape == (batch,)
    n = C.c_int32(0)
    u0, h0, hn = (np.zeros(n_ctas_max, dtype=np.int32) for _ in range(3))
    nx = np.zeros(batch * kv_heads, dtype=np.int32)
    ch = np.zeros(batch * kv_heads, dtype=np.int32)
    p = lambda a: a.ctypes.data_as(C.POINTER(C.c_int32))
    _check(load_library().mkv_plan_starts(batch, kv_heads, budget, p(lens), n_ctas_max, head_tiles, C.byref(n), p(u0),
                                          p(h0), p(hn), p(nx), p(ch)), "mkv_plan_starts")
    return u0[: n.value].copy(), h0[: n.value].copy(), hn[: n.value].copy(), nx, ch


def _check(code, where):
    if code != 0:
        raise MkvError(code, where)


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p(0)


class MomentKV:
    """One mkv context plus the torch tensor that backs its workspace."""

    def __init__(self, layers, q_heads, kv_heads, head_dim, budget, beta, batch, max_prefill, kv_dtype=MKV_BF16,
                 out_dtype=None, score_mode=MKV_SCORE_GROUP_MEAN, kernel=MKV_KERNEL_AUTO, flags=0, device=0):
        import torch

        self._L = load_library()
        self._ctx = C.c_void_p(0)
        if not torch.cuda.is_available():
            raise RuntimeError("MomentKV needs a CUDA device: the decode path has no CPU implementation")
        self.torch = torch
        self.layers, self.q_heads, self.kv_heads, self.head_dim = layers, q_heads, kv_heads, head_dim
        self.batch, self.budget, self.beta, self.max_prefill = batch, budget, beta, max_prefill
        self.budget_max = budget
        self.kv_dtype = kv_dtype
        self.out_dtype = kv_dtype if out_dtype is None else out_dtype
        self.device = torch.device("cuda", device)
        nbytes = workspace_bytes(layers, batch, q_heads, kv_heads, head_dim, budget, max_prefill, kv_dtype, score_mode)
        if nbytes == 0:
            raise MkvError(1, "mkv_workspace_bytes")
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        off = (-self.workspace.data_ptr()) % 256
        self._ws_ptr = self.workspace.data_ptr() + off
        self.workspace_bytes = nbytes
        torch.cuda.synchronize(self.device)
        ctx = C.c_void_p(0)
        _check(self._L.mkv_create(layers, q_heads, kv_heads, head_dim, budget, float(beta), batch, max_prefill,
                                  kv_dtype, self.out_dtype, score_mode, kernel, flags, C.c_void_p(self._ws_ptr),
                                  nbytes, device, C.byref(ctx)), "mkv_create")
        self._ctx = ctx

    # -- lifetime
    def close(self):
        if getattr(self, "_ctx", None) is not None and self._ctx.value:
            self._L.mkv_destroy(self._ctx)
            self._ctx = C.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _stream(self, stream):
        if stream is None:
            stream = self.torch.cuda.current_stream(self.device)
        return C.c_void_p(stream.cuda_stream)

    def torch_kv_dtype(self):
        return self.torch.bfloat16 if self.kv_dtype == MKV_BF16 else self.torch.float32

    def torch_out_dtype(self):
        return self.torch.bfloat16 if self.out_dtype == MKV_BF16 else self.torch.float32

    # -- the calls of the C ABI
    def prefill(self, layer, K, V, prefill_lens, stream=None):
        """K, V: device tensors [batch, kv_heads, src_rows, head_dim] (kv dtype); prefill_lens: ints."""
        lens = np.ascontiguousarray(prefill_lens, dtype=np.int32)
        assert lens.shape == (self.batch,)
        src_rows = int(K.shape[2]) if K is not None else 0
        if K is not None:
            assert K.is_contiguous() and V.is_contiguous() and K.dtype == self.torch_kv_dtype()
            assert tuple(K.shape) == (self.batch, self.kv_heads, src_rows, self.head_dim) == tuple(V.shape)
        _check(self._L.mkv_prefill(self._ctx, layer, _ptr(K), _ptr(V), lens.ctypes.data_as(C.POINTER(C.c_int32)),
                                   src_rows, self._stream(stream)), "mkv_prefill")

    def prefill_units(self, layer, K, V, unit_lens, stream=None):
        """As prefill, with one length per (sequence, KV head): unit_lens [batch, kv_heads] ints."""
        lens = np.ascontiguousarray(unit_lens, dtype=np.int32).reshape(-1)
        assert lens.shape == (self.batch * self.kv_heads,)
        src_rows = int(K.shape[2])
        assert K.is_contiguous() and V.is_contiguous() and K.dtype == self.torch_kv_dtype()
        assert tuple(K.shape) == (self.batch, self.kv_heads, src_rows, self.head_dim) == tuple(V.shape)
        _check(self._L.mkv_prefill_units(self._ctx, layer, _ptr(K), _ptr(V), lens.ctypes.data_as(C.POINTER(C.c_int32)),
                                         src_rows, self._stream(stream)), "mkv_prefill_units")

    def decode_step(self, layer, q, k_new, v_new, out, stream=None):
        _check(self._L.mkv_decode_step(self._ctx, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out),
                                       self._stream(stream)), "mkv_decode_step")

    def decode_step_host(self, layer, q, k_new, v_new, out, stream=None):
        """Same with (pinned) host tensors."""
        _check(self._L.mkv_decode_step_host(self._ctx, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out),
                                            self._stream(stream)), "mkv_decode_step_host")

    def attend_only(self, layer, q, out, stream=None):
        _check(self._L.mkv_attend_only(self._ctx, layer, _ptr(q), _ptr(out), self._stream(stream)), "mkv_attend_only")

    def decode_step_layers(self, layer0, n_layers, q, k_new, v_new, out, stream=None):
        """One launch for layers [layer0, layer0 + n_layers); tensors stacked by layer in front."""
        _check(self._L.mkv_decode_step_layers(self._ctx, layer0, n_layers, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out),
                                              self._stream(stream)), "mkv_decode_step_layers")

    def attend_only_layers(self, layer0, n_layers, q, out, stream=None):
        _check(self._L.mkv_attend_only_layers(self._ctx, layer0, n_layers, _ptr(q), _ptr(out), self._stream(stream)),
               "mkv_attend_only_layers")

    def set_option(self, option, value):
        _check(self._L.mkv_set_option(self._ctx, int(option), int(value)), "mkv_set_option")

    def grid(self, layer):
        """(CTAs of the layer's launches, the bound the grid was sized under)."""
        n, nmax = C.c_int32(0), C.c_int32(0)
        _check(self._L.mkv_get_grid(self._ctx, layer, C.byref(n), C.byref(nmax)), "mkv_get_grid")
        return int(n.value), int(nmax.value)

    def debug_inject(self, layer, what, b=0, g=0):
        _check(self._L.mkv_debug_inject(self._ctx, layer, what, b, g), "mkv_debug_inject")

    def set_budget(self, budget):
        _check(self._L.mkv_set_budget(self._ctx, int(budget)), "mkv_set_budget")
        self.budget = int(budget)

    def reset(self):
        _check(self._L.mkv_reset(self._ctx), "mkv_reset")

    def status_sync(self, stream=None):
        _check(self._L.mkv_status_sync(self._ctx, self._stream(stream)), "mkv_status_sync")

    def launch_count(self) -> int:
        return int(self._L.mkv_launch_count(self._ctx))

    # -- inspection
    def decode_state(self, layer, b, g):
        cap = self.budget_cap()
        n = C.c_int32(0)
        pos = np.zeros(cap, dtype=np.int32)
        sc = np.zeros(cap, dtype=np.float32)
        _check(self._L.mkv_get_decode_state(self._ctx, layer, b, g, C.byref(n), pos.ctypes.data_as(C.POINTER(C.c_int32)),
                                            sc.ctypes.data_as(C.POINTER(C.c_float)), cap), "mkv_get_decode_state")
        return pos[: n.value].copy(), sc[: n.value].copy()

    def last_evicted(self, layer, b, g):
        cap = self.budget_cap()
        k = C.c_int32(0)
        pos = np.zeros(cap, dtype=np.int32)
        sc = np.zeros(cap, dtype=np.float32)
        _check(self._L.mkv_get_last_evicted(self._ctx, layer, b, g, C.byref(k), pos.ctypes.data_as(C.POINTER(C.c_int32)),
                                            sc.ctypes.data_as(C.POINTER(C.c_float)), cap), "mkv_get_last_evicted")
        return pos[: k.value].copy(), sc[: k.value].copy()

    def last_probs(self, layer, b, g, with_pos=False):
        cap = self.budget_cap()
        n = C.c_int32(0)
        ab = np.zeros(cap, dtype=np.float32)
        pos = np.zeros(cap, dtype=np.int32)
        _check(self._L.mkv_get_last_probs(self._ctx, layer, b, g, C.byref(n), ab.ctypes.data_as(C.POINTER(C.c_float)),
                                          pos.ctypes.data_as(C.POINTER(C.c_int32)), cap), "mkv_get_last_probs")
        if with_pos:
            return ab[: n.value].copy(), pos[: n.value].copy()
        return ab[: n.value].copy()

    def recency_diagnostics(self, layer, window, mass, count, curve, stream=None):
        """mass: float32 [units], count: int32 [units], curve: float32 [units, window] device tensors."""
        _check(self._L.mkv_recency_diagnostics(self._ctx, layer, int(window), _ptr(mass), _ptr(count), _ptr(curve),
                                               self._stream(stream)), "mkv_recency_diagnostics")

    def read_kv(self, layer, b, g, pool):
        """Rows of a pool as float64 numpy arrays [n, head_dim] (exact: widening only)."""
        cap = self.max_prefill if pool == 0 else self.budget_cap()
        n = C.c_int32(0)
        es = 2 if self.kv_dtype == MKV_BF16 else 4
        raw_k = np.zeros((max(cap, 1), self.head_dim * es), dtype=np.uint8)
        raw_v = np.zeros_like(raw_k)
        _check(self._L.mkv_read_kv(self._ctx, layer, b, g, pool, C.byref(n), raw_k.ctypes.data_as(C.c_void_p),
                                   raw_v.ctypes.data_as(C.c_void_p), cap), "mkv_read_kv")

        def widen(raw):
            raw = raw[: n.value]
            if self.kv_dtype == MKV_BF16:
                u = raw.view(np.uint16).astype(np.uint32) << 16
                return u.view(np.float32).astype(np.float64)
            return raw.view(np.float32).astype(np.float64)

        return widen(raw_k), widen(raw_v)

    def step_count(self, layer) -> int:
        s = C.c_int64(0)
        _check(self._L.mkv_get_step(self._ctx, layer, C.byref(s)), "mkv_get_step")
        return int(s.value)

    def budget_cap(self) -> int:
        """Rows per decode pool: the largest budget plus the fresh token's slot."""
        return self.budget_max + 1
