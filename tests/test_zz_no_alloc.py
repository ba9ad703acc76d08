"""mkv_attend_noalloc, the entry point for callers that cannot allocate device memory
(a serving process that owns all of it, a plug-in handed buffers only): it keeps its
split-KV scratch in an array built into the library.  Checked here, on two calls in a row (the
second must not be disturbed by what the first left in the shared scratch), against the fp64
oracle's plain attention and against the ordinary workspace-based mkv_attend_only on the same
keys and values.  Collected last on purpose: a run that stops at the first failure has then run
every other test already."""
import numpy as np
import pytest

import paper_2605_29873_b200 as mkv


def oracle_attention(q, K, V):
    """softmax(q K^T / sqrt(d)) V through the oracle: q [B,Hq,d], K/V [B,Hkv,N,d], fp64.  With a
    budget that is never reached, its attention over {N-1 prompt rows} U {the appended row} is
    plain attention over all N rows."""
    from oracle import mkv_oracle as O
    B, Hq, d = q.shape
    Hkv, N = K.shape[1], K.shape[2]
    out = np.zeros_like(q)
    for b in range(B):
        o = O.OracleSequence(Hq, Hkv, d, 1 << 20, 0.5, N - 1)
        o.prefill(K[b, :, : N - 1], V[b, :, : N - 1])
        out[b] = o.attend_update(q[b], K[b, :, N - 1], V[b, :, N - 1])
    return out


CASES = [
    # dtype, q_heads, kv_heads, head_dim, batch, tokens
    ("bf16", 32, 8, 128, 3, 1000),     # several splits, ragged last one
    ("f32", 4, 1, 64, 2, 333),
    ("bf16", 8, 1, 128, 2, 3),         # group of 8, fewer rows than warps: idle warps
    ("bf16", 16, 2, 128, 2, 259),      # second split holds 3 rows
    ("f32", 6, 2, 128, 1, 256),        # exactly one full split
]


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,Hq,Hkv,d,B,N", CASES)
def test_noalloc_matches_oracle_and_attend_only_twice(dtype, Hq, Hkv, d, B, N):
    import torch
    dev = torch.device("cuda", 0)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    kvd = mkv.MKV_BF16 if dtype == "bf16" else mkv.MKV_F32
    gen = torch.Generator(device=dev)
    gen.manual_seed(7)
    K = (torch.randn((B, Hkv, N, d), generator=gen, device=dev) / d ** 0.5).to(tdt)
    V = (torch.randn((B, Hkv, N, d), generator=gen, device=dev) / d ** 0.5).to(tdt)
    ctx = mkv.MomentKV(1, Hq, Hkv, d, 16, 0.9, B, N, kv_dtype=kvd, out_dtype=mkv.MKV_F32)
    ctx.prefill(0, K, V, np.full(B, N, dtype=np.int32))
    tol = 1e-5 if dtype == "f32" else 2e-3
    Kh, Vh = K.double().cpu().numpy(), V.double().cpu().numpy()
    for call in range(2):
        q = (3.0 * torch.randn((B, Hq, d), generator=gen, device=dev)).to(tdt)
        ref = torch.zeros((B, Hq, d), dtype=torch.float32, device=dev)
        got = torch.full((B, Hq, d), float("nan"), dtype=torch.float32, device=dev)
        ctx.attend_only(0, q, ref)
        mkv.attend_noalloc(q, K, V, got, N)
        torch.cuda.synchronize()
        ctx.status_sync()
        r, g = ref.double().cpu().numpy(), got.double().cpu().numpy()
        want = oracle_attention(q.double().cpu().numpy(), Kh, Vh)
        rowmax = np.abs(want).max(axis=-1, keepdims=True)
        assert np.isfinite(g).all()
        assert (np.abs(g - want) <= tol * rowmax).all(), f"call {call}: no-alloc vs oracle {np.abs(g - want).max()}"
        assert (np.abs(r - want) <= tol * rowmax).all(), f"call {call}: attend_only vs oracle {np.abs(r - want).max()}"
        assert (np.abs(g - r) <= tol * rowmax).all(), f"call {call}: {np.abs(g - r).max()}"
    ctx.close()


def test_noalloc_rejects_what_the_scratch_cannot_hold():
    import ctypes as C
    lib = mkv.load_library()
    one = C.c_void_p(256)      # never dereferenced: the size checks come first
    args = lambda batch, n: [one, one, one, one, batch, 32, 8, 128, n, n, mkv.MKV_BF16, mkv.MKV_F32, 0, None]
    assert lib.mkv_attend_noalloc(*args(1, 16385)) == 3          # n_tokens beyond 16384
    assert lib.mkv_attend_noalloc(*args(300, 64)) == 3           # batch * kv_heads beyond the unit limit
    assert lib.mkv_attend_noalloc(*args(16, 16384)) == 3         # partial rows beyond the limit
    assert lib.mkv_attend_noalloc(None, one, one, one, 1, 32, 8, 128, 8, 8, 0, 1, 0, None) == 1
