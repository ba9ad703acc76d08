"""The C-ABI library without a GPU: it loads, exports every declared symbol, its host
arithmetic is right, and it refuses to run without a device (no fallback)."""
import ctypes as C
import os
import re

import pytest

import paper_2605_29873_b200 as mkv
from paper_2605_29873_b200 import build as mkv_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    mkv_build.build_library()
    return mkv.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "mkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mkv_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/mkv.h but not exported"
    assert sorted(mkv.EXPORTED_SYMBOLS) == names


def test_status_strings(lib):
    assert mkv.status_string(0) == "ok"
    assert len({mkv.status_string(i) for i in range(9)}) == 9


def test_kv_sizing_matches_the_papers_figure(lib):
    """Sec. 1: an 8B model's 16-bit KV cache takes exactly 128 KB per token and nearly
    13 GB for 100K tokens (fixture tests/golden/kv_sizing.txt)."""
    vals = {}
    for line in open(os.path.join(ROOT, "tests", "golden", "kv_sizing.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            vals[k] = int(v)
    per_tok = mkv.kv_bytes_per_token(32, 8, 128, mkv.MKV_BF16)
    assert per_tok == vals["bytes_per_token"] == 128 * 1024
    assert round(per_tok * vals["tokens"] / 1e9) == vals["approx_gigabytes"]
    # the workspace grows by that per cached token (plus < 10 % of split-KV scratch)
    a = mkv.workspace_bytes(32, 4, 32, 8, 128, 2048, 2048)
    b = mkv.workspace_bytes(32, 4, 32, 8, 128, 2048, 4096)
    assert (b - a) // (4 * 2048) >= per_tok
    assert (b - a) // (4 * 2048) < per_tok * 1.10


def test_workspace_bytes_rejects_bad_shapes(lib):
    ok = mkv.workspace_bytes(1, 1, 4, 1, 64, 64, 64, mkv.MKV_F32)
    assert ok > 0 and ok % 256 == 0
    assert mkv.workspace_bytes(1, 1, 5, 2, 64, 64, 64) == 0      # q_heads % kv_heads
    assert mkv.workspace_bytes(1, 1, 4, 1, 96, 64, 64) == 0      # head_dim
    assert mkv.workspace_bytes(0, 1, 4, 1, 64, 64, 64) == 0
    assert mkv.workspace_bytes(1, 1, 4, 1, 64, 0, 64) == 0       # budget >= 1
    assert mkv.workspace_bytes(1, 1, 64, 1, 64, 64, 64) == 0     # group > 8
    assert mkv.workspace_bytes(1, 1, 9, 1, 64, 64, 64) == 0      # (the sizing call and mkv_create agree)
    assert mkv.workspace_bytes(1, 1, 8, 1, 64, 64, 64) > 0


def test_create_validates_then_fails_loudly_without_a_gpu(lib):
    import torch
    ctx = C.c_void_p(0)
    fake = C.c_void_p(1 << 20)   # aligned, never dereferenced by the argument checks
    n = mkv.workspace_bytes(1, 1, 4, 1, 64, 64, 64, mkv.MKV_F32)
    args = lambda **kw: [kw.get("layers", 1), 4, 1, 64, 64, C.c_float(kw.get("beta", 0.9)), 1, 64, mkv.MKV_F32,
                         kw.get("out", mkv.MKV_F32), 0, 0, 0, kw.get("ws", fake), kw.get("n", n), 0, C.byref(ctx)]
    assert lib.mkv_create(*args(beta=1.5)) == 1
    assert lib.mkv_create(*args(out=mkv.MKV_BF16)) == 1           # fp32 cache needs fp32 out
    assert lib.mkv_create(*args(ws=C.c_void_p(0))) == 1
    assert lib.mkv_create(*args(ws=C.c_void_p((1 << 20) + 8))) == 4
    assert lib.mkv_create(*args(n=n - 1)) == 4
    if not torch.cuda.is_available():
        assert lib.mkv_create(*args()) == 6                       # MKV_ERR_CUDA: no device, no fallback
        with pytest.raises(RuntimeError):
            mkv.MomentKV(1, 4, 1, 64, 64, 0.9, 1, 64, kv_dtype=mkv.MKV_F32)
    assert lib.mkv_decode_step(None, 0, None, None, None, None, None) == 1
    lib.mkv_destroy(None)


def test_start_table_invariants(lib):
    """mkv_plan_starts: CTAs are spread over the units in tile order, reserved tiles are
    disjoint prefill tiles, a unit's counter starts right behind them, and the CTAs starting in
    a unit plus the pulls of its counter fit the 64 partial results a unit has room for."""
    import numpy as np
    from workloads.synthetic import CONFIGS
    cases = [(CONFIGS["llama_b16"].prefill_lens(), 8, 1024, 296), (np.array([64], dtype=np.int32), 1, 64, 296),
             (np.array([0, 5, 4096], dtype=np.int32), 4, 128, 296), (np.full(64, 512, dtype=np.int32), 4, 2048, 296),
             (np.array([100000], dtype=np.int32), 2, 16, 7), (np.array([100000], dtype=np.int32), 2, 16, 296),
             (np.array([30000, 100, 100, 50000], dtype=np.int32), 1, 4096, 2048)]
    for lens, hkv, budget, nmax in cases:
        B = len(lens)
        u0, h0, hn, nx, ch = mkv.plan_starts(B, hkv, budget, lens, nmax)
        U = B * hkv
        tiles = np.array([-(-int(lens[u // hkv]) // 64) + -(-budget // 64) for u in range(U)])
        assert 1 <= len(u0) <= nmax and len(u0) <= max(1, tiles.sum() // 2)
        assert (np.diff(u0) >= 0).all() and u0.min() >= 0 and u0.max() < U
        # proportional spread: CTA c starts in the unit that holds tile position c * T / n
        begin = np.concatenate([[0], np.cumsum(tiles)])
        for c in range(len(u0)):
            t0 = tiles.sum() * c // len(u0)
            assert begin[u0[c]] <= t0 < begin[u0[c] + 1]
        assert set(hn.tolist()) <= {0, 3}
        # another reservation size: same spread, reserved ranges of that size
        u0b, h0b, hnb, nxb, _ = mkv.plan_starts(B, hkv, budget, lens, nmax, head_tiles=7)
        assert (u0b == u0).all() and set(hnb.tolist()) <= {0, 7} and (nxb % 7 == 0).all()
        assert (mkv.plan_starts(B, hkv, budget, lens, nmax, head_tiles=0)[2] == 0).all()
        for u in range(U):
            mine = np.where(u0 == u)[0]
            got = sorted((int(h0[c]), int(hn[c])) for c in mine if hn[c] > 0)
            # reserved ranges tile [0, next0) without gaps, all inside the prefill tiles
            assert [g[0] for g in got] == list(range(0, 3 * len(got), 3))
            assert nx[u] == 3 * len(got) <= -(-int(lens[u // hkv]) // 64)
            assert len(mine) <= 32 and ch[u] >= 2
            assert len(mine) + -(-int(tiles[u] - nx[u]) // int(ch[u])) <= 64 - 8


def test_reproducible_mode_ranges_cover_every_tile_once(lib):
    """mkv_plan_ranges: the CTAs' ranges tile the global tile sequence without gap or overlap,
    a unit's partial slots (CTA index minus the unit's first CTA) are 0..visits-1 with at most 64
    visits, and every CTA has work."""
    import numpy as np
    from workloads.synthetic import CONFIGS
    cases = [(CONFIGS["llama_b16"].prefill_lens(), 8, 1024, 296), (np.array([64], dtype=np.int32), 1, 64, 296),
             (np.array([0, 5, 4096], dtype=np.int32), 4, 128, 148), (np.full(64, 512, dtype=np.int32), 4, 2048, 296),
             (np.array([100000], dtype=np.int32), 2, 16, 296), (np.array([0], dtype=np.int32), 1, 1, 296)]
    for lens, hkv, budget, nmax in cases:
        B, U = len(lens), len(lens) * hkv
        t0, tb, uc = mkv.plan_ranges(B, hkv, budget, lens, nmax)
        n = len(t0) - 1
        tiles = np.array([-(-int(lens[u // hkv]) // 64) + -(-budget // 64) for u in range(U)])
        assert (np.diff(tb) == tiles).all() and tb[0] == 0
        assert 1 <= n <= nmax and t0[0] == 0 and t0[-1] == tiles.sum() and (np.diff(t0) >= 1).all()
        for u in range(U):
            touching = [c for c in range(n) if t0[c] < tb[u + 1] and t0[c + 1] > tb[u]]
            assert touching == list(range(uc[u], uc[u] + len(touching))) and 1 <= len(touching) <= 64


def test_grid_limit_clamps_to_what_is_resident(lib):
    """The grid never exceeds SM count x resident CTAs per SM (the kernels' CTAs wait on one
    another), never the design point, never 2048; a kernel that does not fit gives 0."""
    assert mkv.grid_limit(148, 2, 2) == 296
    assert mkv.grid_limit(148, 1, 2) == 148          # a deeper ring: one CTA per SM fits
    assert mkv.grid_limit(148, 5, 2) == 296          # more would fit, the design point stands
    assert mkv.grid_limit(148, 16, 8) == 1184
    assert mkv.grid_limit(1000, 8, 8) == 2048
    assert mkv.grid_limit(148, 0, 2) == 0 and mkv.grid_limit(0, 2, 2) == 0


def test_new_calls_check_their_arguments(lib):
    one = C.c_void_p(256)
    assert lib.mkv_set_option(None, 1, 3) == 1
    assert lib.mkv_decode_step_layers(None, 0, 1, one, one, one, one, None) == 1
    assert lib.mkv_attend_only_layers(None, 0, 1, one, one, None) == 1
    assert lib.mkv_debug_inject(None, 0, 0, 0, 0) == 1
    n, m = C.c_int32(0), C.c_int32(0)
    assert lib.mkv_get_grid(None, 0, C.byref(n), C.byref(m)) == 1
