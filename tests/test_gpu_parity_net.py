"""CUDA path vs fp64 oracle: the entry points, instantiations, limits and sizes that the main
parity file does not reach (needs a B200).  Everything goes through the C ABI."""
import numpy as np
import pytest

import paper_2605_29873_b200 as mkv
from oracle import mkv_oracle as O
from tests.parity_harness import FLUSH_ATOL, ParityReport, lockstep, make_context, prefill_both, to_device
from workloads.synthetic import CONFIGS, BatchStream, round_bf16

pytestmark = pytest.mark.gpu


def plain_attention_by_oracle(q, K, V, Hq, Hkv, d):
    """softmax(q K^T / sqrt(d)) V (Eq. 2) through the oracle: with a budget no step reaches,
    Algorithm 1's attention over {N-1 prompt rows} U {the appended row} is plain attention over
    all N rows (the oracle is pinned to the library routine in exactly this case).
    q [Hq,d]; K, V [Hkv,N,d] -> [Hq,d]."""
    N = K.shape[1]
    o = O.OracleSequence(Hq, Hkv, d, 1 << 20, 0.5, N - 1)
    o.prefill(K[:, : N - 1], V[:, : N - 1])
    return o.attend_update(q, K[:, N - 1], V[:, N - 1])


def assert_rows_close(got, ref, tol, what):
    rowmax = np.abs(ref).max(axis=-1, keepdims=True)
    err = np.abs(got - ref)
    assert np.isfinite(got).all(), what
    assert (err <= tol * rowmax).all(), (what, float((err / rowmax).max()))


# ----------------------------------------------------------------------------- (a) plain attention
@pytest.mark.parametrize("case", ["bf16_mma", "bf16_simt", "f32"])
def test_attend_only_is_plain_attention_over_both_pools(case):
    """mkv_attend_only (the denominator of the overhead figure) against Eq. 2 over prompt pool U
    decode pool, after decode steps that filled the pool and evicted from it; ragged batch, several
    tiles and splits.  It must leave the state alone."""
    import torch
    if case == "f32":
        w = CONFIGS["tiny"].with_(q_heads=6, kv_heads=2, batch=3, prefill=(30, 200), steps=90, budget=70, variant="hot")
        kernel, tol = mkv.MKV_KERNEL_AUTO, 1e-5
    else:
        w = CONFIGS["llama_b16"].with_(batch=4, prefill=(90, 700), steps=180, budget=150, variant="hot", n_heavy=4)
        kernel, tol = (mkv.MKV_KERNEL_MMA if case == "bf16_mma" else mkv.MKV_KERNEL_SIMT), 2e-3
    ctx = make_context(w, kernel=kernel)
    stream = BatchStream(w, 0)
    oracles, (Ks, Vs) = prefill_both(ctx, w, stream)
    out = torch.zeros((w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=ctx.device)
    rng = np.random.default_rng(3)
    rep = ParityReport()
    for phase, steps in enumerate((0, 37, w.steps - 37)):     # empty pool, ramp, full pool after evictions
        if steps:
            rep = lockstep(ctx, w, stream, oracles, steps, report=rep, check_state_every=0)
            assert rep.ok(), rep.failures[:5]
        before = [ctx.decode_state(0, b, g) for b in range(w.batch) for g in range(w.kv_heads)]
        q = 2.0 * np.sqrt(w.head_dim) * rng.standard_normal((w.batch, w.q_heads, w.head_dim))
        q = round_bf16(q) if w.dtype == "bf16" else q.astype(np.float32).astype(np.float64)
        ctx.attend_only(0, to_device(q, torch, ctx.torch_kv_dtype(), ctx.device), out)
        ctx.status_sync()
        got = out.double().cpu().numpy()
        for b in range(w.batch):
            Kd, Vd = zip(*(oracles[b].decode_kv(g) for g in range(w.kv_heads)))
            Kall = np.concatenate([Ks[b], np.stack(Kd)], axis=1)
            Vall = np.concatenate([Vs[b], np.stack(Vd)], axis=1)
            ref = plain_attention_by_oracle(q[b], Kall, Vall, w.q_heads, w.kv_heads, w.head_dim)
            assert_rows_close(got[b], ref, tol, (case, phase, b))
        after = [ctx.decode_state(0, b, g) for b in range(w.batch) for g in range(w.kv_heads)]
        for (p0, s0), (p1, s1) in zip(before, after):
            np.testing.assert_array_equal(p0, p1)
            np.testing.assert_array_equal(s0, s1)
    assert ctx.step_count(0) == w.steps and rep.evictions > 0
    ctx.close()


# ----------------------------------------------------------------------------- (b) config 2 as written
def test_llama_b1_real_recipe_heavy_hitters_survive_the_dips():
    """The second configuration exactly as specified: one Llama-shaped layer, bf16, prefill 1024,
    4096 decode steps, budget 512, beta 0.9, 16 heavy hitters per KV head whose alignment with
    the queries is on for 50 steps and off for 20 (Sec. 3.1: attention to important tokens
    dips and comes back).  Parity with the oracle over the whole run; at the end every planted
    heavy hitter is still cached (Sec. 4.2: the momentum score carries it through the dips),
    while the same run with beta = 0 -- the score is the current attention only -- has lost
    heavy hitters during dips."""
    import torch
    w = CONFIGS["llama_b1"]
    assert (w.variant, w.prefill, w.budget, w.n_heavy, w.steps, w.beta) == ("literal", 1024, 512, 16, 4096, 0.9)
    ctx = make_context(w)
    stream = BatchStream(w, 0)
    oracles, _ = prefill_both(ctx, w, stream)
    rep = lockstep(ctx, w, stream, oracles, w.steps, check_state_every=64)
    assert rep.ok(), rep.failures[:5]
    assert rep.max_out_err <= 2e-3 and rep.max_score_err <= 1e-4
    heavy = set(int(t) for t in w.heavy_steps())
    for g in range(w.kv_heads):
        pos, _ = ctx.decode_state(0, 0, g)
        assert len(pos) == w.budget and heavy <= set(pos.tolist()), (g, sorted(heavy - set(pos.tolist())))
        assert heavy <= set(oracles[0].decode_state(g)[0].tolist())
    ctx.close()
    # the same inputs under an instantaneous-attention policy
    w0 = w.with_(beta=0.0)
    ctx0 = make_context(w0)
    stream0 = BatchStream(w0, 0)
    oracles0, _ = prefill_both(ctx0, w0, stream0)
    dt = ctx0.torch_kv_dtype()
    out = torch.zeros((1, w.q_heads, w.head_dim), dtype=torch.float32, device=ctx0.device)
    done = 0
    while done < w.steps:
        qs, ks, vs = stream0.next(256)
        qd, kd, vd = (to_device(a, torch, dt, ctx0.device) for a in (qs, ks, vs))
        for i in range(256):
            ctx0.decode_step(0, qd[i], kd[i], vd[i], out)
        done += 256
    ctx0.status_sync()
    lost = sum(len(heavy - set(ctx0.decode_state(0, 0, g)[0].tolist())) for g in range(w.kv_heads))
    ctx0.close()
    assert lost > 0, "beta = 0 was expected to lose heavy hitters during their dips"


# ----------------------------------------------------------------------------- (c) beta limits, flush rule
@pytest.mark.parametrize("beta", [0.0, 1.0])
@pytest.mark.parametrize("shape,mode", [("bf16", "group"), ("bf16", "layer"), ("f32", "group"), ("f32", "layer")])
def test_beta_limits(beta, shape, mode):
    """Eq. 5 at its limits on the GPU: beta = 0 (the score is the attention of the current step)
    and beta = 1 (the plain running sum), in both score modes and on both kernels."""
    if shape == "bf16":
        w = CONFIGS["llama_b1"].with_(batch=2, prefill=(100, 300), steps=200, budget=80, variant="hot", n_heavy=3, beta=beta)
    else:
        w = CONFIGS["tiny"].with_(q_heads=6, kv_heads=2, batch=2, prefill=70, steps=200, budget=48, variant="hot", beta=beta)
    smode, omode = ((mkv.MKV_SCORE_LAYER_MEAN, O.LAYER_MEAN) if mode == "layer" else (mkv.MKV_SCORE_GROUP_MEAN, O.GROUP_MEAN))
    ctx = make_context(w, score_mode=smode)
    stream = BatchStream(w, 0)
    oracles, _ = prefill_both(ctx, w, stream, mode=omode)
    rep = lockstep(ctx, w, stream, oracles, w.steps)
    ctx.close()
    assert rep.ok(), rep.failures[:5]
    assert rep.max_out_err <= (2e-3 if shape == "bf16" else 1e-5) and rep.max_score_err <= 1e-4
    assert rep.evicted_not_newest > 10


class SharpStream(BatchStream):
    """The same draws with the queries scaled by a power of two (exact in every dtype): logits
    hundreds apart, so that most probabilities are far below what fp32 can hold."""

    def next(self, n):
        q, k, v = super().next(n)
        return q * 16.0, k, v


@pytest.mark.parametrize("shape,beta", [("bf16", 0.0), ("bf16", 0.9), ("f32", 0.0)])
def test_one_hot_attention_flushes_probabilities_to_zero(shape, beta):
    """Nearly one-hot attention.  The GPU forms probabilities in fp32 (2^(s-M), flushed to zero
    below 2^-126), the oracle in fp64, where the same probability is 1e-50 or 1e-200.  The rule
    (see the harness): scores agree to 1e-4 relative plus 2^-100 absolute, tokens whose scores
    were flushed tie at zero and are evicted oldest first, which the free-running comparison
    accepts as a tie at the cutoff; the teacher-forced selection stays bit exact.
    Logits of this size (up to about 300 in log2 units, against 20 in the workloads) also carry
    300 * 2^-24 = 2e-5 of fp32 rounding each, i.e. that much relative error in EVERY probability,
    so the relative tolerances are widened tenfold for this test alone (fp32 `out` 1e-4, scores
    1e-3); the standard ones assume the workloads' logit range."""
    if shape == "bf16":
        w = CONFIGS["llama_b1"].with_(batch=2, prefill=(60, 200), steps=120, budget=50, variant="hot", n_heavy=2, beta=beta)
    else:
        w = CONFIGS["tiny"].with_(batch=2, prefill=70, steps=120, budget=40, variant="hot", beta=beta)
    ctx = make_context(w)
    stream = SharpStream(w, 0)
    oracles, _ = prefill_both(ctx, w, stream)
    tol_out = 2e-3 if shape == "bf16" else 1e-4
    rep = lockstep(ctx, w, stream, oracles, w.steps, tol_out=tol_out, tol_score=1e-3)
    zeros = sum(int((ctx.decode_state(0, b, g)[1] == 0.0).sum()) for b in range(w.batch) for g in range(w.kv_heads))
    tiny = sum(int((oracles[b].decode_state(g)[1] < FLUSH_ATOL).sum()) for b in range(w.batch) for g in range(w.kv_heads))
    ctx.close()
    assert rep.ok(), rep.failures[:5]
    assert rep.max_out_err <= tol_out and rep.max_score_err <= 1e-3
    if beta == 0.0:
        assert zeros > 0 and tiny >= zeros      # the case the rule exists for did occur


# ----------------------------------------------------------------------------- (d) instantiations
SWEEP = [  # (dtype, q_heads, kv_heads, head_dim, kernel)
    ("bf16", 2, 2, 128, "mma"), ("bf16", 4, 2, 128, "mma"), ("bf16", 10, 2, 128, "mma"), ("bf16", 12, 2, 128, "mma"),
    ("bf16", 16, 2, 128, "mma"),
    ("bf16", 2, 2, 128, "simt"), ("bf16", 4, 2, 128, "simt"), ("bf16", 10, 2, 128, "simt"), ("bf16", 12, 2, 128, "simt"),
    ("bf16", 16, 2, 128, "simt"),
    ("bf16", 8, 2, 64, "simt"), ("bf16", 14, 2, 64, "simt"), ("f32", 6, 2, 128, "simt"), ("f32", 8, 1, 128, "simt"),
    ("f32", 5, 5, 64, "simt"),
]


@pytest.mark.parametrize("dtype,Hq,Hkv,d,kernel", SWEEP)
def test_every_group_size_and_element_type(dtype, Hq, Hkv, d, kernel):
    """Group sizes 1, 2, 5, 6, 8 on both kernels (8 = every row of the tensor-core kernel's head
    tile and of the tail's staging live), bf16 with head_dim 64 and fp32 with head_dim 128 on the
    scalar kernel: each is its own template instantiation."""
    w = CONFIGS["tiny"].with_(q_heads=Hq, kv_heads=Hkv, head_dim=d, dtype=dtype, batch=2, prefill=(40, 210), steps=110,
                              budget=45, variant="hot", n_heavy=2, shared_direction=False)
    ctx = make_context(w, kernel=mkv.MKV_KERNEL_MMA if kernel == "mma" else mkv.MKV_KERNEL_SIMT)
    stream = BatchStream(w, 0)
    oracles, _ = prefill_both(ctx, w, stream)
    rep = lockstep(ctx, w, stream, oracles, w.steps, check_state_every=2)
    ctx.close()
    assert rep.ok(), rep.failures[:5]
    assert rep.max_out_err <= (2e-3 if dtype == "bf16" else 1e-5) and rep.max_score_err <= 1e-4
    assert rep.evictions == (w.steps - w.budget) * w.batch * Hkv


@pytest.mark.parametrize("kernel", ["mma", "simt"])
@pytest.mark.parametrize("mode", ["group", "layer"])
def test_budget_of_one_token(kernel, mode):
    """B_d = 1: the pool holds one token and the fresh one; every step decides between the two."""
    w = CONFIGS["llama_b1"].with_(batch=2, prefill=(70, 130), steps=60, budget=1, variant="hot", n_heavy=0)
    smode, omode = ((mkv.MKV_SCORE_LAYER_MEAN, O.LAYER_MEAN) if mode == "layer" else (mkv.MKV_SCORE_GROUP_MEAN, O.GROUP_MEAN))
    ctx = make_context(w, kernel=mkv.MKV_KERNEL_MMA if kernel == "mma" else mkv.MKV_KERNEL_SIMT, score_mode=smode)
    stream = BatchStream(w, 0)
    oracles, _ = prefill_both(ctx, w, stream, mode=omode)
    rep = lockstep(ctx, w, stream, oracles, w.steps)
    ctx.close()
    assert rep.ok(), rep.failures[:5]
    assert rep.evictions == (w.steps - 1) * w.batch * w.kv_heads and 0 < rep.evicted_not_newest < rep.evictions


# ----------------------------------------------------------------------------- (e) bf16 output
@pytest.mark.parametrize("mode", ["group", "layer"])
def test_bf16_out_is_the_rounding_of_the_fp32_result(mode):
    """The bf16 `out` of the benchmark's configuration: the fp32-`out` context is held to 2e-3 of
    the row maximum against the oracle, and the bf16-`out` context, fed the same steps, must
    store exactly the round-to-nearest-even bf16 of those fp32 values.  Both contexts run in the
    reproducible mode, so that the values before the store are the same bits."""
    import torch
    w = CONFIGS["llama_b16"].with_(batch=3, prefill=(90, 500), steps=130, budget=60, variant="hot", n_heavy=3)
    smode, omode = ((mkv.MKV_SCORE_LAYER_MEAN, O.LAYER_MEAN) if mode == "layer" else (mkv.MKV_SCORE_GROUP_MEAN, O.GROUP_MEAN))
    a = make_context(w, out_f32=True, score_mode=smode, flags=mkv.MKV_FLAG_REPRODUCIBLE)
    b = make_context(w, out_f32=False, score_mode=smode, flags=mkv.MKV_FLAG_REPRODUCIBLE)
    sa, sb = BatchStream(w, 0), BatchStream(w, 0)
    oracles, _ = prefill_both(a, w, sa, mode=omode)
    prefill_both(b, w, sb, mode=omode)
    dt, dev = a.torch_kv_dtype(), a.device
    out_a = torch.zeros((w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=dev)
    out_b = torch.zeros((w.batch, w.q_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
    qs, ks, vs = sa.next(w.steps)
    qd, kd, vd = (to_device(x, torch, dt, dev) for x in (qs, ks, vs))
    for i in range(w.steps):
        a.decode_step(0, qd[i], kd[i], vd[i], out_a)
        b.decode_step(0, qd[i], kd[i], vd[i], out_b)
        assert torch.equal(out_a.to(torch.bfloat16), out_b), f"step {i}: bf16 out is not the rounding of the fp32 out"
        got = out_a.double().cpu().numpy()
        for s in range(w.batch):
            ref = oracles[s].attend_update(qs[i, s], ks[i, s], vs[i, s])
            assert_rows_close(got[s], ref, 2e-3, (i, s))
            oracles[s].evict(force=[a.last_evicted(0, s, g)[0].astype(np.int64) for g in range(w.kv_heads)])
    a.status_sync(); b.status_sync()
    a.close(); b.close()


# ----------------------------------------------------------------------------- (f) full sizes, several steps
FULL_SIZE_CASES = {
    # name: (workload, layers, layer-wide score mode)
    "llama_b16": (lambda: CONFIGS["llama_b16"], 1, False),
    "llama_b16_layer_mean": (lambda: CONFIGS["llama_b16"], 1, True),
    "llama_stack_two_layers": (lambda: CONFIGS["llama_stack"], 2, False),
    "qwen_b64_budget128_beta0.8": (lambda: CONFIGS["qwen_b64"].with_(budget=128, beta=0.8), 1, False),
    "qwen_b64_budget1024_beta0.99": (lambda: CONFIGS["qwen_b64"].with_(budget=1024, beta=0.99), 1, False),
    "qwen_b64_budget2048_never_evicts": (lambda: CONFIGS["qwen_b64"].with_(budget=2048, beta=0.9), 1, False),
}


@pytest.mark.parametrize("case", sorted(FULL_SIZE_CASES))
def test_full_size_eight_steps_against_the_oracle(case):
    """The benchmark configurations at their full sizes (batch, prompt lengths, budget: the grid,
    the start table and the work sharing that the bench times, with the bench's early-input
    overlap), run to steady state with device-generated inputs.  Sampled sequences then get an
    oracle each, loaded with the state read back from the GPU, and eight further steps are
    compared one by one: `out`, every score, the evicted tokens.  The sweep's budget-2048 cell
    never evicts (the budget is the whole run: the full-cache mode of the paper's comparison):
    there the pool grows through all eight steps."""
    import torch
    make_w, layers, layer_mean = FULL_SIZE_CASES[case]
    w = make_w()
    lens = w.prefill_lens()
    B, Hq, Hkv, d = w.batch, w.q_heads, w.kv_heads, w.head_dim
    dev = torch.device("cuda", 0)
    ctx = mkv.MomentKV(layers, Hq, Hkv, d, w.budget, w.beta, B, int(lens.max()), out_dtype=mkv.MKV_F32,
                       score_mode=mkv.MKV_SCORE_LAYER_MEAN if layer_mean else mkv.MKV_SCORE_GROUP_MEAN,
                       flags=mkv.MKV_FLAG_INPUTS_READY)
    gen = torch.Generator(device=dev)
    gen.manual_seed(11)
    for layer in range(layers):
        K = (torch.randn((B, Hkv, int(lens.max()), d), generator=gen, device=dev) / d ** 0.5).bfloat16()
        V = (torch.randn((B, Hkv, int(lens.max()), d), generator=gen, device=dev) / d ** 0.5).bfloat16()
        ctx.prefill(layer, K, V, lens)
        torch.cuda.synchronize()
        del K, V
    out = torch.zeros((B, Hq, d), dtype=torch.float32, device=dev)
    ring = 32
    qs = (2.0 * torch.randn((ring, B, Hq, d), generator=gen, device=dev)).bfloat16()
    ks = (torch.randn((ring, B, Hkv, d), generator=gen, device=dev) / d ** 0.5).bfloat16()
    vs = (torch.randn((ring, B, Hkv, d), generator=gen, device=dev) / d ** 0.5).bfloat16()
    torch.cuda.synchronize()
    never = w.budget >= w.steps
    steps = (w.steps - 8) if never else (w.budget + 40)
    for i in range(steps):
        for layer in range(layers):
            ctx.decode_step(layer, qs[(i + layer) % ring], ks[(i + layer) % ring], vs[(i + layer) % ring], out)
    ctx.status_sync()
    layer = layers - 1
    seqs = sorted({0, B // 2, B - 1, int(np.argmax(lens)), int(np.argmin(lens))})
    mode = O.LAYER_MEAN if layer_mean else O.GROUP_MEAN
    oracles = {}
    for b in seqs:
        o = O.OracleSequence(Hq, Hkv, d, w.budget, w.beta, int(lens[b]), mode)
        Kp, Vp = zip(*(ctx.read_kv(layer, b, g, 0) for g in range(Hkv)))
        o.prefill(np.stack(Kp), np.stack(Vp))
        for g in range(Hkv):
            Kd, Vd = ctx.read_kv(layer, b, g, 1)
            pos, sc = ctx.decode_state(layer, b, g)
            assert len(pos) == min(steps, w.budget)
            o.load_decode_state(g, Kd, Vd, sc.astype(np.float64), pos, steps)
        oracles[b] = o
    near_ties = 0
    for j in range(8):
        i = steps + j
        for l2 in range(layers):
            ctx.decode_step(l2, qs[(i + l2) % ring], ks[(i + l2) % ring], vs[(i + l2) % ring], out)
        ctx.status_sync()
        r = (i + layer) % ring
        got = out.double().cpu().numpy()
        qh, kh, vh = (x[r].double().cpu().numpy() for x in (qs, ks, vs))
        for b in seqs:
            o = oracles[b]
            ref = o.attend_update(qh[b], kh[b], vh[b])
            assert_rows_close(got[b], ref, 2e-3, (case, j, b))
            force = []
            for g in range(Hkv):
                ev_pos, ev_sc = ctx.last_evicted(layer, b, g)
                choice = o.choose(g)
                assert len(ev_pos) == len(choice) == (0 if never else 1)
                g_pos, g_sc = ctx.decode_state(layer, b, g)
                all_pos = np.concatenate([g_pos, ev_pos]).astype(np.int64)
                all_sc = np.concatenate([g_sc, ev_sc]).astype(np.float64)
                o_pos, o_sc, _ = o.decode_state(g)
                order, oorder = np.argsort(all_pos), np.argsort(o_pos)
                np.testing.assert_array_equal(all_pos[order], o_pos[oorder])
                assert (np.abs(all_sc[order] - o_sc[oorder]) <= 1e-4 * o_sc[oorder] + FLUSH_ATOL).all(), (case, j, b, g)
                want = all_pos[O.select(all_sc, all_pos, len(ev_pos))]      # integer selection on the GPU's scores
                assert sorted(want.tolist()) == sorted(ev_pos.tolist())
                if set(ev_pos.tolist()) != set(choice.tolist()):
                    cut = np.sort(o_sc)[len(choice) - 1]
                    smap = dict(zip(o_pos.tolist(), o_sc.tolist()))
                    assert all(abs(smap[p] - cut) <= 1e-5 * cut + FLUSH_ATOL for p in set(ev_pos.tolist()) ^ set(choice.tolist()))
                    near_ties += 1
                force.append(ev_pos.astype(np.int64))
            o.evict(force=force)
    ctx.close()
    assert near_ties <= 4
