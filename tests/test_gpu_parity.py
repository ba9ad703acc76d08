"""CUDA path vs fp64 oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest

import paper_2605_29873_b200 as mkv
from tests.parity_harness import ParityReport, lockstep, make_context, prefill_both
from workloads.synthetic import CONFIGS, BatchStream

pytestmark = pytest.mark.gpu


def run_case(w, steps, kernel=mkv.MKV_KERNEL_AUTO, out_f32=True, sequences=None, host_api=False, check_every=1):
    ctx = make_context(w, kernel=kernel, out_f32=out_f32, sequences=sequences)
    stream = BatchStream(w, 0, sequences)
    oracles, _ = prefill_both(ctx, w, stream)
    rep = lockstep(ctx, w, stream, oracles, steps, host_api=host_api, check_state_every=check_every)
    # frozen prefill pool: bytes unchanged after the run (Sec. 4.2 "Prefill pool (frozen)")
    Ks, Vs = BatchStream(w, 0, sequences).prefill()
    for b in range(len(oracles)):
        for g in range(w.kv_heads):
            K, V = ctx.read_kv(0, b, g, 0)
            np.testing.assert_array_equal(K, Ks[b][g])
            np.testing.assert_array_equal(V, Vs[b][g])
            Kd, Vd = ctx.read_kv(0, b, g, 1)
            pos, _ = ctx.decode_state(0, b, g)
            oK, oV = oracles[b].decode_kv(g)
            opos = oracles[b].decode_state(g)[0]
            assert len(pos) <= w.budget
            order, oorder = np.argsort(pos), np.argsort(opos)
            np.testing.assert_array_equal(pos[order], opos[oorder])
            np.testing.assert_array_equal(Kd[order], oK[oorder])      # rows moved by compaction: bit exact
            np.testing.assert_array_equal(Vd[order], oV[oorder])
    assert ctx.step_count(0) == steps
    ctx.close()
    return rep


@pytest.mark.parametrize("variant", ["literal", "hot"])
def test_tiny_fp32_full_run(variant):
    """Config 1: fp32, 4/1 heads, d 64, 512 steps, budget 64 -- every step, every score."""
    w = CONFIGS["tiny"].with_(variant=variant)
    rep = run_case(w, w.steps)
    assert rep.ok(), rep.failures[:5]
    assert rep.max_out_err <= 1e-5 and rep.max_score_err <= 1e-4
    assert rep.evictions == w.steps - w.budget
    if variant == "hot":
        assert rep.evicted_not_newest > 50     # compaction really moves rows


@pytest.mark.parametrize("kernel", [mkv.MKV_KERNEL_SIMT, mkv.MKV_KERNEL_AUTO])
def test_llama_layer_bf16_reduced(kernel):
    """Config 2 shape (32/8 heads, d 128, bf16), shortened: ragged prefill spanning several
    tiles and items, decode pool filling then evicting."""
    w = CONFIGS["llama_b1"].with_(prefill=333, steps=400, budget=150, variant="hot", n_heavy=4)
    rep = run_case(w, w.steps, kernel=kernel)
    assert rep.ok(), rep.failures[:5]
    assert rep.max_out_err <= 2e-3 and rep.max_score_err <= 1e-4
    assert rep.evicted_not_newest > 20


def test_ragged_batch_bf16():
    """Headline shape reduced: several sequences with different prefill lengths (ragged tails in
    both pools, units of different size sharing the CTAs), tensor-core kernel."""
    w = CONFIGS["llama_b16"].with_(batch=5, prefill=(90, 700), steps=300, budget=140, variant="hot", n_heavy=4)
    rep = run_case(w, w.steps, check_every=3)
    assert rep.ok(), rep.failures[:5]
    assert rep.max_out_err <= 2e-3 and rep.max_score_err <= 1e-4
    assert rep.evicted_not_newest > 50


def test_few_long_units_share_many_ctas():
    """One sequence with a long prompt: eight units of ~320 tiles draw the whole grid, about 31
    CTAs each, and every visit of a unit delivers one partial result; the start table must keep
    visits within the room a unit has for them (no device-check status, results as the oracle's)."""
    w = CONFIGS["llama_b1"].with_(prefill=20000, steps=45, budget=30, variant="hot", n_heavy=2)
    rep = run_case(w, w.steps, check_every=5)
    assert rep.ok(), rep.failures[:5]
    assert rep.max_out_err <= 2e-3 and rep.max_score_err <= 1e-4


def test_headline_sequences_through_ramp_and_steady_state():
    """Two sequences of the headline workload at its real sizes (prefill 654 and 926 tokens of the
    U[512,4096] draw, budget 1024, bf16), free-running against the oracle from the empty pool
    through the whole ramp and 160 evicting steps: drift of the scores over more than a thousand
    steps of Eq. 5 and every eviction at the full budget."""
    w = CONFIGS["llama_b16"].with_(variant="hot")
    rep = run_case(w, w.budget + 160, sequences=[9, 8], check_every=16)
    assert rep.ok(), rep.failures[:5]
    assert rep.max_out_err <= 2e-3 and rep.max_score_err <= 1e-4
    assert rep.evictions == 2 * w.kv_heads * 160


@pytest.mark.parametrize("budget,beta", [(128, 0.8), (128, 0.99), (512, 0.8), (512, 0.99)])
def test_qwen_sweep_cells_one_sequence(budget, beta):
    """Cells of the G=7 sweep at their real sizes (28/4 heads, prefill 512, the cell's budget and
    momentum factor), one sequence each, free-running through the ramp and 100 evicting steps.
    beta only enters Eq. 5, so the cells differ in how fast old attention fades: 0.99 keeps
    scores of very different ages close together, 0.8 forgets within a few steps."""
    w = CONFIGS["qwen_b64"].with_(budget=budget, beta=beta, variant="hot")
    rep = run_case(w, budget + 100, sequences=[3], check_every=8)
    assert rep.ok(), rep.failures[:5]
    assert rep.max_out_err <= 2e-3 and rep.max_score_err <= 1e-4
    assert rep.evictions == w.kv_heads * 100


def test_qwen_group7_bf16():
    """GQA group 7 (28 query heads on 4 KV heads): the padded head rows of the tensor-core
    kernel and the 8-head staging of the tail."""
    w = CONFIGS["qwen_b64"].with_(batch=3, prefill=210, steps=240, budget=100, variant="hot", n_heavy=4)
    rep = run_case(w, w.steps, check_every=2)
    assert rep.ok(), rep.failures[:5]
    assert rep.max_out_err <= 2e-3 and rep.max_score_err <= 1e-4
    assert rep.evicted_not_newest > 20


def test_empty_prefill_and_bf16_out_through_host_api():
    """No prompt at all (the decode pool is the whole cache), bf16 output, host-buffer entry
    point: covers the unit with nothing cached at the first step.  The host buffers are pinned
    (the kernel writes `out` into them directly), then pinned and packed (one input copy), then
    pageable (staged copies both ways)."""
    w = CONFIGS["llama_b1"].with_(prefill=0, steps=150, budget=40, variant="hot", n_heavy=2)
    ctx = make_context(w, out_f32=False)
    stream = BatchStream(w, 0)
    oracles, _ = prefill_both(ctx, w, stream)
    rep = lockstep(ctx, w, stream, oracles, 70, host_api=True)
    rep = lockstep(ctx, w, stream, oracles, 40, host_api=True, host_packed=True, report=rep)
    rep = lockstep(ctx, w, stream, oracles, w.steps - 110, host_api=True, host_pinned=False, report=rep)
    ctx.close()
    assert rep.ok(), rep.failures[:5]
    assert rep.evictions == (w.steps - w.budget) * w.kv_heads


@pytest.mark.parametrize("kernel", [mkv.MKV_KERNEL_SIMT, mkv.MKV_KERNEL_AUTO])
def test_budget_shrink_evicts_many_at_once(kernel):
    """mkv_set_budget below the current count: the next step evicts overflow > 1 tokens (the
    general arg-min of Eq. 8: radix select, ordered hole filling)."""
    w = CONFIGS["llama_b1"].with_(prefill=130, steps=200, budget=120, variant="hot", n_heavy=3)
    ctx = make_context(w, kernel=kernel)
    stream = BatchStream(w, 0)
    oracles, _ = prefill_both(ctx, w, stream)
    rep = lockstep(ctx, w, stream, oracles, 150)
    ctx.set_budget(67)
    for o in oracles:
        o.set_budget(67)
    rep = lockstep(ctx, w, stream, oracles, 50, report=rep)
    for g in range(w.kv_heads):
        pos, _ = ctx.decode_state(0, 0, g)
        assert len(pos) == 67
    ctx.close()
    assert rep.ok(), rep.failures[:5]
    assert rep.max_out_err <= 2e-3 and rep.max_score_err <= 1e-4


def test_two_layers_keep_independent_state():
    """Steps on two layers interleaved (each layer has its own pools, scores and counters)."""
    w = CONFIGS["llama_b1"].with_(prefill=200, steps=120, budget=50, variant="hot", n_heavy=2)
    ctx = make_context(w, layers=2)
    streams = [BatchStream(w.with_(seed=s), 0) for s in (0, 1)]
    oracles = [prefill_both(ctx, w, streams[l], layer=l)[0] for l in (0, 1)]
    reps = [ParityReport(), ParityReport()]
    for _ in range(6):
        for l in (0, 1):
            lockstep(ctx, w, streams[l], oracles[l], 20, layer=l, report=reps[l], chunk=20)
    ctx.close()
    for rep in reps:
        assert rep.ok(), rep.failures[:5]
        assert rep.steps == 120 and rep.evictions > 0


@pytest.mark.parametrize("shape", ["llama_bf16", "small_f32"])
def test_layer_mean_mode_scores_over_all_heads(shape):
    """MKV_SCORE_LAYER_MEAN with several KV heads (Eq. 4 as printed: the mean runs over all H
    heads, one importance vector per sequence, every KV head evicts the same tokens)."""
    from oracle import mkv_oracle as O
    if shape == "llama_bf16":
        w = CONFIGS["llama_b1"].with_(batch=2, prefill=(100, 300), steps=220, budget=90, variant="hot", n_heavy=3)
    else:
        w = CONFIGS["tiny"].with_(q_heads=6, kv_heads=2, batch=2, prefill=70, steps=200, budget=48, variant="hot")
    ctx = make_context(w, score_mode=mkv.MKV_SCORE_LAYER_MEAN)
    stream = BatchStream(w, 0)
    oracles, _ = prefill_both(ctx, w, stream, mode=O.LAYER_MEAN)
    rep = lockstep(ctx, w, stream, oracles, 150)
    ctx.set_budget(w.budget - 20)                   # one step with overflow > 1 as well
    for o in oracles:
        o.set_budget(w.budget - 20)
    rep = lockstep(ctx, w, stream, oracles, w.steps - 150, report=rep)
    for b in range(w.batch):
        ref_pos, ref_sc = ctx.decode_state(0, b, 0)
        for g in range(1, w.kv_heads):               # identical token sets and scores in every KV head
            pos, sc = ctx.decode_state(0, b, g)
            np.testing.assert_array_equal(pos, ref_pos)
            np.testing.assert_array_equal(sc, ref_sc)
    ctx.close()
    assert rep.ok(), rep.failures[:5]
    assert rep.max_out_err <= (2e-3 if w.dtype == "bf16" else 1e-5) and rep.max_score_err <= 1e-4
    assert rep.evicted_not_newest > 20


def test_error_paths_return_status_codes():
    """Misuse is answered with a status code on the host, never with a device fault."""
    import torch
    w = CONFIGS["llama_b1"].with_(prefill=100, budget=32)
    ctx = make_context(w)
    dev = ctx.device
    q = torch.zeros((1, w.q_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
    kv = torch.zeros((1, w.kv_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
    out = torch.zeros((1, w.q_heads, w.head_dim), dtype=torch.float32, device=dev)
    with pytest.raises(mkv.MkvError) as e:
        ctx.decode_step(0, q, kv, kv, out)                       # before any prefill
    assert e.value.code == 2
    K = torch.zeros((1, w.kv_heads, 200, w.head_dim), dtype=torch.bfloat16, device=dev)
    with pytest.raises(mkv.MkvError) as e:
        ctx.prefill(0, K, K, np.array([150], dtype=np.int32))    # longer than max_prefill (100)
    assert e.value.code == 3
    with pytest.raises(mkv.MkvError) as e:
        ctx.prefill(1, K, K, np.array([50], dtype=np.int32))     # no such layer
    assert e.value.code == 1
    ctx.prefill(0, K, K, np.array([100], dtype=np.int32))
    with pytest.raises(mkv.MkvError) as e:
        ctx.set_budget(33)                                       # above the budget given at creation
    assert e.value.code == 3
    flat = torch.zeros(q.numel() + 8, dtype=torch.bfloat16, device=dev)
    with pytest.raises(mkv.MkvError) as e:
        ctx.decode_step(0, flat[1:1 + q.numel()].view_as(q), kv, kv, out)    # 2-byte aligned query
    assert e.value.code == 1
    ctx.decode_step(0, q, kv, kv, out)                           # and the context still works
    ctx.status_sync()
    assert ctx.step_count(0) == 1
    ctx.reset()
    with pytest.raises(mkv.MkvError) as e:
        ctx.attend_only(0, q, out)                               # reset: back to "not prefilled"
    assert e.value.code == 2
    ctx.close()


@pytest.mark.parametrize("mode", ["group", "layer"])
def test_head_averaged_probabilities_match_eq4(mode):
    """MKV_FLAG_RECORD_PROBS: the head-averaged attention of every decode token (Eq. 4), fresh
    token included, read back after each step and compared with the oracle's, in both score
    modes.  Their sum over the decode pool is at most 1 (the rest went to the prefill pool)."""
    import torch
    from oracle import mkv_oracle as O
    w = CONFIGS["llama_b1"].with_(prefill=150, steps=90, budget=60, variant="hot", n_heavy=2)
    smode = mkv.MKV_SCORE_LAYER_MEAN if mode == "layer" else mkv.MKV_SCORE_GROUP_MEAN
    ctx = make_context(w, record_probs=True, score_mode=smode)
    stream = BatchStream(w, 0)
    oracles, _ = prefill_both(ctx, w, stream, mode=O.LAYER_MEAN if mode == "layer" else O.GROUP_MEAN)
    dt = ctx.torch_kv_dtype()
    out = torch.zeros((1, w.q_heads, w.head_dim), dtype=torch.float32, device=ctx.device)
    qs, ks, vs = stream.next(w.steps)
    worst = 0.0
    for i in range(w.steps):
        ctx.decode_step(0, *(torch.from_numpy(np.ascontiguousarray(a[i], dtype=np.float32)).to(ctx.device, dt)
                             for a in (qs, ks, vs)), out)
        oracles[0].attend_update(qs[i, 0], ks[i, 0], vs[i, 0])
        for g in range(w.kv_heads):
            got = ctx.last_probs(0, 0, g).astype(np.float64)          # slot order before this step's eviction
            _, _, o_ab = oracles[0].decode_state(g)                   # oracle: insertion order, before evict()
            assert len(got) == len(o_ab) and got.sum() <= 1.0 + 1e-5 and (got > 0).all()
            # compare as multisets keyed by value order: slot order differs from insertion order
            np.testing.assert_allclose(np.sort(got), np.sort(o_ab), rtol=2e-4, atol=1e-9)
            worst = max(worst, float(np.abs(np.sort(got) - np.sort(o_ab)).max()))
        # keep the oracle in step with the GPU's eviction choice
        oracles[0].evict(force=[ctx.last_evicted(0, 0, g)[0].astype(np.int64) for g in range(w.kv_heads)])
    ctx.close()
    assert worst < 1e-4


def test_per_head_prefill_lengths_like_a_compressed_prompt():
    """mkv_prefill_units: every (sequence, KV head) unit keeps its own number of prompt rows and
    the two layers differ as well -- the shape of a prefill pool that a per-head / per-layer
    compressor has thinned out (the paper's plug-in setting, Sec. 6.3).  In the group score mode
    each unit is an independent instance of Algorithm 1, so the oracle is one single-KV-head
    instance per unit."""
    import torch
    from oracle import mkv_oracle as O
    rng = np.random.default_rng(5)
    B, Hq, Hkv, d, budget, beta, steps, Lmax = 2, 32, 8, 128, 70, 0.9, 130, 400
    G = Hq // Hkv
    from workloads.synthetic import round_bf16
    ctx = mkv.MomentKV(2, Hq, Hkv, d, budget, beta, B, Lmax, out_dtype=mkv.MKV_F32)
    dev = ctx.device
    oracles = {}
    for layer, hi in ((0, Lmax), (1, 120)):                      # the second layer keeps far fewer rows
        lens = rng.integers(0, hi + 1, size=(B, Hkv)).astype(np.int32)
        lens[0, 0] = 0                                           # one unit with no prompt rows at all
        K = round_bf16(rng.standard_normal((B, Hkv, Lmax, d)) / np.sqrt(d))
        V = round_bf16(rng.standard_normal((B, Hkv, Lmax, d)) / np.sqrt(d))
        ctx.prefill_units(layer, torch.from_numpy(K.astype(np.float32)).to(dev, torch.bfloat16),
                          torch.from_numpy(V.astype(np.float32)).to(dev, torch.bfloat16), lens)
        for b in range(B):
            for g in range(Hkv):
                o = O.OracleSequence(G, 1, d, budget, beta, int(lens[b, g]))
                o.prefill(K[b, g:g + 1, :lens[b, g]], V[b, g:g + 1, :lens[b, g]])
                oracles[(layer, b, g)] = o
    out = torch.zeros((B, Hq, d), dtype=torch.float32, device=dev)
    worst_out = worst_sc = 0.0
    for t in range(steps):
        for layer in (0, 1):
            q = round_bf16(4.0 * rng.standard_normal((B, Hq, d)))
            k = round_bf16(rng.standard_normal((B, Hkv, d)) / np.sqrt(d) + 0.05 * q.reshape(B, Hkv, G, d).mean(2))
            v = round_bf16(rng.standard_normal((B, Hkv, d)) / np.sqrt(d))
            ctx.decode_step(layer, *(torch.from_numpy(a.astype(np.float32)).to(dev, torch.bfloat16) for a in (q, k, v)), out)
            got = out.double().cpu().numpy()
            for b in range(B):
                for g in range(Hkv):
                    o = oracles[(layer, b, g)]
                    ref = o.attend_update(q[b, g * G:(g + 1) * G], k[b, g:g + 1], v[b, g:g + 1])
                    rowmax = np.abs(ref).max(axis=1, keepdims=True)
                    err = np.abs(got[b, g * G:(g + 1) * G] - ref) / rowmax
                    worst_out = max(worst_out, float(err.max()))
                    ev_pos, _ = ctx.last_evicted(layer, b, g)
                    choice = o.choose(0)
                    if sorted(ev_pos.tolist()) != sorted(choice.tolist()):
                        # tolerated only as a near tie at the cutoff (never seen on this seed)
                        o_pos, o_sc, _ = o.decode_state(0)
                        cut = np.sort(o_sc)[len(choice) - 1]
                        smap = dict(zip(o_pos.tolist(), o_sc.tolist()))
                        assert all(abs(smap[p] - cut) <= 1e-5 * cut for p in set(ev_pos.tolist()) ^ set(choice.tolist()))
                    o.evict(force=[ev_pos.astype(np.int64)])
                    if t % 10 == 9:
                        pos, sc = ctx.decode_state(layer, b, g)
                        o_pos, o_sc, _ = o.decode_state(0)
                        assert sorted(pos.tolist()) == sorted(o_pos.tolist())
                        rel = np.abs(sc[np.argsort(pos)] - o_sc[np.argsort(o_pos)]) / o_sc[np.argsort(o_pos)]
                        worst_sc = max(worst_sc, float(rel.max()))
    ctx.status_sync()
    ctx.close()
    assert worst_out <= 2e-3 and worst_sc <= 1e-4, (worst_out, worst_sc)


@pytest.mark.parametrize("case", ["mma_group", "simt_f32", "mma_layer"])
def test_recorded_steps_replay_as_a_cuda_graph(case):
    """A recorded sequence of decode steps (an odd number, so consecutive replays start on
    alternating copies of the work-sharing counters) replays as a CUDA graph: outputs of every
    step and the pool after every replay against the oracle run step by step (Algorithm 1)."""
    import torch
    from oracle import mkv_oracle as O
    mode, omode = mkv.MKV_SCORE_GROUP_MEAN, O.GROUP_MEAN
    if case == "simt_f32":
        w = CONFIGS["tiny"].with_(q_heads=6, kv_heads=2, batch=2, prefill=70, steps=64, budget=24, variant="hot")
    else:
        w = CONFIGS["llama_b1"].with_(batch=3, prefill=(100, 400), steps=64, budget=40, variant="hot", n_heavy=3)
        if case == "mma_layer":
            mode, omode = mkv.MKV_SCORE_LAYER_MEAN, O.LAYER_MEAN
    ctx = make_context(w, score_mode=mode)
    stream = BatchStream(w, 0)
    oracles, _ = prefill_both(ctx, w, stream, mode=omode)
    rep = lockstep(ctx, w, stream, oracles, 35)          # eager steps first: the pool is nearly full
    assert rep.ok(), rep.failures[:5]
    dt, dev, n_rec = ctx.torch_kv_dtype(), ctx.device, 3
    B = len(oracles)
    q_s = torch.zeros((n_rec, B, w.q_heads, w.head_dim), dtype=dt, device=dev)
    k_s = torch.zeros((n_rec, B, w.kv_heads, w.head_dim), dtype=dt, device=dev)
    v_s = torch.zeros_like(k_s)
    out_s = torch.zeros((n_rec, B, w.q_heads, w.head_dim), dtype=torch.float32, device=dev)
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    recorded = False
    tol = 1e-5 if w.dtype == "f32" else 2e-3
    for replay in range(5):
        qs, ks, vs = stream.next(n_rec)
        q_s.copy_(torch.from_numpy(np.ascontiguousarray(qs, dtype=np.float32)).to(dev, dt))
        k_s.copy_(torch.from_numpy(np.ascontiguousarray(ks, dtype=np.float32)).to(dev, dt))
        v_s.copy_(torch.from_numpy(np.ascontiguousarray(vs, dtype=np.float32)).to(dev, dt))
        torch.cuda.synchronize()
        if not recorded:                                  # recording runs nothing: replay it below
            with torch.cuda.graph(graph, stream=side):
                for i in range(n_rec):
                    ctx.decode_step(0, q_s[i], k_s[i], v_s[i], out_s[i])
            recorded = True
        graph.replay()
        torch.cuda.synchronize()
        got = out_s.to(torch.float64).cpu().numpy()
        for i in range(n_rec):
            for b in range(B):
                ref = oracles[b].attend_update(qs[i, b], ks[i, b], vs[i, b])
                oracles[b].evict()
                rowmax = np.abs(ref).max(axis=1)
                assert (np.abs(got[i, b] - ref).max(axis=1) <= tol * rowmax).all(), (replay, i, b)
        for b in range(B):
            for g in range(w.kv_heads):
                pos, sc = ctx.decode_state(0, b, g)
                opos, osc, _ = oracles[b].decode_state(g)
                order, oorder = np.argsort(pos), np.argsort(opos)
                np.testing.assert_array_equal(pos[order], opos[oorder])
                np.testing.assert_allclose(sc[order], osc[oorder], rtol=1e-4)
    ctx.status_sync()
    ctx.close()


@pytest.mark.parametrize("mode", ["group", "layer"])
def test_recency_window_diagnostics(mode):
    """mkv_recency_diagnostics (Sec. 3.2 / Sec. 7.1 analysis) against the oracle: the attention
    mass of the last W decoded tokens, their number, and the cumulative share of the most attended
    ones.  Two comparisons per step: the oracle fed the GPU's own recorded probabilities and
    position ids (sorting, windowing and summation: 1e-6), and the oracle fed its own fp64
    probabilities (the whole chain: the tolerance of the recorded probabilities, 3e-4)."""
    import torch
    from oracle import mkv_diagnostics as D
    from oracle import mkv_oracle as O
    w = CONFIGS["llama_b1"].with_(batch=2, prefill=(60, 150), steps=100, budget=70, variant="hot", n_heavy=2)
    smode = mkv.MKV_SCORE_LAYER_MEAN if mode == "layer" else mkv.MKV_SCORE_GROUP_MEAN
    ctx = make_context(w, record_probs=True, score_mode=smode)
    stream = BatchStream(w, 0)
    oracles, _ = prefill_both(ctx, w, stream, mode=O.LAYER_MEAN if mode == "layer" else O.GROUP_MEAN)
    dt, dev = ctx.torch_kv_dtype(), ctx.device
    B, U = w.batch, w.batch * w.kv_heads
    out = torch.zeros((B, w.q_heads, w.head_dim), dtype=torch.float32, device=dev)
    qs, ks, vs = stream.next(w.steps)
    windows = [1, 16, 256]                               # one token; inside the pool; wider than the pool
    bufs = {W: (torch.full((U,), -1.0, device=dev), torch.full((U,), -1, dtype=torch.int32, device=dev),
                torch.full((U, W), -1.0, device=dev)) for W in windows}
    # before the first step everything is zero
    ctx.recency_diagnostics(0, 16, *bufs[16])
    torch.cuda.synchronize()
    assert not bufs[16][0].any() and not bufs[16][1].any() and not bufs[16][2].any()
    checked = 0
    for i in range(w.steps):
        ctx.decode_step(0, *(torch.from_numpy(np.ascontiguousarray(a[i], dtype=np.float32)).to(dev, dt)
                             for a in (qs, ks, vs)), out)
        for b in range(B):
            oracles[b].attend_update(qs[i, b], ks[i, b], vs[i, b])
        if i % 7 == 0 or i >= w.steps - 3:
            for W in windows:
                ctx.recency_diagnostics(0, W, *bufs[W])
            torch.cuda.synchronize()
            for W in windows:
                mass, count, curve = (x.cpu().numpy() for x in bufs[W])
                for b in range(B):
                    for g in range(w.kv_heads):
                        u = b * w.kv_heads + g
                        g_ab, g_pos = ctx.last_probs(0, b, g, with_pos=True)
                        m1, c1, cv1 = D.recency_window(g_ab, g_pos, i, W)          # GPU's own inputs
                        o_pos, _, o_ab = oracles[b].decode_state(g)
                        m2, c2, cv2 = D.recency_window(o_ab, o_pos, i, W)          # the oracle's
                        assert count[u] == c1 == c2 <= min(W, len(o_pos))
                        assert mass[u] == pytest.approx(m1, rel=1e-6) and mass[u] == pytest.approx(m2, rel=3e-4)
                        np.testing.assert_allclose(curve[u, :c1], cv1, rtol=1e-6, atol=1e-7)
                        np.testing.assert_allclose(curve[u, :c1], cv2, rtol=3e-4, atol=1e-6)
                        assert not curve[u, c1:].any()
                        checked += 1
        for b in range(B):   # keep the oracle in step with the GPU's eviction choice
            oracles[b].evict(force=[ctx.last_evicted(0, b, g)[0].astype(np.int64) for g in range(w.kv_heads)])
    # argument and state errors
    with pytest.raises(mkv.MkvError):
        ctx.recency_diagnostics(0, 0, *bufs[16])
    ctx.close()
    plain = make_context(w)                              # probabilities not recorded
    with pytest.raises(mkv.MkvError):
        plain.recency_diagnostics(0, 16, *bufs[16])
    plain.close()
    assert checked > 100
