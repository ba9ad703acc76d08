"""Launch modes of the CUDA path against the oracle (needs a B200): several layers per launch,
the early-input overlap, the reproducible mode, ring depths that change the grid, and the error
path of the bounded waits."""
import numpy as np
import pytest

import paper_2605_29873_b200 as mkv
from oracle import mkv_oracle as O
from tests.parity_harness import ParityReport, lockstep, make_context, prefill_both, to_device
from workloads.synthetic import CONFIGS, BatchStream

pytestmark = pytest.mark.gpu


def stacked_inputs(streams, n, torch, dt, dev):
    """n steps of every layer's stream: numpy [n, layers, B, ...] and device tensors of the same shape."""
    qs, ks, vs = zip(*(s.next(n) for s in streams))
    qs, ks, vs = (np.stack(a, axis=1) for a in (qs, ks, vs))
    return (qs, ks, vs), tuple(to_device(a, torch, dt, dev) for a in (qs, ks, vs))


def check_layers_step(ctx, w, oracles, layers, got, q, k, v, tol, where, score_check):
    """One step of every layer in `layers` on the oracle side; compares `out`, the eviction (near
    ties tolerated as in the harness) and, when asked, every score."""
    for li, layer in enumerate(layers):
        for b in range(w.batch):
            o = oracles[layer][b]
            ref = o.attend_update(q[li, b], k[li, b], v[li, b])
            rowmax = np.abs(ref).max(axis=1)
            err = np.abs(got[li, b] - ref).max(axis=1)
            assert (err <= tol * rowmax).all(), (where, layer, b, float((err / rowmax).max()))
            force = []
            for g in range(w.kv_heads):
                ev_pos, _ = ctx.last_evicted(layer, b, g)
                choice = o.choose(g)
                assert len(ev_pos) == len(choice), (where, layer, b, g)
                if set(ev_pos.tolist()) != set(choice.tolist()):
                    o_pos, o_sc, _ = o.decode_state(g)
                    cut = np.sort(o_sc)[len(choice) - 1]
                    smap = dict(zip(o_pos.tolist(), o_sc.tolist()))
                    assert all(abs(smap[p] - cut) <= 1e-5 * cut for p in set(ev_pos.tolist()) ^ set(choice.tolist()))
                force.append(ev_pos.astype(np.int64))
            o.evict(force=force)
            if score_check:
                for g in range(w.kv_heads):
                    pos, sc = ctx.decode_state(layer, b, g)
                    o_pos, o_sc, _ = o.decode_state(g)
                    order, oorder = np.argsort(pos), np.argsort(o_pos)
                    np.testing.assert_array_equal(pos[order], o_pos[oorder])
                    np.testing.assert_allclose(sc[order], o_sc[oorder], rtol=1e-4)


@pytest.mark.parametrize("case", ["two_layers_mma", "five_layers_mma_layer_mean", "three_layers_f32"])
def test_several_layers_in_one_launch(case):
    """mkv_decode_step_layers: Algorithm 1 is per layer and the layers' inputs are independent,
    so one launch steps a run of layers.  Every layer has its own prompt lengths and its own
    oracle; ranges and single-layer calls are mixed (they use different launch plans over the same
    state), and mkv_attend_only_layers is plain attention over every layer's pools."""
    import torch
    if case == "three_layers_f32":
        w = CONFIGS["tiny"].with_(q_heads=6, kv_heads=2, batch=2, prefill=(20, 120), steps=90, budget=30, variant="hot")
        n_layers, smode, omode, tol = 3, mkv.MKV_SCORE_GROUP_MEAN, O.GROUP_MEAN, 1e-5
    else:
        w = CONFIGS["llama_b1"].with_(batch=2, prefill=(60, 420), steps=90, budget=40, variant="hot", n_heavy=2)
        n_layers = 2 if case == "two_layers_mma" else 5
        smode, omode = ((mkv.MKV_SCORE_LAYER_MEAN, O.LAYER_MEAN) if case.endswith("layer_mean")
                        else (mkv.MKV_SCORE_GROUP_MEAN, O.GROUP_MEAN))
        tol = 2e-3
    # every layer draws its own prompt lengths (seed) and its own inputs
    ws = [w.with_(seed=10 + l) for l in range(n_layers)]
    max_pre = max(int(x.prefill_lens().max()) for x in ws)
    kv_dtype = mkv.MKV_BF16 if w.dtype == "bf16" else mkv.MKV_F32
    ctx = mkv.MomentKV(n_layers, w.q_heads, w.kv_heads, w.head_dim, w.budget, w.beta, w.batch, max_pre, kv_dtype=kv_dtype,
                       out_dtype=mkv.MKV_F32, score_mode=smode)
    streams = [BatchStream(ws[l], l) for l in range(n_layers)]
    oracles = [prefill_both(ctx, ws[l], streams[l], layer=l, mode=omode)[0] for l in range(n_layers)]
    dt, dev = ctx.torch_kv_dtype(), ctx.device
    out = torch.zeros((n_layers, w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=dev)
    launches0 = ctx.launch_count()
    (qs, ks, vs), (qd, kd, vd) = stacked_inputs(streams, w.steps, torch, dt, dev)
    all_layers = list(range(n_layers))
    for i in range(w.steps):
        if i % 10 == 7:
            # the same step as one call per layer, and (for the last layers) as a shorter range
            ctx.decode_step(0, qd[i, 0], kd[i, 0], vd[i, 0], out[0])
            ctx.decode_step_layers(1, n_layers - 1, qd[i, 1:], kd[i, 1:], vd[i, 1:], out[1:])
        else:
            ctx.decode_step_layers(0, n_layers, qd[i], kd[i], vd[i], out)
        got = out.double().cpu().numpy()
        check_layers_step(ctx, w, oracles, all_layers, got, qs[i], ks[i], vs[i], tol, i, score_check=(i % 6 == 0))
    ctx.status_sync()
    assert ctx.launch_count() - launches0 == w.steps + w.steps // 10       # one launch per range step
    for l in range(n_layers):
        assert ctx.step_count(l) == w.steps
    # plain attention over every layer's pools with one launch
    rng = np.random.default_rng(5)
    q = 2.0 * np.sqrt(w.head_dim) * rng.standard_normal((n_layers, w.batch, w.q_heads, w.head_dim))
    q = to_device(q, torch, dt, "cpu").double().numpy()          # on the dtype's grid
    ctx.attend_only_layers(0, n_layers, to_device(q, torch, dt, dev), out)
    ctx.status_sync()
    got = out.double().cpu().numpy()
    Ks = [BatchStream(ws[l], l).prefill() for l in range(n_layers)]
    for l in range(n_layers):
        for b in range(w.batch):
            Kd, Vd = zip(*(oracles[l][b].decode_kv(g) for g in range(w.kv_heads)))
            Kall = np.concatenate([Ks[l][0][b], np.stack(Kd)], axis=1)
            Vall = np.concatenate([Ks[l][1][b], np.stack(Vd)], axis=1)
            N = Kall.shape[1]
            o = O.OracleSequence(w.q_heads, w.kv_heads, w.head_dim, 1 << 20, 0.5, N - 1)
            o.prefill(Kall[:, : N - 1], Vall[:, : N - 1])
            ref = o.attend_update(q[l, b], Kall[:, N - 1], Vall[:, N - 1])
            rowmax = np.abs(ref).max(axis=1, keepdims=True)
            assert (np.abs(got[l, b] - ref) <= tol * rowmax).all(), (l, b)
    # argument checks
    with pytest.raises(mkv.MkvError) as e:
        ctx.decode_step_layers(1, n_layers, qd[0], kd[0], vd[0], out)       # range beyond the last layer
    assert e.value.code == 1
    ctx.close()


def test_layer_ranges_replay_as_a_cuda_graph():
    """Recorded several-layer steps replay as a CUDA graph (the range's launch plan is built by the
    eager calls before the recording)."""
    import torch
    w = CONFIGS["llama_b1"].with_(batch=2, prefill=(80, 300), steps=40, budget=24, variant="hot", n_heavy=2)
    n_layers, n_rec = 3, 3
    ws = [w.with_(seed=30 + l) for l in range(n_layers)]
    max_pre = max(int(x.prefill_lens().max()) for x in ws)
    ctx = mkv.MomentKV(n_layers, w.q_heads, w.kv_heads, w.head_dim, w.budget, w.beta, w.batch, max_pre, out_dtype=mkv.MKV_F32)
    streams = [BatchStream(ws[l], l) for l in range(n_layers)]
    oracles = [prefill_both(ctx, ws[l], streams[l], layer=l)[0] for l in range(n_layers)]
    dt, dev = ctx.torch_kv_dtype(), ctx.device
    out = torch.zeros((n_layers, w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=dev)
    (qs, ks, vs), (qd, kd, vd) = stacked_inputs(streams, 20, torch, dt, dev)
    for i in range(20):                                   # eager: builds the plan, nearly fills the pool
        ctx.decode_step_layers(0, n_layers, qd[i], kd[i], vd[i], out)
        check_layers_step(ctx, w, oracles, list(range(n_layers)), out.double().cpu().numpy(), qs[i], ks[i], vs[i], 2e-3, i, False)
    q_s, k_s, v_s = (torch.zeros((n_rec,) + tuple(x.shape[1:]), dtype=dt, device=dev) for x in (qd, kd, vd))
    out_s = torch.zeros((n_rec,) + tuple(out.shape), dtype=torch.float32, device=dev)
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        for j in range(n_rec):
            ctx.decode_step_layers(0, n_layers, q_s[j], k_s[j], v_s[j], out_s[j])
    for replay in range(5):
        (qs, ks, vs), (qd, kd, vd) = stacked_inputs(streams, n_rec, torch, dt, dev)
        q_s.copy_(qd); k_s.copy_(kd); v_s.copy_(vd)
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        got = out_s.double().cpu().numpy()
        for j in range(n_rec):
            # evictions of the steps inside a replay cannot be read back one by one: the oracle
            # takes its own choice and the pools are compared after the replay
            for l in range(n_layers):
                for b in range(w.batch):
                    ref = oracles[l][b].attend_update(qs[j, l, b], ks[j, l, b], vs[j, l, b])
                    oracles[l][b].evict()
                    rowmax = np.abs(ref).max(axis=1)
                    assert (np.abs(got[j, l, b] - ref).max(axis=1) <= 2e-3 * rowmax).all(), (replay, j, l, b)
        for l in range(n_layers):
            for b in range(w.batch):
                for g in range(w.kv_heads):
                    pos, sc = ctx.decode_state(l, b, g)
                    o_pos, o_sc, _ = oracles[l][b].decode_state(g)
                    np.testing.assert_array_equal(np.sort(pos), np.sort(o_pos))
                    np.testing.assert_allclose(sc[np.argsort(pos)], o_sc[np.argsort(o_pos)], rtol=1e-4)
    ctx.status_sync()
    ctx.close()


@pytest.mark.parametrize("head_tiles", [4, 9])
@pytest.mark.parametrize("mode", ["group", "layer"])
def test_early_inputs_overlap_keeps_parity(mode, head_tiles):
    """MKV_FLAG_INPUTS_READY: the consumers start on the CTA's reserved prompt tiles before the
    previous step of the stream has ended.  Steps are enqueued back to back, many per
    synchronisation, so that consecutive launches really overlap; every step's `out` and the final
    pools are compared with the oracle."""
    import torch
    w = CONFIGS["llama_b16"].with_(batch=6, prefill=(300, 2500), steps=200, budget=96, variant="hot", n_heavy=3)
    smode, omode = ((mkv.MKV_SCORE_LAYER_MEAN, O.LAYER_MEAN) if mode == "layer" else (mkv.MKV_SCORE_GROUP_MEAN, O.GROUP_MEAN))
    ctx = make_context(w, score_mode=smode, flags=mkv.MKV_FLAG_INPUTS_READY)
    ctx.set_option(mkv.MKV_OPT_HEAD_TILES, head_tiles)
    stream = BatchStream(w, 0)
    oracles, _ = prefill_both(ctx, w, stream, mode=omode)
    dt, dev = ctx.torch_kv_dtype(), ctx.device
    burst = 25
    outs = torch.zeros((burst, w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=dev)
    near = 0
    for start in range(0, w.steps, burst):
        qs, ks, vs = stream.next(burst)
        qd, kd, vd = (to_device(a, torch, dt, dev) for a in (qs, ks, vs))
        torch.cuda.synchronize()                          # the inputs are final before any step is enqueued
        for j in range(burst):
            ctx.decode_step(0, qd[j], kd[j], vd[j], outs[j])
        ctx.status_sync()
        got = outs.double().cpu().numpy()
        for j in range(burst):
            for b in range(w.batch):
                ref = oracles[b].attend_update(qs[j, b], ks[j, b], vs[j, b])
                rowmax = np.abs(ref).max(axis=1)
                assert (np.abs(got[j, b] - ref).max(axis=1) <= 2e-3 * rowmax).all(), (start + j, b)
                oracles[b].evict()
        # the pools after the burst (a near tie inside a burst would show here)
        for b in range(w.batch):
            for g in range(w.kv_heads):
                pos, sc = ctx.decode_state(0, b, g)
                o_pos, o_sc, _ = oracles[b].decode_state(g)
                if sorted(pos.tolist()) != sorted(o_pos.tolist()):
                    near += 1
                    continue
                np.testing.assert_allclose(sc[np.argsort(pos)], o_sc[np.argsort(o_pos)], rtol=1e-4)
        assert near == 0, "eviction sets differ after a burst"
    ctx.close()


@pytest.mark.parametrize("mode", ["group", "layer"])
@pytest.mark.parametrize("n_layers", [2, 3])
def test_steps_of_different_layers_run_side_by_side(mode, n_layers):
    """With MKV_FLAG_INPUTS_READY a step on another layer than the previous one does not wait for
    it: it streams alongside (its own pools and counters, the other set of scratch) and only
    completes behind it.  Layers are cycled back to back, many steps per synchronisation, each
    step with an output buffer of its own; every output and, after every burst, every pool and
    score is compared with the per-layer oracles.  With two layers a step's successor-but-one is
    the same layer again, which must see the step complete."""
    import torch
    w = CONFIGS["llama_b16"].with_(batch=5, prefill=(300, 2500), steps=120, budget=64, variant="hot", n_heavy=3)
    smode, omode = ((mkv.MKV_SCORE_LAYER_MEAN, O.LAYER_MEAN) if mode == "layer" else (mkv.MKV_SCORE_GROUP_MEAN, O.GROUP_MEAN))
    ws = [w.with_(seed=50 + l) for l in range(n_layers)]
    max_pre = max(int(x.prefill_lens().max()) for x in ws)
    ctx = mkv.MomentKV(n_layers, w.q_heads, w.kv_heads, w.head_dim, w.budget, w.beta, w.batch, max_pre, out_dtype=mkv.MKV_F32,
                       score_mode=smode, flags=mkv.MKV_FLAG_INPUTS_READY)
    streams = [BatchStream(ws[l], l) for l in range(n_layers)]
    oracles = [prefill_both(ctx, ws[l], streams[l], layer=l, mode=omode)[0] for l in range(n_layers)]
    dt, dev = ctx.torch_kv_dtype(), ctx.device
    burst = 20
    outs = torch.zeros((burst, n_layers, w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=dev)
    for start in range(0, w.steps, burst):
        (qs, ks, vs), (qd, kd, vd) = stacked_inputs(streams, burst, torch, dt, dev)
        torch.cuda.synchronize()                          # the inputs are final before any step is enqueued
        for j in range(burst):
            for l in range(n_layers):
                ctx.decode_step(l, qd[j, l], kd[j, l], vd[j, l], outs[j, l])
        ctx.status_sync()
        got = outs.double().cpu().numpy()
        for j in range(burst):
            for l in range(n_layers):
                for b in range(w.batch):
                    ref = oracles[l][b].attend_update(qs[j, l, b], ks[j, l, b], vs[j, l, b])
                    rowmax = np.abs(ref).max(axis=1)
                    assert (np.abs(got[j, l, b] - ref).max(axis=1) <= 2e-3 * rowmax).all(), (start + j, l, b)
                    oracles[l][b].evict()
        for l in range(n_layers):
            for b in range(w.batch):
                for g in range(w.kv_heads):
                    pos, sc = ctx.decode_state(l, b, g)
                    o_pos, o_sc, _ = oracles[l][b].decode_state(g)
                    np.testing.assert_array_equal(np.sort(pos), np.sort(o_pos))
                    np.testing.assert_allclose(sc[np.argsort(pos)], o_sc[np.argsort(o_pos)], rtol=1e-4)
    for l in range(n_layers):
        assert ctx.step_count(l) == w.steps
    ctx.close()


@pytest.mark.parametrize("case", ["mma_group", "mma_layer", "simt_f32", "simt_f32_layer"])
def test_reproducible_mode_gives_the_same_bits_twice(case):
    """MKV_FLAG_REPRODUCIBLE: two contexts fed the same 300 steps (ragged batch, evictions of all
    ages) agree bit for bit in every `out`, every score, every position id and every pool row --
    and with the oracle within the usual tolerances.  Without the flag the work sharing is decided
    by counters at run time and the last bits of the sums may differ; with it a difference between
    two runs means a race."""
    import torch
    if case.startswith("simt"):
        w = CONFIGS["tiny"].with_(q_heads=6, kv_heads=2, batch=3, prefill=(20, 150), steps=300, budget=40, variant="hot")
    else:
        w = CONFIGS["llama_b16"].with_(batch=5, prefill=(90, 700), steps=300, budget=140, variant="hot", n_heavy=4)
    smode, omode = ((mkv.MKV_SCORE_LAYER_MEAN, O.LAYER_MEAN) if case.endswith("layer") else (mkv.MKV_SCORE_GROUP_MEAN, O.GROUP_MEAN))
    ctxs = [make_context(w, score_mode=smode, flags=mkv.MKV_FLAG_REPRODUCIBLE) for _ in range(2)]
    stream = BatchStream(w, 0)
    oracles, _ = prefill_both(ctxs[0], w, stream, mode=omode)
    prefill_both(ctxs[1], w, BatchStream(w, 0), mode=omode)
    dt, dev = ctxs[0].torch_kv_dtype(), ctxs[0].device
    outs = [torch.zeros((w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=dev) for _ in range(2)]
    tol = 1e-5 if w.dtype == "f32" else 2e-3
    qs, ks, vs = stream.next(w.steps)
    qd, kd, vd = (to_device(a, torch, dt, dev) for a in (qs, ks, vs))
    for i in range(w.steps):
        for c in range(2):
            ctxs[c].decode_step(0, qd[i], kd[i], vd[i], outs[c])
        assert torch.equal(outs[0], outs[1]), f"step {i}: outputs differ between two runs"
        if i % 3 == 0 or i >= w.steps - 5:
            got = outs[0].double().cpu().numpy()
        for b in range(w.batch):
            ref = oracles[b].attend_update(qs[i, b], ks[i, b], vs[i, b])
            if i % 3 == 0 or i >= w.steps - 5:
                rowmax = np.abs(ref).max(axis=1)
                assert (np.abs(got[b] - ref).max(axis=1) <= tol * rowmax).all(), (i, b)
            oracles[b].evict(force=[ctxs[0].last_evicted(0, b, g)[0].astype(np.int64) for g in range(w.kv_heads)])
        if i % 25 == 24 or i == w.steps - 1:
            for b in range(w.batch):
                for g in range(w.kv_heads):
                    (p0, s0), (p1, s1) = (c.decode_state(0, b, g) for c in ctxs)
                    np.testing.assert_array_equal(p0, p1)                      # same slots, not only same sets
                    np.testing.assert_array_equal(s0.view(np.uint32), s1.view(np.uint32))
                    for pool in (0, 1):
                        (K0, V0), (K1, V1) = (c.read_kv(0, b, g, pool) for c in ctxs)
                        np.testing.assert_array_equal(K0, K1)
                        np.testing.assert_array_equal(V0, V1)
                    o_pos, o_sc, _ = oracles[b].decode_state(g)
                    np.testing.assert_array_equal(np.sort(p0), np.sort(o_pos))
                    np.testing.assert_allclose(s0[np.argsort(p0)], o_sc[np.argsort(o_pos)], rtol=1e-4)
    for c in ctxs:
        c.status_sync()
        c.close()


def test_reproducible_mode_with_launches_side_by_side():
    """Both flags together: launches on different layers overlap in time, but each has its own
    scratch and a fixed partition, so two contexts stepped the same way still agree bit for bit
    (outputs of every step, pools and scores of both layers at the end)."""
    import torch
    w = CONFIGS["llama_b16"].with_(batch=4, prefill=(200, 1500), steps=80, budget=48, variant="hot", n_heavy=2)
    n_layers = 2
    ws = [w.with_(seed=70 + l) for l in range(n_layers)]
    max_pre = max(int(x.prefill_lens().max()) for x in ws)
    flags = mkv.MKV_FLAG_REPRODUCIBLE | mkv.MKV_FLAG_INPUTS_READY
    ctxs = [mkv.MomentKV(n_layers, w.q_heads, w.kv_heads, w.head_dim, w.budget, w.beta, w.batch, max_pre,
                         out_dtype=mkv.MKV_F32, flags=flags) for _ in range(2)]
    streams = [BatchStream(ws[l], l) for l in range(n_layers)]
    oracles = [prefill_both(ctxs[0], ws[l], streams[l], layer=l)[0] for l in range(n_layers)]
    for l in range(n_layers):
        prefill_both(ctxs[1], ws[l], BatchStream(ws[l], l), layer=l)
    dt, dev = ctxs[0].torch_kv_dtype(), ctxs[0].device
    burst = 20
    outs = [torch.zeros((burst, n_layers, w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=dev) for _ in range(2)]
    for start in range(0, w.steps, burst):
        (qs, ks, vs), (qd, kd, vd) = stacked_inputs(streams, burst, torch, dt, dev)
        torch.cuda.synchronize()
        for c in range(2):
            for j in range(burst):
                for l in range(n_layers):
                    ctxs[c].decode_step(l, qd[j, l], kd[j, l], vd[j, l], outs[c][j, l])
            ctxs[c].status_sync()
        assert torch.equal(outs[0], outs[1]), f"steps {start}..: outputs differ between two runs"
        got = outs[0].double().cpu().numpy()
        for j in range(burst):
            for l in range(n_layers):
                for b in range(w.batch):
                    ref = oracles[l][b].attend_update(qs[j, l, b], ks[j, l, b], vs[j, l, b])
                    rowmax = np.abs(ref).max(axis=1)
                    assert (np.abs(got[j, l, b] - ref).max(axis=1) <= 2e-3 * rowmax).all(), (start + j, l, b)
                    oracles[l][b].evict()
    for l in range(n_layers):
        for b in range(w.batch):
            for g in range(w.kv_heads):
                (p0, s0), (p1, s1) = (c.decode_state(l, b, g) for c in ctxs)
                np.testing.assert_array_equal(p0, p1)
                np.testing.assert_array_equal(s0.view(np.uint32), s1.view(np.uint32))
                (K0, V0), (K1, V1) = (c.read_kv(l, b, g, 1) for c in ctxs)
                np.testing.assert_array_equal(K0, K1)
                np.testing.assert_array_equal(V0, V1)
    for c in ctxs:
        c.close()


@pytest.mark.parametrize("stages", [2, 5])
def test_ring_depth_resizes_the_grid(stages):
    """MKV_OPT_RING_STAGES: with five 32 KB stages only one CTA of the tensor-core kernel fits an
    SM, and the grid must shrink to one CTA per SM -- its CTAs wait on one another, so a grid that
    is not resident as a whole would run into the wait limit.  Parity holds at either depth."""
    import torch
    w = CONFIGS["llama_b16"].with_(batch=5, prefill=(200, 3000), steps=150, budget=70, variant="hot", n_heavy=3)
    ctx = make_context(w)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert ctx.grid(0)[1] == 2 * sms
    ctx.set_option(mkv.MKV_OPT_RING_STAGES, stages)
    assert ctx.grid(0) == (0, (1 if stages == 5 else 2) * sms)       # not prefilled any more; new bound
    with pytest.raises(mkv.MkvError) as e:
        ctx.set_option(mkv.MKV_OPT_RING_STAGES, 7)                    # does not fit the shared memory
    assert e.value.code == 1
    stream = BatchStream(w, 0)
    oracles, _ = prefill_both(ctx, w, stream)
    assert 0 < ctx.grid(0)[0] <= ctx.grid(0)[1]
    rep = lockstep(ctx, w, stream, oracles, w.steps, check_state_every=3)
    ctx.close()
    assert rep.ok(), rep.failures[:5]
    assert rep.max_out_err <= 2e-3 and rep.max_score_err <= 1e-4


def test_a_wait_that_runs_out_ends_the_step_with_a_status():
    """The error path of the kernel's bounded waits, made to happen from the host: one tile of one
    unit is marked as never delivered, so that unit's finishing part waits for a count that cannot
    come, gives up at the wait limit (set to 20 ms here) and the step ends with MKV_ERR_TIMEOUT in
    the sticky status.  Nothing traps and nothing spins without bound.  After mkv_reset and a new
    prefill the context passes a parity run again."""
    import time
    import torch
    w = CONFIGS["llama_b1"].with_(batch=2, prefill=(100, 260), steps=60, budget=30, variant="hot", n_heavy=2)
    ctx = make_context(w, kernel=mkv.MKV_KERNEL_MMA)
    ctx.set_option(mkv.MKV_OPT_WAIT_LIMIT_US, 20000)
    stream = BatchStream(w, 0)
    oracles, _ = prefill_both(ctx, w, stream)
    rep = lockstep(ctx, w, stream, oracles, 20)
    assert rep.ok(), rep.failures[:5]
    ctx.debug_inject(0, mkv.MKV_INJECT_LOST_TILE, 1, 3)
    dt, dev = ctx.torch_kv_dtype(), ctx.device
    qs, ks, vs = stream.next(1)
    out = torch.zeros((w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=dev)
    t0 = time.perf_counter()
    ctx.decode_step(0, *(to_device(a[0], torch, dt, dev) for a in (qs, ks, vs)), out)
    with pytest.raises(mkv.MkvError) as e:
        ctx.status_sync()
    elapsed = time.perf_counter() - t0
    assert e.value.code == 7                                          # MKV_ERR_TIMEOUT
    assert 0.015 < elapsed < 1.5                                      # it waited for the limit, not for 2 s
    with pytest.raises(mkv.MkvError):
        ctx.status_sync()                                             # sticky until reset
    ctx.reset()
    ctx.status_sync()
    stream = BatchStream(w, 0)
    oracles, _ = prefill_both(ctx, w, stream)
    rep = lockstep(ctx, w, stream, oracles, w.steps)
    ctx.close()
    assert rep.ok(), rep.failures[:5]
    assert rep.evictions == (w.steps - w.budget) * w.batch * w.kv_heads
