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
