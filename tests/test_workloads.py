"""The synthetic input generator: determinism, shapes, dtype grid (CPU only)."""
import numpy as np

from workloads.synthetic import CONFIGS, BatchStream, SequenceStream, round_bf16


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -7, -3.14159, 0.0])
    r = round_bf16(x)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0 + 2 ** -6 and r[3] == 1.0 + 2 ** -7
    assert abs(r[4] + 3.14159) <= 2 ** -7 and r[5] == 0.0
    # values are on the bf16 grid: low 16 bits of the fp32 pattern are zero
    assert not (r.astype(np.float32).view(np.uint32) & 0xFFFF).any()


def test_streams_are_deterministic_and_chunking_invariant():
    w = CONFIGS["llama_b1"].with_(steps=64)
    a = SequenceStream(w, 0, 0, prefill_len=16)
    b = SequenceStream(w, 0, 0, prefill_len=16)
    qa, ka, va = a.next(24)
    parts = [b.next(8) for _ in range(3)]
    np.testing.assert_array_equal(qa, np.concatenate([p[0] for p in parts]))
    np.testing.assert_array_equal(ka, np.concatenate([p[1] for p in parts]))
    np.testing.assert_array_equal(va, np.concatenate([p[2] for p in parts]))
    assert qa.shape == (24, 32, 128) and ka.shape == (24, 8, 128)


def test_config_shapes_and_heavy_hitters():
    w = CONFIGS["llama_b16"]
    lens = w.prefill_lens()
    assert lens.shape == (16,) and lens.min() >= 512 and lens.max() <= 4096
    np.testing.assert_array_equal(lens, w.prefill_lens())
    t = CONFIGS["tiny"]
    s = SequenceStream(t, 0, 0)
    q, k, v = s.next(t.steps)
    for j, tj in enumerate(t.heavy_steps()):
        np.testing.assert_allclose(np.linalg.norm(k[tj, 0]), t.hh_scale, rtol=1e-6)
    bs = BatchStream(CONFIGS["qwen_b64"].with_(batch=3, steps=4))
    q, k, v = bs.next(4)
    assert q.shape == (4, 3, 28, 128) and k.shape == (4, 3, 4, 128)


def test_algorithmic_bytes_of_the_headline_step():
    """The roofline numerator: K and V of every cached token once per KV head, the appended rows,
    the scores read and written, q and out, and one row moved per unit -- 237.8 MB for the
    headline workload, written out here term by term."""
    import bench
    w = CONFIGS["llama_b16"]
    lens = w.prefill_lens()
    assert int(lens.sum()) == 41292
    n, units = w.budget + 1, w.batch * w.kv_heads
    want = (w.kv_heads * (int(lens.sum()) + w.batch * n) * 512     # K+V rows streamed
            + units * 512                                           # fresh rows appended
            + units * n * 8                                         # scores read and written
            + 2 * w.batch * w.q_heads * w.head_dim * 2              # q in, out back (bf16)
            + units * 1 * 2 * 520)                                  # one token moved per unit
    assert want == 237816832
    assert bench.algorithmic_bytes_per_step(w, lens, n, 1) == want
