"""The seeded input generators: determinism, shapes and the planted structure."""
import numpy as np

from paper_2602_02199_b200 import synth


def test_bf16_round_to_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.0e-40, 65504.0], np.float32)
    b = synth.f32_to_bf16_bits(x)
    back = synth.bf16_bits_to_f32(b)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 ties up to 1 + 2^-6
    assert back[0] == 1.0 and back[1] == 1.0 and back[2] == 1.015625 and back[3] == -2.5
    assert abs(back[5] - 65504.0) <= 256.0


def test_deterministic_and_blockwise():
    w = synth.workload("tiny")
    k1, v1 = synth.kv_block(w, 0, 0, 2)
    k2, v2 = synth.kv_block(w, 0, 0, 2)
    assert (k1 == k2).all() and (v1 == v2).all()
    assert k1.shape == (8, 1024, 128) and k1.dtype == np.uint16
    ks, vs = synth.kv_blocks(w, 0, 0, 1, 2)
    assert (ks[:, 1024:] == k1).all() and (vs[:, 1024:] == v1).all()
    k3, _ = synth.kv_block(w, 0, 1, 2)
    assert (k3 != k1).any()
    assert synth.q_window(w, 0, 0).shape == (32, 32, 128)
    assert synth.hyperplanes(w).shape == (128, 128)


def test_needles_have_cosine_0p9_with_a_window_query():
    w = synth.workload("tiny")
    pos = synth.needle_positions(w, 0, 0)
    assert len(pos) == 8 and (np.diff(pos) > 0).all()
    q = synth.bf16_bits_to_f32(synth.q_window(w, 0, 0)).astype(np.float64)
    t = int(pos[0] // w.block_size)
    k, _ = synth.kv_block(w, 0, 0, t)
    kf = synth.bf16_bits_to_f32(k).astype(np.float64)
    j = int(pos[0] - t * w.block_size)
    for h in range(w.n_kv_heads):
        qs = q[h * w.group:(h + 1) * w.group].reshape(-1, 128)
        cos = (qs @ kf[h, j]) / (np.linalg.norm(qs, axis=1) * np.linalg.norm(kf[h, j]))
        assert abs(cos.max() - 0.9) < 0.01


def test_rope_preserves_norms_and_outliers_scale_rows():
    w = synth.workload("llama8b_64k").with_(block_size=256, context_len=1024)
    k, v = synth.kv_block(w, 0, 0, 1)
    w0 = w.with_(rope_base=0.0)
    k0, v0 = synth.kv_block(w0, 0, 0, 1)
    n1 = np.linalg.norm(synth.bf16_bits_to_f32(k).astype(np.float64), axis=2)
    n0 = np.linalg.norm(synth.bf16_bits_to_f32(k0).astype(np.float64), axis=2)
    np.testing.assert_allclose(n1, n0, rtol=5e-3)
    assert (v == v0).all()
    assert (n0.max(axis=1) > 4 * np.median(n0, axis=1)).all()     # 8x outlier tokens present
