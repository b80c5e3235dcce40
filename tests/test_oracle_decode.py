"""Pins for the oracle's decode-phase attention over the kept tokens (Section 3: the selected
tokens stay in the cache and serve the decoding phase)."""
import math
import struct

import numpy as np

from oracle import laser_kv_oracle as O
from paper_2602_02199_b200 import synth


def _bf16(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _scalar(bits: int) -> float:
    return struct.unpack("<f", struct.pack("<I", int(bits) << 16))[0]


def test_hand_case_two_entries():
    # q = (1, 0); keys (ln 3, 0) and (0, 5) with scale 1 give logits ln 3 and 0 -> weights 3/4, 1/4
    # (ln 3 is not a bf16 value, so take the weights from the rounded key)
    q = _bf16([[1.0, 0.0]])
    k = _bf16([[math.log(3.0), 0.0], [0.0, 5.0]])
    v = _bf16([[2.0, -4.0], [10.0, 8.0]])
    a = math.exp(_scalar(k[0, 0]))
    want = np.array([(a * 2.0 + 10.0) / (a + 1.0), (a * -4.0 + 8.0) / (a + 1.0)])
    got = O.decode_attention(q, k, v, scale=1.0)
    assert got.shape == (1, 2)
    np.testing.assert_allclose(got[0], want, rtol=1e-14)
    assert abs(a - 3.0) < 0.02                     # the example is the 3:1 case up to bf16 rounding


def test_matches_scalar_loops_and_default_scale():
    rng = np.random.default_rng(5)
    G, n, d = 3, 7, 8
    q = _bf16(rng.standard_normal((G, d)))
    k = _bf16(rng.standard_normal((n, d)))
    v = _bf16(rng.standard_normal((n, d)))
    got = O.decode_attention(q, k, v)              # default scale 1/sqrt(d)
    for g in range(G):
        logits = []
        for i in range(n):
            acc = 0.0
            for c in range(d):
                acc += _scalar(q[g, c]) * _scalar(k[i, c])
            logits.append(acc / math.sqrt(d))
        z = sum(math.exp(x) for x in logits)
        for c in range(d):
            want = sum(math.exp(logits[i]) / z * _scalar(v[i, c]) for i in range(n))
            assert abs(got[g, c] - want) < 1e-12


def test_single_entry_returns_its_value_and_identical_keys_give_the_mean():
    rng = np.random.default_rng(6)
    q = _bf16(rng.standard_normal((2, 16)))
    k1 = _bf16(rng.standard_normal((1, 16)))
    v1 = _bf16(rng.standard_normal((1, 16)))
    got = O.decode_attention(q, k1, v1)
    np.testing.assert_allclose(got, np.repeat(O.bf16_bits_to_f64(v1), 2, axis=0), rtol=0, atol=0)
    k = np.repeat(k1, 5, axis=0)
    v = _bf16(rng.standard_normal((5, 16)))
    got = O.decode_attention(q, k, v)
    np.testing.assert_allclose(got, np.repeat(O.bf16_bits_to_f64(v).mean(axis=0)[None], 2, axis=0), rtol=1e-14)


def test_output_is_a_convex_combination_and_order_of_entries_does_not_matter():
    rng = np.random.default_rng(7)
    q = _bf16(rng.standard_normal((4, 32)) * 3)
    k = _bf16(rng.standard_normal((50, 32)) * 3)
    v = _bf16(rng.standard_normal((50, 32)))
    got = O.decode_attention(q, k, v)
    vf = O.bf16_bits_to_f64(v)
    assert (got <= vf.max(axis=0) + 1e-12).all() and (got >= vf.min(axis=0) - 1e-12).all()
    perm = rng.permutation(50)
    np.testing.assert_allclose(O.decode_attention(q, k[perm], v[perm]), got, rtol=1e-12, atol=1e-14)
    # a transposed operand or a softmax over the wrong axis breaks this: value columns are independent
    np.testing.assert_allclose(O.decode_attention(q, k, v[:, :5]), got[:, :5], rtol=1e-12, atol=1e-14)


def test_large_logits_concentrate_on_the_aligned_entry_without_overflow():
    d = 128
    base = np.zeros((6, d), np.float32)
    for i in range(6):
        base[i, i] = 40.0
    q = _bf16(base[2:3] * 2)                         # logit 3200/sqrt(128) ~ 283 for entry 2, 0 elsewhere
    v = _bf16(np.arange(6 * d, dtype=np.float32).reshape(6, d) % 17)
    got = O.decode_attention(q, _bf16(base), v)
    assert np.isfinite(got).all()
    np.testing.assert_allclose(got[0], O.bf16_bits_to_f64(v[2]), rtol=1e-12, atol=1e-100)


def test_matches_the_library_attention_routine():
    """Plain softmax attention is a library routine: torch's scaled_dot_product_attention in float64."""
    import torch
    rng = np.random.default_rng(9)
    G, n, d = 4, 300, 128
    q = _bf16(rng.standard_normal((G, d)))
    k = _bf16(rng.standard_normal((n, d)) * 2)
    v = _bf16(rng.standard_normal((n, d)))
    tq, tk, tv = (torch.from_numpy(O.bf16_bits_to_f64(x)) for x in (q, k, v))
    want = torch.nn.functional.scaled_dot_product_attention(tq[None], tk[None], tv[None])[0].numpy()
    np.testing.assert_allclose(O.decode_attention(q, k, v), want, rtol=1e-11, atol=1e-13)
    want2 = torch.nn.functional.scaled_dot_product_attention(tq[None], tk[None], tv[None], scale=0.3)[0].numpy()
    np.testing.assert_allclose(O.decode_attention(q, k, v, scale=0.3), want2, rtol=1e-11, atol=1e-13)
