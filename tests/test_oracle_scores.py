"""Pins for the oracle's window attention scores (Section 3.3 "Precision", Algorithm 1 line 3)."""
import math
import struct

import numpy as np

from oracle import laser_kv_oracle as O
from paper_2602_02199_b200 import synth


def _bf16(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _decode_scalar(bits: int) -> float:
    """bfloat16 bit pattern -> Python float through the binary32 encoding (independent of numpy)."""
    return struct.unpack("<f", struct.pack("<I", int(bits) << 16))[0]


def _scores_python_loops(q_bits, k_bits, scale):
    """Definition written as scalar loops: softmax over keys per query, then sum over queries."""
    nq, d = q_bits.shape
    S = k_bits.shape[0]
    out = [0.0] * S
    for qi in range(nq):
        logits = []
        for j in range(S):
            acc = 0.0
            for c in range(d):
                acc += _decode_scalar(q_bits[qi, c]) * _decode_scalar(k_bits[j, c])
            logits.append(acc * scale)
        m = max(logits)
        e = [math.exp(x - m) for x in logits]
        z = math.fsum(e)
        for j in range(S):
            out[j] += e[j] / z
    return np.array(out)


def test_decode_known_bit_patterns():
    bits = np.array([0x3F80, 0xBF80, 0x4000, 0x3F00, 0x0000, 0x8000, 0x4049, 0x7F7F], np.uint16)
    want = [1.0, -1.0, 2.0, 0.5, 0.0, -0.0, 3.140625, 3.3895313892515355e38]
    got = O.bf16_bits_to_f64(bits)
    assert got.tolist() == want
    assert math.copysign(1.0, got[5]) == -1.0


def test_hand_case_d2_s4_w1():
    # q = (1, 0), keys (2,0), (0,3), (-2,1), (1,1); scale 1: logits 2, 0, -2, 1.
    q = _bf16([[1.0, 0.0]])
    k = _bf16([[2.0, 0.0], [0.0, 3.0], [-2.0, 1.0], [1.0, 1.0]])
    z = math.exp(2) + 1.0 + math.exp(-2) + math.exp(1)
    want = np.array([math.exp(2), 1.0, math.exp(-2), math.exp(1)]) / z
    got = O.window_scores(q, k, scale=1.0)
    np.testing.assert_allclose(got, want, rtol=1e-14)
    # default scale is 1/sqrt(d) = 1/sqrt(2)
    s = 1 / math.sqrt(2)
    z = sum(math.exp(x * s) for x in (2, 0, -2, 1))
    want = np.array([math.exp(x * s) for x in (2, 0, -2, 1)]) / z
    np.testing.assert_allclose(O.window_scores(q, k), want, rtol=1e-14)


def test_matches_scalar_loops_on_small_random_input():
    rng = np.random.default_rng(7)
    q = _bf16(rng.standard_normal((6, 16)))
    k = _bf16(rng.standard_normal((37, 16)) * 2.0)
    want = _scores_python_loops(q, k, 0.25)
    np.testing.assert_allclose(O.window_scores(q, k, scale=0.25), want, rtol=1e-12)
    # not symmetric in its operands: swapping q and k is a different, differently shaped result
    assert O.window_scores(k, q, scale=0.25).shape == (6,)


def test_rows_sum_to_one_so_total_is_query_count():
    rng = np.random.default_rng(3)
    for nq, S in ((128, 1024), (5, 33)):
        q = _bf16(rng.standard_normal((nq, 128)))
        k = _bf16(rng.standard_normal((S, 128)))
        s = O.window_scores(q, k)
        assert s.shape == (S,)
        assert abs(s.sum() - nq) < 1e-9 * nq
        assert (s > 0).all()


def test_identical_keys_give_uniform_scores():
    rng = np.random.default_rng(5)
    q = _bf16(rng.standard_normal((8, 128)))
    k = np.tile(_bf16(rng.standard_normal((1, 128))), (64, 1))
    np.testing.assert_allclose(O.window_scores(q, k), np.full(64, 8 / 64), rtol=1e-13)


def test_large_logits_do_not_overflow_and_concentrate_on_argmax():
    q = _bf16(np.full((1, 128), 16.0))
    k = _bf16(np.stack([np.full(128, 16.0), np.full(128, 8.0), np.zeros(128)]))
    s = O.window_scores(q, k, scale=1.0)            # logits 32768, 16384, 0
    assert np.isfinite(s).all()
    np.testing.assert_allclose(s, [1.0, 0.0, 0.0], atol=1e-300)


def test_aligned_key_ranks_first():
    # A key at cosine 0.9 with one window query and typical norm outranks random keys for the
    # softmax mass of that query (what the planted needles rely on).
    w = synth.workload("tiny")
    q = synth.q_window(w, 0, 0)
    k, _ = synth.kv_block(w, 0, 0, 0)
    G = w.group
    s = O.window_scores(q[0:G].reshape(G * w.window, w.head_dim), k[0])
    pos = synth.needle_positions(w, 0, 0)
    here = pos[pos < w.block_size]
    if here.size:
        rank = (s > s[here[0]]).sum()
        assert rank < 32


def test_matches_the_library_softmax_routine():
    """Column sums of scipy's softmax over the keys (a library routine) are the window scores."""
    from scipy.special import softmax
    rng = np.random.default_rng(21)
    q = _bf16(rng.standard_normal((24, 128)))
    k = _bf16(rng.standard_normal((200, 128)) * 1.5)
    logits = (O.bf16_bits_to_f64(q) @ O.bf16_bits_to_f64(k).T) / math.sqrt(128)
    want = softmax(logits, axis=1).sum(axis=0)
    np.testing.assert_allclose(O.window_scores(q, k), want, rtol=1e-12)
