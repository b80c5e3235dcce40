"""Pins for the closed-form recall score (Section 3.3 "Recall": ranking by the theoretical hash
collision probability), the expectation of Algorithm 1's collision fraction."""
import math

import numpy as np

from oracle import laser_kv_oracle as O
from paper_2602_02199_b200 import synth


def _bf16(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def test_special_angles():
    q = _bf16([[1.0, 0.0]])
    k = _bf16([[2.0, 0.0],      # same direction: never separated
               [0.0, 3.0],      # orthogonal: each hyperplane separates with probability 1/2
               [-1.0, 0.0],     # opposite: always separated
               [1.0, 1.0],      # 45 degrees: (3/4)^K
               [-1.0, 1.0]])    # 135 degrees: (1/4)^K
    for K in (1, 4, 10):
        got = O.collision_probability(q, k, K)
        np.testing.assert_allclose(got, [1.0, 0.5 ** K, 0.0, 0.75 ** K, 0.25 ** K], rtol=1e-12, atol=1e-15)


def test_mean_over_queries_and_scale_invariance():
    rng = np.random.default_rng(3)
    q = _bf16(rng.standard_normal((5, 16)))
    k = _bf16(rng.standard_normal((9, 16)))
    got = O.collision_probability(q, k, 6)
    per_query = np.stack([O.collision_probability(q[i:i + 1], k, 6) for i in range(5)])
    np.testing.assert_allclose(got, per_query.mean(axis=0), rtol=1e-13)
    # powers of two scale bf16 values exactly; angles do not change
    k4 = _bf16(synth.bf16_bits_to_f32(k) * 4.0)
    q8 = _bf16(synth.bf16_bits_to_f32(q) * 0.125)
    np.testing.assert_allclose(O.collision_probability(q8, k4, 6), got, rtol=1e-12)
    # scalar loops: a transposed operand or a wrong normalisation fails here
    for j in (0, 4, 8):
        acc = 0.0
        for i in range(5):
            a = synth.bf16_bits_to_f32(q[i]).astype(np.float64)
            b = synth.bf16_bits_to_f32(k[j]).astype(np.float64)
            cosv = float(a @ b) / math.sqrt(float(a @ a) * float(b @ b))
            acc += (1.0 - math.acos(cosv) / math.pi) ** 6
        assert abs(got[j] - acc / 5) < 1e-13


def test_is_the_expectation_of_the_empirical_collision_fraction():
    """Algorithm 1's S_lsh over many independent tables converges to the closed form."""
    rng = np.random.default_rng(11)
    d, K, L, nq, S = 32, 4, 8192, 3, 24
    q = _bf16(rng.standard_normal((nq, d)))
    base = rng.standard_normal((S, d))
    base[:8] = synth.bf16_bits_to_f32(q[0]) * 0.7 + 0.5 * base[:8]      # some keys close to a query
    k = _bf16(base)
    P = _bf16(rng.standard_normal((L * K, d)))
    qb, _ = O.simhash_buckets(q, P, K, L)
    kb, _ = O.simhash_buckets(k, P, K, L)
    frac = O.collision_counts(qb, kb) / float(L * nq)
    want = O.collision_probability(q, k, K)
    # per key the fraction is a mean of L*nq indicators (independent over tables): 5 sigma
    sigma = np.sqrt(np.maximum(want * (1 - want), 1e-6) / L)
    assert (np.abs(frac - want) < 5 * sigma + 1e-3).all(), np.abs(frac - want).max()
    assert np.corrcoef(frac, want)[0, 1] > 0.99


def test_zero_vectors_count_as_orthogonal():
    q = _bf16([[0.0, 0.0], [1.0, 0.0]])
    k = _bf16([[0.0, 0.0], [1.0, 0.0]])
    got = O.collision_probability(q, k, 2)
    np.testing.assert_allclose(got, [(0.25 + 0.25) / 2, (0.25 + 1.0) / 2], rtol=1e-14)
