"""Pins for SimHash signatures and collision counts (Section 3.3 "Recall", Algorithm 1 line 6)."""
import math

import numpy as np

from oracle import laser_kv_oracle as O
from paper_2602_02199_b200 import synth


def _bf16(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def test_axis_aligned_hand_case():
    # 2 tables x 2 bits in d = 4; hyperplanes e0, e1 | e2, -e3.
    P = _bf16([[1, 0, 0, 0], [0, 1, 0, 0], [0, 0, 1, 0], [0, 0, 0, -1]])
    X = _bf16([[1, 1, 1, 1],      # t0: bits (1,1) -> 3 ; t1: bits (1, 0) -> 1
               [-1, 2, -3, -4],   # t0: (0,1) -> 2      ; t1: (0, 1) -> 2
               [0, -1, 0, 0]])    # t0: (1,0) -> 1 (zero projection counts as >= 0); t1: (1,1) -> 3
    b, m = O.simhash_buckets(X, P, n_bits=2, n_tables=2)
    assert b.tolist() == [[3, 1], [2, 2], [1, 3]]
    assert m.tolist() == [[1.0, 1.0], [1.0, 3.0], [0.0, 0.0]]


def test_positive_scaling_keeps_buckets_and_negation_complements():
    rng = np.random.default_rng(11)
    P = _bf16(rng.standard_normal((8 * 6, 32)))
    Xf = rng.standard_normal((50, 32)).astype(np.float32)
    X = _bf16(Xf)
    b, m = O.simhash_buckets(X, P, 6, 8)
    X4 = _bf16(synth.bf16_bits_to_f32(X) * 4.0)           # exact power-of-two scaling in bf16
    b4, _ = O.simhash_buckets(X4, P, 6, 8)
    assert (b4 == b).all()
    Xn = X ^ np.uint16(0x8000)                             # exact negation
    bn, _ = O.simhash_buckets(Xn, P, 6, 8)
    away = m > 0
    assert (bn[away] == (63 - b[away])).all()


def test_projection_matches_scalar_dot_and_is_not_transposed():
    rng = np.random.default_rng(2)
    P = _bf16(rng.standard_normal((12, 8)))
    X = _bf16(rng.standard_normal((5, 8)))
    proj = O.simhash_projections(X, P)
    assert proj.shape == (5, 12)
    Pf, Xf = O.bf16_bits_to_f64(P), O.bf16_bits_to_f64(X)
    for i in range(5):
        for mm in range(12):
            assert abs(proj[i, mm] - math.fsum(Xf[i, c] * Pf[mm, c] for c in range(8))) < 1e-12
    # bit b of table r is hyperplane r*K + b, least significant bit first
    b, _ = O.simhash_buckets(X, P, n_bits=3, n_tables=4)
    for i in range(5):
        for r in range(4):
            want = sum(int(proj[i, r * 3 + bb] >= 0) << bb for bb in range(3))
            assert b[i, r] == want


def test_collision_rate_follows_angle_law():
    # P[h(x) = h(y)] for one K-bit SimHash table is (1 - theta/pi)^K (Goemans-Williamson sign
    # agreement, independent bits): cos 0.9 -> 0.8564^8 = 0.2894; orthogonal pairs -> 2^-K.
    rng = np.random.default_rng(1234)
    d, K, L = 128, 8, 4096
    P = _bf16(rng.standard_normal((K * L, d)))
    x = rng.standard_normal(d)
    x /= np.linalg.norm(x)
    u = rng.standard_normal(d)
    u -= (u @ x) * x
    u /= np.linalg.norm(u)
    for cos in (0.9, 0.5, 0.0):
        y = cos * x + math.sqrt(1 - cos * cos) * u
        bx, _ = O.simhash_buckets(_bf16(x[None] * 8), P, K, L)
        by, _ = O.simhash_buckets(_bf16(y[None] * 8), P, K, L)
        rate = (bx == by).mean()
        p = (1 - math.acos(cos) / math.pi) ** K
        sigma = math.sqrt(p * (1 - p) / L)
        assert abs(rate - p) < 4 * sigma + 2e-3, (cos, rate, p)


def _counts_python_loops(qb, kb):
    out = [0] * len(kb)
    for j in range(len(kb)):
        for qi in range(len(qb)):
            for r in range(len(qb[0])):
                if qb[qi][r] == kb[j][r]:
                    out[j] += 1
    return out


def test_counts_three_formulations_agree():
    rng = np.random.default_rng(9)
    nq, S, L, K = 24, 200, 16, 4
    qb = rng.integers(0, 1 << K, (nq, L))
    kb = rng.integers(0, 1 << K, (S, L))
    got = O.collision_counts(qb, kb)
    # (a) scalar triple loop
    assert got.tolist() == _counts_python_loops(qb.tolist(), kb.tolist())
    # (b) L*nq minus the number of differing tables (XOR, nonzero test)
    differing = ((qb[None, :, :] ^ kb[:, None, :]) != 0).sum(axis=(1, 2))
    assert (got == nq * L - differing).all()
    # (c) query-bucket histogram lookups
    hist = np.zeros((L, 1 << K), np.int64)
    for r in range(L):
        np.add.at(hist[r], qb[:, r], 1)
    via_hist = hist[np.arange(L)[None, :], kb].sum(axis=1)
    assert (got == via_hist).all()


def test_counts_symmetric_and_bounded():
    rng = np.random.default_rng(10)
    a = rng.integers(0, 8, (13, 6))
    b = rng.integers(0, 8, (17, 6))
    # total collisions are the same whichever side is called "queries"
    assert O.collision_counts(a, b).sum() == O.collision_counts(b, a).sum()
    pair = np.array([[(a[i] == b[j]).sum() for j in range(17)] for i in range(13)])
    assert (O.collision_counts(a, b) == pair.sum(axis=0)).all()
    assert (O.collision_counts(b, a) == pair.sum(axis=1)).all()
    same = O.collision_counts(a, a)
    assert (same >= 6).all() and (same <= 13 * 6).all()       # a key always collides with itself
