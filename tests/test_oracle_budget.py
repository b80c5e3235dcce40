"""Pins for the oracle's budget arithmetic (Appendix B Eq. 1, Section 3.1, Algorithm 1 l.4/7)."""
import os
from fractions import Fraction

import pytest

from oracle import laser_kv_oracle as O


def _rows(path):
    with open(path) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line.split()


def test_budget_matches_hand_values(golden_dir):
    n = 0
    for S, L, r, B in _rows(os.path.join(golden_dir, "budget_eq1.txt")):
        assert O.budget(int(L), int(S), float(r)) == int(B)
        n += 1
    assert n >= 8


def test_budget_exact_rational_sweep():
    # Eq. 1 evaluated in exact rational arithmetic; r is a binary fraction so the double
    # evaluation must agree wherever the quotient is not within 1e-9 of an integer.
    for S in (512, 1024, 4096, 8192, 5000):
        for L in (4096, 16384, 65536, 131072, 100000, 1 << 20):
            for r in (0.25, 0.5, 0.125):
                exact = Fraction(2) * Fraction(r) * S * L / (S + L)
                assert O.budget(L, S, r) == exact.numerator // exact.denominator


def test_budget_is_harmonic_mean_scaled():
    # B = r * harmonic_mean(S, L) rounded down; symmetric in (S, L); S == L gives r*S.
    assert O.budget(4096, 4096, 0.25) == 1024
    assert O.budget(16384, 4096) == O.budget(4096, 16384)
    assert O.budget(10**9, 4096, 0.25) == 2047      # L -> inf: 2 r S = 2048, approached from below


def test_partition_matches_hand_values(golden_dir):
    for B, n, alpha, a, loc, bl, ke, kl in _rows(os.path.join(golden_dir, "partition_sec3_1.txt")):
        assert O.partition(int(B), int(n), float(alpha)) == (int(a), int(loc), int(bl), int(ke), int(kl))


def test_partition_keep_count_is_budget():
    for B in range(0, 300, 7):
        for n in (2, 3, 4, 8, 16):
            for alpha in (0.0, 0.25, 0.5, 0.75, 1.0):
                a, loc, bl, ke, kl = O.partition(B, n, alpha)
                assert a == loc == B // n
                assert a + loc + ke + kl == B and bl == ke + kl
                assert 0 <= ke <= bl
                if alpha == 1.0:
                    assert kl == 0
                if alpha == 0.0:
                    assert ke == 0


def test_partition_rejects_bad_arguments():
    with pytest.raises(ValueError):
        O.partition(100, 1, 0.5)
    with pytest.raises(ValueError):
        O.partition(100, 4, 1.5)
    with pytest.raises(ValueError):
        O.budget(0, 4096)
