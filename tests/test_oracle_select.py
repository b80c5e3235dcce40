"""Pins for the two-stage top-k (Algorithm 1 lines 4-8), the partition's keep count
(Section 3.1) and the append-only cache (Sections 1 and 3)."""
import itertools

import numpy as np
import pytest

from oracle import laser_kv_oracle as O
from paper_2602_02199_b200 import synth


def _brute_topk(cands, score, k):
    """Exhaustive: the k-subset that is lexicographically best under (score desc, index asc)."""
    best = None
    for sub in itertools.combinations(cands, k):
        rest = [c for c in cands if c not in sub]
        ok = all((score[s] > score[r]) or (score[s] == score[r] and s < r) for s in sub for r in rest)
        if ok:
            assert best is None, "the tie rule must make the answer unique"
            best = sub
    return list(best)


def test_topk_exhaustive_on_tiny_inputs():
    rng = np.random.default_rng(0)
    for trial in range(40):
        n = int(rng.integers(1, 11))
        score = rng.integers(0, 4, n + 3).astype(float)          # many ties
        cands = np.sort(rng.choice(n + 3, n, replace=False))
        for k in range(0, n + 1):
            got = O.topk_lower_index(cands, score, k).tolist()
            assert got == sorted(_brute_topk(list(cands), score, k))


def test_topk_hand_case_with_ties():
    score = np.array([5.0, 1.0, 5.0, 3.0, 5.0, 3.0])
    c = np.arange(6)
    assert O.topk_lower_index(c, score, 2).tolist() == [0, 2]
    assert O.topk_lower_index(c, score, 4).tolist() == [0, 2, 3, 4]
    assert O.topk_lower_index(c[1:], score, 3).tolist() == [2, 3, 4]
    assert O.topk_lower_index(c, score, 0).tolist() == []
    assert O.topk_lower_index(c, score, 99).tolist() == [0, 1, 2, 3, 4, 5]


def _random_case(rng, S, a):
    s_exact = rng.random(S)
    counts = rng.integers(0, 6, S)
    return s_exact, counts


def test_two_stage_invariants_and_brute_force():
    rng = np.random.default_rng(1)
    for trial in range(30):
        S, a = 16, int(rng.integers(0, 4))
        s_exact, counts = _random_case(rng, S, a)
        n_c = S - 2 * a
        k_e = int(rng.integers(0, n_c + 1))
        k_l = int(rng.integers(0, n_c - k_e + 1))
        ke, kl, idx = O.select_indices(s_exact, counts, S, a, k_e, k_l)
        cand = list(range(a, S - a))
        assert len(ke) == k_e and len(kl) == k_l
        assert set(ke) <= set(cand) and set(kl) <= set(cand) - set(ke)
        assert ke.tolist() == sorted(_brute_topk(cand, s_exact, k_e))
        resid = [c for c in cand if c not in set(ke.tolist())]
        assert kl.tolist() == sorted(_brute_topk(resid, counts.astype(float), k_l))
        assert len(idx) == 2 * a + k_e + k_l and (np.diff(idx) > 0).all()
        assert idx[:a].tolist() == list(range(a)) and idx[len(idx) - a:].tolist() == list(range(S - a, S))
        # composite-key form: top-(k_e+k_l) of 2*[j in K_exact] + count/(max_count+1)
        comp = 2.0 * np.isin(np.arange(S), ke) + counts / (counts.max() + 1.0)
        assert O.topk_lower_index(np.array(cand), comp, k_e + k_l).tolist() == sorted(ke.tolist() + kl.tolist())


def test_alpha_one_is_pure_attention_topk_and_alpha_zero_pure_lsh():
    rng = np.random.default_rng(2)
    w = synth.workload("tiny").with_(block_size=256, context_len=1024, window=8)
    k, _ = synth.kv_block(w, 0, 0, 1)
    q = synth.q_window(w, 0, 0)
    P = synth.hyperplanes(w)
    B = 100
    r1 = O.select_block(k, q, P, n_bits=8, n_tables=16, B=B, n=4, alpha=1.0)
    r0 = O.select_block(k, q, P, n_bits=8, n_tables=16, B=B, n=4, alpha=0.0)
    a, _, b_long, _, _ = O.partition(B, 4, 1.0)
    cand = np.arange(a, 256 - a)
    for h in range(w.n_kv_heads):
        assert len(r1.k_lsh[h]) == 0 and len(r0.k_exact[h]) == 0
        assert r1.k_exact[h].tolist() == O.topk_lower_index(cand, r1.s_exact[h], b_long).tolist()
        assert r0.k_lsh[h].tolist() == O.topk_lower_index(cand, r0.counts[h], b_long).tolist()
        # descending-sort definition, written independently
        order = sorted(cand.tolist(), key=lambda j: (-r1.s_exact[h][j], j))[:b_long]
        assert r1.k_exact[h].tolist() == sorted(order)


def test_keep_count_equals_budget_and_n2_keeps_only_syntactic_set():
    w = synth.workload("tiny").with_(block_size=128, context_len=512, window=4)
    k, _ = synth.kv_block(w, 0, 0, 0)
    q = synth.q_window(w, 0, 0)
    P = synth.hyperplanes(w)
    for B, n in ((40, 4), (41, 4), (40, 2), (64, 8), (0, 4)):
        r = O.select_block(k, q, P, n_bits=8, n_tables=16, B=B, n=n, alpha=0.75)
        assert r.idx.shape == (w.n_kv_heads, B)
        for h in range(w.n_kv_heads):
            assert len(set(r.idx[h].tolist())) == B
            if B:
                assert (np.diff(r.idx[h]) > 0).all() or B == 1
        if n == 2:
            a = B // 2
            assert r.idx[0].tolist() == list(range(a)) + list(range(128 - a, 128))


def test_unpicked_candidates_never_beat_picked_ones():
    w = synth.workload("tiny").with_(block_size=256, context_len=1024, window=8)
    k, _ = synth.kv_block(w, 0, 0, 2)
    r = O.select_block(k, synth.q_window(w, 0, 0), synth.hyperplanes(w), n_bits=8, n_tables=16,
                       B=96, n=4, alpha=0.5)
    a = 24
    for h in range(w.n_kv_heads):
        cand = set(range(a, 256 - a))
        ke, kl = set(r.k_exact[h].tolist()), set(r.k_lsh[h].tolist())
        rest = cand - ke
        assert min(r.s_exact[h][list(ke)]) >= max(r.s_exact[h][list(rest)])
        rest2 = rest - kl
        assert min(r.counts[h][list(kl)]) >= max(r.counts[h][list(rest2)])


def test_cache_is_append_only_with_increasing_positions():
    w = synth.workload("tiny").with_(block_size=128, context_len=512, window=4)
    q, P = synth.q_window(w, 0, 0), synth.hyperplanes(w)
    B = 32
    cache = O.AppendOnlyCache(w.n_kv_heads, w.head_dim, capacity=4 * B)
    for t in range(4):
        k, v = synth.kv_block(w, 0, 0, t)
        r = O.select_block(k, q, P, n_bits=8, n_tables=16, B=B, n=4)
        before = (cache.K.copy(), cache.V.copy(), cache.pos.copy(), cache.length)
        cache.append(k, v, r.idx, t * 128)
        assert cache.length == before[3] + B
        n0 = before[3]
        assert (cache.K[:, :n0] == before[0][:, :n0]).all()
        assert (cache.V[:, :n0] == before[1][:, :n0]).all()
        assert (cache.pos[:, :n0] == before[2][:, :n0]).all()
        for h in range(w.n_kv_heads):
            p = cache.pos[h, n0:n0 + B]
            assert (p >= t * 128).all() and (p < (t + 1) * 128).all()
            assert (cache.K[h, n0:n0 + B] == k[h, p - t * 128]).all()
            assert (cache.V[h, n0:n0 + B] == v[h, p - t * 128]).all()
    for h in range(w.n_kv_heads):
        assert (np.diff(cache.pos[h, :cache.length]) > 0).all()
    with pytest.raises(ValueError):
        cache.append(k, v, r.idx, 4 * 128)


def _small_layers(n_layers, seed=3, S=96, hkv=2, hq=4, W=8, K=4, L=8):
    w = synth.workload("tiny").with_(name="cons", n_layers=n_layers, n_q_heads=hq, n_kv_heads=hkv, window=W,
                                     lsh_bits=K, lsh_tables=L, block_size=S, context_len=2 * S, seed=seed)
    ks = [synth.kv_block(w, l, 0, 1)[0] for l in range(n_layers)]
    qs = [synth.q_window(w, l, 0) for l in range(n_layers)]
    return w, ks, qs, synth.hyperplanes(w)


def test_consensus_reduces_to_the_single_head_rule():
    # one layer with one KV head: the consensus sums are that head's own scores and counts
    w, ks, qs, P = _small_layers(1, hkv=1, hq=2)
    r = O.select_block(ks[0], qs[0], P, n_bits=4, n_tables=8, B=40, n=4)
    s, c, k_ex, k_ls, idx = O.select_block_consensus(ks, qs, P, n_bits=4, n_tables=8, B=40, n=4)
    assert (s == r.s_exact[0]).all() and (c == r.counts[0]).all()
    assert idx.tolist() == r.idx[0].tolist() and k_ex.tolist() == r.k_exact[0].tolist()


def test_consensus_sums_over_heads_and_layers():
    w, ks, qs, P = _small_layers(3)
    s, c, k_ex, k_ls, idx = O.select_block_consensus(ks, qs, P, n_bits=4, n_tables=8, B=40, n=4)
    # plain definition: add every (layer, head) array, then run the two-stage rule once
    s_ref = np.zeros(96)
    c_ref = np.zeros(96, np.int64)
    for l in range(3):
        r = O.select_block(ks[l], qs[l], P, n_bits=4, n_tables=8, B=40, n=4)
        s_ref += r.s_exact.sum(axis=0)
        c_ref += r.counts.sum(axis=0)
    assert np.allclose(s, s_ref, rtol=1e-13, atol=0) and (c == c_ref).all()
    # every softmax row sums to one: the block total is (layers * query heads * window)
    assert abs(s.sum() - 3 * 4 * 8) < 1e-9
    a, _, _, k_e, k_l = O.partition(40, 4)
    assert len(idx) == 40 and len(k_ex) == k_e and len(k_ls) == k_l
    assert idx.tolist() == O.select_indices(s_ref, c_ref, 96, a, k_e, k_l)[2].tolist()
    # the order of layers does not matter beyond rounding; counts are exact
    s2, c2, *_ = O.select_block_consensus(ks[::-1], qs[::-1], P, n_bits=4, n_tables=8, B=40, n=4)
    assert np.allclose(s2, s, rtol=1e-13, atol=0) and (c2 == c).all()


def test_consensus_of_identical_layers_keeps_the_selection():
    # the same layer repeated: sums scale by the repeat count, the chosen set does not change
    w, ks, qs, P = _small_layers(1)
    one = O.select_block_consensus(ks, qs, P, n_bits=4, n_tables=8, B=40, n=4)
    four = O.select_block_consensus(ks * 4, qs * 4, P, n_bits=4, n_tables=8, B=40, n=4)
    assert np.allclose(four[0], 4 * one[0], rtol=1e-13, atol=0) and (four[1] == 4 * one[1]).all()
    assert four[4].tolist() == one[4].tolist()
