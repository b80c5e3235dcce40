"""Pins for the oracle's look-back rule (Section 3.2, block processing and boundary smoothing): the
held-back tail of block t-1 is scored with block t's keys against block t's window and pruned only
then. Checked against the plain rule (empty local window), exhaustive search, a hand case worked
out below, and the keep-count / append-only invariants."""
import itertools
import math

import numpy as np
import pytest

from oracle import laser_kv_oracle as O
from paper_2602_02199_b200 import synth


def _bf16(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _small(S=64, seed=11, **kw):
    w = synth.workload("tiny").with_(name="lb", n_q_heads=4, n_kv_heads=2, window=4, lsh_bits=4, lsh_tables=8,
                                     block_size=S, context_len=4 * S, seed=seed, **kw)
    return w, synth.hyperplanes(w)


def test_partition_of_a_lookback_step():
    # first block: the plain recall budget; later blocks: the window's released entries join it
    assert O.lookback_partition(3855, 4, 0.75, 0) == (963, 963, 1929, 1446, 483)
    assert O.lookback_partition(3855, 4, 0.75, 963) == (963, 963, 3855 - 963, math.floor(0.75 * 2892), 2892 - 2169)
    assert O.lookback_partition(40, 2, 0.75, 20) == (20, 20, 20, 15, 5)            # n = 2: only released entries
    assert O.lookback_partition(6, 8, 0.5, 0) == (0, 0, 6, 3, 3)                   # empty window: plain rule
    # a short last block (budget 100, a = 25) after full blocks that held 963 tokens back
    assert O.lookback_partition(100, 4, 0.5, 963) == (25, 25, 50 + 963, 506, 507)


def test_empty_local_window_reduces_to_the_plain_rule():
    w, P = _small()
    q = synth.q_window(w, 0, 0)
    for t in range(3):
        k, _ = synth.kv_block(w, 0, 0, t)
        plain = O.select_block(k, q, P, n_bits=4, n_tables=8, B=6, n=8, alpha=0.5)      # a = floor(6/8) = 0
        prev = None if t == 0 else np.zeros((2, 0, 128), np.uint16)
        lb = O.select_block_lookback(prev, k, q, P, n_bits=4, n_tables=8, B=6, n=8, alpha=0.5)
        assert lb.offset == 0 and (lb.idx == plain.idx).all()
        assert np.allclose(lb.s_exact, plain.s_exact, rtol=1e-13) and (lb.counts == plain.counts).all()


def test_first_block_keeps_anchors_and_plain_picks_and_holds_its_tail_back():
    w, P = _small()
    k, _ = synth.kv_block(w, 0, 0, 0)
    q = synth.q_window(w, 0, 0)
    B, n = 24, 4
    plain = O.select_block(k, q, P, n_bits=4, n_tables=8, B=B, n=n)
    lb = O.select_block_lookback(None, k, q, P, n_bits=4, n_tables=8, B=B, n=n)
    a = B // n
    for h in range(2):
        # the plain list minus its local window [S - a, S)
        assert lb.idx[h].tolist() == [j for j in plain.idx[h].tolist() if j < 64 - a]
    assert lb.idx.shape == (2, B - a)


def _brute_two_stage(cand, s, c, k_e, k_l):
    def best(cs, score, k):
        for sub in itertools.combinations(cs, k):
            rest = [x for x in cs if x not in sub]
            if all((score[u] > score[v]) or (score[u] == score[v] and u < v) for u in sub for v in rest):
                return list(sub)
        raise AssertionError
    ke = best(cand, s, k_e)
    kl = best([x for x in cand if x not in ke], c, k_l)
    return ke, kl


def test_later_blocks_against_exhaustive_search_over_the_candidate_set():
    # tiny blocks so that every subset can be tried: S = 12, a = 2 -> scored keys 14, candidates
    # {0, 1} (the held-back tail) + {4, ..., 11} minus the block's own tail {12, 13}
    w, P = _small(S=12, seed=5)
    q = synth.q_window(w, 0, 0)
    B, n = 8, 4                                       # a = 2, later blocks: B_long = 6, k_e = 4, k_l = 2
    k0, _ = synth.kv_block(w, 0, 0, 0)
    k1, _ = synth.kv_block(w, 0, 0, 1)
    r = O.select_block_lookback(k0[:, 10:], k1, q, P, n_bits=4, n_tables=8, B=B, n=n)
    assert r.offset == -2 and r.s_exact.shape == (2, 14)
    cand = [0, 1] + list(range(4, 12))
    for h in range(2):
        ke, kl = _brute_two_stage(cand, r.s_exact[h], r.counts[h].astype(float), 4, 2)
        assert r.k_exact[h].tolist() == sorted(ke) and r.k_lsh[h].tolist() == sorted(kl)
        assert r.idx[h].tolist() == sorted([2, 3] + ke + kl)
        # one softmax over all 14 scored keys: the total is the number of window queries of the group
        assert abs(r.s_exact[h].sum() - 2 * 4) < 1e-9
        # the scores are those of the plain definition on the concatenated keys
        both = np.concatenate([k0[h, 10:], k1[h]], axis=0)
        np.testing.assert_allclose(r.s_exact[h], O.window_scores(O.group_queries(q, 2, h), both), rtol=1e-13)


def test_hand_case_a_tail_token_survives_only_if_the_next_window_attends_to_it():
    # d = 2, one head, one window query per call, S = 6, B = 4, n = 4 -> a = 1, alpha = 1 (scores only).
    # Block 0 keys: tokens 0..5; token 5 is its tail. Call 1's window is q = (4, 0) (scale 1):
    #   held-back token 5 = (2, 0)  -> logit 8
    #   block 1 tokens 6..11 = (0,0), (1,0), (0,1), (-1,0), (0.5,0), (0,0): logits 0, 4, 0, -4, 2, 0
    # Scored keys in order: [5 | 6 7 8 9 10 11]; anchors = {6}; block 1's tail {11} is held back;
    # candidates = {5, 7, 8, 9, 10}; B_long = B - a = 3 -> the three largest logits: 5 (8), 7 (4), 10 (2).
    q1 = _bf16([[[4.0, 0.0]]])
    tail0 = _bf16([[[2.0, 0.0]]])
    blk1 = _bf16([[[0, 0], [1, 0], [0, 1], [-1, 0], [0.5, 0], [0, 0]]])
    P = _bf16([[1.0, 0.0], [0.0, 1.0]])
    r = O.select_block_lookback(tail0, blk1, q1, P, n_bits=1, n_tables=2, B=4, n=4, alpha=1.0, scale=1.0)
    assert r.offset == -1
    assert r.idx[0].tolist() == [0, 1, 2, 5]                 # scored-key indices: token 5, 6 (anchor), 7, 10
    z = sum(math.exp(v) for v in (8, 0, 4, 0, -4, 2, 0))
    np.testing.assert_allclose(r.s_exact[0], [math.exp(v) / z for v in (8, 0, 4, 0, -4, 2, 0)], rtol=1e-12)
    # the same tail token under a window that ignores it, q = (-4, 0). Logits: token 5: -8 | 6: 0 (anchor),
    # 7: -4, 8: 0, 9: 4, 10: -2, 11: 0 (held back, not a candidate). Candidates {5, 7, 8, 9, 10} -> the three
    # largest: 9 (4), 8 (0), 10 (-2): token 5 is pruned and its entry goes to a token of block 1.
    q1b = _bf16([[[-4.0, 0.0]]])
    r2 = O.select_block_lookback(tail0, blk1, q1b, P, n_bits=1, n_tables=2, B=4, n=4, alpha=1.0, scale=1.0)
    assert r2.idx[0].tolist() == [1, 3, 4, 5]                # scored-key indices of tokens 6, 8, 9, 10
    # without look-back block 0 would have kept token 5 unconditionally (its local window) and block 1
    # would have kept only B_long = 2 of its middle tokens
    plain = O.select_block(blk1, q1b, P, n_bits=1, n_tables=2, B=4, n=4, alpha=1.0, scale=1.0)
    assert plain.idx[0].tolist() == [0, 2, 3, 5]             # anchor 6, picks 8 and 9, local window 11


def test_prefill_keep_counts_order_and_append_only():
    w, P = _small(S=64, seed=3)
    B, n = 24, 4
    a = B // n
    run = O.LookbackPrefill(2, 128, capacity=4 * B, n_bits=4, n_tables=8, B=B, n=n)
    lens = []
    prev = None
    for t in range(4):
        k, v = synth.kv_block(w, 0, 0, t)
        q = synth.q_window(w.with_(seed=100 + t), 0, 0)      # every block brings its own window
        run.step(k, v, q, P)
        c = run.cache
        lens.append(c.length)
        if prev is not None:                                  # entries already written never change
            m = prev[3]
            assert (c.K[:, :m] == prev[0][:, :m]).all() and (c.V[:, :m] == prev[1][:, :m]).all()
            assert (c.pos[:, :m] == prev[2][:, :m]).all()
        prev = (c.K.copy(), c.V.copy(), c.pos.copy(), c.length)
    assert lens == [B - a, 2 * B - a, 3 * B - a, 4 * B - a]
    run.close()
    c = run.cache
    assert c.length == 4 * B                                  # the same total as without look-back
    assert (c.K[:, :prev[3]] == prev[0][:, :prev[3]]).all()
    K_all = np.concatenate([synth.kv_block(w, 0, 0, t)[0] for t in range(4)], axis=1)
    V_all = np.concatenate([synth.kv_block(w, 0, 0, t)[1] for t in range(4)], axis=1)
    for h in range(2):
        p = c.pos[h, :c.length]
        assert (np.diff(p) > 0).all()                         # ascending absolute positions
        assert (c.K[h, :c.length] == K_all[h, p]).all() and (c.V[h, :c.length] == V_all[h, p]).all()
        # every block's anchors are there, and so is the last block's tail
        for t in range(4):
            assert set(range(t * 64, t * 64 + a)) <= set(p.tolist())
        assert set(range(4 * 64 - a, 4 * 64)) <= set(p.tolist())
    with pytest.raises(ValueError):
        run.step(*synth.kv_block(w, 0, 0, 0), synth.q_window(w, 0, 0), P)


def test_short_last_block_plain_rule_and_lookback_totals():
    # plain rule: a last block of S_t tokens runs with B_t = min(B, S_t)
    assert O.tail_budget(24, 40) == 24 and O.tail_budget(24, 10) == 10 and O.tail_budget(24, 24) == 24
    w, P = _small(S=64, seed=9)
    q = synth.q_window(w, 0, 0)
    k, v = synth.kv_block(w, 0, 0, 2)
    for S_t in (40, 10, 1):
        Bt = O.tail_budget(24, S_t)
        r = O.select_block(k[:, :S_t], q, P, n_bits=4, n_tables=8, B=Bt, n=4)
        assert r.idx.shape == (2, Bt) and (r.idx < S_t).all()
        if S_t <= 24:                                       # fewer tokens than the budget: all of them are kept
            assert r.idx[0].tolist() == list(range(S_t))
    # look-back with a short last block: the cache ends with (full blocks) * B + B_t entries
    B, n = 24, 4
    for S_t in (40, 10):
        run = O.LookbackPrefill(2, 128, capacity=4 * B, n_bits=4, n_tables=8, B=B, n=n)
        for t in range(2):
            kk, vv = synth.kv_block(w, 0, 0, t)
            run.step(kk, vv, q, P)
        run.step(k[:, :S_t], v[:, :S_t], q, P)
        with pytest.raises(ValueError):
            run.step(k, v, q, P)                            # nothing follows a short block
        run.close()
        Bt = O.tail_budget(B, S_t)
        assert run.cache.length == 2 * B + Bt
        for h in range(2):
            p = run.cache.pos[h, :run.cache.length]
            assert (np.diff(p) > 0).all() and p[-1] == 2 * 64 + S_t - 1
            if S_t <= B:                                    # every token of the short block is there
                assert set(range(128, 128 + S_t)) <= set(p.tolist())
