"""Pins for the oracle's grouped-query convention: query heads h*G .. h*G+G-1 score KV head h
(Section 3.3 "Precision": the attention of the window queries summed over the heads that share
the keys). Two independent statements of the convention meet here: the explicit head lists of
this file, and the needle generator of ``synth`` (written on its own), whose planted keys are
aligned with a window query of exactly that group."""
import math

import numpy as np

from oracle import laser_kv_oracle as O
from paper_2602_02199_b200 import synth


def _bf16(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _softmax_sum_scalar(queries, keys, scale):
    """sum over the listed queries of softmax_j(<q, k_j> * scale), plain Python floats."""
    out = [0.0] * len(keys)
    for q in queries:
        logits = [scale * sum(a * b for a, b in zip(q, k)) for k in keys]
        m = max(logits)
        e = [math.exp(v - m) for v in logits]
        z = sum(e)
        for j, v in enumerate(e):
            out[j] += v / z
    return out


def test_hand_case_lists_the_query_heads_of_each_kv_head():
    # H_q = 6, H_kv = 2, G = 3, W = 1, d = 2. Every query head points somewhere else, so any other
    # assignment of query heads to KV heads changes the scores visibly.
    q = np.array([[[2.0, 0.0]], [[0.0, 2.0]], [[-2.0, 0.0]],          # heads 0, 1, 2 -> KV head 0
                  [[0.0, -2.0]], [[1.0, 1.0]], [[-1.0, 1.0]]])        # heads 3, 4, 5 -> KV head 1
    k = np.array([[[1.0, 0.0], [0.0, 1.0], [-1.0, -1.0], [0.5, 0.5]],
                  [[1.0, 0.0], [0.0, 1.0], [-1.0, -1.0], [0.5, 0.5]]])
    P = _bf16(np.array([[1.0, 0.0], [0.0, 1.0]]))
    r = O.select_block(_bf16(k), _bf16(q), P, n_bits=1, n_tables=2, B=4, n=4, alpha=1.0, scale=1.0)
    keys = k[0].tolist()
    want0 = _softmax_sum_scalar([q[0, 0].tolist(), q[1, 0].tolist(), q[2, 0].tolist()], keys, 1.0)
    want1 = _softmax_sum_scalar([q[3, 0].tolist(), q[4, 0].tolist(), q[5, 0].tolist()], keys, 1.0)
    np.testing.assert_allclose(r.s_exact[0], want0, rtol=1e-12)
    np.testing.assert_allclose(r.s_exact[1], want1, rtol=1e-12)
    # the interleaved assignment (heads 0, 2, 4 -> KV head 0) is a different function of the inputs
    wrong0 = _softmax_sum_scalar([q[0, 0].tolist(), q[2, 0].tolist(), q[4, 0].tolist()], keys, 1.0)
    assert max(abs(a - b) for a, b in zip(want0, wrong0)) > 0.1


def test_select_block_scores_equal_window_scores_on_listed_heads():
    w = synth.workload("tiny").with_(name="grp", n_q_heads=12, n_kv_heads=4, window=8, block_size=96,
                                     context_len=192, lsh_bits=4, lsh_tables=8)
    G = 3
    k, _ = synth.kv_block(w, 0, 0, 1)
    q = synth.q_window(w, 0, 0)
    P = synth.hyperplanes(w)
    r = O.select_block(k, q, P, n_bits=4, n_tables=8, B=40, n=4)
    for h in range(4):
        rows = np.concatenate([q[h * G + 0], q[h * G + 1], q[h * G + 2]], axis=0)   # heads listed one by one
        assert (O.group_queries(q, 4, h) == rows).all()
        np.testing.assert_allclose(r.s_exact[h], O.window_scores(rows, k[h]), rtol=1e-13)
        qb, _ = O.simhash_buckets(rows, P, 4, 8)
        assert (r.query_buckets[h] == qb).all()
        kb, _ = O.simhash_buckets(k[h], P, 4, 8)
        assert (r.counts[h] == O.collision_counts(qb, kb)).all()
        # a different assignment of heads gives different scores on this input
        other = np.concatenate([q[(h + 4 * g) % 12] for g in range(G)], axis=0)
        assert np.abs(O.window_scores(other, k[h]) - r.s_exact[h]).max() > 1e-3


def test_oracle_keeps_every_planted_needle_in_the_head_it_was_aligned_to():
    # synth plants, for every KV head h, a key with cosine 0.9 to a window query drawn from query
    # heads h*G .. h*G+G-1. That key must dominate that query's softmax in head h - and only there.
    w = synth.workload("tiny")                     # 8 needles over 4 blocks of 1024, G = 4, W = 32
    G, S = w.group, w.block_size
    q = synth.q_window(w, 0, 0)
    P = synth.hyperplanes(w)
    B = O.budget(w.context_len, S, w.ratio)
    pos = synth.needle_positions(w, 0, 0)
    assert pos.size == 8
    seen = 0
    for t in range(w.n_blocks):
        here = pos[(pos >= t * S) & (pos < (t + 1) * S)] - t * S
        if not here.size:
            continue
        k, _ = synth.kv_block(w, 0, 0, t)
        r = O.select_block(k, q, P, n_bits=w.lsh_bits, n_tables=w.lsh_tables, B=B, n=w.protection_divisor,
                           alpha=1.0)
        for h in range(w.n_kv_heads):
            order = np.argsort(-r.s_exact[h], kind="stable")
            top = set(order[:here.size].tolist())
            for j in here:
                assert int(j) in top, (t, h, int(j))              # the needles are the head's top scores
                assert int(j) in set(r.idx[h].tolist())            # and are kept
                # the needle takes most of one query's probability mass: its score exceeds the
                # uniform share G*W/S by far more than any ordinary key's
                assert r.s_exact[h][j] > 0.5 + G * w.window / S
                seen += 1
    assert seen == 8 * w.n_kv_heads
