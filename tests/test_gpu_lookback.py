"""Look-back boundary smoothing (Section 3.2) on the GPU against the oracle's rule: the held-back
tail of block t-1 is scored with block t's keys and pruned then; the call pattern (all blocks at
once, block by block) does not change a byte of the cache."""
import numpy as np
import pytest

from oracle import laser_kv_oracle as O
from paper_2602_02199_b200 import synth

from parity_util import check_segment, to_np

pytestmark = pytest.mark.gpu


def _setup(w, nb, B, debug=1, lookback=1):
    import torch
    from paper_2602_02199_b200 import binding as Bn
    Ks, Vs, Qs = [], [], []
    for b in range(w.batch):
        k, v = synth.kv_blocks(w, 0, b, 0, nb)
        Ks.append(k); Vs.append(v); Qs.append(synth.q_window(w, 0, b))
    K, V, Q = np.stack(Ks), np.stack(Vs), np.stack(Qs)
    P = synth.hyperplanes(w)
    dev = torch.device("cuda", 0)
    t = dict(K=torch.from_numpy(K.view(np.int16)).to(dev), V=torch.from_numpy(V.view(np.int16)).to(dev),
             Q=torch.from_numpy(Q.view(np.int16)).to(dev), P=torch.from_numpy(P.view(np.int16)).to(dev))

    def engine():
        cfg = Bn.make_config(n_layers=1, batch=w.batch, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads,
                             block_size=w.block_size, window=w.window, max_blocks=nb, max_blocks_per_call=nb,
                             lsh_bits=w.lsh_bits, lsh_tables=w.lsh_tables, protection_divisor=w.protection_divisor,
                             budget_per_block=B, alpha=w.alpha, debug=debug, lookback=lookback)
        return Bn.LaserKV(cfg, t["P"])
    return K, V, Q, P, t, engine


def _blocks(t, S, b0, n):
    return t["K"][:, :, b0 * S:(b0 + n) * S], t["V"][:, :, b0 * S:(b0 + n) * S]


def _check_pass(w, eng, K, Q, P, B, first_block, n_blocks):
    """The debug view of the last pass (blocks first_block .. first_block + n_blocks - 1) against the oracle."""
    S, n = w.block_size, w.protection_divisor
    first = first_block == 0
    a, _, b_long, k_e, k_l = O.lookback_partition(B, n, w.alpha, 0 if first else B // n)
    dbg = eng.laser_kv_debug_view()
    off = 0 if first else a
    assert dbg.segment_keys == S + off and dbg.segment_shift == off
    s_all, c_all, idx_all = to_np(dbg.s_exact), to_np(dbg.counts), to_np(dbg.idx)
    qc_all, kc_all, lse_all = to_np(dbg.query_buckets), to_np(dbg.key_buckets), to_np(dbg.lse2)
    cand = np.concatenate([np.arange(0, off), np.arange(off + a, off + S - a)])
    kept = np.arange(off, off + a)
    n_out = a + b_long
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            for i in range(n_blocks):
                t = first_block + i
                scored = K[b, h, t * S - off:(t + 1) * S]
                check_segment(k_bits=scored, q_bits_group=O.group_queries(Q[b], w.n_kv_heads, h), p_bits=P,
                              n_bits=w.lsh_bits, n_tables=w.lsh_tables, S=S + off, anchors=a, k_exact=k_e, k_lsh=k_l,
                              scale=None, s_gpu=s_all[b, h, i], counts_gpu=c_all[b, h, i], idx_gpu=idx_all[b, h, i][:n_out],
                              qcodes_gpu=qc_all[b, h], kcodes_gpu=kc_all[b, h, i], lse2_gpu=lse_all[b, h, i],
                              what=f"lookback b{b} h{h} t{t}", cand=cand, kept=kept)
    return idx_all[..., :n_out].astype(np.int64)


@pytest.mark.parametrize("name,S,nb,B", [
    ("tiny", 512, 4, 200),                  # a = 50: the later segments have 562 keys, 4.4 tiles
    ("qwen7b_128k", 520, 3, 160),           # GQA 7, n = 8 -> a = 20, batch 2
    ("tiny", 256, 3, 128),                  # n = 4, a = 32
])
def test_lookback_select_against_oracle_and_call_patterns(name, S, nb, B):
    import torch
    w = synth.workload(name).with_(name=f"lb_{name}", block_size=S, context_len=nb * S, n_layers=1,
                                   batch=2 if name != "tiny" else 1, needles="uniform:4",
                                   lsh_bits=8, lsh_tables=16)
    K, V, Q, P, t, engine = _setup(w, nb, B)
    a = B // w.protection_divisor
    # pattern 1: the first block, then all the others in one call; every pass is checked in full
    e1 = engine()
    kb, vb = _blocks(t, S, 0, 1)
    e1.laser_kv_select_block(0, kb, vb, t["Q"], 1)
    e1.laser_kv_poll_status()
    idx0 = _check_pass(w, e1, K, Q, P, B, 0, 1)
    assert e1.laser_kv_cache_view(0)[3] == B - a
    kb, vb = _blocks(t, S, 1, nb - 1)
    e1.laser_kv_select_block(0, kb, vb, t["Q"], nb - 1)
    e1.laser_kv_poll_status()
    idx1 = _check_pass(w, e1, K, Q, P, B, 1, nb - 1)
    assert e1.laser_kv_cache_view(0)[3] == nb * B - a
    e1.laser_kv_lookback_close(0, t["K"][:, :, nb * S - a:], t["V"][:, :, nb * S - a:])
    e1.laser_kv_poll_status()
    Kc, Vc, pos, n = e1.laser_kv_cache_view(0)
    assert n == nb * B
    Kc, Vc, pos = to_np(Kc).view(np.uint16), to_np(Vc).view(np.uint16), to_np(pos)
    # the cache holds, in position order, the rows named by the GPU's own index lists, then the last tail
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            want = [idx0[b, h, 0]] + [t_ * S - a + idx1[b, h, t_ - 1] for t_ in range(1, nb)] + [np.arange(nb * S - a, nb * S)]
            want = np.concatenate(want)
            assert (pos[b, h, :n] == want).all() and (np.diff(want) > 0).all()
            assert (Kc[b, h, :n] == K[b, h, want]).all() and (Vc[b, h, :n] == V[b, h, want]).all()
    # patterns 2 and 3: everything in one call; block by block. Same bytes.
    for pattern in ("one call", "block by block"):
        e = engine()
        if pattern == "one call":
            e.laser_kv_select_block(0, t["K"], t["V"], t["Q"], nb)
        else:
            for i in range(nb):
                kb, vb = _blocks(t, S, i, 1)
                e.laser_kv_select_block(0, kb, vb, t["Q"], 1)
        e.laser_kv_lookback_close(0, t["K"][:, :, nb * S - a:], t["V"][:, :, nb * S - a:])
        e.laser_kv_poll_status()
        for x, y in zip(e.laser_kv_cache_view(0)[:3], e1.laser_kv_cache_view(0)[:3]):
            assert torch.equal(x[:, :, :n], y[:, :, :n]), pattern
        assert e.laser_kv_cache_view(0)[3] == n


def test_lookback_state_errors_and_reset():
    from paper_2602_02199_b200 import binding as Bn
    w = synth.workload("tiny").with_(name="lb_state", block_size=256, context_len=512, n_layers=1)
    K, V, Q, P, t, engine = _setup(w, 2, 96, debug=0)
    e = engine()
    tail = (t["K"][:, :, 512 - 24:], t["V"][:, :, 512 - 24:])
    with pytest.raises(Bn.LaserKVError) as err:          # nothing to close yet
        e.laser_kv_lookback_close(0, *tail)
    assert err.value.status == Bn.ERR_STATE
    e.laser_kv_select_block(0, t["K"], t["V"], t["Q"], 2)
    e.laser_kv_lookback_close(0, *tail)
    assert e.laser_kv_cache_view(0)[3] == 2 * 96
    for call in (lambda: e.laser_kv_lookback_close(0, *tail), lambda: e.laser_kv_select_block(0, t["K"], t["V"], t["Q"], 1)):
        with pytest.raises(Bn.LaserKVError) as err:      # a closed layer takes nothing more
            call()
        assert err.value.status == Bn.ERR_STATE
    e.laser_kv_reset(0)
    e.laser_kv_select_block(0, t["K"][:, :, :256], t["V"][:, :, :256], t["Q"], 1)
    assert e.laser_kv_cache_view(0)[3] == 96 - 24
    e.laser_kv_poll_status()
    # a handle without look-back refuses the close
    K2, V2, Q2, P2, t2, engine0 = _setup(w, 2, 96, debug=0, lookback=0)
    e0 = engine0()
    e0.laser_kv_select_block(0, t2["K"], t2["V"], t2["Q"], 2)
    with pytest.raises(Bn.LaserKVError) as err:
        e0.laser_kv_lookback_close(0, *tail)
    assert err.value.status == Bn.ERR_STATE


@pytest.mark.parametrize("lookback,S_t", [(0, 200), (0, 72), (0, 8), (1, 200), (1, 72), (1, 1)])
def test_short_last_block(lookback, S_t):
    """Two whole blocks and a last one of S_t < S tokens (S_t above and below the budget, and tiny):
    the short block runs with B_t = min(B, S_t); under look-back it also decides about the held-back
    tokens of the block before it."""
    import torch
    from paper_2602_02199_b200 import binding as Bn
    S, B, nb = 256, 96, 3
    w = synth.workload("tiny").with_(name=f"tail{lookback}_{S_t}", block_size=S, context_len=nb * S, n_layers=1,
                                     needles="uniform:3", lsh_bits=8, lsh_tables=16)
    K, V, Q, P, t, engine = _setup(w, nb, B, lookback=lookback)
    n, a = w.protection_divisor, B // w.protection_divisor
    T = 2 * S + S_t
    e = engine()
    e.laser_kv_select_block(0, t["K"][:, :, :2 * S], t["V"][:, :, :2 * S], t["Q"], 2)
    e.laser_kv_select_tail(0, t["K"][:, :, 2 * S:T], t["V"][:, :, 2 * S:T], t["Q"], S_t)
    e.laser_kv_poll_status()
    B_t = O.tail_budget(B, S_t)
    a_t = B_t // n
    released = a if lookback else 0
    _, _, b_long, k_e, k_l = O.lookback_partition(B_t, n, w.alpha, released) if lookback else (0, 0) + O.partition(B_t, n, w.alpha)[2:]
    dbg = e.laser_kv_debug_view()
    assert dbg.segment_keys == S_t + released and dbg.segment_shift == released
    s_all, c_all, idx_all = to_np(dbg.s_exact), to_np(dbg.counts), to_np(dbg.idx)
    qc_all, kc_all, lse_all = to_np(dbg.query_buckets), to_np(dbg.key_buckets), to_np(dbg.lse2)
    if lookback:
        cand = np.concatenate([np.arange(0, released), np.arange(released + a_t, released + S_t - a_t)])
        kept = np.arange(released, released + a_t)
    else:
        cand = np.arange(a_t, S_t - a_t)
        kept = np.concatenate([np.arange(a_t), np.arange(S_t - a_t, S_t)])
    n_out = len(kept) + k_e + k_l
    assert n_out == (B_t - a_t + released if lookback else B_t)
    for h in range(w.n_kv_heads):
        scored = K[0, h, 2 * S - released:T]
        if n_out:
            check_segment(k_bits=scored, q_bits_group=O.group_queries(Q[0], w.n_kv_heads, h), p_bits=P, n_bits=w.lsh_bits,
                          n_tables=w.lsh_tables, S=S_t + released, anchors=a_t, k_exact=k_e, k_lsh=k_l, scale=None,
                          s_gpu=s_all[0, h, 0], counts_gpu=c_all[0, h, 0], idx_gpu=idx_all[0, h, 0][:n_out],
                          qcodes_gpu=qc_all[0, h], kcodes_gpu=kc_all[0, h, 0], lse2_gpu=lse_all[0, h, 0],
                          what=f"tail h{h}", cand=cand, kept=kept)
    if lookback:
        e.laser_kv_lookback_close(0, t["K"][:, :, T - a_t:T], t["V"][:, :, T - a_t:T])
        e.laser_kv_poll_status()
    Kc, Vc, pos, length = e.laser_kv_cache_view(0)
    assert length == 2 * B + B_t
    Kc, Vc, pos = to_np(Kc).view(np.uint16), to_np(Vc).view(np.uint16), to_np(pos)
    for h in range(w.n_kv_heads):
        p = pos[0, h, :length].astype(np.int64)
        assert (np.diff(p) > 0).all() and p[-1] == T - 1 and (p < T).all()
        assert (Kc[0, h, :length] == K[0, h, p]).all() and (Vc[0, h, :length] == V[0, h, p]).all()
        if S_t <= B:                                            # a short block no larger than the budget is kept whole
            assert set(range(2 * S, T)) <= set(p.tolist())
    with pytest.raises(Bn.LaserKVError) as err:                # nothing follows a short block
        e.laser_kv_select_block(0, t["K"][:, :, :S], t["V"][:, :, :S], t["Q"], 1)
    assert err.value.status == Bn.ERR_STATE
