"""Consensus aggregation on the GPU (step-level entry points through the C ABI) against the oracle:
per-head scores and collision counts, their sums over heads and layers, the shared index set and
the gather of every head with that set."""
import numpy as np
import pytest

from oracle import laser_kv_oracle as O
from paper_2602_02199_b200 import synth

from parity_util import SCORE_ATOL, SCORE_RTOL, to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,S,nb,n_layers", [("tiny", 520, 3, 2), ("qwen7b_128k", 392, 2, 3)])
def test_consensus_pipeline_against_oracle(name, S, nb, n_layers):
    import torch
    from paper_2602_02199_b200 import binding as Bn
    w = synth.workload(name).with_(block_size=S, context_len=nb * S, batch=1, n_layers=n_layers, lsh_tables=16,
                                   needles="uniform:4")
    B = Bn.laser_kv_budget(w.context_len, S, w.ratio)
    a, _, _, k_e, k_l = O.partition(B, w.protection_divisor, w.alpha)
    P = synth.hyperplanes(w)
    tP = torch.from_numpy(P.view(np.int16)).cuda()
    s_acc = c_acc = None
    Ks, Vs, Qs = [], [], []
    for layer in range(n_layers):
        K, V = synth.kv_blocks(w, layer, 0, 0, nb)
        Q = synth.q_window(w, layer, 0)
        Ks.append(K); Vs.append(V); Qs.append(Q)
        tK = torch.from_numpy(K.view(np.int16)).cuda()[None]
        tQ = torch.from_numpy(Q.view(np.int16)).cuda()[None]
        s = Bn.laser_kv_window_scores(tK, tQ, S, nb)
        c, scratch = Bn.laser_kv_collision_counts(tK, tQ, tP, S, nb, w.lsh_bits, w.lsh_tables)
        torch.cuda.synchronize()
        assert int(to_np(scratch[:4]).view(np.int32)[0]) == 0          # status word
        # the counts of every head are exact (signatures are exact up to the 1e-6 exemption, which
        # these inputs do not hit: checked below through the oracle's min |projection|)
        cn = to_np(c)
        for h in (0, w.n_kv_heads - 1):
            for t in range(nb):
                r = O.select_block(K[h:h + 1, t * S:(t + 1) * S], Q[h * w.group:(h + 1) * w.group], P,
                                   n_bits=w.lsh_bits, n_tables=w.lsh_tables, B=B, n=w.protection_divisor)
                assert min(r.key_min_abs.min(), r.query_min_abs.min()) > 1e-6
                assert (cn[0, h, t] == r.counts[0]).all(), (layer, h, t)
        s_acc, c_acc = Bn.laser_kv_consensus_accumulate(s, c, s_acc, c_acc, carry=layer > 0)
    idx = Bn.laser_kv_two_stage_topk(s_acc.view(nb, S), c_acc.view(nb, S), a, k_e, k_l)
    torch.cuda.synchronize()
    s_np, c_np, idx_np = to_np(s_acc)[0], to_np(c_acc)[0], to_np(idx)
    for t in range(nb):
        ks = [K[:, t * S:(t + 1) * S] for K in Ks]
        s_ref, c_ref, k_ex, k_ls, idx_ref = O.select_block_consensus(ks, Qs, P, n_bits=w.lsh_bits, n_tables=w.lsh_tables,
                                                                     B=B, n=w.protection_divisor, alpha=w.alpha)
        assert (c_np[t] == c_ref).all()
        err = np.abs(s_np[t] - s_ref)
        assert (err <= SCORE_RTOL * np.abs(s_ref) + SCORE_ATOL * n_layers * w.n_kv_heads).all(), err.max()
        # the GPU's own sums decide its picks exactly as the two-stage rule says
        own = O.select_indices(s_np[t].astype(np.float64), c_np[t].astype(np.int64), S, a, k_e, k_l)
        assert (idx_np[t] == own[2]).all()
        # against the oracle's picks only tokens within the tolerance band of the k_e-th score may differ
        if k_e > 0:
            cand = np.arange(a, S - a)
            kth = np.sort(s_ref[cand])[::-1][k_e - 1]
            diff = np.setxor1d(own[0], k_ex)
            assert (np.abs(s_ref[diff] - kth) <= 1e-3 * abs(kth) + SCORE_ATOL * n_layers * w.n_kv_heads).all()
    # one index set for every head: gather head by head into a [H_kv][nb*B] cache
    layer = n_layers - 1
    tK = torch.from_numpy(Ks[layer].view(np.int16)).cuda()
    tV = torch.from_numpy(Vs[layer].view(np.int16)).cuda()
    Kd = torch.zeros((w.n_kv_heads, nb * B, 128), dtype=torch.int16, device="cuda")
    Vd = torch.zeros_like(Kd)
    pos = torch.full((w.n_kv_heads, nb * B), -1, dtype=torch.int32, device="cuda")
    bad = torch.zeros(w.n_kv_heads, dtype=torch.int32, device="cuda")
    for h in range(w.n_kv_heads):
        # segments = the blocks of head h: sources S rows apart, destinations B rows apart
        Bn.laser_kv_gather_append(tK[h].view(nb, S, 128), tV[h].view(nb, S, 128), idx, Kd[h].view(nb, B, 128),
                                  Vd[h].view(nb, B, 128), pos[h].view(nb, B), 0, 0, bad[h:h + 1])
    torch.cuda.synchronize()
    assert int(bad.abs().sum()) == 0
    Kd, Vd, pos = to_np(Kd).view(np.uint16), to_np(Vd).view(np.uint16), to_np(pos)
    for h in range(w.n_kv_heads):
        for t in range(nb):
            rows = t * S + idx_np[t]
            assert (Kd[h, t * B:(t + 1) * B] == Ks[layer][h, rows]).all()
            assert (Vd[h, t * B:(t + 1) * B] == Vs[layer][h, rows]).all()
            assert (pos[h, t * B:(t + 1) * B] == idx_np[t]).all()
