"""Closed-form recall score (theoretical collision probability) on the GPU, through the C ABI,
against the oracle, and the two-stage top-k ranked by it."""
import numpy as np
import pytest

from oracle import laser_kv_oracle as O
from paper_2602_02199_b200 import synth

from parity_util import to_np

pytestmark = pytest.mark.gpu

# fp32 chain: cosine from an fp32-accumulated dot product and two fp32 norms (relative 1e-6),
# acos, log2 and exp2 approximations of a few ulp, K <= 12: relative 1e-4 at worst away from
# cos = +-1; the bound leaves a factor of ten.
TH_RTOL, TH_ATOL = 1e-3, 1e-6


@pytest.mark.parametrize("name,S,nb,batch", [
    ("tiny", 520, 3, 1),              # G*W = 128, ragged last tile, a block shorter than a CTA's run of tiles
    ("llama8b_32k", 1096, 2, 2),      # G*W = 256, RoPE, two CTAs per block, batch 2
    ("qwen7b_128k", 392, 2, 1),       # G = 7, G*W = 224
])
def test_collision_probability_against_oracle(name, S, nb, batch):
    import torch
    from paper_2602_02199_b200 import binding as Bn
    w = synth.workload(name).with_(block_size=S, context_len=nb * S, batch=batch, n_layers=1, needles="uniform:4")
    Ks, Qs = [], []
    for b in range(batch):
        k, _ = synth.kv_blocks(w, 0, b, 0, nb)
        Ks.append(k); Qs.append(synth.q_window(w, 0, b))
    K, Q = np.stack(Ks), np.stack(Qs)
    tK = torch.from_numpy(K.view(np.int16)).cuda()
    tQ = torch.from_numpy(Q.view(np.int16)).cuda()
    p, scratch = Bn.laser_kv_collision_probability(tK, tQ, S, nb, w.lsh_bits)
    torch.cuda.synchronize()
    assert int(to_np(scratch[:4]).view(np.int32)[0]) == 0
    got = to_np(p)
    G = w.group
    for b in range(batch):
        for h in range(w.n_kv_heads):
            q = O.group_queries(Q[b], w.n_kv_heads, h)
            for t in range(nb):
                want = O.collision_probability(q, K[b, h, t * S:(t + 1) * S], w.lsh_bits)
                err = np.abs(got[b, h, t] - want)
                assert (err <= TH_RTOL * want + TH_ATOL).all(), (b, h, t, err.max())
    # the recall stage ranked by it: the float bit patterns serve as the stage's keys
    B = Bn.laser_kv_budget(w.context_len, S, w.ratio)
    a, _, _, k_e, k_l = O.partition(B, w.protection_divisor, w.alpha)
    s = Bn.laser_kv_window_scores(tK, tQ, S, nb)
    idx = Bn.laser_kv_two_stage_topk(s.view(-1, S), p.view(torch.int32).view(-1, S), a, k_e, k_l)
    torch.cuda.synchronize()
    s_np, idx_np = to_np(s).reshape(-1, S), to_np(idx)
    p_np = got.reshape(-1, S)
    for seg in range(0, s_np.shape[0], 3):
        own = O.select_indices(s_np[seg].astype(np.float64), p_np[seg].astype(np.float64), S, a, k_e, k_l)
        assert (idx_np[seg] == own[2]).all(), seg


@pytest.mark.parametrize("K", [6, 7, 33])      # 6: u^K by multiplication; 7, 33: the run-time form
def test_collision_probability_special_vectors(K):
    """Keys equal to, orthogonal to and opposite to the only query direction, and a zero key."""
    import torch
    from paper_2602_02199_b200 import binding as Bn
    S, W = 64, 16
    q = np.zeros((1, 1, W, 128), np.float32)
    q[..., 0] = 2.0                                                   # every window query along e0
    k = np.zeros((1, 1, S, 128), np.float32)
    k[0, 0, 0, 0] = 3.0                                               # same direction -> 1
    k[0, 0, 1, 1] = 5.0                                               # orthogonal -> 2^-K
    k[0, 0, 2, 0] = -1.0                                              # opposite -> 0
    k[0, 0, 3, 0] = 1.0; k[0, 0, 3, 1] = 1.0                          # 45 degrees -> (3/4)^K
    tK = torch.from_numpy(synth.f32_to_bf16_bits(k).view(np.int16)).cuda()
    tQ = torch.from_numpy(synth.f32_to_bf16_bits(q).view(np.int16)).cuda()
    p, _ = Bn.laser_kv_collision_probability(tK, tQ, S, 1, K)
    got = to_np(p)[0, 0, 0]
    np.testing.assert_allclose(got[:4], [1.0, 0.5 ** K, 0.0, 0.75 ** K], rtol=2e-5, atol=1e-7)
    np.testing.assert_allclose(got[4:], 0.5 ** K, rtol=2e-5)         # zero keys count as orthogonal
