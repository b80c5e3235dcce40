"""Per-layer budgets on the same kernels: every layer keeps its own number of tokens per block,
split by the protection divisor and alpha like the configured budget."""
import numpy as np
import pytest

from oracle import laser_kv_oracle as O
from paper_2602_02199_b200 import synth

from parity_util import to_np

pytestmark = pytest.mark.gpu


def test_layers_with_different_budgets():
    import torch
    from paper_2602_02199_b200 import binding as Bn
    S, nb, n_layers = 520, 3, 4
    w = synth.workload("tiny").with_(block_size=S, context_len=nb * S, n_layers=n_layers, lsh_tables=16, needles="uniform:4")
    B_max = 260
    budgets = [B_max, 130, 24, 0]
    dev = torch.device("cuda", 0)
    P = torch.from_numpy(synth.hyperplanes(w).view(np.int16)).to(dev)
    cfg = Bn.make_config(n_layers=n_layers, batch=1, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, block_size=S,
                         window=w.window, max_blocks=nb, max_blocks_per_call=nb, lsh_bits=w.lsh_bits, lsh_tables=w.lsh_tables,
                         protection_divisor=w.protection_divisor, budget_per_block=B_max, alpha=w.alpha, debug=1)
    eng = Bn.LaserKV(cfg, P)
    with pytest.raises(Bn.LaserKVError) as e:
        eng.laser_kv_set_layer_budget(1, B_max + 1)
    assert e.value.status == Bn.ERR_INVALID_ARG
    for layer in range(1, n_layers):
        eng.laser_kv_set_layer_budget(layer, budgets[layer])
    G = w.group
    for layer in range(n_layers):
        B = budgets[layer]
        a, _, _, k_e, k_l = O.partition(B, w.protection_divisor, w.alpha)
        K, V = synth.kv_blocks(w, layer, 0, 0, nb)
        Q = synth.q_window(w, layer, 0)
        tK, tV, tQ = (torch.from_numpy(x.view(np.int16)).to(dev)[None] for x in (K, V, Q))
        eng.laser_kv_select_block(layer, tK, tV, tQ, nb)
        eng.laser_kv_poll_status()
        Kc, Vc, pos, n = eng.laser_kv_cache_view(layer)
        assert n == nb * B
        if B == 0:
            with pytest.raises(Bn.LaserKVError) as e:
                eng.laser_kv_decode_attention(layer, tQ[:, :, 0, :])
            assert e.value.status == Bn.ERR_STATE
            continue
        dbg = eng.laser_kv_debug_view()
        s_all, c_all, idx_all = to_np(dbg.s_exact), to_np(dbg.counts), to_np(dbg.idx)
        assert idx_all.shape[-1] == B
        Kc, Vc, pos = to_np(Kc).view(np.uint16), to_np(Vc).view(np.uint16), to_np(pos)
        for h in range(w.n_kv_heads):
            for t in range(nb):
                # the kept set is the two-stage rule with this layer's partition on the GPU's own scores
                want = O.select_indices(s_all[0, h, t].astype(np.float64), c_all[0, h, t].astype(np.int64), S, a, k_e, k_l)[2]
                assert (idx_all[0, h, t] == want).all(), (layer, h, t)
                sl = slice(t * B, (t + 1) * B)
                assert (pos[0, h, sl] == t * S + want).all()
                assert (Kc[0, h, sl] == K[h, t * S + want]).all() and (Vc[0, h, sl] == V[h, t * S + want]).all()
        # scores agree with the oracle as in the single-budget path (one segment)
        r = O.select_block(K[:, :S], Q, synth.hyperplanes(w), n_bits=w.lsh_bits, n_tables=w.lsh_tables, B=B,
                           n=w.protection_divisor, alpha=w.alpha)
        assert (np.abs(s_all[0, 0, 0] - r.s_exact[0]) <= 1e-3 * np.abs(r.s_exact[0]) + 1e-5).all()
        # decode attention runs over this layer's shorter cache
        qd = tQ[:, :, w.window - 1, :]
        out = to_np(eng.laser_kv_decode_attention(layer, qd))
        eng.laser_kv_poll_status()
        for h in (0, w.n_kv_heads - 1):
            ref = O.decode_attention(Q[h * G:(h + 1) * G, w.window - 1], Kc[0, h, :n], Vc[0, h, :n])
            err = np.abs(out[0, h * G:(h + 1) * G] - ref)
            assert (err <= 1e-3 * np.abs(ref) + 1e-4).all()
    # a layer that holds blocks keeps its budget until it is reset
    with pytest.raises(Bn.LaserKVError) as e:
        eng.laser_kv_set_layer_budget(1, 64)
    assert e.value.status == Bn.ERR_STATE
    eng.laser_kv_reset(1)
    eng.laser_kv_set_layer_budget(1, 64)
    assert eng.laser_kv_cache_view(1)[3] == 0
