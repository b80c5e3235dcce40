"""Decode-phase attention over the compacted cache on the GPU (through the C ABI) against the oracle:
the oracle selects with its own rule, appends into its own cache and attends over it in fp64."""
import numpy as np
import pytest

from oracle import laser_kv_oracle as O
from paper_2602_02199_b200 import synth

from parity_util import run_workload_layer, to_np

pytestmark = pytest.mark.gpu

# fp32 products and sums of bf16 inputs against fp64: the relative error of a softmax-weighted mean
# of len terms stays far below 1e-3; the absolute term covers outputs that cancel to nearly zero.
DEC_RTOL, DEC_ATOL = 1e-3, 1e-4


def _oracle_cache(w, run, b):
    """The oracle's own selection and append for sequence b of the run's inputs."""
    S, nb = w.block_size, run["n_blocks"]
    cache = O.AppendOnlyCache(w.n_kv_heads, w.head_dim, nb * run["B"])
    K, V, Q, P = run["K"][b], run["V"][b], run["Q"][b], run["P"]
    for t in range(nb):
        r = O.select_block(K[:, t * S:(t + 1) * S], Q, P,
                           n_bits=w.lsh_bits, n_tables=w.lsh_tables, B=run["B"], n=w.protection_divisor,
                           alpha=w.alpha)
        cache.append(K[:, t * S:(t + 1) * S], V[:, t * S:(t + 1) * S], r.idx, t * S)
    return cache


@pytest.mark.parametrize("name,S,nb,batch,budget,strided,scale", [
    ("tiny", 520, 3, 1, None, True, None),             # G = 4, one ragged tile per split
    ("llama8b_32k", 1032, 2, 2, None, False, None),    # G = 4, two sequences
    ("qwen7b_128k", 776, 3, 2, None, True, None),      # G = 7: two sets of heads
    # budget = block size keeps every token, so the kept set has no near-ties to depend on
    ("tiny", 1016, 9, 1, 1016, False, None),           # several tiles per split: the ring wraps, ragged tail
    ("qwen7b_128k", 1016, 12, 1, 1016, True, None),    # the same for two sets of heads
    ("tiny", 1016, 9, 1, 1016, False, 6.0),            # logits hundreds apart: the reference maximum is raised late
])
def test_decode_attention_against_oracle(name, S, nb, batch, budget, strided, scale):
    import torch
    w = synth.workload(name).with_(block_size=S, context_len=nb * S, batch=batch, n_layers=1, lsh_tables=16,
                                   needles="uniform:4")
    run = run_workload_layer(w, 0, n_blocks=nb, debug=0, budget=budget)
    eng = run["engine"]
    rng = np.random.default_rng(1234)
    if strided:
        # the last window query of every head, read in place through the strides
        tq = run["tQ"][:, :, w.window - 1, :]
        q_bits = run["Q"][:, :, w.window - 1, :]
    else:
        q_bits = synth.f32_to_bf16_bits((rng.standard_normal((batch, w.n_q_heads, 128)) * 1.5).astype(np.float32))
        tq = torch.from_numpy(q_bits.view(np.int16)).cuda()
    out = eng.laser_kv_decode_attention(0, tq, softmax_scale=0.0 if scale is None else scale)
    eng.laser_kv_poll_status()
    got = to_np(out)
    _, _, pos, length = eng.laser_kv_cache_view(0)
    pos = to_np(pos)
    assert length == nb * run["B"]
    G = w.group
    for b in range(batch):
        cache = _oracle_cache(w, run, b)
        assert cache.length == length
        assert (pos[b, :, :length] == cache.pos[:, :length]).all()       # same tokens kept, same order
        for h in range(w.n_kv_heads):
            want = O.decode_attention(q_bits[b, h * G:(h + 1) * G], cache.K[h, :length], cache.V[h, :length], scale=scale)
            err = np.abs(got[b, h * G:(h + 1) * G] - want)
            assert (err <= DEC_RTOL * np.abs(want) + DEC_ATOL).all(), (b, h, err.max())


@pytest.mark.parametrize("S,B,nb,G", [(64, 8, 1, 1), (64, 8, 3, 2), (128, 40, 2, 8)])
def test_decode_attention_on_caches_shorter_than_a_tile(S, B, nb, G):
    """8, 24 and 80 entries per head (less than, and just over, one 64-row tile); G = 1, 2, 8."""
    import torch
    H = 2
    w = synth.workload("tiny").with_(block_size=S, context_len=nb * S, n_q_heads=H * G, n_kv_heads=H, window=16 // G if G < 8 else 2,
                                     lsh_tables=8, needles="none")
    run = run_workload_layer(w, 0, n_blocks=nb, debug=0, budget=B)
    eng = run["engine"]
    rng = np.random.default_rng(7)
    q_bits = synth.f32_to_bf16_bits(rng.standard_normal((1, H * G, 128)).astype(np.float32))
    out = eng.laser_kv_decode_attention(0, torch.from_numpy(q_bits.view(np.int16)).cuda())
    eng.laser_kv_poll_status()
    got = to_np(out)
    cache = _oracle_cache(w, run, 0)
    assert cache.length == nb * B
    for h in range(H):
        want = O.decode_attention(q_bits[0, h * G:(h + 1) * G], cache.K[h, :cache.length], cache.V[h, :cache.length])
        err = np.abs(got[0, h * G:(h + 1) * G] - want)
        assert (err <= DEC_RTOL * np.abs(want) + DEC_ATOL).all(), (h, err.max())


def test_decode_attention_reports_an_empty_cache():
    import torch
    from paper_2602_02199_b200 import binding as Bn
    w = synth.workload("tiny").with_(block_size=256, context_len=512, lsh_tables=8)
    tP = torch.from_numpy(synth.hyperplanes(w).view(np.int16)).cuda()
    cfg = Bn.make_config(n_layers=1, batch=1, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, block_size=256,
                         window=w.window, max_blocks=2, max_blocks_per_call=2, lsh_bits=w.lsh_bits, lsh_tables=8,
                         protection_divisor=4, budget_per_block=64, alpha=0.75, debug=0)
    eng = Bn.LaserKV(cfg, tP)
    q = torch.zeros(1, w.n_q_heads, 128, dtype=torch.int16, device="cuda")
    with pytest.raises(Bn.LaserKVError) as e:
        eng.laser_kv_decode_attention(0, q)
    assert e.value.status == Bn.ERR_STATE
