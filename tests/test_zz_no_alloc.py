"""The allocation-free window-score entry point against the ordinary one.

laser_kv_window_scores_static is for callers that may not allocate device memory (a plugin in
an engine whose pool owns the GPU, a latency-critical loop that cannot afford cudaMalloc's
synchronisation): its scratch is a 2 MiB array inside the library. It runs the same two
kernels as laser_kv_window_scores, so on the same inputs the two must agree within the score
tolerance of the parity tests. The test makes two calls in a row with different shapes, so the
second call starts from the first call's leftovers in the shared array, reads the status word
that these calls keep inside the library, compares sampled heads with the fp64 oracle, and checks
that sizes beyond the array are refused. This file sorts last on purpose: a run that stops at the first
failure has then already run every other test.
"""
import gc

import numpy as np
import pytest

from oracle import laser_kv_oracle as O
from paper_2602_02199_b200 import synth

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-3, 1e-5     # the score tolerance used by the parity tests


def _inputs(name, S, nb, first_block):
    import torch
    w = synth.workload(name).with_(block_size=S, context_len=16 * S, batch=1)
    K, _ = synth.kv_blocks(w, 0, 0, first_block, nb)
    Q = synth.q_window(w, 0, 0)
    return (torch.from_numpy(K.view(np.int16)).cuda()[None], torch.from_numpy(Q.view(np.int16)).cuda()[None], K, Q)


def test_static_scratch_variant_matches_caller_scratch_variant_twice_in_a_row():
    import torch
    from paper_2602_02199_b200 import binding as Bn
    assert Bn.laser_kv_window_scores_static_max_bytes() == 2 << 20
    # first call: 8 KV heads x 5 blocks of 4096 keys (two key splits per block), 256 queries per head;
    # second call: 4 KV heads x 3 ragged blocks of 1000 keys, 224 queries per head. The shapes differ so
    # that partials left in the shared array by the first call would show up in the second.
    for name, S, nb, first in (("llama8b_128k", 4096, 5, 0), ("qwen7b_128k", 1000, 3, 4)):
        tK, tQ, K, Q = _inputs(name, S, nb, first)
        want = Bn.laser_kv_window_scores(tK, tQ, S, nb)
        out = torch.full((1, tK.shape[1], nb, S), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        # tensors of earlier tests may be freed by the garbage collector at any moment: count torch's
        # allocations (a number that only grows) instead of comparing the bytes in use, and look at
        # the driver's own figure for what the library could have taken behind torch's back
        gc.collect()
        allocs = lambda: torch.cuda.memory_stats().get("allocation.all.allocated", 0)
        before, free_before = allocs(), torch.cuda.mem_get_info()[0]
        Bn.laser_kv_window_scores_static(tK, tQ, S, nb, out)
        torch.cuda.synchronize()
        assert allocs() == before
        assert torch.cuda.mem_get_info()[0] >= free_before
        got, ref = out.cpu().numpy(), want.cpu().numpy()
        assert np.isfinite(got).all()
        assert (np.abs(got - ref) <= RTOL * np.abs(ref) + ATOL).all()
        # each query's probabilities sum to one: the block total is the number of window queries
        np.testing.assert_allclose(got.sum(axis=3), tQ.shape[1] // tK.shape[1] * tQ.shape[2], rtol=2e-3)
        # no kernel of the call gave up a wait (the word sits in the library's array; this reads it)
        Bn.laser_kv_window_scores_static_status()
        assert allocs() == before
        # and against the oracle itself, for the first and the last head of the last block
        n_kv = tK.shape[1]
        for h in (0, n_kv - 1):
            ref64 = O.window_scores(O.group_queries(Q, n_kv, h), K[h, (nb - 1) * S:nb * S])
            assert (np.abs(got[0, h, nb - 1] - ref64) <= RTOL * np.abs(ref64) + ATOL).all()


def test_static_scratch_variant_rejects_sizes_beyond_its_array():
    import torch
    from paper_2602_02199_b200 import binding as Bn
    # 8 heads x 64 blocks of 8192 keys need ~4.7 MiB of partials: more than the built-in 2 MiB
    assert Bn.laser_kv_window_scores_scratch_bytes(1, 32, 8, 8192, 64, 64) > Bn.laser_kv_window_scores_static_max_bytes()
    # the size check comes before anything is read, so small stand-in buffers are enough here
    K = torch.zeros((1, 8, 128, 128), dtype=torch.int16, device="cuda")
    Q = torch.zeros((1, 32, 64, 128), dtype=torch.int16, device="cuda")
    out = torch.zeros((1, 8, 1, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(Bn.LaserKVError) as e:
        Bn.laser_kv_window_scores_static(K, Q, 8192, 64, out)
    assert e.value.status == Bn.ERR_CAPACITY and "2097152" in str(e.value)
    # the headline layer (16 blocks) fits
    assert Bn.laser_kv_window_scores_scratch_bytes(1, 32, 8, 8192, 64, 16) <= Bn.laser_kv_window_scores_static_max_bytes()
