"""The host-buffer entry point (pinned host K, V, Q in, appended positions out) against the
device-buffer entry point on the same inputs: identical cache bytes, identical positions."""
import numpy as np
import pytest

from paper_2602_02199_b200 import synth

from parity_util import to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("nb,batch,pin_v", [(1, 1, True), (5, 2, True), (8, 1, True), (5, 2, False)])
def test_host_path_equals_device_path(nb, batch, pin_v):
    """Four calls with different inputs append behind one another. pin_v: the kept V rows are read in
    place from pinned memory; otherwise V is pageable and staged. Two sets of staging buffers are used
    alternately and the calls are queued back to back, so the copies of a call run under the tail of
    the previous call: a copy that overtook a reader would change the cache."""
    import torch
    from paper_2602_02199_b200 import binding as Bn
    S, n_calls = 264, 4
    w = synth.workload("tiny").with_(block_size=S, context_len=nb * S, batch=batch, lsh_tables=16, needles="uniform:4")
    B = Bn.laser_kv_budget(w.context_len, S, w.ratio)
    dev = torch.device("cuda", 0)
    P = torch.from_numpy(synth.hyperplanes(w).view(np.int16)).to(dev)
    cfg = Bn.make_config(n_layers=1, batch=batch, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, block_size=S,
                         window=w.window, max_blocks=n_calls * nb, max_blocks_per_call=nb, lsh_bits=w.lsh_bits,
                         lsh_tables=w.lsh_tables, protection_divisor=w.protection_divisor, budget_per_block=B)
    inputs = []
    for call in range(n_calls):                            # a different synthetic layer per call
        Ks, Vs, Qs = [], [], []
        for b in range(batch):
            k, v = synth.kv_blocks(w, call, b, 0, nb)
            Ks.append(k); Vs.append(v); Qs.append(synth.q_window(w, call, b))
        hK = torch.from_numpy(np.stack(Ks).view(np.int16)).pin_memory()
        hV = torch.from_numpy(np.stack(Vs).view(np.int16))
        if pin_v:
            hV = hV.pin_memory()
        hQ = torch.from_numpy(np.stack(Qs).view(np.int16)).pin_memory()
        inputs.append((hK, hV, hQ))
    ref = Bn.LaserKV(cfg, P)
    for hK, hV, hQ in inputs:
        ref.laser_kv_select_block(0, hK.to(dev), hV.to(dev), hQ.to(dev), nb)
    ref.laser_kv_poll_status()
    Kr, Vr, pr, n = ref.laser_kv_cache_view(0)
    assert n == n_calls * nb * B

    eng = Bn.LaserKV(cfg, P)
    stages = [[torch.empty_like(x, device=dev) for x in inputs[0]] for _ in range(2)]
    pos_hosts = [torch.full((batch, w.n_kv_heads, nb * B), -1, dtype=torch.int32).pin_memory() for _ in range(n_calls)]
    for call, (hK, hV, hQ) in enumerate(inputs):
        stage = stages[call % 2]
        eng.laser_kv_select_block_host(0, hK, hV, hQ, stage[0], stage[1], stage[2], nb, pos_hosts[call])
    eng.laser_kv_poll_status()
    torch.cuda.synchronize()
    Kc, Vc, pc, m = eng.laser_kv_cache_view(0)
    assert m == n
    assert (to_np(Kc[:, :, :n]) == to_np(Kr[:, :, :n])).all()
    assert (to_np(Vc[:, :, :n]) == to_np(Vr[:, :, :n])).all()
    assert (to_np(pc[:, :, :n]) == to_np(pr[:, :, :n])).all()
    for call in range(n_calls):
        sl = slice(call * nb * B, (call + 1) * nb * B)
        assert (pos_hosts[call].numpy() == to_np(pr[:, :, sl])).all()

    # one set of staging buffers for every call: each call's copies wait for the previous call
    eng.laser_kv_reset(0)
    for call, (hK, hV, hQ) in enumerate(inputs):
        eng.laser_kv_select_block_host(0, hK, hV, hQ, stages[0][0], stages[0][1], stages[0][2], nb, pos_hosts[call])
    eng.laser_kv_poll_status()
    torch.cuda.synchronize()
    Kc, Vc, pc, m = eng.laser_kv_cache_view(0)
    assert m == n and (to_np(Kc[:, :, :n]) == to_np(Kr[:, :, :n])).all() and (to_np(Vc[:, :, :n]) == to_np(Vr[:, :, :n])).all()
    assert (to_np(pc[:, :, :n]) == to_np(pr[:, :, :n])).all()
