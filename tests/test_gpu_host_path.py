"""The host-buffer entry point (pinned host K, V, Q in, appended positions out) against the
device-buffer entry point on the same inputs: identical cache bytes, identical positions."""
import numpy as np
import pytest

from paper_2602_02199_b200 import synth

from parity_util import to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("nb,batch,pin_v", [(1, 1, True), (5, 2, True), (8, 1, True), (5, 2, False)])
def test_host_path_equals_device_path(nb, batch, pin_v):
    """pin_v: the kept V rows are read in place from pinned memory; otherwise V is pageable and staged."""
    import torch
    from paper_2602_02199_b200 import binding as Bn
    S = 264
    w = synth.workload("tiny").with_(block_size=S, context_len=nb * S, batch=batch, lsh_tables=16, needles="uniform:4")
    B = Bn.laser_kv_budget(w.context_len, S, w.ratio)
    dev = torch.device("cuda", 0)
    P = torch.from_numpy(synth.hyperplanes(w).view(np.int16)).to(dev)
    cfg = Bn.make_config(n_layers=1, batch=batch, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, block_size=S,
                         window=w.window, max_blocks=2 * nb, max_blocks_per_call=nb, lsh_bits=w.lsh_bits,
                         lsh_tables=w.lsh_tables, protection_divisor=w.protection_divisor, budget_per_block=B)
    Ks, Vs, Qs = [], [], []
    for b in range(batch):
        k, v = synth.kv_blocks(w, 0, b, 0, nb)
        Ks.append(k); Vs.append(v); Qs.append(synth.q_window(w, 0, b))
    hK = torch.from_numpy(np.stack(Ks).view(np.int16)).pin_memory()
    hV = torch.from_numpy(np.stack(Vs).view(np.int16))
    if pin_v:
        hV = hV.pin_memory()
    hQ = torch.from_numpy(np.stack(Qs).view(np.int16)).pin_memory()
    ref = Bn.LaserKV(cfg, P)
    ref.laser_kv_select_block(0, hK.to(dev), hV.to(dev), hQ.to(dev), nb)
    ref.laser_kv_poll_status()
    Kr, Vr, pr, n = ref.laser_kv_cache_view(0)
    assert n == nb * B

    eng = Bn.LaserKV(cfg, P)
    stage = [torch.empty_like(x, device=dev) for x in (hK, hV, hQ)]
    pos_host = torch.full((batch, w.n_kv_heads, nb * B), -1, dtype=torch.int32).pin_memory()
    for call in range(2):                                  # the second call appends behind the first
        eng.laser_kv_select_block_host(0, hK, hV, hQ, stage[0], stage[1], stage[2], nb, pos_host)
        eng.laser_kv_poll_status()
        torch.cuda.synchronize()
        Kc, Vc, pc, m = eng.laser_kv_cache_view(0)
        assert m == (call + 1) * nb * B
        sl = slice(call * nb * B, (call + 1) * nb * B)
        assert (to_np(Kc[:, :, sl]) == to_np(Kr[:, :, :n])).all()
        assert (to_np(Vc[:, :, sl]) == to_np(Vr[:, :, :n])).all()
        assert (to_np(pc[:, :, sl]) == to_np(pr[:, :, :n]) + call * nb * S).all()
        assert (pos_host.numpy() == to_np(pc[:, :, sl])).all()
