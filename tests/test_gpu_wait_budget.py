"""The give-up path of the bounded device-side waits, reached on purpose.

Every hand-off wait inside the streaming kernels has a poll budget; laser_kv_set_wait_budget shrinks
it to a few polls, so that the waits run out although nothing is wrong: every role records the
timeout and returns, copies and tensor-core work already in flight are still waited for with the
full budget, the tensor memory is freed and the kernel ends normally. Nothing hangs, traps or
faults: the host only sees LASER_KV_ERR_TIMEOUT from laser_kv_poll_status, and the next ordinary
call on the same handle gives the same bytes as a handle that never saw a timeout.
"""
import numpy as np
import pytest

from paper_2602_02199_b200 import synth

from parity_util import check_run, run_workload_layer, to_np

pytestmark = pytest.mark.gpu


def test_waits_that_run_out_report_timeout_and_leave_the_handle_usable():
    import torch
    from paper_2602_02199_b200 import binding as Bn
    w = synth.workload("tiny").with_(block_size=512, context_len=2048)
    ref = run_workload_layer(w, 0, n_blocks=4)
    check_run(w, ref)                                   # the reference run itself matches the oracle
    run = run_workload_layer(w, 0, n_blocks=4, inputs_of=ref)
    eng = run["engine"]
    eng.laser_kv_reset(0)
    eng.laser_kv_set_wait_budget(2)                     # two polls: no hand-off can complete in time
    eng.laser_kv_select_block(0, run["tK"], run["tV"], run["tQ"], 4)
    with pytest.raises(Bn.LaserKVError) as e:
        eng.laser_kv_poll_status()
    assert e.value.status == Bn.ERR_TIMEOUT
    eng.laser_kv_poll_status()                          # the word was cleared by the read
    # back to the built-in budgets: same handle, same inputs, same bytes as the untouched handle
    eng.laser_kv_set_wait_budget(0)
    eng.laser_kv_reset(0)
    eng.laser_kv_select_block(0, run["tK"], run["tV"], run["tQ"], 4)
    eng.laser_kv_poll_status()
    n = 4 * run["B"]
    for x, y in zip(eng.laser_kv_cache_view(0)[:3], ref["engine"].laser_kv_cache_view(0)[:3]):
        assert torch.equal(x[:, :, :n], y[:, :, :n])
    d1, d0 = eng.laser_kv_debug_view(), ref["engine"].laser_kv_debug_view()
    assert torch.equal(d1.s_exact, d0.s_exact) and torch.equal(d1.counts, d0.counts) and torch.equal(d1.idx, d0.idx)
