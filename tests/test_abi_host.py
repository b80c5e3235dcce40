"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, does the budget arithmetic of the paper, validates configurations, and fails
loudly (no CPU fallback) when there is no CUDA device."""
import ctypes as C
import os
import re

import pytest

from paper_2602_02199_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _have_gpu():
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False


def _cfg(**kw):
    base = dict(n_layers=2, batch=1, n_q_heads=32, n_kv_heads=8, block_size=1024, window=32, max_blocks=4,
                max_blocks_per_call=4, lsh_bits=8, lsh_tables=16, protection_divisor=4, context_len=4096)
    base.update(kw)
    return B.make_config(**base)


def test_library_exports_every_declared_symbol():
    lib = B.load()
    header = open(os.path.join(ROOT, "include", "laser_kv.h")).read()
    declared = set(re.findall(r"\b(laser_kv_[a-z_0-9]+)\s*\(", header))
    declared -= {"laser_kv_status_t", "laser_kv_handle_t"}
    assert declared == set(B.EXPORTS), declared ^ set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_budget_and_partition_match_golden(golden_dir):
    for line in open(os.path.join(golden_dir, "budget_eq1.txt")):
        if line.strip() and not line.startswith("#"):
            S, L, r, want = line.split()
            assert B.laser_kv_budget(int(L), int(S), float(r)) == int(want)
    for line in open(os.path.join(golden_dir, "partition_sec3_1.txt")):
        if line.strip() and not line.startswith("#"):
            Bv, n, alpha, a, loc, bl, ke, kl = line.split()
            assert B.laser_kv_partition(int(Bv), int(n), float(alpha)) == (int(a), int(loc), int(ke), int(kl))
    assert B.laser_kv_budget(0, 4096) == -1
    with pytest.raises(B.LaserKVError) as e:
        B.laser_kv_partition(100, 1, 0.5)
    assert e.value.status == B.ERR_INVALID_ARG


def test_query_sizes_and_validation():
    cb, wb = B.laser_kv_query_sizes(_cfg())
    # cache: 2 layers x 8 heads x (4 blocks x 409) entries x (256 B K + 256 B V + 4 B pos)
    assert cb >= 2 * 8 * 4 * 409 * 516 and cb < 2 * 8 * 4 * 409 * 516 + 4096
    assert wb > 0 and wb % 256 == 0
    for bad, status in ((dict(head_dim=64), B.ERR_UNSUPPORTED), (dict(protection_divisor=1), B.ERR_INVALID_ARG),
                        (dict(n_q_heads=30), B.ERR_INVALID_ARG), (dict(lsh_bits=13), B.ERR_UNSUPPORTED),
                        (dict(window=100), B.ERR_UNSUPPORTED),
                        (dict(budget_per_block=2000), B.ERR_INVALID_ARG), (dict(alpha=1.5), B.ERR_INVALID_ARG),
                        (dict(block_size=1001), B.ERR_UNSUPPORTED), (dict(context_len=0), B.ERR_INVALID_ARG)):
        with pytest.raises(B.LaserKVError) as e:
            B.laser_kv_query_sizes(_cfg(**bad))
        assert e.value.status == status, bad
    assert B.load().laser_kv_status_string(B.ERR_TIMEOUT) == b"device-side wait timed out"


def test_null_and_misaligned_arguments_are_rejected():
    lib = B.load()
    cfg = _cfg()
    h = C.c_void_p()
    assert lib.laser_kv_init(C.byref(cfg), None, None, 0, None, 0, C.byref(h)) == B.ERR_INVALID_ARG
    assert lib.laser_kv_init(C.byref(cfg), 0x1000, 0x1010, 1 << 40, 0x2000, 1 << 40, C.byref(h)) == B.ERR_ALIGNMENT
    assert lib.laser_kv_init(C.byref(cfg), 0x1000, 0x1100, 16, 0x2000, 16, C.byref(h)) == B.ERR_CAPACITY
    assert lib.laser_kv_select_block(None, 0, None, None, None, None, None, 1, None) == B.ERR_INVALID_ARG
    assert lib.laser_kv_two_stage_topk(None, None, 1, 8, 1, 1, 1, None, None) == B.ERR_INVALID_ARG
    assert lib.laser_kv_gather_append(None, None, 0, 0, 8, None, 1, 1, None, None, 0, 8, None, 0, 0, 0, None, None) == B.ERR_INVALID_ARG
    # entries that do not fit the destination are refused before anything is launched
    assert lib.laser_kv_gather_append(0x1000, 0x2000, 1024, 128, 8, 0x3000, 1, 5, 0x4000, 0x5000, 1024, 8, 0x6000, 8, 4, 0,
                                      0x7000, None) == B.ERR_CAPACITY
    assert lib.laser_kv_gather_append(0x1000, 0x2000, 1024, 128, -1, 0x3000, 1, 5, 0x4000, 0x5000, 1024, 8, 0x6000, 8, 0, 0,
                                      0x7000, None) == B.ERR_INVALID_ARG
    assert lib.laser_kv_set_wait_budget(None, 5) == B.ERR_INVALID_ARG
    assert lib.laser_kv_get_counters(None, None) == B.ERR_INVALID_ARG
    assert b"NULL" in lib.laser_kv_last_error(None)
    # the entry points beside the hot path validate before they touch the device
    assert lib.laser_kv_decode_attention(None, 0, None, None, 0.0, None, None, 0, None) == B.ERR_INVALID_ARG
    assert lib.laser_kv_decode_attention_scratch_bytes(None) == 0
    ks, qs = (C.c_int64 * 3)(0, 1024 * 128, 128), (C.c_int64 * 3)(0, 64 * 128, 128)
    cp = lib.laser_kv_collision_probability
    assert cp(None, None, ks, qs, 1, 4, 1, 1024, 64, 1, 10, None, 0, None, None) == B.ERR_INVALID_ARG
    assert cp(0x1000, 0x2000, ks, qs, 1, 4, 1, 1024, 64, 1, 0, 0x3000, 256, 0x4000, None) == B.ERR_INVALID_ARG    # K = 0
    assert cp(0x1000, 0x2000, ks, qs, 1, 4, 1, 1024, 72, 1, 10, 0x3000, 256, 0x4000, None) == B.ERR_UNSUPPORTED   # G*W = 288
    assert cp(0x1008, 0x2000, ks, qs, 1, 4, 1, 1024, 64, 1, 10, 0x3000, 256, 0x4000, None) == B.ERR_ALIGNMENT
    assert cp(0x1000, 0x2000, ks, qs, 1, 4, 1, 1024, 64, 1, 10, 0x3000, 16, 0x4000, None) == B.ERR_CAPACITY
    bad = (C.c_int64 * 3)(0, 1024 * 128, 100)
    assert cp(0x1000, 0x2000, bad, qs, 1, 4, 1, 1024, 64, 1, 10, 0x3000, 256, 0x4000, None) == B.ERR_ALIGNMENT


@pytest.mark.skipif(_have_gpu(), reason="checks the no-GPU failure path")
def test_init_fails_loudly_without_a_gpu():
    lib = B.load()
    cfg = _cfg()
    h = C.c_void_p()
    st = lib.laser_kv_init(C.byref(cfg), 0x1000, 0x10000, 1 << 40, 0x20000, 1 << 40, C.byref(h))
    assert st == B.ERR_CUDA and not h.value
    assert b"no CPU path" in lib.laser_kv_last_error(None)
