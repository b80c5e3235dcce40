"""CUDA path vs the fp64 oracle, element by element, through the C ABI."""
import numpy as np
import pytest

from oracle import laser_kv_oracle as O
from paper_2602_02199_b200 import synth

from parity_util import check_run, run_workload_layer, to_np

pytestmark = pytest.mark.gpu


def test_tiny_config_all_blocks_all_heads():
    w = synth.workload("tiny")
    run = run_workload_layer(w, 0)
    stats = check_run(w, run)
    assert len(stats) == 8 * 4


@pytest.mark.parametrize("S,B,n,alpha", [
    (1000, 300, 4, 0.75),      # ragged: last key tile has 104 keys
    (136, 40, 4, 0.5),         # one full tile + 8 keys
    (512, 128, 2, 0.75),       # n = 2: empty recall budget
    (512, 129, 2, 0.75),       # n = 2 with an odd budget: one LSH pick
    (640, 200, 4, 1.0),        # LSH stage disabled: pure attention top-k
    (640, 200, 4, 0.0),        # exact stage disabled: pure LSH top-k
    (384, 384, 4, 0.75),       # keep everything
    (256, 2, 4, 0.75),         # no anchors, one pick per stage.. (B_long = 2)
])
def test_shrunken_and_degenerate_shapes(S, B, n, alpha):
    w = synth.workload("tiny").with_(name=f"s{S}", block_size=S, context_len=3 * S, protection_divisor=n,
                                     alpha=alpha)
    run = run_workload_layer(w, 0, budget=B, alpha=alpha)
    check_run(w, run, alpha=alpha)


def test_gqa7_k10_shape_with_rope_and_batch():
    # Qwen-like group of 7 (G*W = 224), 10-bit tables, two sequences
    w = synth.workload("qwen7b_128k").with_(name="qwen_small", batch=2, block_size=520, context_len=4 * 520,
                                            lsh_bits=10, lsh_tables=16, needles="uniform:4", n_layers=1)
    run = run_workload_layer(w, 0)
    check_run(w, run)


@pytest.mark.parametrize("K,L,hq,hkv,W,S", [
    (4, 8, 2, 2, 16, 264),       # G*W = 16: three of the four score groups have no columns
    (6, 24, 4, 2, 24, 392),      # G*W = 48, 6-bit tables, 24 tables in chunks of 8
    (12, 8, 8, 2, 64, 520),      # G*W = 256, 12-bit tables, one chunk
    (12, 16, 4, 4, 32, 136),     # 12-bit tables in one chunk of 16: two accumulator buffers of 192 columns
    (8, 32, 6, 2, 48, 648),      # G*W = 144: two query row blocks, the second one ragged; chunk of 32 tables
    (10, 8, 16, 2, 16, 1032),    # G = 8, W = 16
    (7, 12, 4, 2, 32, 392),      # odd bits (padded to 8 with a repeat of the first hyperplane), 12 tables (padded to 16)
    (5, 3, 8, 2, 16, 264),       # 5 bits -> 6, 3 tables -> 8
    (1, 20, 4, 4, 16, 136),      # one bit per table -> 4, 20 tables -> 24
    (11, 9, 4, 2, 64, 520),      # 11 bits -> 12, 9 tables -> 16
    (9, 64, 8, 2, 32, 648),      # 9 bits -> 10, tables already a multiple of eight
    (8, 16, 8, 2, 128, 520),     # G*W = 512: the window is scored in two parts of 64 positions
    (10, 8, 6, 2, 96, 392),      # G*W = 288: two parts of 48 positions (144 queries each)
    (8, 8, 8, 1, 128, 264),      # G*W = 1024: four parts of 32 positions
])
def test_hash_and_group_geometries(K, L, hq, hkv, W, S):
    w = synth.workload("tiny").with_(name=f"geo{K}_{L}_{hq}_{hkv}_{W}", n_q_heads=hq, n_kv_heads=hkv, window=W,
                                     lsh_bits=K, lsh_tables=L, block_size=S, context_len=3 * S,
                                     needles="uniform:3")
    run = run_workload_layer(w, 0)
    check_run(w, run)


def test_outlier_tokens_and_n_sweep():
    for n in (2, 4, 8):
        w = synth.workload("llama8b_64k").with_(name=f"out{n}", block_size=768, context_len=2 * 768,
                                                protection_divisor=n, n_layers=1)
        run = run_workload_layer(w, 0)
        check_run(w, run)


def test_token_major_layout_gives_identical_results():
    w = synth.workload("tiny").with_(block_size=256, context_len=1024)
    r1 = run_workload_layer(w, 0)
    r2 = run_workload_layer(w, 0, layout="bshd")
    d1, d2 = r1["engine"].laser_kv_debug_view(), r2["engine"].laser_kv_debug_view()
    assert (to_np(d1.idx) == to_np(d2.idx)).all()
    assert (to_np(d1.counts) == to_np(d2.counts)).all()
    assert (to_np(d1.s_exact) == to_np(d2.s_exact)).all()
    check_run(w, r2)


def test_append_only_across_calls_and_capacity():
    import torch
    from paper_2602_02199_b200 import binding as Bn
    w = synth.workload("tiny").with_(block_size=256, context_len=1024, n_layers=2)
    B = Bn.laser_kv_budget(w.context_len, w.block_size)
    dev = torch.device("cuda", 0)
    P = torch.from_numpy(synth.hyperplanes(w).view(np.int16)).to(dev)
    cfg = Bn.make_config(n_layers=2, batch=1, n_q_heads=32, n_kv_heads=8, block_size=256, window=32, max_blocks=4,
                         max_blocks_per_call=4, lsh_bits=8, lsh_tables=16, protection_divisor=4,
                         budget_per_block=B)
    one = Bn.LaserKV(cfg, P)
    inc = Bn.LaserKV(cfg, P)
    K, V = synth.kv_blocks(w, 1, 0, 0, 4)
    Q = synth.q_window(w, 1, 0)
    tK = torch.from_numpy(K.view(np.int16)).to(dev)[None]
    tV = torch.from_numpy(V.view(np.int16)).to(dev)[None]
    tQ = torch.from_numpy(Q.view(np.int16)).to(dev)[None]
    one.laser_kv_select_block(1, tK, tV, tQ, 4)
    one.laser_kv_poll_status()
    Kc1, Vc1, p1, n1 = one.laser_kv_cache_view(1)
    assert n1 == 4 * B and one.laser_kv_cache_view(0)[3] == 0
    prev = None
    for t in range(4):
        sl = slice(t * 256, (t + 1) * 256)
        inc.laser_kv_select_block(1, tK[:, :, sl], tV[:, :, sl], tQ, 1)
        inc.laser_kv_poll_status()
        Kc, Vc, p, n = inc.laser_kv_cache_view(1)
        assert n == (t + 1) * B
        snap = (to_np(Kc[:, :, :n]).copy(), to_np(Vc[:, :, :n]).copy(), to_np(p[:, :, :n]).copy())
        if prev is not None:       # earlier entries never change
            m = prev[2].shape[2]
            assert (snap[0][:, :, :m] == prev[0]).all() and (snap[1][:, :, :m] == prev[1]).all()
            assert (snap[2][:, :, :m] == prev[2]).all()
        prev = snap
    assert (prev[0] == to_np(Kc1[:, :, :n1])).all() and (prev[1] == to_np(Vc1[:, :, :n1])).all()
    assert (prev[2] == to_np(p1[:, :, :n1])).all()
    with pytest.raises(Bn.LaserKVError) as e:
        inc.laser_kv_select_block(1, tK[:, :, :256], tV[:, :, :256], tQ, 1)
    assert e.value.status == Bn.ERR_CAPACITY
    assert inc.laser_kv_cache_view(1)[3] == 4 * B
    inc.laser_kv_reset(1)
    assert inc.laser_kv_cache_view(1)[3] == 0


def test_counters_follow_the_calls():
    w = synth.workload("tiny").with_(block_size=256, context_len=1024)
    run = run_workload_layer(w, 0, debug=0)
    c = run["engine"].laser_kv_get_counters()
    B, S, nb, hk = run["B"], 256, 4, w.n_kv_heads
    assert c["select_calls"] == 1 and c["blocks"] == nb and c["tokens"] == nb * S
    assert c["entries_appended"] == hk * nb * B
    want = hk * nb * S * 256 + w.n_q_heads * w.window * 256 + w.lsh_tables * w.lsh_bits * 256 + hk * nb * B * (4 * 256 + 4)
    assert c["algorithmic_bytes"] == want


def test_same_inputs_twice_give_identical_bytes():
    w = synth.workload("tiny").with_(block_size=512, context_len=1024)
    r1 = run_workload_layer(w, 0)
    r2 = run_workload_layer(w, 0)
    for a, b in zip(r1["engine"].laser_kv_cache_view(0)[:3], r2["engine"].laser_kv_cache_view(0)[:3]):
        n = r1["n_blocks"] * r1["B"]
        assert (to_np(a[:, :, :n]) == to_np(b[:, :, :n])).all()


@pytest.mark.parametrize("debug", [0, 1])
def test_back_to_back_calls_on_small_grids_repeat_bit_for_bit(debug):
    """The log-sum-exp, score and projection kernels of a call start before the kernel ahead of them
    has finished. On grids this small (a few CTAs per kernel) all of them are on the GPU at once, so
    a kernel that read something too early would see it half written. Forty calls are queued without
    a host synchronisation between them, alternating between two inputs; every call's appended rows
    and positions must equal those of the same input run alone on a fresh handle."""
    import torch
    from paper_2602_02199_b200 import binding as Bn
    for S, nb, hkv, G, W, K, L in ((264, 1, 2, 4, 32, 8, 16), (136, 3, 1, 7, 16, 10, 8), (1024, 2, 4, 2, 64, 6, 24)):
        w = synth.workload("tiny").with_(name=f"b2b{S}", block_size=S, context_len=nb * S, n_q_heads=hkv * G, n_kv_heads=hkv,
                                         window=W, lsh_bits=K, lsh_tables=L, needles="uniform:2")
        ref = [run_workload_layer(w, layer, debug=debug) for layer in (0, 1)]
        B, n = ref[0]["B"], nb * ref[0]["B"]
        want = [[to_np(x[:, :, :n]).copy() for x in r["engine"].laser_kv_cache_view(0)[:3]] for r in ref]
        cfg = Bn.make_config(n_layers=1, batch=w.batch, n_q_heads=w.n_q_heads, n_kv_heads=hkv, block_size=S, window=W,
                             max_blocks=40 * nb, max_blocks_per_call=nb, lsh_bits=K, lsh_tables=L,
                             protection_divisor=w.protection_divisor, budget_per_block=B, alpha=w.alpha, debug=debug)
        eng = Bn.LaserKV(cfg, ref[0]["tP"])
        for call in range(40):                               # queued back to back, no synchronisation
            r = ref[call % 2]
            eng.laser_kv_select_block(0, r["tK"], r["tV"], r["tQ"], nb)
        eng.laser_kv_poll_status()
        Kc, Vc, pc, m = eng.laser_kv_cache_view(0)
        assert m == 40 * n
        Kc, Vc, pc = to_np(Kc), to_np(Vc), to_np(pc)
        for call in range(40):
            sl = slice(call * n, (call + 1) * n)
            wk, wv, wp = want[call % 2]
            assert (Kc[:, :, sl] == wk).all() and (Vc[:, :, sl] == wv).all(), (S, call)
            assert (pc[:, :, sl] - call * nb * S == wp).all(), (S, call)


@pytest.mark.parametrize("alpha", [1.0, 0.0])
def test_single_stage_policies_skip_the_unused_stage_and_keep_the_cache(alpha):
    # alpha = 1 (exact attention only) and alpha = 0 (LSH only): without the debug view the unused
    # stage is not computed; the cache must equal the one of the run that computed everything
    w = synth.workload("tiny").with_(block_size=640, context_len=1280, alpha=alpha)
    full = run_workload_layer(w, 0, alpha=alpha, debug=1)
    check_run(w, full, alpha=alpha)
    lean = run_workload_layer(w, 0, alpha=alpha, debug=0)
    n = full["n_blocks"] * full["B"]
    for x, y in zip(full["engine"].laser_kv_cache_view(0)[:3], lean["engine"].laser_kv_cache_view(0)[:3]):
        assert (to_np(x[:, :, :n]) == to_np(y[:, :, :n])).all()


def test_two_stage_topk_entry_point_against_oracle():
    import torch
    from paper_2602_02199_b200 import binding as Bn
    rng = np.random.default_rng(5)
    for S, a, ke, kl in ((1024, 100, 150, 60), (8192, 963, 1446, 483), (200, 0, 200, 0), (200, 0, 0, 200),
                         (333 * 8, 17, 1, 1), (4096, 455, 0, 0), (16384, 2000, 3000, 1000)):
        n_seg = 5
        # quantised scores and small integer counts: many exact ties in both stages
        s = (rng.integers(0, 50, (n_seg, S)) / 64.0).astype(np.float32)
        s[0] = rng.random(S).astype(np.float32)
        s[1, :] = 0.25
        c = rng.integers(0, 7, (n_seg, S)).astype(np.int32)
        c[2, :] = 3
        idx = Bn.laser_kv_two_stage_topk(torch.from_numpy(s).cuda(), torch.from_numpy(c).cuda(), a, ke, kl)
        torch.cuda.synchronize()
        idx = to_np(idx)
        for g in range(n_seg):
            want = O.select_indices(s[g].astype(np.float64), c[g].astype(np.int64), S, a, ke, kl)[2]
            assert (idx[g] == want).all(), (S, a, ke, kl, g)


def test_window_scores_entry_point_against_oracle():
    import torch
    from paper_2602_02199_b200 import binding as Bn
    from parity_util import SCORE_ATOL, SCORE_RTOL
    for name, S, nb in (("tiny", 1024, 2), ("qwen7b_128k", 1000, 3), ("llama8b_128k", 4096, 2)):
        w = synth.workload(name).with_(block_size=S, context_len=8 * S, batch=1)
        K, _ = synth.kv_blocks(w, 0, 0, 2, nb)
        Q = synth.q_window(w, 0, 0)
        tK = torch.from_numpy(K.view(np.int16)).cuda()[None]
        tQ = torch.from_numpy(Q.view(np.int16)).cuda()[None]
        for scale in (0.0, 0.05):
            out = to_np(Bn.laser_kv_window_scores(tK, tQ, S, nb, softmax_scale=scale))
            torch.cuda.synchronize()
            G = w.group
            for h in (0, w.n_kv_heads - 1):
                for t in range(nb):
                    want = O.window_scores(O.group_queries(Q, w.n_kv_heads, h), K[h, t * S:(t + 1) * S],
                                           None if scale == 0.0 else scale)
                    err = np.abs(out[0, h, t] - want)
                    assert (err <= SCORE_RTOL * np.abs(want) + SCORE_ATOL).all(), (name, h, t, err.max())
    assert Bn.laser_kv_window_scores_scratch_bytes(1, 32, 8, 8192, 64, 16) > 0
    with pytest.raises(Bn.LaserKVError) as e:
        Bn.laser_kv_window_scores(tK, tQ, S, nb, scratch=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == Bn.ERR_CAPACITY


def test_gather_append_entry_point_bit_exact():
    import torch
    from paper_2602_02199_b200 import binding as Bn
    rng = np.random.default_rng(6)
    n_seg, rows, cap, keep = 3, 500, 700, 123
    K = rng.integers(0, 65536, (n_seg, rows, 128)).astype(np.uint16)
    V = rng.integers(0, 65536, (n_seg, rows, 128)).astype(np.uint16)
    idx = np.stack([np.sort(rng.choice(rows, keep, replace=False)) for _ in range(n_seg)]).astype(np.int32)
    Kd = torch.zeros((n_seg, cap, 128), dtype=torch.int16, device="cuda")
    Vd = torch.zeros_like(Kd)
    pos = torch.full((n_seg, cap), -1, dtype=torch.int32, device="cuda")
    tK, tV = torch.from_numpy(K.view(np.int16)).cuda(), torch.from_numpy(V.view(np.int16)).cuda()
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    Bn.laser_kv_gather_append(tK, tV, torch.from_numpy(idx).cuda(), Kd, Vd, pos, 200, 5000, status)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    Kn, Vn, pn = to_np(Kd).view(np.uint16), to_np(Vd).view(np.uint16), to_np(pos)
    for g in range(n_seg):
        assert (Kn[g, 200:200 + keep] == K[g, idx[g]]).all() and (Vn[g, 200:200 + keep] == V[g, idx[g]]).all()
        assert (pn[g, 200:200 + keep] == 5000 + idx[g]).all()
        assert (Kn[g, :200] == 0).all() and (Kn[g, 200 + keep:] == 0).all() and (pn[g, :200] == -1).all()
    # indices outside the source segment are never dereferenced: their entries are skipped and the
    # status word says so; every valid entry is still copied
    bad = idx.copy()
    bad[1, 7], bad[2, 100], bad[0, keep - 1] = rows, -1, 2 ** 30
    Kd.zero_(); Vd.zero_(); pos.fill_(-1)
    Bn.laser_kv_gather_append(tK, tV, torch.from_numpy(bad).cuda(), Kd, Vd, pos, 200, 5000, status)
    torch.cuda.synchronize()
    assert int(status[0]) == Bn.ERR_INVALID_ARG
    Kn, pn = to_np(Kd).view(np.uint16), to_np(pos)
    for g in range(n_seg):
        ok = (bad[g] >= 0) & (bad[g] < rows)
        assert (Kn[g, 200:200 + keep][ok] == K[g, bad[g][ok]]).all() and (pn[g, 200:200 + keep][ok] == 5000 + bad[g][ok]).all()
        assert (Kn[g, 200:200 + keep][~ok] == 0).all() and (pn[g, 200:200 + keep][~ok] == -1).all()
    with pytest.raises(Bn.LaserKVError) as e:      # entries beyond the destination's capacity
        Bn.laser_kv_gather_append(tK, tV, torch.from_numpy(idx).cuda(), Kd, Vd, pos, cap - keep + 1, 0, status)
    assert e.value.status == Bn.ERR_CAPACITY


def test_headline_config_full_size_sampled_segments():
    import torch
    # 128k context, 16 blocks of 8192 in one call (the launch shape the benchmark times); the
    # oracle checks sampled (head, block) segments in full and the cache of every segment.
    w = synth.workload("llama8b_128k")
    run = run_workload_layer(w, 3, debug=1)
    segs = [(0, 0, 0), (0, 3, 1), (0, 5, 7), (0, 7, 15), (0, 2, 11)]   # blocks holding needles included
    check_run(w, run, segments=segs)
    # the benchmarked path keeps no per-key bucket ids (debug = 0), which is another branch of the
    # projection epilogue: its cache must equal, bit for bit, the one the oracle has just checked
    lean = run_workload_layer(w, 3, debug=0, inputs_of=run)
    n = run["n_blocks"] * run["B"]
    for x, y in zip(run["engine"].laser_kv_cache_view(0)[:3], lean["engine"].laser_kv_cache_view(0)[:3]):
        assert torch.equal(x[:, :, :n], y[:, :, :n])
    d1, d0 = run["engine"].laser_kv_debug_view(), lean["engine"].laser_kv_debug_view()
    assert torch.equal(d1.counts, d0.counts) and torch.equal(d1.s_exact, d0.s_exact) and torch.equal(d1.idx, d0.idx)


@pytest.mark.parametrize("name,n_blocks,segs", [
    ("llama8b_32k", 8, [(0, 1, 0), (0, 6, 5)]),
    ("qwen7b_128k", 6, [(0, 0, 0), (2, 3, 4), (3, 1, 5)]),
])
def test_other_configs_sampled_segments(name, n_blocks, segs):
    w = synth.workload(name)
    run = run_workload_layer(w, 1, n_blocks=n_blocks)
    check_run(w, run, segments=segs)


def test_64k_config_n_sweep_sampled_segments():
    for n, seg in ((2, (0, 0, 1)), (4, (0, 4, 0)), (8, (0, 7, 2))):
        w = synth.workload("llama8b_64k").with_(protection_divisor=n)
        run = run_workload_layer(w, 2, n_blocks=3)
        check_run(w, run, segments=[seg])
