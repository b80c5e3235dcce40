"""Shared pieces of the GPU parity tests: run the CUDA path through the C ABI on seeded inputs
and compare every stage with the fp64 oracle under the stated tolerances.

Tolerances (from the benchmark spec of this path):
  scores            |gpu - oracle| <= 1e-3 * |oracle| + 1e-5   (bf16 inputs, fp32 accumulation)
  signature bits    exact except bits whose oracle projection has |p| < 1e-6
  collision counts  exact given the (validated) GPU signatures
  index sets        exact-stage picks may differ from the oracle's only in tokens whose oracle
                    score is within 1e-3 relative of the oracle's k-th score; the LSH stage is
                    replayed on the GPU's exact picks and must match exactly; the kept list is
                    ascending and has exactly B entries
  cache rows        bit-exact copies of the source rows named by the GPU's own indices
"""
from __future__ import annotations

import numpy as np

from oracle import laser_kv_oracle as O
from paper_2602_02199_b200 import synth

SCORE_RTOL, SCORE_ATOL = 1e-3, 1e-5
SIGN_EXEMPT = 1e-6


def codes_to_bits(codes: np.ndarray, n_bits: int) -> np.ndarray:
    """Library bucket code (first hyperplane of the table = most significant bit) -> bits
    [..., n_bits] with bit b of the table at index b."""
    codes = codes.astype(np.int64) & 0xFFFF
    shifts = (n_bits - 1 - np.arange(n_bits))
    return (codes[..., None] >> shifts) & 1


def bits_to_lsb_bucket(bits: np.ndarray) -> np.ndarray:
    """bits [..., K] -> the oracle's bucket id convention (bit b has weight 2**b)."""
    w = 1 << np.arange(bits.shape[-1], dtype=np.int64)
    return (bits * w).sum(axis=-1)


def check_signatures(codes_gpu: np.ndarray, x_bits: np.ndarray, p_bits: np.ndarray, n_bits: int,
                     n_tables: int, what: str):
    """codes_gpu [N, L] (library codes) vs oracle signs of x [N, d]. Returns the GPU's buckets in
    the oracle's convention and the number of exempted bit differences."""
    proj = O.simhash_projections(x_bits, p_bits).reshape(x_bits.shape[0], n_tables, n_bits)
    want = (proj >= 0.0).astype(np.int64)
    # the library pads a table to an even number (>= 4) of bits and the tables to a multiple of eight:
    # a code has code_bits = even(max(n_bits, 4)) bits of which the first n_bits are the table's own
    code_bits = max(4, (n_bits + 1) // 2 * 2)
    got = codes_to_bits(codes_gpu[:, :n_tables], code_bits)[..., :n_bits]
    diff = got != want
    bad = diff & (np.abs(proj) >= SIGN_EXEMPT)
    assert not bad.any(), f"{what}: {int(bad.sum())} signature bits differ outside |proj| < 1e-6 " \
                          f"(first at {np.argwhere(bad)[0].tolist()}, proj {proj[tuple(np.argwhere(bad)[0])]})"
    return bits_to_lsb_bucket(got), int(diff.sum())


def check_segment(*, k_bits, q_bits_group, p_bits, n_bits, n_tables, S, anchors, k_exact, k_lsh,
                  scale, s_gpu, counts_gpu, idx_gpu, qcodes_gpu, kcodes_gpu=None, lse2_gpu=None,
                  what="segment", cand=None, kept=None):
    """One (sequence, KV head, block): k_bits [S, d] (the scored keys), q_bits_group [G*W, d]; GPU
    arrays already on the host. By default the candidates are [anchors, S - anchors) and the rest is
    kept (Section 3.1); `cand` and `kept` (ascending index arrays) override that (look-back).
    Returns a small dict of statistics."""
    stats = {}
    # --- scores ---
    s_or = O.window_scores(q_bits_group, k_bits, scale)
    err = np.abs(s_gpu.astype(np.float64) - s_or)
    tol = SCORE_RTOL * np.abs(s_or) + SCORE_ATOL
    assert (err <= tol).all(), f"{what}: score error {err.max():.3e} at {int(err.argmax())} exceeds tolerance"
    stats["score_max_rel"] = float((err / np.maximum(np.abs(s_or), 1e-30)).max())
    if lse2_gpu is not None:
        q = O.bf16_bits_to_f64(q_bits_group)
        k = O.bf16_bits_to_f64(k_bits)
        sc = (1.0 / np.sqrt(k.shape[1])) if scale is None else scale
        logits = (q @ k.T) * sc
        m = logits.max(axis=1)
        lse2 = (m + np.log(np.exp(logits - m[:, None]).sum(axis=1))) / np.log(2.0)
        assert np.abs(lse2_gpu - lse2).max() < 2e-4 * max(1.0, np.abs(lse2).max()), f"{what}: log-sum-exp mismatch"
    # --- signatures and counts ---
    qb, nq_ex = check_signatures(qcodes_gpu, q_bits_group, p_bits, n_bits, n_tables, what + " queries")
    stats["exempt_query_bits"] = nq_ex        # differences that check_signatures allowed (|proj| < 1e-6)
    if kcodes_gpu is not None:
        kb, nk_ex = check_signatures(kcodes_gpu, k_bits, p_bits, n_bits, n_tables, what + " keys")
        stats["exempt_bits"] = nk_ex + nq_ex
    else:
        kb, _ = O.simhash_buckets(k_bits, p_bits, n_bits, n_tables)
    counts_or = O.collision_counts(qb, kb)
    if kcodes_gpu is not None:
        assert (counts_gpu.astype(np.int64) == counts_or).all(), \
            f"{what}: {int((counts_gpu != counts_or).sum())} collision counts differ"
    else:
        # without the GPU's key signatures a count may differ only through an exempt sign
        bad = counts_gpu.astype(np.int64) != counts_or
        if bad.any():
            _, mabs = O.simhash_buckets(k_bits[bad], p_bits, n_bits, n_tables)
            assert (mabs.min(axis=1) < SIGN_EXEMPT).all(), f"{what}: collision counts differ"
    # --- selection ---
    if cand is None:
        cand = np.arange(anchors, S - anchors)
        kept = np.concatenate([np.arange(anchors), np.arange(S - anchors, S)])
    B = len(kept) + k_exact + k_lsh
    assert idx_gpu.shape == (B,)
    if B > 1:
        assert (np.diff(idx_gpu) > 0).all(), f"{what}: kept indices not strictly ascending"
    # what the selector must produce from the GPU's own scores and counts (bit-exact)
    ke_g = O.topk_lower_index(cand, s_gpu.astype(np.float64), k_exact)
    resid = np.setdiff1d(cand, ke_g, assume_unique=True)
    kl_g = O.topk_lower_index(resid, counts_gpu.astype(np.int64), k_lsh)
    want_idx = np.sort(np.concatenate([kept, ke_g, kl_g]))
    assert (idx_gpu.astype(np.int64) == want_idx).all(), f"{what}: kept index list differs from the two-stage rule"
    # the GPU's exact picks against the oracle's: only boundary tokens may differ
    ke_o = O.topk_lower_index(cand, s_or, k_exact)
    sym = np.setxor1d(ke_g, ke_o)
    if sym.size:
        kth = np.sort(s_or[cand])[::-1][k_exact - 1]
        rel = np.abs(s_or[sym] - kth) / abs(kth)
        assert (rel <= SCORE_RTOL).all(), f"{what}: exact-stage picks differ away from the k-th boundary ({rel.max():.2e})"
    stats["exact_stage_swaps"] = int(sym.size // 2)
    # LSH stage replayed on the GPU's exact picks with the oracle's counts (exact match required)
    kl_o = O.topk_lower_index(resid, counts_or, k_lsh)
    assert (kl_o == kl_g).all(), f"{what}: LSH-stage picks differ"
    return stats


def to_np(t):
    return t.detach().cpu().numpy()


def run_workload_layer(w: synth.Workload, layer: int, *, first_block=0, n_blocks=None, debug=1,
                       layout="bhsd", budget=None, alpha=None, inputs_of=None):
    """Generates one layer's inputs on the host (or takes the host and device tensors of an earlier
    run, ``inputs_of``), runs one select call on the GPU and returns everything the checks need."""
    import torch
    from paper_2602_02199_b200 import binding as Bn
    n_blocks = w.n_blocks if n_blocks is None else n_blocks
    S, d = w.block_size, w.head_dim
    dev = torch.device("cuda", 0)
    if inputs_of is not None:
        K, V, Q, P = (inputs_of[k] for k in ("K", "V", "Q", "P"))
        tK, tV, tQ, tP = (inputs_of[k] for k in ("tK", "tV", "tQ", "tP"))
    else:
        Ks, Vs, Qs = [], [], []
        for b in range(w.batch):
            k, v = synth.kv_blocks(w, layer, b, first_block, n_blocks)
            Ks.append(k); Vs.append(v); Qs.append(synth.q_window(w, layer, b))
        K = np.stack(Ks); V = np.stack(Vs); Q = np.stack(Qs)          # [batch][H][T][d]
        P = synth.hyperplanes(w)
        tK = torch.from_numpy(K.view(np.int16)).to(dev)
        tV = torch.from_numpy(V.view(np.int16)).to(dev)
        tQ = torch.from_numpy(Q.view(np.int16)).to(dev)
        tP = torch.from_numpy(P.view(np.int16)).to(dev)
    if layout == "bshd":      # token-major storage, viewed as [batch][H][T][d]
        tK = tK.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        tV = tV.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    B = budget if budget is not None else Bn.laser_kv_budget(w.context_len, S, w.ratio)
    cfg = Bn.make_config(n_layers=1, batch=w.batch, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads,
                         block_size=S, window=w.window, max_blocks=n_blocks, max_blocks_per_call=n_blocks,
                         lsh_bits=w.lsh_bits, lsh_tables=w.lsh_tables, protection_divisor=w.protection_divisor,
                         budget_per_block=B, alpha=w.alpha if alpha is None else alpha, debug=debug)
    eng = Bn.LaserKV(cfg, tP)
    eng.laser_kv_select_block(0, tK, tV, tQ, n_blocks)
    eng.laser_kv_poll_status()
    return dict(engine=eng, K=K, V=V, Q=Q, P=P, B=B, n_blocks=n_blocks, tK=tK, tV=tV, tQ=tQ, tP=tP)


def check_run(w: synth.Workload, run, segments=None, alpha=None):
    """Compares the chosen (b, h, t) segments (default: all) of a run with the oracle and checks the
    cache contents for every segment."""
    eng = run["engine"]
    dbg = eng.laser_kv_debug_view()
    S, G, W = w.block_size, w.group, w.window
    nb, B = run["n_blocks"], run["B"]
    a, _, _, ke, kl = O.partition(B, w.protection_divisor, w.alpha if alpha is None else alpha)
    s_all, c_all, idx_all = to_np(dbg.s_exact), to_np(dbg.counts), to_np(dbg.idx)
    qc_all = to_np(dbg.query_buckets)
    kc_all = to_np(dbg.key_buckets) if dbg.key_buckets is not None else None
    lse_all = to_np(dbg.lse2)
    if dbg.window_part != W:
        # a wide window is scored in parts: the library orders the group's queries (part, head, position
        # in the part); bring its per-query arrays into the oracle's (head, position) order
        Wp = dbg.window_part
        order = np.array([(r // (G * Wp)) * Wp + ((r % (G * Wp)) // Wp) * W + (r % Wp) for r in range(G * W)])
        inv = np.argsort(order)
        qc_all, lse_all = qc_all[:, :, inv], lse_all[..., inv]
    if segments is None:
        segments = [(b, h, t) for b in range(w.batch) for h in range(w.n_kv_heads) for t in range(nb)]
    stats = []
    for (b, h, t) in segments:
        kb = run["K"][b, h, t * S:(t + 1) * S]
        qg = O.group_queries(run["Q"][b], w.n_kv_heads, h)     # the oracle's own grouping of the query heads
        stats.append(check_segment(
            k_bits=kb, q_bits_group=qg, p_bits=run["P"], n_bits=w.lsh_bits, n_tables=w.lsh_tables, S=S,
            anchors=a, k_exact=ke, k_lsh=kl, scale=None, s_gpu=s_all[b, h, t], counts_gpu=c_all[b, h, t],
            idx_gpu=idx_all[b, h, t][:B], qcodes_gpu=qc_all[b, h],
            kcodes_gpu=None if kc_all is None else kc_all[b, h, t], lse2_gpu=lse_all[b, h, t],
            what=f"{w.name} b{b} h{h} t{t}"))
    # cache: rows named by the GPU's own indices, bit-exact, for every segment
    Kc, Vc, pos, length = eng.laser_kv_cache_view(0)
    assert length == nb * B
    Kc, Vc, pos = to_np(Kc).view(np.uint16), to_np(Vc).view(np.uint16), to_np(pos)
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            for t in range(nb):
                ids = idx_all[b, h, t][:B].astype(np.int64)
                sl = slice(t * B, (t + 1) * B)
                assert (pos[b, h, sl] == t * S + ids).all()
                assert (Kc[b, h, sl] == run["K"][b, h, t * S + ids]).all()
                assert (Vc[b, h, sl] == run["V"][b, h, t * S + ids]).all()
            if length > 1:
                assert (np.diff(pos[b, h, :length]) > 0).all()
    return stats
