"""Seeded sweeps over random geometries (sizes, group shapes, table shapes, budgets, policies): the
select call, decode attention and the closed-form recall score against the oracle."""
import numpy as np
import pytest

from oracle import laser_kv_oracle as O
from paper_2602_02199_b200 import synth

from parity_util import check_run, run_workload_layer, to_np

pytestmark = pytest.mark.gpu


def _group_and_window(rng):
    G = int(rng.choice([1, 2, 3, 4, 5, 7, 8]))
    windows = [w for w in (2, 4, 8, 16, 32, 48, 64, 128) if (G * w) % 16 == 0 and G * w <= 256]
    return G, int(rng.choice(windows))


@pytest.mark.parametrize("seed", [11, 12, 13, 14])
def test_select_call_on_random_geometries(seed):
    rng = np.random.default_rng(seed)
    for case in range(10):
        G, W = _group_and_window(rng)
        hkv = int(rng.choice([1, 2, 4]))
        S, nb, batch = int(rng.integers(8, 190)) * 8, int(rng.integers(1, 4)), int(rng.integers(1, 3))
        w = synth.workload("tiny").with_(
            name=f"sweep{seed}_{case}", n_q_heads=hkv * G, n_kv_heads=hkv, window=W,
            lsh_bits=int(rng.choice([4, 6, 8, 10, 12])), lsh_tables=int(rng.choice([8, 16, 24, 32])), block_size=S,
            context_len=nb * S, batch=batch, protection_divisor=int(rng.choice([2, 3, 4, 8])),
            alpha=float(rng.choice([0.0, 0.25, 0.5, 0.75, 1.0])), ratio=float(rng.choice([0.1, 0.25, 0.5])),
            needles="uniform:2", rope_base=float(rng.choice([0.0, 10000.0])))
        run = run_workload_layer(w, 0)
        segs = [(b, h, t) for b in range(batch) for h in range(hkv) for t in range(nb)]
        if len(segs) > 4:
            segs = [segs[i] for i in rng.choice(len(segs), 4, replace=False)]
        check_run(w, run, segments=segs)


@pytest.mark.parametrize("seed", [31, 32])
def test_select_call_on_random_hash_shapes(seed):
    """Any number of bits per table up to 12 and any number of tables (the library pads inside)."""
    rng = np.random.default_rng(seed)
    for case in range(8):
        G, W = _group_and_window(rng)
        hkv = int(rng.choice([1, 2]))
        S, nb = int(rng.integers(8, 120)) * 8, int(rng.integers(1, 3))
        w = synth.workload("tiny").with_(
            name=f"hash{seed}_{case}", n_q_heads=hkv * G, n_kv_heads=hkv, window=W,
            lsh_bits=int(rng.integers(1, 13)), lsh_tables=int(rng.integers(1, 41)), block_size=S,
            context_len=nb * S, protection_divisor=int(rng.choice([2, 4, 8])),
            alpha=float(rng.choice([0.0, 0.5, 0.75])), needles="uniform:2")
        run = run_workload_layer(w, 0)
        check_run(w, run, segments=[(0, int(rng.integers(hkv)), int(rng.integers(nb)))])


@pytest.mark.parametrize("seed", [21, 22])
def test_decode_and_closed_form_score_on_random_geometries(seed):
    import torch
    from paper_2602_02199_b200 import binding as Bn
    rng = np.random.default_rng(seed)
    for case in range(10):
        G, W = _group_and_window(rng)
        hkv = int(rng.choice([1, 2, 4]))
        S, nb, batch = int(rng.integers(8, 160)) * 8, int(rng.integers(1, 9)), int(rng.integers(1, 3))
        K = int(rng.choice([4, 6, 7, 8, 10, 12, 20]))
        w = synth.workload("tiny").with_(name=f"sweepd{seed}_{case}", n_q_heads=hkv * G, n_kv_heads=hkv, window=W,
                                         lsh_bits=8, lsh_tables=8, block_size=S, context_len=nb * S, batch=batch,
                                         needles="none")
        # a budget of the whole block keeps every token: the cache is the input, in order
        run = run_workload_layer(w, 0, n_blocks=nb, debug=0, budget=S)
        eng = run["engine"]
        scale = float(rng.choice([0.0, 0.0, 2.0]))
        qb = synth.f32_to_bf16_bits(rng.standard_normal((batch, hkv * G, 128)).astype(np.float32))
        out = to_np(eng.laser_kv_decode_attention(0, torch.from_numpy(qb.view(np.int16)).cuda(), softmax_scale=scale))
        eng.laser_kv_poll_status()
        for b in range(batch):
            for h in range(hkv):
                want = O.decode_attention(qb[b, h * G:(h + 1) * G], run["K"][b, h], run["V"][b, h], scale=scale or None)
                err = np.abs(out[b, h * G:(h + 1) * G] - want)
                assert (err <= 1e-3 * np.abs(want) + 1e-4).all(), (case, b, h, err.max())
        p, scratch = Bn.laser_kv_collision_probability(run["tK"], run["tQ"], S, nb, K)
        torch.cuda.synchronize()
        assert int(to_np(scratch[:4]).view(np.int32)[0]) == 0
        p = to_np(p)
        for _ in range(3):
            b, h, t = int(rng.integers(batch)), int(rng.integers(hkv)), int(rng.integers(nb))
            q = O.group_queries(run["Q"][b], hkv, h)
            want = O.collision_probability(q, run["K"][b, h, t * S:(t + 1) * S], K)
            err = np.abs(p[b, h, t] - want)
            assert (err <= 1e-3 * want + 1e-6).all(), (case, b, h, t, err.max())


def test_select_call_at_the_largest_block_size():
    """block_size 16384 (the limit of the selection kernel's shared memory), two blocks, 12-bit tables."""
    w = synth.workload("tiny").with_(name="maxblock", n_q_heads=8, n_kv_heads=2, window=64, lsh_bits=12, lsh_tables=8,
                                     block_size=16384, context_len=2 * 16384, needles="uniform:6", rope_base=500000.0)
    run = run_workload_layer(w, 0)
    check_run(w, run, segments=[(0, 0, 0), (0, 1, 1)])


@pytest.mark.parametrize("name,alpha", [("tiny", 0.75), ("tiny", 1.0), ("llama8b_32k", 0.75), ("qwen7b_128k", 0.75)])
def test_planted_needles_stay_in_every_heads_cache(name, alpha):
    """The synthetic contexts plant keys with cosine 0.9 to a window query of each KV head's group:
    the exact stage must keep all of them, whatever else it keeps (a functional check of the selection
    on needle-like structure, not an accuracy figure)."""
    w = synth.workload(name).with_(alpha=alpha)
    run = run_workload_layer(w, 0, debug=0, alpha=alpha)
    _, _, pos, n = run["engine"].laser_kv_cache_view(0)
    pos = to_np(pos)[:, :, :n]
    for b in range(w.batch):
        needles = synth.needle_positions(w, 0, b)
        assert len(needles) > 0
        for h in range(w.n_kv_heads):
            assert np.isin(needles, pos[b, h]).all(), (b, h)
