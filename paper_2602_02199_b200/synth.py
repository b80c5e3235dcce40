"""Seeded synthetic inputs shaped like long-context prefill activations.

These generators serve the tests, the smoke check and the benchmark. They hold none of the
selection method's arithmetic: they only draw random tensors (counter-based Philox streams
keyed by what the tensor is), apply the structure the workloads call for (per-channel
log-normal scales, rotary position embedding, planted "needle" keys, magnitude outliers) and
round once to bfloat16. The same bits are handed to the CUDA path and to the CPU oracle.

Every tensor can be produced block by block, so a single block of a 128k-token context can be
regenerated on the host without materialising the rest.

Real activations (the paper evaluates Llama-3.1-8B-Instruct and a 1M-context Llama-3-8B variant
on a long-context QA suite, Section 4) are not available offline; these inputs stand in for them.
"""
from __future__ import annotations

import hashlib
import math
from dataclasses import dataclass, replace

import numpy as np

__all__ = ["Workload", "WORKLOADS", "workload", "f32_to_bf16_bits", "bf16_bits_to_f32",
           "hyperplanes", "q_window", "kv_block", "kv_blocks", "needle_positions"]


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    context_len: int
    block_size: int
    window: int
    lsh_bits: int            # K: sign bits per table
    lsh_tables: int          # L: tables (the paper's R hash rounds)
    protection_divisor: int  # n (Section 3.1)
    alpha: float = 0.75      # exact share of the recall budget (Section 4.2)
    ratio: float = 0.25      # compression ratio r (Appendix B)
    rope_base: float = 0.0   # 0 = no rotary embedding
    needles: str = "none"    # "uniform:<m>" | "depths" | "none"
    outlier_frac: float = 0.0
    outlier_gain: float = 8.0
    seed: int = 2602_02199

    @property
    def n_blocks(self) -> int:
        return self.context_len // self.block_size

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


WORKLOADS = {
    # tiny single layer; the case the oracle finishes in seconds
    "tiny": Workload("tiny", 1, 1, 32, 8, 128, 4096, 1024, 32, 8, 16, 4, needles="uniform:8"),
    # Llama-3-8B-shaped, 32k context
    "llama8b_32k": Workload("llama8b_32k", 32, 1, 32, 8, 128, 32768, 4096, 64, 10, 32, 4,
                            rope_base=500000.0, needles="uniform:64"),
    # same shape at 64k with magnitude outliers; n is swept by the caller
    "llama8b_64k": Workload("llama8b_64k", 32, 1, 32, 8, 128, 65536, 8192, 64, 10, 32, 4,
                            rope_base=500000.0, outlier_frac=0.01),
    # the headline: 128k context
    "llama8b_128k": Workload("llama8b_128k", 32, 1, 32, 8, 128, 131072, 8192, 64, 10, 64, 4,
                             rope_base=500000.0, needles="depths"),
    # Qwen2-7B-shaped, four independent sequences
    "qwen7b_128k": Workload("qwen7b_128k", 28, 4, 28, 4, 128, 131072, 4096, 32, 8, 32, 8,
                            rope_base=1000000.0, needles="uniform:16"),
}


def workload(name: str) -> Workload:
    return WORKLOADS[name]


# ----------------------------------------------------------------------------------------------
# bfloat16 <-> float32 bit conversion (round to nearest even)
# ----------------------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------------------------
# counter-based streams
# ----------------------------------------------------------------------------------------------
def _stream(w: Workload, *what) -> np.random.Generator:
    """An independent Philox stream named by (workload seed, name, what...)."""
    tag = repr((w.seed, w.name) + tuple(what)).encode()
    digest = hashlib.blake2b(tag, digest_size=16).digest()
    key = np.frombuffer(digest, dtype=np.uint64).copy()
    return np.random.Generator(np.random.Philox(key=key))


def _channel_scales(w: Workload, layer: int, tensor: str, n_heads: int) -> np.ndarray:
    """Per-(head, channel) log-normal(0, 0.5) gains: a few channels carry most of the energy."""
    g = _stream(w, "scales", layer, tensor)
    return np.exp(0.5 * g.standard_normal((n_heads, w.head_dim))).astype(np.float32)


def _rope(x: np.ndarray, positions: np.ndarray, base: float) -> np.ndarray:
    """Rotary embedding, rotate-half pairing (i, i + d/2). x: [..., T, d], positions: [T]."""
    d = x.shape[-1]
    half = d // 2
    inv_freq = base ** (-np.arange(half, dtype=np.float64) * 2.0 / d)
    ang = positions.astype(np.float64)[:, None] * inv_freq[None, :]
    cos = np.cos(ang).astype(np.float32)
    sin = np.sin(ang).astype(np.float32)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * cos - x2 * sin, x2 * cos + x1 * sin], axis=-1)


def hyperplanes(w: Workload) -> np.ndarray:
    """Gaussian SimHash hyperplanes, bf16 bits [L*K, d]; row r*K + b is bit b of table r.
    One set is shared by all layers, heads and sequences."""
    g = _stream(w, "hyperplanes")
    p = g.standard_normal((w.lsh_tables * w.lsh_bits, w.head_dim), dtype=np.float32)
    return f32_to_bf16_bits(p)


def _q_window_f32(w: Workload, layer: int, seq: int) -> np.ndarray:
    g = _stream(w, "q", layer, seq)
    q = g.standard_normal((w.n_q_heads, w.window, w.head_dim), dtype=np.float32)
    q *= _channel_scales(w, layer, "q", w.n_q_heads)[:, None, :]
    if w.rope_base > 0:
        pos = np.arange(w.context_len, w.context_len + w.window)
        q = _rope(q, pos, w.rope_base)
    return q


def q_window(w: Workload, layer: int, seq: int) -> np.ndarray:
    """Observation-window queries, bf16 bits [H_q, W, d]; rotated at positions L .. L+W-1."""
    return f32_to_bf16_bits(_q_window_f32(w, layer, seq))


def needle_positions(w: Workload, layer: int, seq: int) -> np.ndarray:
    """Absolute token positions of the planted needle keys (same for every KV head)."""
    if w.needles == "none":
        return np.zeros(0, dtype=np.int64)
    if w.needles == "depths":
        return np.array([int(round(0.1 * i * w.context_len)) for i in range(1, 10)], dtype=np.int64)
    kind, m = w.needles.split(":")
    assert kind == "uniform"
    g = _stream(w, "needle_pos", layer, seq)
    return np.sort(g.choice(w.context_len, size=int(m), replace=False)).astype(np.int64)


def kv_block(w: Workload, layer: int, seq: int, block: int):
    """Keys and values of one block, bf16 bits, each [H_kv, S, d].

    K, V ~ N(0,1) times per-(head, channel) log-normal gains; a fraction ``outlier_frac`` of
    tokens has both rows multiplied by ``outlier_gain``; keys are rotated at their absolute
    positions; needle keys are then overwritten with ||k||_rms * (0.9 q^ + sqrt(0.19) u^) for a
    randomly chosen window query q of the KV head's group and a random unit u orthogonal to q.
    """
    S, d, hk = w.block_size, w.head_dim, w.n_kv_heads
    g = _stream(w, "kv", layer, seq, block)
    k = g.standard_normal((hk, S, d), dtype=np.float32)
    v = g.standard_normal((hk, S, d), dtype=np.float32)
    k *= _channel_scales(w, layer, "k", hk)[:, None, :]
    v *= _channel_scales(w, layer, "v", hk)[:, None, :]
    if w.outlier_frac > 0:
        hot = g.random(S) < w.outlier_frac
        k[:, hot, :] *= w.outlier_gain
        v[:, hot, :] *= w.outlier_gain
    start = block * S
    if w.rope_base > 0:
        k = _rope(k, np.arange(start, start + S), w.rope_base)
    pos = needle_positions(w, layer, seq)
    here = pos[(pos >= start) & (pos < start + S)]
    if here.size:
        q = _q_window_f32(w, layer, seq)
        # the planted keys must be aligned with what the kernels see: bf16-rounded queries
        q = bf16_bits_to_f32(f32_to_bf16_bits(q)).astype(np.float64)
        G = w.group
        rms = np.sqrt((k.astype(np.float64) ** 2).sum(axis=2).mean(axis=1))      # [H_kv]
        for p in here:
            gp = _stream(w, "needle", layer, seq, int(p))
            for h in range(hk):
                qi = q[h * G + int(gp.integers(G)), int(gp.integers(w.window))]
                qh = qi / np.linalg.norm(qi)
                u = gp.standard_normal(d)
                u -= (u @ qh) * qh
                u /= np.linalg.norm(u)
                k[h, p - start] = (rms[h] * (0.9 * qh + math.sqrt(1.0 - 0.81) * u)).astype(np.float32)
    return f32_to_bf16_bits(k), f32_to_bf16_bits(v)


def kv_blocks(w: Workload, layer: int, seq: int, first_block: int, n_blocks: int):
    """Consecutive blocks concatenated along the token axis: [H_kv, n_blocks*S, d] each."""
    ks, vs = zip(*(kv_block(w, layer, seq, t) for t in range(first_block, first_block + n_blocks)))
    return np.concatenate(ks, axis=1), np.concatenate(vs, axis=1)
