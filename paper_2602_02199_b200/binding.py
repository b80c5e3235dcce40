"""ctypes binding of liblaserkv.so: the same names as include/laser_kv.h, argument marshalling
only. PyTorch appears here solely as the owner of device memory and streams."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

from . import build as _build

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CAPACITY, ERR_ALIGNMENT, ERR_CUDA, ERR_TIMEOUT, ERR_STATE = range(8)

EXPORTS = [
    "laser_kv_budget", "laser_kv_partition", "laser_kv_query_sizes", "laser_kv_init",
    "laser_kv_select_block", "laser_kv_select_block_host", "laser_kv_cache_view",
    "laser_kv_debug_view", "laser_kv_poll_status", "laser_kv_reset", "laser_kv_destroy",
    "laser_kv_status_string", "laser_kv_last_error", "laser_kv_launch_count",
    "laser_kv_two_stage_topk", "laser_kv_gather_append", "laser_kv_profile_enable",
    "laser_kv_profile_read", "laser_kv_window_scores", "laser_kv_window_scores_scratch_bytes",
    "laser_kv_window_scores_static", "laser_kv_window_scores_static_max_bytes",
    "laser_kv_collision_counts", "laser_kv_collision_counts_scratch_bytes", "laser_kv_consensus_accumulate",
    "laser_kv_decode_attention", "laser_kv_decode_attention_scratch_bytes", "laser_kv_collision_probability",
    "laser_kv_set_layer_budget", "laser_kv_set_wait_budget", "laser_kv_window_scores_static_status",
    "laser_kv_lookback_close", "laser_kv_select_tail", "laser_kv_get_counters",
]


class Config(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("batch", C.c_int32), ("n_q_heads", C.c_int32),
        ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("block_size", C.c_int32),
        ("window", C.c_int32), ("max_blocks", C.c_int32), ("max_blocks_per_call", C.c_int32),
        ("lsh_bits", C.c_int32), ("lsh_tables", C.c_int32), ("protection_divisor", C.c_int32),
        ("budget_per_block", C.c_int32), ("debug", C.c_int32), ("context_len", C.c_int64),
        ("ratio", C.c_double), ("alpha", C.c_double), ("softmax_scale", C.c_float),
        ("device", C.c_int32), ("lookback", C.c_int32),
    ]


class View(C.Structure):
    _fields_ = [("K", C.c_void_p), ("V", C.c_void_p), ("pos", C.c_void_p), ("len", C.c_int64),
                ("cap", C.c_int64), ("kv_strides", C.c_int64 * 3), ("pos_strides", C.c_int64 * 2)]


class Debug(C.Structure):
    _fields_ = [("s_exact", C.c_void_p), ("counts", C.c_void_p), ("lse2", C.c_void_p),
                ("query_buckets", C.c_void_p), ("key_buckets", C.c_void_p), ("hist", C.c_void_p),
                ("idx", C.c_void_p), ("n_blocks", C.c_int32), ("batch", C.c_int32),
                ("n_kv_heads", C.c_int32), ("block_size", C.c_int32), ("budget", C.c_int32),
                ("gw", C.c_int32), ("lsh_tables", C.c_int32), ("lsh_bits", C.c_int32),
                ("n_sign_fixups", C.c_int32), ("segment_keys", C.c_int32), ("segment_shift", C.c_int32),
                ("window_part", C.c_int32)]


class Counters(C.Structure):
    _fields_ = [("select_calls", C.c_int64), ("blocks", C.c_int64), ("tokens", C.c_int64),
                ("entries_appended", C.c_int64), ("algorithmic_bytes", C.c_int64)]


class LaserKVError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"laser_kv status {status}: {message}")
        self.status = status


_lib = None


def lib_path() -> str:
    return _build.LIB


def load(build_if_missing: bool = True) -> C.CDLL:
    """Loads the shared library (building it with nvcc first if its sources are newer)."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing:
        _build.build()      # a no-op when the library is newer than its sources; a failed rebuild raises
    if not os.path.exists(_build.LIB):
        raise RuntimeError(f"{_build.LIB} is missing: build it with python -m paper_2602_02199_b200.build")
    lib = C.CDLL(_build.LIB)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    p = C.POINTER
    lib.laser_kv_budget.restype = i32
    lib.laser_kv_budget.argtypes = [i64, i32, C.c_double]
    lib.laser_kv_partition.restype = i32
    lib.laser_kv_partition.argtypes = [i32, i32, C.c_double, p(i32), p(i32), p(i32), p(i32)]
    lib.laser_kv_query_sizes.restype = i32
    lib.laser_kv_query_sizes.argtypes = [p(Config), p(sz), p(sz)]
    lib.laser_kv_init.restype = i32
    lib.laser_kv_init.argtypes = [p(Config), vp, vp, sz, vp, sz, p(vp)]
    lib.laser_kv_select_block.restype = i32
    lib.laser_kv_select_block.argtypes = [vp, i32, vp, vp, vp, p(i64), p(i64), i32, vp]
    lib.laser_kv_select_block_host.restype = i32
    lib.laser_kv_select_block_host.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, i32, vp, vp]
    lib.laser_kv_cache_view.restype = i32
    lib.laser_kv_cache_view.argtypes = [vp, i32, p(View)]
    lib.laser_kv_debug_view.restype = i32
    lib.laser_kv_debug_view.argtypes = [vp, p(Debug)]
    lib.laser_kv_poll_status.restype = i32
    lib.laser_kv_poll_status.argtypes = [vp, vp]
    lib.laser_kv_reset.restype = i32
    lib.laser_kv_reset.argtypes = [vp, i32]
    lib.laser_kv_destroy.restype = None
    lib.laser_kv_destroy.argtypes = [vp]
    lib.laser_kv_status_string.restype = C.c_char_p
    lib.laser_kv_status_string.argtypes = [i32]
    lib.laser_kv_last_error.restype = C.c_char_p
    lib.laser_kv_last_error.argtypes = [vp]
    lib.laser_kv_launch_count.restype = i64
    lib.laser_kv_launch_count.argtypes = []
    lib.laser_kv_two_stage_topk.restype = i32
    lib.laser_kv_two_stage_topk.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp, vp]
    lib.laser_kv_gather_append.restype = i32
    lib.laser_kv_gather_append.argtypes = [vp, vp, i64, i64, i32, vp, i32, i32, vp, vp, i64, i64, vp, i64, i64, i32, vp, vp]
    lib.laser_kv_get_counters.restype = i32
    lib.laser_kv_get_counters.argtypes = [vp, p(Counters)]
    lib.laser_kv_select_tail.restype = i32
    lib.laser_kv_select_tail.argtypes = [vp, i32, vp, vp, vp, p(i64), p(i64), i32, vp]
    lib.laser_kv_lookback_close.restype = i32
    lib.laser_kv_lookback_close.argtypes = [vp, i32, vp, vp, p(i64), vp]
    lib.laser_kv_set_wait_budget.restype = i32
    lib.laser_kv_set_wait_budget.argtypes = [vp, C.c_uint32]
    lib.laser_kv_window_scores_static_status.restype = i32
    lib.laser_kv_window_scores_static_status.argtypes = [vp]
    lib.laser_kv_profile_enable.restype = i32
    lib.laser_kv_profile_enable.argtypes = [vp, i32]
    lib.laser_kv_profile_read.restype = i32
    lib.laser_kv_profile_read.argtypes = [vp, p(i32), p(C.c_char_p), p(C.c_float), p(i32)]
    lib.laser_kv_window_scores_scratch_bytes.restype = sz
    lib.laser_kv_window_scores_scratch_bytes.argtypes = [i32] * 6
    lib.laser_kv_window_scores.restype = i32
    lib.laser_kv_window_scores.argtypes = [vp, vp, p(i64), p(i64), i32, i32, i32, i32, i32, i32, C.c_float, vp, sz,
                                           vp, vp]
    lib.laser_kv_window_scores_static_max_bytes.restype = sz
    lib.laser_kv_window_scores_static_max_bytes.argtypes = []
    lib.laser_kv_window_scores_static.restype = i32
    lib.laser_kv_window_scores_static.argtypes = [vp, vp, p(i64), p(i64), i32, i32, i32, i32, i32, i32, C.c_float,
                                                  vp, vp]
    lib.laser_kv_collision_counts_scratch_bytes.restype = sz
    lib.laser_kv_collision_counts_scratch_bytes.argtypes = [i32] * 8
    lib.laser_kv_collision_counts.restype = i32
    lib.laser_kv_collision_counts.argtypes = [vp, vp, vp, p(i64), p(i64), i32, i32, i32, i32, i32, i32, i32, i32, vp, sz,
                                              vp, vp]
    lib.laser_kv_consensus_accumulate.restype = i32
    lib.laser_kv_consensus_accumulate.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp, vp, vp]
    lib.laser_kv_set_layer_budget.restype = i32
    lib.laser_kv_set_layer_budget.argtypes = [vp, i32, i32]
    lib.laser_kv_collision_probability.restype = i32
    lib.laser_kv_collision_probability.argtypes = [vp, vp, p(i64), p(i64), i32, i32, i32, i32, i32, i32, i32, vp, sz, vp, vp]
    lib.laser_kv_decode_attention_scratch_bytes.restype = sz
    lib.laser_kv_decode_attention_scratch_bytes.argtypes = [vp]
    lib.laser_kv_decode_attention.restype = i32
    lib.laser_kv_decode_attention.argtypes = [vp, i32, vp, p(i64), C.c_float, vp, vp, sz, vp]
    _lib = lib
    return lib


def _check(status: int, handle=None):
    if status != OK:
        msg = load().laser_kv_last_error(handle)
        raise LaserKVError(status, (msg or b"").decode() or load().laser_kv_status_string(status).decode())


# ---- host-only helpers ---------------------------------------------------------------------------
def laser_kv_budget(context_len: int, block_size: int, ratio: float = 0.25) -> int:
    return int(load().laser_kv_budget(context_len, block_size, ratio))


def laser_kv_partition(B: int, n: int, alpha: float = 0.75):
    a, l, ke, kl = C.c_int32(), C.c_int32(), C.c_int32(), C.c_int32()
    _check(load().laser_kv_partition(B, n, alpha, C.byref(a), C.byref(l), C.byref(ke), C.byref(kl)))
    return a.value, l.value, ke.value, kl.value


def laser_kv_query_sizes(cfg: Config):
    cb, wb = C.c_size_t(), C.c_size_t()
    _check(load().laser_kv_query_sizes(C.byref(cfg), C.byref(cb), C.byref(wb)))
    return cb.value, wb.value


def laser_kv_launch_count() -> int:
    return int(load().laser_kv_launch_count())


def make_config(*, n_layers, batch, n_q_heads, n_kv_heads, block_size, window, max_blocks,
                max_blocks_per_call, lsh_bits, lsh_tables, protection_divisor, budget_per_block=0,
                context_len=0, ratio=0.25, alpha=0.75, softmax_scale=0.0, debug=0, device=0,
                head_dim=128, lookback=0) -> Config:
    return Config(n_layers, batch, n_q_heads, n_kv_heads, head_dim, block_size, window, max_blocks,
                  max_blocks_per_call, lsh_bits, lsh_tables, protection_divisor, budget_per_block,
                  debug, context_len, ratio, alpha, softmax_scale, device, lookback)


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def _stream_ptr(stream) -> int:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream)
    return int(getattr(stream, "cuda_stream", stream))


@dataclass
class DebugTensors:
    s_exact: object
    counts: object
    lse2: object
    query_buckets: object
    key_buckets: object
    hist: object
    idx: object
    n_sign_fixups: int
    segment_keys: int = 0
    segment_shift: int = 0
    window_part: int = 0


class LaserKV:
    """A handle plus the torch tensors that back its cache and workspace."""

    def __init__(self, cfg: Config, hyperplanes):
        import torch
        self._torch = torch
        self.lib = load()
        self.cfg = cfg
        self.device = torch.device("cuda", cfg.device)
        cb, wb = laser_kv_query_sizes(cfg)
        self.cache_mem = torch.empty(cb, dtype=torch.uint8, device=self.device)
        self.workspace = torch.empty(wb, dtype=torch.uint8, device=self.device)
        self.hyperplanes = hyperplanes
        assert hyperplanes.is_cuda and hyperplanes.is_contiguous() and hyperplanes.element_size() == 2
        h = C.c_void_p()
        _check(self.lib.laser_kv_init(C.byref(cfg), _ptr(hyperplanes), _ptr(self.cache_mem), cb,
                                      _ptr(self.workspace), wb, C.byref(h)))
        self.handle = h
        a, _, ke, kl = laser_kv_partition(self.budget, cfg.protection_divisor,
                                          0.75 if cfg.alpha < 0 else cfg.alpha)
        self.anchors, self.k_exact, self.k_lsh = a, ke, kl

    @property
    def budget(self) -> int:
        c = self.cfg
        if c.budget_per_block:
            return c.budget_per_block
        return laser_kv_budget(c.context_len, c.block_size, c.ratio or 0.25)

    def close(self):
        if getattr(self, "handle", None):
            self.lib.laser_kv_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the calls of the header ----
    def laser_kv_select_block(self, layer, K_blk, V_blk, Q_win, n_blocks, stream=None):
        """K_blk, V_blk: [batch][H_kv][n_blocks*S][d]-indexable 2-byte tensors (any strides with a
        contiguous last dim); Q_win: [batch][H_q][W][d]."""
        ks = (C.c_int64 * 3)(*K_blk.stride()[:3])
        assert tuple(V_blk.stride()) == tuple(K_blk.stride()) and K_blk.stride(3) == 1
        qs = (C.c_int64 * 3)(*Q_win.stride()[:3])
        _check(self.lib.laser_kv_select_block(self.handle, layer, _ptr(K_blk), _ptr(V_blk), _ptr(Q_win),
                                              ks, qs, n_blocks, _stream_ptr(stream)), self.handle)

    def laser_kv_select_block_host(self, layer, K_host, V_host, Q_host, K_stage, V_stage, Q_stage,
                                   n_blocks, pos_out_host=None, stream=None):
        _check(self.lib.laser_kv_select_block_host(self.handle, layer, _ptr(K_host), _ptr(V_host),
                                                   _ptr(Q_host), _ptr(K_stage), _ptr(V_stage),
                                                   _ptr(Q_stage), n_blocks, _ptr(pos_out_host),
                                                   _stream_ptr(stream)), self.handle)

    def laser_kv_select_tail(self, layer, K_blk, V_blk, Q_win, n_tokens, stream=None):
        """A last block of n_tokens < block_size tokens: K_blk, V_blk [batch][H_kv][n_tokens][d]."""
        ks = (C.c_int64 * 3)(*K_blk.stride()[:3])
        assert tuple(V_blk.stride()) == tuple(K_blk.stride()) and K_blk.stride(3) == 1
        qs = (C.c_int64 * 3)(*Q_win.stride()[:3])
        _check(self.lib.laser_kv_select_tail(self.handle, layer, _ptr(K_blk), _ptr(V_blk), _ptr(Q_win),
                                             ks, qs, n_tokens, _stream_ptr(stream)), self.handle)

    def laser_kv_lookback_close(self, layer, K_tail, V_tail, stream=None):
        """K_tail, V_tail: [batch][H_kv][a][d] views of the last block's last a = floor(B/n) rows."""
        ks = (C.c_int64 * 3)(*K_tail.stride()[:3])
        assert tuple(V_tail.stride()) == tuple(K_tail.stride())
        _check(self.lib.laser_kv_lookback_close(self.handle, layer, _ptr(K_tail), _ptr(V_tail), ks,
                                                _stream_ptr(stream)), self.handle)

    def laser_kv_cache_view(self, layer):
        """Returns (K, V, pos, len) as torch views [batch][H_kv][cap][d] / [batch][H_kv][cap]."""
        torch = self._torch
        v = View()
        _check(self.lib.laser_kv_cache_view(self.handle, layer, C.byref(v)), self.handle)
        c = self.cfg
        n = c.batch * c.n_kv_heads * v.cap
        base = self.cache_mem.data_ptr()
        k = self.cache_mem[v.K - base: v.K - base + n * 256].view(torch.int16).view(c.batch, c.n_kv_heads, v.cap, 128)
        vv = self.cache_mem[v.V - base: v.V - base + n * 256].view(torch.int16).view(c.batch, c.n_kv_heads, v.cap, 128)
        p = self.cache_mem[v.pos - base: v.pos - base + n * 4].view(torch.int32).view(c.batch, c.n_kv_heads, v.cap)
        return k, vv, p, int(v.len)

    def laser_kv_debug_view(self) -> DebugTensors:
        torch = self._torch
        d = Debug()
        _check(self.lib.laser_kv_debug_view(self.handle, C.byref(d)), self.handle)
        base = self.workspace.data_ptr()
        nseg = d.batch * d.n_kv_heads * d.n_blocks
        S, L = d.segment_keys, d.lsh_tables

        def view(ptr, nbytes, dtype, shape):
            if not ptr:
                return None
            return self.workspace[ptr - base: ptr - base + nbytes].view(dtype).view(*shape)

        shp = (d.batch, d.n_kv_heads, d.n_blocks)
        return DebugTensors(
            s_exact=view(d.s_exact, nseg * S * 4, torch.float32, shp + (S,)),
            counts=view(d.counts, nseg * S * 4, torch.int32, shp + (S,)),
            lse2=view(d.lse2, nseg * d.gw * 4, torch.float32, shp + (d.gw,)),
            query_buckets=view(d.query_buckets, d.batch * d.n_kv_heads * d.gw * L * 2, torch.int16,
                               (d.batch, d.n_kv_heads, d.gw, L)),
            key_buckets=view(d.key_buckets, nseg * S * L * 2, torch.int16, shp + (S, L)),
            hist=view(d.hist, d.batch * d.n_kv_heads * L * (2 << d.lsh_bits), torch.int16,
                      (d.batch, d.n_kv_heads, L, 1 << d.lsh_bits)),
            idx=view(d.idx, nseg * max(d.budget, 1) * 4, torch.int32, shp + (max(d.budget, 1),)),
            n_sign_fixups=int(d.n_sign_fixups), segment_keys=int(d.segment_keys), segment_shift=int(d.segment_shift),
            window_part=int(d.window_part))

    def laser_kv_decode_attention(self, layer, Q_dec, softmax_scale=0.0, out=None, stream=None):
        """Q_dec: [batch][H_q][d] 2-byte tensor (contiguous last dim) -> fp32 [batch][H_q][d]."""
        torch = self._torch
        c = self.cfg
        assert Q_dec.stride(2) == 1 and Q_dec.element_size() == 2
        if getattr(self, "_decode_scratch", None) is None:
            nbytes = int(self.lib.laser_kv_decode_attention_scratch_bytes(self.handle))
            self._decode_scratch = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        if out is None:
            out = torch.empty(c.batch, c.n_q_heads, 128, dtype=torch.float32, device=self.device)
        qs = (C.c_int64 * 2)(*Q_dec.stride()[:2])
        _check(self.lib.laser_kv_decode_attention(self.handle, layer, _ptr(Q_dec), qs, softmax_scale, _ptr(out),
                                                  _ptr(self._decode_scratch), self._decode_scratch.numel(),
                                                  _stream_ptr(stream)), self.handle)
        return out

    def laser_kv_poll_status(self, stream=None):
        _check(self.lib.laser_kv_poll_status(self.handle, _stream_ptr(stream)), self.handle)

    def laser_kv_profile_enable(self, on=True):
        _check(self.lib.laser_kv_profile_enable(self.handle, 1 if on else 0), self.handle)

    def laser_kv_profile_read(self):
        """-> {kernel name: (total device ms, launches)} since profiling was enabled."""
        n = C.c_int32()
        names = (C.c_char_p * 16)()
        ms = (C.c_float * 16)()
        cnt = (C.c_int32 * 16)()
        _check(self.lib.laser_kv_profile_read(self.handle, C.byref(n), names, ms, cnt), self.handle)
        return {names[i].decode(): (float(ms[i]), int(cnt[i])) for i in range(n.value)}

    def laser_kv_set_layer_budget(self, layer, budget_per_block):
        _check(self.lib.laser_kv_set_layer_budget(self.handle, layer, budget_per_block), self.handle)

    def laser_kv_get_counters(self):
        c = Counters()
        _check(self.lib.laser_kv_get_counters(self.handle, C.byref(c)), self.handle)
        return {k: int(getattr(c, k)) for k, _ in Counters._fields_}

    def laser_kv_set_wait_budget(self, max_polls):
        _check(self.lib.laser_kv_set_wait_budget(self.handle, max_polls), self.handle)

    def laser_kv_reset(self, layer=-1):
        _check(self.lib.laser_kv_reset(self.handle, layer), self.handle)


def laser_kv_two_stage_topk(s_exact, counts, anchors, k_exact, k_lsh, stream=None):
    """s_exact fp32 [n_seg][S], counts int32 [n_seg][S] (device) -> idx int32 [n_seg][B]."""
    import torch
    n_seg, S = s_exact.shape
    B = 2 * anchors + k_exact + k_lsh
    idx = torch.empty((n_seg, B), dtype=torch.int32, device=s_exact.device)
    _check(load().laser_kv_two_stage_topk(_ptr(s_exact), _ptr(counts), n_seg, S, anchors, k_exact, k_lsh,
                                          _ptr(idx), _stream_ptr(stream)))
    return idx


def laser_kv_gather_append(K_src, V_src, idx, K_dst, V_dst, pos_out, dst_offset, pos_base, status, stream=None):
    """K_src, V_src [n_seg][rows][128]; idx int32 [n_seg][n_keep]; K_dst, V_dst [n_seg][cap][128];
    pos_out int32 [n_seg][cap]; status int32 device tensor of one element (0 afterwards unless an
    index was out of range)."""
    n_seg, n_keep = idx.shape
    _check(load().laser_kv_gather_append(_ptr(K_src), _ptr(V_src), K_src.stride(0), K_src.stride(1), K_src.shape[1],
                                         _ptr(idx), n_seg, n_keep, _ptr(K_dst), _ptr(V_dst), K_dst.stride(0),
                                         K_dst.shape[1], _ptr(pos_out), pos_out.stride(0), dst_offset, pos_base,
                                         _ptr(status), _stream_ptr(stream)))


def laser_kv_window_scores_scratch_bytes(batch, n_q_heads, n_kv_heads, block_size, window, n_blocks) -> int:
    return int(load().laser_kv_window_scores_scratch_bytes(batch, n_q_heads, n_kv_heads, block_size, window, n_blocks))


def laser_kv_window_scores(K_blk, Q_win, block_size, n_blocks, softmax_scale=0.0, scratch=None, stream=None):
    """K_blk [batch][H_kv][n_blocks*S][128], Q_win [batch][H_q][W][128] (2-byte device tensors) ->
    S_exact fp32 [batch][H_kv][n_blocks][S]. `scratch` (uint8 device tensor) is allocated by torch
    when not given."""
    import torch
    batch, h_kv = K_blk.shape[0], K_blk.shape[1]
    h_q, window = Q_win.shape[1], Q_win.shape[2]
    need = laser_kv_window_scores_scratch_bytes(batch, h_q, h_kv, block_size, window, n_blocks)
    if scratch is None:
        scratch = torch.empty(max(need, 256), dtype=torch.uint8, device=K_blk.device)
    out = torch.empty((batch, h_kv, n_blocks, block_size), dtype=torch.float32, device=K_blk.device)
    ks = (C.c_int64 * 3)(*K_blk.stride()[:3])
    qs = (C.c_int64 * 3)(*Q_win.stride()[:3])
    _check(load().laser_kv_window_scores(_ptr(K_blk), _ptr(Q_win), ks, qs, batch, h_q, h_kv, block_size, window,
                                         n_blocks, softmax_scale, _ptr(scratch), scratch.numel(), _ptr(out),
                                         _stream_ptr(stream)))
    return out


def laser_kv_collision_counts(K_blk, Q_win, hyperplanes, block_size, n_blocks, lsh_bits, lsh_tables, scratch=None,
                              stream=None):
    """K_blk [batch][H_kv][n_blocks*S][128], Q_win [batch][H_q][W][128], hyperplanes [L*K][128] (2-byte
    device tensors) -> collision counts int32 [batch][H_kv][n_blocks][S]. Returns (counts, scratch); the
    first int of scratch is the status word. `scratch` is allocated by torch when not given."""
    import torch
    batch, h_kv = K_blk.shape[0], K_blk.shape[1]
    h_q, window = Q_win.shape[1], Q_win.shape[2]
    need = int(load().laser_kv_collision_counts_scratch_bytes(batch, h_q, h_kv, block_size, window, n_blocks,
                                                              lsh_bits, lsh_tables))
    if scratch is None:
        scratch = torch.empty(max(need, 256), dtype=torch.uint8, device=K_blk.device)
    out = torch.empty((batch, h_kv, n_blocks, block_size), dtype=torch.int32, device=K_blk.device)
    ks = (C.c_int64 * 3)(*K_blk.stride()[:3])
    qs = (C.c_int64 * 3)(*Q_win.stride()[:3])
    _check(load().laser_kv_collision_counts(_ptr(K_blk), _ptr(Q_win), _ptr(hyperplanes), ks, qs, batch, h_q, h_kv,
                                            block_size, window, n_blocks, lsh_bits, lsh_tables, _ptr(scratch),
                                            scratch.numel(), _ptr(out), _stream_ptr(stream)))
    return out, scratch


def laser_kv_collision_probability(K_blk, Q_win, block_size, n_blocks, lsh_bits, scratch=None, stream=None):
    """K_blk [batch][H_kv][n_blocks*S][128], Q_win [batch][H_q][W][128] (2-byte device tensors) -> the
    closed-form recall score fp32 [batch][H_kv][n_blocks][S]. Returns (p, scratch); the first int of
    scratch is the status word. `p.view(torch.int32)` serves as `counts` of laser_kv_two_stage_topk."""
    import torch
    batch, h_kv = K_blk.shape[0], K_blk.shape[1]
    h_q, window = Q_win.shape[1], Q_win.shape[2]
    if scratch is None:
        scratch = torch.empty(256, dtype=torch.uint8, device=K_blk.device)
    out = torch.empty((batch, h_kv, n_blocks, block_size), dtype=torch.float32, device=K_blk.device)
    ks = (C.c_int64 * 3)(*K_blk.stride()[:3])
    qs = (C.c_int64 * 3)(*Q_win.stride()[:3])
    _check(load().laser_kv_collision_probability(_ptr(K_blk), _ptr(Q_win), ks, qs, batch, h_q, h_kv, block_size, window,
                                                 n_blocks, lsh_bits, _ptr(scratch), scratch.numel(), _ptr(out),
                                                 _stream_ptr(stream)))
    return out, scratch


def laser_kv_consensus_accumulate(s_exact, counts, s_acc=None, c_acc=None, carry=False, stream=None):
    """Sums [batch][H][n_blocks][S] scores (fp32) and counts (int32) over the heads into
    [batch][n_blocks][S] accumulators; carry=True adds to the given accumulators."""
    import torch
    batch, heads, nb, S = s_exact.shape
    if s_acc is None:
        s_acc = torch.empty((batch, nb, S), dtype=torch.float32, device=s_exact.device)
        c_acc = torch.empty((batch, nb, S), dtype=torch.int32, device=s_exact.device)
    _check(load().laser_kv_consensus_accumulate(_ptr(s_exact), _ptr(counts), batch, heads, nb, S, 1 if carry else 0,
                                                _ptr(s_acc), _ptr(c_acc), _stream_ptr(stream)))
    return s_acc, c_acc


def laser_kv_window_scores_static_max_bytes() -> int:
    return int(load().laser_kv_window_scores_static_max_bytes())


def laser_kv_window_scores_static(K_blk, Q_win, block_size, n_blocks, out, softmax_scale=0.0, stream=None):
    """The window-score step for callers that cannot allocate: inputs and the fp32 output tensor
    `out` [batch][H_kv][n_blocks][S] come from the caller, the scratch is the library's built-in
    2 MiB array. This wrapper allocates nothing either. Calls sharing a device must not overlap."""
    batch, h_kv = K_blk.shape[0], K_blk.shape[1]
    h_q, window = Q_win.shape[1], Q_win.shape[2]
    ks = (C.c_int64 * 3)(*K_blk.stride()[:3])
    qs = (C.c_int64 * 3)(*Q_win.stride()[:3])
    _check(load().laser_kv_window_scores_static(_ptr(K_blk), _ptr(Q_win), ks, qs, batch, h_q, h_kv, block_size,
                                                window, n_blocks, softmax_scale, _ptr(out), _stream_ptr(stream)))
    return out


def laser_kv_window_scores_static_status(stream=None):
    """Raises LaserKVError if a kernel of an earlier laser_kv_window_scores_static call on the current
    device recorded an error (and clears it); synchronises the stream."""
    _check(load().laser_kv_window_scores_static_status(_stream_ptr(stream)))
