// Key-streaming tensor-core kernels for the two dense contractions of the selection path:
//   * the window-score contraction Q_win . K^T  (Section 3.3 "Precision", Algorithm 1 line 3)
//   * the hyperplane projection K . P^T         (Section 3.3 "Recall", hash functions h_r)
// One warp-specialised skeleton serves three passes. A CTA keeps one small operand stationary
// in shared memory (the group's window queries, or a chunk of hyperplanes with the matching
// slice of the query-bucket histogram) and streams 128-key tiles of one (sequence, KV head,
// block) through a TMA -> tcgen05.mma -> TMEM -> register pipeline:
//
//   kLse   : D[query][key]; every thread owns one query row and keeps an online
//            (max, sum-exp2) pair over the CTA's keys -> per-split partials of log-sum-exp.
//   kScore : D[key][query]; every thread owns one key and sums exp2(s - lse_q) over the
//            group's queries -> S_exact[key].
//   kProj  : D[key][hyperplane]; every thread owns one key, packs sign bits into K-bit bucket
//            ids, looks the buckets up in the query-bucket histogram (count of window queries
//            per bucket) and adds the collisions to count[key]. Signs decided by a projection
//            that is tiny relative to the key's other projections are queued for an exact
//            recomputation.
//
// Warp roles (320 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner,
// warps 2..9 = two epilogue groups of four warps (TMEM lane quarter = warp_id % 4) that split
// the accumulator columns of every tile.
#pragma once
#include "ptx.cuh"

namespace lkv {

constexpr int kTileKeys = 128;                 // keys per streamed tile (UMMA M or N)
constexpr int kAtomCols = 64;                  // bf16 elements per 128-byte swizzle row
constexpr int kTileAtomBytes = kTileKeys * 128;  // one 64-column half of a key tile
constexpr int kTileBytes = 2 * kTileAtomBytes;   // 128 keys x 128 dims bf16
constexpr int kStages = 4;
constexpr int kStreamThreads = 320;
constexpr int kEpilogueThreads = 256;
constexpr int kXwgBytes = 2048;                // exchange area between the two epilogue groups
constexpr int kTmemCols = 512;
constexpr int kAccStride = 256;                // TMEM columns per accumulator buffer
constexpr int kMaxStatRows = 256;

enum StreamMode { kLse = 0, kScore = 1, kProj = 2 };

enum : int { kStatusOk = 0, kStatusCapacity = 3, kStatusTimeout = 6 };

template <int N> struct IntTag { static constexpr int value = N; };

// Walks the 32-bit columns [c_begin, c_end) of the calling thread's TMEM lane (c_begin a multiple
// of 32, length a multiple of 16 and at most 128) in chunks of 32 (a last chunk of 16), loading
// chunk i+1 while f(values, first column, IntTag<count>) works on chunk i.
template <class F>
__device__ __forceinline__ void walk_columns(uint32_t taddr, int c_begin, int c_end, F&& f) {
  const int n = c_end - c_begin;
  if (n <= 0) return;
  uint32_t va[32], vb[32];
  if (n >= 32) { tmem_ld_x32(taddr + c_begin, va); tmem_wait_ld_dep32(va); }
  else { tmem_ld_x16(taddr + c_begin, va); tmem_wait_ld_dep16(va); }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int off = i * 32;
    if (off < n) {
      uint32_t* cur = (i & 1) ? vb : va;
      uint32_t* nxt = (i & 1) ? va : vb;
      const int rest = n - off - 32;       // columns after this chunk
      if (rest >= 32) tmem_ld_x32(taddr + c_begin + off + 32, nxt);
      else if (rest > 0) tmem_ld_x16(taddr + c_begin + off + 32, nxt);
      if (n - off >= 32) f(cur, c_begin + off, IntTag<32>{});
      else f(cur, c_begin + off, IntTag<16>{});
      if (rest >= 32) tmem_wait_ld_dep32(nxt);
      else if (rest > 0) tmem_wait_ld_dep16(nxt);
    }
  }
}


struct StreamArgs {
  // problem geometry
  int S;               // keys per block
  int nb;              // blocks in this call
  int t0, tn;          // block range [t0, t0 + tn) handled by this launch
  int H_kv, batch;
  int G, W, GW;        // GQA group size, window, G*W
  int tiles_per_cta;   // key tiles per CTA
  int n_split;         // CTAs along the keys of one block
  int stat_rows;       // rows of the stationary operand (GW, or tables_per_chunk * lsh_bits)
  int stat_rows_alloc; // rows reserved per 64-column half in shared memory (multiple of 8)
  int n_chunks, tables_per_chunk, lsh_bits, lsh_tables;
  float scale_log2e;   // softmax scale * log2(e)
  // buffers (device)
  float2* lse_part;        // [seg][n_split][GW]  (max, sum) in the log2 domain
  float* lse2;             // [seg][GW]
  float* s_exact;          // [seg][S]
  uint32_t* counts;        // [seg][S]
  const uint16_t* hist;    // [batch][H_kv][L][2^K]
  uint16_t* key_buckets;   // [seg][S][L] or nullptr
  int4* fix_items;         // (seg, key, table, provisional bucket)
  int* fix_count;
  int fix_cap;
  int* status;
};

__device__ __forceinline__ void record_status(int* status, int code) {
  atomicCAS(status, kStatusOk, code);
}

// Loads the 32-bit columns [CB, CE) of the calling thread's TMEM lane into r[0 .. CE-CB) as a
// sequence of power-of-two loads, each starting at a multiple of its own width.
template <int CB, int CE>
__device__ __forceinline__ void tmem_ld_range(uint32_t taddr, uint32_t* r) {
  if constexpr (CB < CE) {
    constexpr int W = (CB % 32 == 0 && CB + 32 <= CE) ? 32
                    : (CB % 16 == 0 && CB + 16 <= CE) ? 16
                    : (CB % 8 == 0 && CB + 8 <= CE)   ? 8
                    : (CB % 4 == 0 && CB + 4 <= CE)   ? 4
                    : (CB % 2 == 0 && CB + 2 <= CE)   ? 2 : 1;
    tmem_ld_cols<W>(taddr + CB, r);
    tmem_ld_range<CB + W, CE>(taddr, r + W);
  }
}

// Tables [T_BEGIN, T_END) of the chunk for the calling thread's key: packs the sign bits of each
// table's K projections into a bucket code, looks the code up in the histogram slice and
// returns the summed collisions. A table whose smallest |projection| is below 2^-15 of the
// largest |projection| among the key's first 16 hyperplanes of the chunk is queued for an exact
// recomputation of its signs. All of the thread's columns are read into registers first and the
// accumulator buffer is handed back to the MMA warp (arrive on `bar_release`) before the
// arithmetic starts; the per-table work is branch-free so that the tables interleave.
template <int KBITS, int T_BEGIN, int T_END>
__device__ __forceinline__ uint32_t proj_tables(uint32_t t_acc, uint32_t bar_release, const uint16_t* hist_s,
                                                const StreamArgs& a, int seg, int key, int table0, bool valid) {
  constexpr int NT = T_END - T_BEGIN;
  constexpr int CB = T_BEGIN * KBITS, CE = T_END * KBITS;
  constexpr uint32_t bucket_mask = (1u << KBITS) - 1u;
  uint32_t v[CE - CB];
  uint32_t v16[16];
  tmem_ld_range<CB, CE>(t_acc, v);
  tmem_ld_x16(t_acc, v16);
  tmem_wait_ld();
  reg_fence<CE - CB>(v);
  reg_fence<16>(v16);
  tc_fence_before();
  mbar_arrive(bar_release);
  float amax = 0.f;
#pragma unroll
  for (int k = 0; k < 16; k += 2) amax = max3_abs(__uint_as_float(v16[k]), __uint_as_float(v16[k + 1]), amax);
  const float tau = amax * (1.0f / 32768.0f);
  uint32_t code[NT];
  float amin[NT];
#pragma unroll
  for (int t = 0; t < NT; ++t) {
    uint32_t neg = 0;
    float mn = INFINITY;
#pragma unroll
    for (int k = 0; k < KBITS; k += 2) {
      const uint32_t x0 = v[t * KBITS + k], x1 = v[t * KBITS + k + 1];
      neg = __funnelshift_l(x0, neg, 1);                   // (neg << 1) | sign(x0)
      neg = __funnelshift_l(x1, neg, 1);
      mn = min3_abs(__uint_as_float(x0), __uint_as_float(x1), mn);
    }
    code[t] = (~neg) & bucket_mask;
    amin[t] = mn;
  }
  uint32_t partial = 0;
  float lowest = INFINITY;
#pragma unroll
  for (int t = 0; t < NT; ++t) {
    partial += hist_s[((uint32_t)(T_BEGIN + t) << KBITS) + code[t]];
    lowest = fminf(lowest, amin[t]);
  }
  if (valid && (a.key_buckets != nullptr || !(lowest >= tau))) {
#pragma unroll
    for (int t = 0; t < NT; ++t) {
      const int r = table0 + T_BEGIN + t;
      if (a.key_buckets) a.key_buckets[((size_t)seg * a.S + key) * a.lsh_tables + r] = (uint16_t)code[t];
      if (!(amin[t] >= tau)) {
        const int slot = atomicAdd(a.fix_count, 1);
        if (slot < a.fix_cap) a.fix_items[slot] = make_int4(seg, key, r, (int)code[t]);
        else record_status(a.status, kStatusCapacity);
      }
    }
  }
  return partial;
}

struct StreamSmem {
  uint32_t stat, stages, hist, lse, xwg, bars, tmem_slot;  // shared-space byte addresses
};

// Shared memory carve-up, identical on host (sizes) and device (addresses).
__host__ __device__ inline uint32_t stream_smem_bytes(int mode, int stat_rows_alloc,
                                                      int hist_bytes, int GW) {
  uint32_t b = 2u * stat_rows_alloc * 128u + kStages * kTileBytes;
  if (mode == kProj) b += (hist_bytes + 127u) & ~127u;
  if (mode == kScore) b += ((GW * 4u) + 127u) & ~127u;
  b += kXwgBytes;
  b += 256;          // barriers + TMEM slot
  return b + 1024;   // slack for 1024-byte alignment of the base
}

template <int MODE, int KBITS, int TC>
__global__ void __launch_bounds__(kStreamThreads, 1)
stream_kernel(const __grid_constant__ CUtensorMap map_keys,   // K: (d, token, head, batch)
              const __grid_constant__ CUtensorMap map_stat,   // Q: (d, W, H_q, batch) | P: (d, L*K)
              const StreamArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  // ---- which work item -------------------------------------------------------------------
  int bid = blockIdx.x;
  int chunk = 0;
  if (MODE == kProj) { chunk = bid % a.n_chunks; bid /= a.n_chunks; }
  const int split = bid % a.n_split; bid /= a.n_split;
  const int tl = bid % a.tn; bid /= a.tn;
  const int h = bid % a.H_kv;
  const int b = bid / a.H_kv;
  const int t = a.t0 + tl;
  const int seg = (b * a.H_kv + h) * a.nb + t;
  const int tiles_in_block = (a.S + kTileKeys - 1) / kTileKeys;
  const int tile0 = split * a.tiles_per_cta;
  const int ntiles = min(a.tiles_per_cta, tiles_in_block - tile0);

  // ---- shared memory ---------------------------------------------------------------------
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t stat_atom_bytes = a.stat_rows_alloc * 128u;
  StreamSmem sm;
  sm.stat = base;
  sm.stages = sm.stat + 2u * stat_atom_bytes;
  uint32_t cur = sm.stages + kStages * kTileBytes;
  const uint32_t hist_bytes = (MODE == kProj) ? (uint32_t)TC * (2u << KBITS) : 0u;
  sm.hist = cur;
  if (MODE == kProj) cur += (hist_bytes + 127u) & ~127u;
  sm.lse = cur;
  if (MODE == kScore) cur += ((a.GW * 4u) + 127u) & ~127u;
  sm.xwg = cur;
  cur += kXwgBytes;
  sm.bars = cur;
  sm.tmem_slot = cur + 128;
  const uint32_t bar_full = sm.bars;                 // kStages barriers
  const uint32_t bar_empty = sm.bars + 8 * kStages;  // kStages barriers
  const uint32_t bar_tfull = sm.bars + 16 * kStages; // 2 barriers
  const uint32_t bar_tempty = bar_tfull + 16;        // 2 barriers
  const uint32_t bar_stat = bar_tempty + 16;         // 1 barrier
  uint8_t* const gen_base = smem_raw + (base - smem_u32(smem_raw));
  const uint16_t* hist_s = reinterpret_cast<const uint16_t*>(gen_base + (sm.hist - base));
  float* lse_s = reinterpret_cast<float*>(gen_base + (sm.lse - base));
  uint8_t* xwg_s = gen_base + (sm.xwg - base);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen_base + (sm.tmem_slot - base));

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(bar_tfull + 8 * s, 1); mbar_init(bar_tempty + 8 * s, kEpilogueThreads); }
    mbar_init(bar_stat, 1);
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(sm.tmem_slot, kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int nmb = (MODE == kLse) ? (a.GW + 127) / 128 : 1;   // query row blocks of 128

  if (warp == 0) {
    // ================= TMA producer =================
    if (lane == 0) {
      bool ok = true;
      tma_prefetch_desc(&map_keys);
      tma_prefetch_desc(&map_stat);
      // stationary operand (+ histogram slice)
      const uint32_t stat_bytes = 2u * a.stat_rows * 128u;
      mbar_expect_tx(bar_stat, stat_bytes + hist_bytes);
      if (MODE == kProj) {
        const int row0 = chunk * a.stat_rows;
        tma_load_2d(sm.stat, &map_stat, bar_stat, 0, row0);
        tma_load_2d(sm.stat + stat_atom_bytes, &map_stat, bar_stat, kAtomCols, row0);
        const uint16_t* hsrc = a.hist + ((size_t)(b * a.H_kv + h) * a.lsh_tables +
                                         (size_t)chunk * TC) * ((size_t)1 << KBITS);
        bulk_load(sm.hist, hsrc, hist_bytes, bar_stat);
      } else {
        tma_load_4d(sm.stat, &map_stat, bar_stat, 0, 0, h * a.G, b);
        tma_load_4d(sm.stat + stat_atom_bytes, &map_stat, bar_stat, kAtomCols, 0, h * a.G, b);
      }
      int issued = 0;
      for (int i = 0; i < ntiles && ok; ++i) {
        const int s = i % kStages;
        const int round = i / kStages;
        if (round > 0) ok = mbar_wait(bar_empty + 8 * s, (round - 1) & 1);
        if (!ok) break;
        const uint32_t dst = sm.stages + s * kTileBytes;
        const int token = t * a.S + (tile0 + i) * kTileKeys;
        mbar_expect_tx(bar_full + 8 * s, kTileBytes);
        tma_load_4d(dst, &map_keys, bar_full + 8 * s, 0, token, h, b);
        tma_load_4d(dst + kTileAtomBytes, &map_keys, bar_full + 8 * s, kAtomCols, token, h, b);
        issued = i + 1;
      }
      if (!ok) {
        record_status(a.status, kStatusTimeout);
        // let copies already in flight land before the CTA may exit
        for (int i = max(0, issued - kStages); i < issued; ++i)
          mbar_wait(bar_full + 8 * (i % kStages), (i / kStages) & 1);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ================= MMA issuer =================
    if (lane == 0) {
      bool ok = mbar_wait(bar_stat, 0);
      const uint32_t idesc = (MODE == kLse) ? umma_idesc_bf16(128, kTileKeys)
                                            : umma_idesc_bf16(128, a.stat_rows);
      for (int i = 0; i < ntiles && ok; ++i) {
        const int s = i % kStages;
        const int acc = i & 1;
        if (i >= 2) ok = mbar_wait(bar_tempty + 8 * acc, ((i >> 1) - 1) & 1);
        if (ok) ok = mbar_wait(bar_full + 8 * s, (i / kStages) & 1);
        if (!ok) break;
        tc_fence_after();
        const uint32_t tile = sm.stages + s * kTileBytes;
        for (int mb = 0; mb < nmb; ++mb) {
          const uint32_t d = tmem_base + acc * kAccStride + mb * 128;
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint32_t koff = (k & 3) * 32;
            const uint32_t tile_k = tile + (k >> 2) * kTileAtomBytes + koff;
            const uint32_t stat_k = sm.stat + (k >> 2) * stat_atom_bytes + koff;
            if (MODE == kLse) {
              umma_bf16(d, umma_sdesc_sw128(stat_k + mb * (128 * 128)), umma_sdesc_sw128(tile_k),
                        idesc, k > 0);
            } else {
              umma_bf16(d, umma_sdesc_sw128(tile_k), umma_sdesc_sw128(stat_k), idesc, k > 0);
            }
          }
        }
        umma_commit(bar_empty + 8 * s);     // stage reusable once these MMAs have read it
        umma_commit(bar_tfull + 8 * acc);   // accumulator ready for the epilogue
      }
      if (!ok) record_status(a.status, kStatusTimeout);
    }
    __syncwarp();
  } else {
    // ================= epilogue warps: two groups of four =================
    // Both groups cover all 128 TMEM lanes (lane quarter = warp_id % 4); they split the
    // accumulator columns of every tile between them.
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;                   // TMEM lane owned by this thread
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const int etid = threadIdx.x - 64;                     // 0..255
    const int wg = etid >> 7;                              // epilogue group 0 / 1
    bool ok = true;

    if constexpr (MODE == kLse) {
      // group g owns query block g (G*W > 128) or half of the key columns (G*W <= 128)
      const int mb = (nmb == 2) ? wg : 0;
      const int c_begin = (nmb == 2) ? 0 : wg * 64;
      const int c_end = (nmb == 2) ? kTileKeys : wg * 64 + 64;
      float m = -INFINITY, l = 0.f;
      const float c2 = a.scale_log2e;
      for (int i = 0; i < ntiles && ok; ++i) {
        const int acc = i & 1;
        ok = mbar_wait(bar_tfull + 8 * acc, (i >> 1) & 1);
        if (!ok) break;
        tc_fence_after();
        const int nvalid = min(kTileKeys, a.S - (tile0 + i) * kTileKeys);
        const int ce = min(c_end, (nvalid + 15) & ~15);
        walk_columns(t_lane + acc * kAccStride + mb * 128, c_begin, ce, [&](const uint32_t* v, int col0, auto cnt_tag) {
          constexpr int CNT = decltype(cnt_tag)::value;
          const int lim = nvalid - col0;                   // valid columns in this chunk (>= 1)
          float cmax = -INFINITY;
          if (lim >= CNT) {
#pragma unroll
            for (int k = 0; k < CNT; ++k) cmax = fmaxf(cmax, __uint_as_float(v[k]));
            const float m_new = fmaxf(m, cmax * c2);
            float add0 = 0.f, add1 = 0.f;
#pragma unroll
            for (int k = 0; k < CNT; ++k) {
              const float x = fmaf(__uint_as_float(v[k]), c2, -m_new);
              const float e = ((k * 5) % 16 < 5) ? ex2_poly(x) : ex2_approx(x);
              if (k & 1) add1 += e; else add0 += e;
            }
            l = l * ex2_approx(m - m_new) + (add0 + add1);
            m = m_new;
          } else {
#pragma unroll
            for (int k = 0; k < CNT; ++k) if (k < lim) cmax = fmaxf(cmax, __uint_as_float(v[k]));
            const float m_new = fmaxf(m, cmax * c2);
            float add = 0.f;
#pragma unroll
            for (int k = 0; k < CNT; ++k)
              if (k < lim) add += ex2_approx(fmaf(__uint_as_float(v[k]), c2, -m_new));
            l = l * ex2_approx(m - m_new) + add;
            m = m_new;
          }
        });
        tc_fence_before();
        mbar_arrive(bar_tempty + 8 * acc);
      }
      if (nmb == 2) {
        const int q = mb * 128 + row;
        if (ok && q < a.GW) a.lse_part[((size_t)seg * a.n_split + split) * a.GW + q] = make_float2(m, l);
      } else {
        float2* xch = reinterpret_cast<float2*>(xwg_s);
        if (wg == 1) xch[row] = make_float2(m, l);
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (wg == 0 && ok && row < a.GW) {
          const float2 o = xch[row];
          const float mx = fmaxf(m, o.x);
          const float lt = (mx == -INFINITY) ? 0.f : l * ex2_approx(m - mx) + o.y * ex2_approx(o.x - mx);
          a.lse_part[((size_t)seg * a.n_split + split) * a.GW + row] = make_float2(mx, lt);
        }
      }
    } else if constexpr (MODE == kScore) {
      // combine the splits' (max, sum) partials into log2-sum-exp2 per query
      for (int q = etid; q < a.GW; q += 256) {
        const float2* p = a.lse_part + (size_t)seg * a.n_split * a.GW + q;
        float mx = -INFINITY;
        for (int s2 = 0; s2 < a.n_split; ++s2) mx = fmaxf(mx, p[(size_t)s2 * a.GW].x);
        float sum = 0.f;
        for (int s2 = 0; s2 < a.n_split; ++s2) {
          const float2 e = p[(size_t)s2 * a.GW];
          sum += e.y * exp2f(e.x - mx);
        }
        const float r = mx + log2f(sum);
        lse_s[q] = r;
        if (split == 0) a.lse2[(size_t)seg * a.GW + q] = r;
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
      // group 0 sums queries [0, cs), group 1 queries [cs, G*W); both ranges start 32-aligned
      const int cs = ((a.GW / 32 + 1) / 2) * 32;
      const int c_begin = wg ? cs : 0;
      const int c_end = wg ? a.GW : cs;
      const float c2 = a.scale_log2e;
      float* part = reinterpret_cast<float*>(xwg_s);       // [2 accumulators][128 keys]
      for (int i = 0; i < ntiles && ok; ++i) {
        const int acc = i & 1;
        ok = mbar_wait(bar_tfull + 8 * acc, (i >> 1) & 1);
        if (!ok) break;
        tc_fence_after();
        float s0 = 0.f, s1 = 0.f;
        walk_columns(t_lane + acc * kAccStride, c_begin, c_end, [&](const uint32_t* v, int col0, auto cnt_tag) {
          constexpr int CNT = decltype(cnt_tag)::value;
#pragma unroll
          for (int k = 0; k < CNT; k += 4) {
            const float4 ls = *reinterpret_cast<const float4*>(lse_s + col0 + k);
            const float lsv[4] = {ls.x, ls.y, ls.z, ls.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float x = fmaf(__uint_as_float(v[k + e]), c2, -lsv[e]);
              const float ex = (((k + e) * 5) % 16 < 5) ? ex2_poly(x) : ex2_approx(x);
              if (e & 1) s1 += ex; else s0 += ex;
            }
          }
        });
        tc_fence_before();
        mbar_arrive(bar_tempty + 8 * acc);
        const float sum = s0 + s1;
        if (wg == 1) part[acc * 128 + row] = sum;
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (wg == 0) {
          const int key = (tile0 + i) * kTileKeys + row;
          if (key < a.S) a.s_exact[(size_t)seg * a.S + key] = sum + part[acc * 128 + row];
        }
      }
    } else {
      // ---- kProj: sign bits -> bucket codes -> histogram lookups ----
      // Bucket code of a table: bit b of the table (hyperplane r*K + b) sits at position
      // K-1-b, i.e. the first hyperplane is the most significant bit; bit = [projection >= 0].
      // Group 0 handles the chunk's first TC/2 tables, group 1 the rest.
      ok = mbar_wait(bar_stat, 0);   // histogram slice landed (async-proxy writes visible after the wait)
      for (int i = 0; i < ntiles && ok; ++i) {
        const int acc = i & 1;
        ok = mbar_wait(bar_tfull + 8 * acc, (i >> 1) & 1);
        if (!ok) break;
        tc_fence_after();
        const int key = (tile0 + i) * kTileKeys + row;
        const bool valid = key < a.S;
        const uint32_t t_acc = t_lane + acc * kAccStride;
        const uint32_t bar_rel = bar_tempty + 8 * acc;
        uint32_t partial;
        if (wg == 0) partial = proj_tables<KBITS, 0, TC / 2>(t_acc, bar_rel, hist_s, a, seg, key, chunk * TC, valid);
        else partial = proj_tables<KBITS, TC / 2, TC>(t_acc, bar_rel, hist_s, a, seg, key, chunk * TC, valid);
        if (valid) atomicAdd(a.counts + (size_t)seg * a.S + key, partial);
      }
    }
    if (!ok) record_status(a.status, kStatusTimeout);
  }

  // ---- teardown ----------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace lkv
