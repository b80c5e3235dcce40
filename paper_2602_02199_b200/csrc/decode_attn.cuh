// Decode-phase attention over the compacted cache (Section 3: only the selected tokens are kept
// in the KV cache and are used for the decoding phase): for every sequence and query head,
//   out = sum_i softmax_i(<q, k_i> * scale) * v_i     over the cache entries i in [0, len)
// of the query head's KV head. The cache is read once (K and V rows, 256 bytes each): the op is
// bound by HBM bandwidth. All (up to eight) query heads of a GQA group share every row that is
// read; the two small contractions per row (scores, weighted sum of V) run as warp-level
// m16n8k16 bf16 MMAs with the heads on the 8-wide dimension, which keeps the instruction count
// per row far below what the memory pipeline needs (a CUDA-core version of the same loop was
// bound by instruction issue at half the bandwidth). tcgen05 would need M = 128 per instruction
// and a round trip through TMEM and shared memory for the numerators; nothing is gained when the
// tensor pipe is busy 14 % of the time as it is.
//
//   decode_split_kernel   - one CTA per (split of the cache entries, KV head, sequence); the number
//                           of splits fills the GPU exactly once. A producer warp brings tiles of
//                           64 K rows and 64 V rows into a ring of stages with TMA (128-byte
//                           swizzle, rows past the cache length read as zeros); each of four
//                           consumer warps owns 16 rows of every tile: scores S^T = K Q^T,
//                           numerators relative to the warp's running reference maximum (raised
//                           only when a score exceeds it by 2^20), O^T += V^T P^T with the
//                           numerators split into two bf16 terms so that the weights keep
//                           16 mantissa bits. -> partial (max, sum, G x 128 accumulator) per split.
//                           The CTA that finishes last for its (sequence, KV head) merges the
//                           splits' partials in split order and writes the output rows, so the
//                           whole op is one launch.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx.cuh"
#include "stream_gemm.cuh"

namespace lkv {

constexpr int kDecTile = 64;            // cache rows per stage
constexpr int kDecBoxBytes = kDecTile * 128;   // one TMA box: 64 rows x 64 bf16
constexpr int kDecStageBytes = 4 * kDecBoxBytes;   // K cols 0-63, K cols 64-127, V cols 0-63, V cols 64-127
constexpr int kDecStages = 3;
constexpr int kDecWarps = 4;            // consumer warps, 16 rows of every tile each
constexpr int kDecThreads = (kDecWarps + 1) * 32;
constexpr int kDecCtasPerSm = 2;
constexpr int kDecMaxGroup = 8;         // query heads per KV head, at most (the N of the MMA)
constexpr int kDecPartFloats = 128 + 4; // per (split, query head): accumulator, reference max, sum, padding to 16 bytes
constexpr int kDecMaxSplit = 512;
constexpr float kDecRescaleAt = 20.f;   // log2 units a score may exceed the reference maximum by
constexpr int kDecRedStride = 132;      // floats between heads in the merge buffer (bank spread)

struct DecodeArgs {
  const uint16_t* Q;      // decode queries [batch][H_q][128] via strides
  long long qs_b, qs_h;
  float* part;            // [batch][H_kv][n_split][G][132]
  int* counters;          // [batch][H_kv] finished splits; zero between calls
  float* out;             // [batch][H_q][128]
  int H_kv, G, len, n_split;
  float scale_log2e;
  int* status;
};

__host__ __device__ constexpr uint32_t dec_smem_bytes() {
  return kDecStages * kDecStageBytes + (2u * kDecStages + 1u) * 8u + 2u * kDecWarps * 8u * 4u + 1024u;
}

// Byte offset of the 16-byte chunk (0..15 over the 128 dims) of a row inside a K or V tile made
// of two 128-byte-swizzled boxes.
__device__ __forceinline__ uint32_t dec_swz(uint32_t row, uint32_t chunk) {
  return (chunk >> 3) * kDecBoxBytes + row * 128u + (((chunk & 7u) ^ (row & 7u)) << 4);
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t* r) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t* r) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float* d, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// Transposes the 8x8 matrix of 16-bit elements that the warp holds one register per lane.
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
  return y;
}
// (lo, hi) -> two bf16 (round to nearest even), lo in the low half
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t y;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(y) : "f"(hi), "f"(lo));
  return y;
}

// MMA fragment coordinates of a lane: g = lane / 4 (a row of the 16-row operand, a column of B),
// c = lane % 4 (the pair of columns 2c, 2c+1). Scores come out as S^T[key g (+8)][heads 2c, 2c+1];
// the accumulators are O^T[dim 16 mt + g (+8)][heads 2c, 2c+1].
__global__ void __launch_bounds__(kDecThreads, kDecCtasPerSm)
decode_split_kernel(const __grid_constant__ CUtensorMap map_k,    // cache K: (d, len, H_kv, batch), box (64, 64, 1, 1)
                    const __grid_constant__ CUtensorMap map_v,    // cache V, same shape
                    const DecodeArgs a) {
  extern __shared__ uint8_t dsm_raw[];
  const uint32_t base = (smem_u32(dsm_raw) + 1023u) & ~1023u;
  uint8_t* const gen = dsm_raw + (base - smem_u32(dsm_raw));
  const uint32_t sm_bars = base + kDecStages * kDecStageBytes;
  float* wm = reinterpret_cast<float*>(gen + kDecStages * kDecStageBytes + (2 * kDecStages + 1) * 8);   // [warps][8] maxima
  float* wl = wm + kDecWarps * 8;                                                                   // [warps][8] sums
  float* red = reinterpret_cast<float*>(gen);                     // merge buffer over the stages: [warps][8][132]
  auto bar_full = [&](int s) { return sm_bars + 8u * s; };
  auto bar_empty = [&](int s) { return sm_bars + 8u * (kDecStages + s); };

  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, c = lane & 3;
  // splits are whole tiles (the host launches at most one split per tile): no CTA reads rows of
  // its neighbour, and only the cache's last tile is partial
  const int tiles_total = (a.len + kDecTile - 1) / kDecTile;
  const int tile_begin = (int)((long long)split * tiles_total / a.n_split);
  const int n_tiles = (int)((long long)(split + 1) * tiles_total / a.n_split) - tile_begin;
  const int e_begin = tile_begin * kDecTile;
  const int n_rows = min(a.len - e_begin, n_tiles * kDecTile);

  float o[8][4];                 // O^T, eight 16-dim row blocks
  float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;   // heads 2c and 2c+1
#pragma unroll
  for (int mt = 0; mt < 8; ++mt)
#pragma unroll
    for (int i = 0; i < 4; ++i) o[mt][i] = 0.f;

  if (warp == kDecWarps) {
    // ---- producer: one lane sets the barriers up and keeps the ring full --------------------------
    auto issue = [&](int t) {
      const int st = t % kDecStages;
      const uint32_t dst = base + st * kDecStageBytes;
      const int row0 = e_begin + t * kDecTile;
      mbar_expect_tx(bar_full(st), kDecStageBytes);
      tma_load_4d(dst, &map_k, bar_full(st), 0, row0, h, b);
      tma_load_4d(dst + kDecBoxBytes, &map_k, bar_full(st), 64, row0, h, b);
      tma_load_4d(dst + 2 * kDecBoxBytes, &map_v, bar_full(st), 0, row0, h, b);
      tma_load_4d(dst + 3 * kDecBoxBytes, &map_v, bar_full(st), 64, row0, h, b);
    };
    if (lane == 0) {
      for (int s = 0; s < kDecStages; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), kDecWarps); }
      mbar_init(sm_bars + 8u * (2 * kDecStages), 1);               // the merge's bulk copies
      fence_mbar_init();
      // the first tiles are on their way before the other warps have seen the barriers
      for (int t = 0; t < min(n_tiles, kDecStages); ++t) issue(t);
    }
    __syncwarp();
    __syncthreads();                                               // the barriers are set up
    if (lane == 0) {
      for (int t = kDecStages; t < n_tiles; ++t) {
        if (!mbar_wait(bar_empty(t % kDecStages), (uint32_t)(t / kDecStages - 1) & 1u)) {
          record_status(a.status, kStatusTimeout);
          break;
        }
        issue(t);
      }
    }
  } else {
    // ---- consumers ------------------------------------------------------------------------------
    // B fragments of Q^T: head g, dims 16 ks + 2c, +1 and +8, +9 (heads past G are zero rows)
    uint32_t qb[8][2];
    {
      const uint16_t* qrow = a.Q + b * a.qs_b + (long long)(h * a.G + g) * a.qs_h;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        qb[ks][0] = g < a.G ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 2 * c) : 0u;
        qb[ks][1] = g < a.G ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 8 + 2 * c) : 0u;
      }
    }
    __syncthreads();                                               // the barriers are set up
    for (int t = 0; t < n_tiles; ++t) {
      const int st = t % kDecStages;
      if (!__all_sync(0xffffffffu, mbar_wait(bar_full(st), (uint32_t)(t / kDecStages) & 1u))) {   // warp-uniform
        if (lane == 0) record_status(a.status, kStatusTimeout);
        break;
      }
      const int key0 = t * kDecTile + warp * 16;                   // first of the warp's rows, within the split
      if (key0 < n_rows) {
        const uint32_t k_tile = base + st * kDecStageBytes;
        const uint32_t v_tile = k_tile + 2 * kDecBoxBytes;
        // scores of 16 keys x 8 heads; two accumulators shorten the dependency chain
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < 8; ks += 2) {
          uint32_t k0[4], k1[4];
          ldsm_x4(k_tile + dec_swz(warp * 16 + (lane & 15), 2 * ks + (lane >> 4)), k0);
          ldsm_x4(k_tile + dec_swz(warp * 16 + (lane & 15), 2 * ks + 2 + (lane >> 4)), k1);
          mma_bf16(s0, k0, qb[ks][0], qb[ks][1]);
          mma_bf16(s1, k1, qb[ks + 1][0], qb[ks + 1][1]);
        }
        // rows past the cache's end read as zeros: weight 0
        const bool v_lo = key0 + g < n_rows, v_hi = key0 + g + 8 < n_rows;
        const float x0 = v_lo ? (s0[0] + s1[0]) * a.scale_log2e : -INFINITY;   // key g,   head 2c
        const float x1 = v_lo ? (s0[1] + s1[1]) * a.scale_log2e : -INFINITY;   // key g,   head 2c+1
        const float x2 = v_hi ? (s0[2] + s1[2]) * a.scale_log2e : -INFINITY;   // key g+8, head 2c
        const float x3 = v_hi ? (s0[3] + s1[3]) * a.scale_log2e : -INFINITY;   // key g+8, head 2c+1
        const float t_a = fmaxf(x0, x2), t_b = fmaxf(x1, x3);
        if (__any_sync(0xffffffffu, t_a > m_a + kDecRescaleAt || t_b > m_b + kDecRescaleAt)) {
          // raise the reference maxima to the maxima over the warp's 16 keys (lanes with equal c)
          float n_a = t_a, n_b = t_b;
#pragma unroll
          for (int off = 4; off < 32; off <<= 1) {
            n_a = fmaxf(n_a, __shfl_xor_sync(0xffffffffu, n_a, off));
            n_b = fmaxf(n_b, __shfl_xor_sync(0xffffffffu, n_b, off));
          }
          n_a = fmaxf(n_a, m_a);                                  // finite: row key0 is valid
          n_b = fmaxf(n_b, m_b);
          const float f_a = exp2f(m_a - n_a), f_b = exp2f(m_b - n_b);   // 0 on the first raise
          m_a = n_a; m_b = n_b;
          l_a *= f_a; l_b *= f_b;
#pragma unroll
          for (int mt = 0; mt < 8; ++mt) { o[mt][0] *= f_a; o[mt][1] *= f_b; o[mt][2] *= f_a; o[mt][3] *= f_b; }
        }
        const float p0 = exp2f(x0 - m_a), p1 = exp2f(x1 - m_b), p2 = exp2f(x2 - m_a), p3 = exp2f(x3 - m_b);
        l_a += p0 + p2;
        l_b += p1 + p3;
        // numerators as two bf16 terms each; transposed they are the B fragments of P^T
        const uint32_t h01 = pack_bf16x2(p0, p1), h23 = pack_bf16x2(p2, p3);
        const uint32_t r01 = pack_bf16x2(p0 - __uint_as_float(h01 << 16), p1 - __uint_as_float(h01 & 0xFFFF0000u));
        const uint32_t r23 = pack_bf16x2(p2 - __uint_as_float(h23 << 16), p3 - __uint_as_float(h23 & 0xFFFF0000u));
        const uint32_t bh0 = movmatrix_trans(h01), bh1 = movmatrix_trans(h23);
        const uint32_t bl0 = movmatrix_trans(r01), bl1 = movmatrix_trans(r23);
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
          uint32_t vt[4];
          ldsm_x4_trans(v_tile + dec_swz(warp * 16 + (lane & 7) + 8 * (lane >> 4), 2 * mt + ((lane >> 3) & 1)), vt);
          mma_bf16(o[mt], vt, bh0, bh1);
          mma_bf16(o[mt], vt, bl0, bl1);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_empty(st));
    }
    // the warp's sums over its keys: lanes with equal c hold different keys
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
      l_a += __shfl_xor_sync(0xffffffffu, l_a, off);
      l_b += __shfl_xor_sync(0xffffffffu, l_b, off);
    }
    if (g == 0) { wm[warp * 8 + 2 * c] = m_a; wm[warp * 8 + 2 * c + 1] = m_b; }
  }
  __syncthreads();                                                 // every tile is consumed: the stages are free

  // ---- merge the consumer warps (a warp that saw no valid row has max -inf and weight 0) ----------
  if (warp < kDecWarps) {
    float top_a = -INFINITY, top_b = -INFINITY;
#pragma unroll
    for (int wi = 0; wi < kDecWarps; ++wi) { top_a = fmaxf(top_a, wm[wi * 8 + 2 * c]); top_b = fmaxf(top_b, wm[wi * 8 + 2 * c + 1]); }
    const float f_a = m_a == -INFINITY ? 0.f : exp2f(m_a - top_a), f_b = m_b == -INFINITY ? 0.f : exp2f(m_b - top_b);
    if (g == 0) { wl[warp * 8 + 2 * c] = l_a * f_a; wl[warp * 8 + 2 * c + 1] = l_b * f_b; }
    float* dst = red + (warp * 8 + 2 * c) * kDecRedStride;
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      dst[16 * mt + g] = o[mt][0] * f_a;
      dst[kDecRedStride + 16 * mt + g] = o[mt][1] * f_b;
      dst[16 * mt + g + 8] = o[mt][2] * f_a;
      dst[kDecRedStride + 16 * mt + g + 8] = o[mt][3] * f_b;
    }
  }
  __syncthreads();
  float* part = a.part + (((long long)(b * a.H_kv + h) * a.n_split + split) * a.G) * kDecPartFloats;
  for (int i = tid; i < a.G * 128; i += kDecThreads) {
    const int head = i >> 7, d = i & 127;
    float sum = 0.f;
#pragma unroll
    for (int wi = 0; wi < kDecWarps; ++wi) sum += red[(wi * 8 + head) * kDecRedStride + d];
    part[head * kDecPartFloats + d] = sum;
  }
  if (tid < a.G) {
    float top = -INFINITY, l = 0.f;
#pragma unroll
    for (int wi = 0; wi < kDecWarps; ++wi) { top = fmaxf(top, wm[wi * 8 + tid]); l += wl[wi * 8 + tid]; }
    part[tid * kDecPartFloats + 128] = top;
    part[tid * kDecPartFloats + 129] = l;
  }

  // ---- the CTA that finishes last for this (sequence, KV head) merges all splits -----------------
  // The partials of this (sequence, KV head) are contiguous, split-major. The last CTA brings them
  // into the free stage ring with one bulk copy per round (a ring too small for all splits of many
  // heads takes several rounds) while the splits' maxima and sums are read and turned into weights.
  __shared__ int s_last;
  const float* seg = a.part + ((long long)(b * a.H_kv + h) * a.n_split) * a.G * kDecPartFloats;
  const int sstride = a.G * kDecPartFloats;                        // floats between splits
  const int gn = a.G * a.n_split;
  float* wgt = reinterpret_cast<float*>(gen);                      // [G][n_split]
  float* msl = wgt + gn;                                           // [G][n_split][2] maxima and sums
  const uint32_t data_off = ((uint32_t)gn * 12u + 15u) & ~15u;
  const float4* data = reinterpret_cast<const float4*>(gen + data_off);
  // splits per round: a multiple of four (the accumulator of a split is its index modulo four), >= 8
  const int per_round = (int)((kDecStages * kDecStageBytes - data_off) / ((uint32_t)sstride * 4u)) & ~3;
  const uint32_t bar_merge = sm_bars + 8u * (2 * kDecStages);
  auto fetch = [&](int s0, int ns) {                               // one thread
    fence_proxy_async_smem();                                      // the ring was last touched by ordinary accesses
    mbar_expect_tx(bar_merge, (uint32_t)ns * (uint32_t)sstride * 4u);
    bulk_load(base + data_off, seg + (long long)s0 * sstride, (uint32_t)ns * (uint32_t)sstride * 4u, bar_merge);
  };
  __syncthreads();                                                 // the CTA's partial is written ...
  if (tid == 0) {
    __threadfence();                                               // ... and visible before the count goes up
    int* counter = a.counters + b * a.H_kv + h;
    s_last = atomicAdd(counter, 1) == a.n_split - 1;
    if (s_last) {
      *counter = 0;                                                // ready for the next call
      __threadfence();                                             // the other CTAs' partials are visible from here on
      fence_proxy_async_global();                                  // also to the copy engine
      fetch(0, min(per_round, a.n_split));
    }
  }
  __syncthreads();
  if (!s_last) return;
  for (int i = tid; i < gn; i += kDecThreads) {
    const int head = i / a.n_split, s = i - head * a.n_split;
    const float2 v = __ldcg(reinterpret_cast<const float2*>(seg + (long long)s * sstride + head * kDecPartFloats + 128));
    msl[2 * i] = v.x;
    msl[2 * i + 1] = v.y;
  }
  __syncthreads();
  for (int head = warp; head < a.G; head += kDecWarps + 1) {
    const float* ms = msl + 2 * head * a.n_split;
    float top = -INFINITY;
    for (int s = lane; s < a.n_split; s += 32) top = fmaxf(top, ms[2 * s]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) top = fmaxf(top, __shfl_xor_sync(0xffffffffu, top, off));
    float l = 0.f;
    for (int s = lane; s < a.n_split; s += 32) {
      const float ws = exp2f(ms[2 * s] - top);
      wgt[head * a.n_split + s] = ws;
      l += ws * ms[2 * s + 1];
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
    if (lane == 0) wl[head] = l;
  }
  // thread -> up to two (head, four dims) items; four accumulators per item, split s adds to s % 4
  constexpr int kItems = (kDecMaxGroup * 32 + kDecThreads - 1) / kDecThreads;
  float4 acc[kItems][4];
#pragma unroll
  for (int it = 0; it < kItems; ++it)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[it][j] = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s0 = 0; s0 < a.n_split; s0 += per_round) {
    const int ns = min(per_round, a.n_split - s0);
    if (s0 > 0) {
      __syncthreads();                                             // the previous round's rows are read
      if (tid == 0) fetch(s0, ns);
    }
    const bool landed = mbar_wait(bar_merge, (uint32_t)(s0 / per_round) & 1u);
    if (!__syncthreads_and(landed)) {                              // also: the weights are written
      if (tid == 0) record_status(a.status, kStatusTimeout);
      return;
    }
#pragma unroll
    for (int it = 0; it < kItems; ++it) {
      const int i = tid + it * kDecThreads;
      if (i < a.G * 32) {
        const int head = i >> 5, d4 = i & 31;
        const float* w = wgt + head * a.n_split + s0;
        const float4* x = data + head * (kDecPartFloats / 4) + d4;
        const int ns4 = ns & ~3;
        for (int s = 0; s < ns4; s += 4) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float ws = w[s + j];
            const float4 v = x[(s + j) * (sstride / 4)];
            float4& c4 = acc[it][j];
            c4.x = fmaf(ws, v.x, c4.x); c4.y = fmaf(ws, v.y, c4.y); c4.z = fmaf(ws, v.z, c4.z); c4.w = fmaf(ws, v.w, c4.w);
          }
        }
#pragma unroll
        for (int j = 0; j < 3; ++j) {
          if (ns4 + j < ns) {
            const float ws = w[ns4 + j];
            const float4 v = x[(ns4 + j) * (sstride / 4)];
            float4& c4 = acc[it][j];
            c4.x = fmaf(ws, v.x, c4.x); c4.y = fmaf(ws, v.y, c4.y); c4.z = fmaf(ws, v.z, c4.z); c4.w = fmaf(ws, v.w, c4.w);
          }
        }
      }
    }
  }
#pragma unroll
  for (int it = 0; it < kItems; ++it) {
    const int i = tid + it * kDecThreads;
    if (i < a.G * 32) {
      const int head = i >> 5, d4 = i & 31;
      const float inv = 1.f / wl[head];
      const float4* c4 = acc[it];
      float4 r;
      r.x = ((c4[0].x + c4[1].x) + (c4[2].x + c4[3].x)) * inv;
      r.y = ((c4[0].y + c4[1].y) + (c4[2].y + c4[3].y)) * inv;
      r.z = ((c4[0].z + c4[1].z) + (c4[2].z + c4[3].z)) * inv;
      r.w = ((c4[0].w + c4[1].w) + (c4[2].w + c4[3].w)) * inv;
      reinterpret_cast<float4*>(a.out + ((long long)(b * a.H_kv + h) * a.G + head) * 128)[d4] = r;
    }
  }
}

}  // namespace lkv
