// Decode-phase attention over the compacted cache (Section 3: only the selected tokens are kept
// in the KV cache and are used for the decoding phase): for every sequence and query head,
//   out = sum_i softmax_i(<q, k_i> * scale) * v_i     over the cache entries i in [0, len)
// of the query head's KV head. The cache is read once (K and V rows, 256 bytes each): the op is
// bound by HBM bandwidth, so the arithmetic is plain CUDA-core code fed from shared memory by a
// ring of bulk copies, and all query heads of a GQA group share every row that is read.
//
//   decode_split_kernel   - one CTA per (split of the cache entries, KV head, sequence); the number
//                           of splits fills the GPU exactly once. Tiles of 64 K rows and 64 V rows
//                           arrive through cp.async.bulk into a ring of stages; per tile: scores
//                           of the G query heads, softmax numerators relative to a running
//                           reference maximum (raised only when a score exceeds it by 2^20, so the
//                           common tile needs one barrier), weighted sum of the V rows.
//                           -> partial (reference max, sum, G x 128 accumulator) per split.
//   decode_combine_kernel - merges the splits' partials per query head (fixed order).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx.cuh"
#include "stream_gemm.cuh"

namespace lkv {

constexpr int kDecTile = 64;            // cache rows per stage (16 KB of K and 16 KB of V)
constexpr int kDecTileBytes = kDecTile * 256;
constexpr int kDecSetThreads = 256;     // threads that work on one set of up to four query heads
constexpr int kDecMaxGroup = 8;         // query heads per KV head, at most (two sets of four)
constexpr int kDecPartFloats = 128 + 2; // per (split, query head): accumulator, reference max, sum
constexpr int kDecMaxSplit = 512;
constexpr float kDecRescaleAt = 20.f;   // log2 units a score may exceed the reference maximum by

struct DecodeArgs {
  const uint16_t* Kc;     // cache keys   [batch][H_kv][cap][128]
  const uint16_t* Vc;     // cache values [batch][H_kv][cap][128]
  long long seg_stride;   // elements between (sequence, KV head) slabs
  const uint16_t* Q;      // decode queries [batch][H_q][128] via strides
  long long qs_b, qs_h;
  float* part;            // [batch][H_kv][n_split][G][130]
  float* out;             // [batch][H_q][128]
  int H_kv, G, len, n_split;
  float scale_log2e;
  int* status;
};

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ void unpack8(const uint4& w, float* x) {
  x[0] = bf16_lo(w.x); x[1] = bf16_hi(w.x); x[2] = bf16_lo(w.y); x[3] = bf16_hi(w.y);
  x[4] = bf16_lo(w.z); x[5] = bf16_hi(w.z); x[6] = bf16_lo(w.w); x[7] = bf16_hi(w.w);
}

// Shared memory of one CTA: NS stages of (K tile, V tile), then the small arrays.
__host__ __device__ constexpr uint32_t dec_smem_bytes(int gt, int nset, int ns) {
  return (uint32_t)ns * 2u * kDecTileBytes            // stages
         + 2u * 2u * (gt * nset) * kDecTile * 4u      // scores and numerators, double-buffered
         + 2u * (gt * nset) * 4u                      // reference maxima, rescale factors
         + (uint32_t)nset * 8u * gt * 4u              // per-warp sums of numerators
         + (uint32_t)ns * 8u + 16u;                   // mbarriers, failure flag
}

// GT = query heads per set (1, 2 or 4; register arrays are sized by it), NSET = sets (1 or 2; a
// set is 8 warps that walk every tile for their own heads), NS = stages of the ring.
template <int GT, int NSET, int NS>
__global__ void __launch_bounds__(kDecSetThreads * NSET, NSET == 1 ? 2 : 1) decode_split_kernel(const DecodeArgs a) {
  extern __shared__ __align__(128) uint8_t dsm[];
  constexpr int NH = GT * NSET;
  constexpr int NT = kDecSetThreads * NSET;
  uint8_t* tiles = dsm;
  float* sc_s = reinterpret_cast<float*>(dsm + NS * 2 * kDecTileBytes);   // [2][NH][64] scaled scores
  float* sc_p = sc_s + 2 * NH * kDecTile;                                  // [2][NH][64] numerators
  float* m_ref = sc_p + 2 * NH * kDecTile;                                 // [NH]
  float* fac = m_ref + NH;                                                 // [NH]
  float* lred = fac + NH;                                                  // [NSET*8][GT]
  uint64_t* bars = reinterpret_cast<uint64_t*>(lred + NSET * 8 * GT);      // [NS]
  volatile int* failed = reinterpret_cast<volatile int*>(bars + NS);

  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int set = warp >> 3, wset = warp & 7;
  const int l16 = lane & 15, half = lane >> 4;                     // 16 lanes share one cache row
  const int hw = wset * 2 + half;                                  // half-warp within the set
  const int e_begin = (int)((long long)split * a.len / a.n_split);
  const int n_rows = (int)((long long)(split + 1) * a.len / a.n_split) - e_begin;
  const int n_tiles = (n_rows + kDecTile - 1) / kDecTile;
  const uint16_t* Kb = a.Kc + (long long)(b * a.H_kv + h) * a.seg_stride + (long long)e_begin * 128;
  const uint16_t* Vb = a.Vc + (long long)(b * a.H_kv + h) * a.seg_stride + (long long)e_begin * 128;

  if (tid == 0) {
    for (int s = 0; s < NS; ++s) mbar_init(smem_u32(&bars[s]), 1);
    fence_mbar_init();
    *failed = 0;
  }
  if (tid < NH) m_ref[tid] = -INFINITY;
  __syncthreads();
  auto issue = [&](int t) {                                        // one thread: both copies of tile t
    const int st = t % NS;
    const uint32_t bytes = (uint32_t)min(kDecTile, n_rows - t * kDecTile) * 256u;
    const uint32_t bar = smem_u32(&bars[st]);
    mbar_expect_tx(bar, 2u * bytes);
    bulk_load(smem_u32(tiles + st * 2 * kDecTileBytes), Kb + (long long)t * kDecTile * 128, bytes, bar);
    bulk_load(smem_u32(tiles + st * 2 * kDecTileBytes + kDecTileBytes), Vb + (long long)t * kDecTile * 128, bytes, bar);
  };
  if (tid == 0)
    for (int t = 0; t < NS - 1 && t < n_tiles; ++t) issue(t);

  // this lane's 8 dims of every query of the set
  float q[GT][8];
#pragma unroll
  for (int g = 0; g < GT; ++g) {
    if (set * GT + g < a.G) {
      unpack8(*reinterpret_cast<const uint4*>(a.Q + b * a.qs_b + (long long)(h * a.G + set * GT + g) * a.qs_h + l16 * 8), q[g]);
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) q[g][i] = 0.f;
    }
  }
  float2 acc[GT][4];
  float lsum[GT];
#pragma unroll
  for (int g = 0; g < GT; ++g) {
    lsum[g] = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[g][i] = make_float2(0.f, 0.f);
  }

  bool alive = true;
  for (int t = 0; t < n_tiles; ++t) {
    const int st = t % NS, buf = t & 1;
    const int rows_here = min(kDecTile, n_rows - t * kDecTile);
    const uint8_t* kt = tiles + st * 2 * kDecTileBytes + l16 * 16;
    const uint8_t* vt = kt + kDecTileBytes;
    float* s_buf = sc_s + buf * NH * kDecTile;
    float* p_buf = sc_p + buf * NH * kDecTile;
    bool flag = false;
    if (!mbar_wait(smem_u32(&bars[st]), (uint32_t)(t / NS) & 1u)) { *failed = 1; flag = true; }

    // ---- scores: a half-warp per row, four rows per half-warp ----------------------------------
    uint4 w[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) w[r] = *reinterpret_cast<const uint4*>(kt + (hw + 16 * r) * 256);
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int row = hw + 16 * r;
      float k[8];
      unpack8(w[r], k);
      float s[GT];
#pragma unroll
      for (int g = 0; g < GT; ++g) {
        float2 x = make_float2(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 8; i += 2)
          x = __ffma2_rn(make_float2(k[i], k[i + 1]), make_float2(q[g][i], q[g][i + 1]), x);
        s[g] = x.x + x.y;
      }
      // sum over the row's 16 lanes; while more than one head is left, each step also halves the
      // heads a lane keeps, so that the lane ends up with the full sum of one head
      int mine = 0;
      int left = GT;
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) {
        if (left > 1) {
          left >>= 1;
          const bool upper = (lane & off) != 0;
#pragma unroll
          for (int j = 0; j < GT / 2; ++j) {
            if (j < left) {
              const float send = upper ? s[j] : s[j + left];
              const float keep = upper ? s[j + left] : s[j];
              s[j] = keep + __shfl_xor_sync(0xffffffffu, send, off);
            }
          }
          if (upper) mine += left;
        } else {
          s[0] += __shfl_xor_sync(0xffffffffu, s[0], off);
        }
      }
      // lanes that hold the same head hold the same sum; the lowest of them stores it
      constexpr int kDup = 16 / GT;
      const int head = set * GT + mine;
      if ((l16 & (kDup - 1)) == 0 && head < a.G) {
        const float sv = row < rows_here ? s[0] * a.scale_log2e : -INFINITY;   // stale rows of a short tile
        const float m = m_ref[head];
        s_buf[head * kDecTile + row] = sv;
        p_buf[head * kDecTile + row] = exp2f(sv - m);
        flag |= sv > m + kDecRescaleAt;
      }
    }
    const int any = __syncthreads_or(flag);
    // every thread is past the V rows of tile t-1: its stage takes tile t+NS-1
    if (tid == 0 && t + NS - 1 < n_tiles) issue(t + NS - 1);
    if (any) {
      if (*failed) { alive = false; break; }                       // uniform: read after the barrier
      // raise the reference maxima to the tile's maxima: warp g redoes head g's numerators
      if (warp < a.G) {
        const float s0 = s_buf[warp * kDecTile + lane], s1 = s_buf[warp * kDecTile + lane + 32];
        float tm = fmaxf(s0, s1);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, off));
        const float m_old = m_ref[warp];
        const float m_new = fmaxf(m_old, tm);                      // finite: the tile has a valid row
        p_buf[warp * kDecTile + lane] = exp2f(s0 - m_new);
        p_buf[warp * kDecTile + lane + 32] = exp2f(s1 - m_new);
        __syncwarp();
        if (lane == 0) { fac[warp] = exp2f(m_old - m_new); m_ref[warp] = m_new; }
      }
      __syncthreads();
#pragma unroll
      for (int g = 0; g < GT; ++g) {
        if (set * GT + g < a.G) {
          const float f = fac[set * GT + g];
          lsum[g] *= f;
#pragma unroll
          for (int i = 0; i < 4; ++i) { acc[g][i].x *= f; acc[g][i].y *= f; }
        }
      }
    }

    // ---- weighted sum of the tile's V rows: the lane keeps 8 dims for each head of the set ------
#pragma unroll
    for (int r = 0; r < 4; ++r) w[r] = *reinterpret_cast<const uint4*>(vt + (hw + 16 * r) * 256);
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int row = hw + 16 * r;
      if (row < rows_here) {                                       // stale rows may hold anything
        float v[8];
        unpack8(w[r], v);
#pragma unroll
        for (int g = 0; g < GT; ++g) {
          if (set * GT + g < a.G) {
            const float p = p_buf[(set * GT + g) * kDecTile + row];
            const float2 pp = make_float2(p, p);
            lsum[g] += p;
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[g][i] = __ffma2_rn(pp, make_float2(v[2 * i], v[2 * i + 1]), acc[g][i]);
          }
        }
      }
    }
  }
  if (!alive) {                                                    // a copy never arrived: report, write nothing
    if (tid == 0) record_status(a.status, kStatusTimeout);
    return;
  }
  __syncthreads();                                                 // every tile is consumed: the stages are free

  // the two half-warps of a warp hold different rows of the same dims
#pragma unroll
  for (int g = 0; g < GT; ++g) {
    lsum[g] += __shfl_xor_sync(0xffffffffu, lsum[g], 16);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      acc[g][i].x += __shfl_xor_sync(0xffffffffu, acc[g][i].x, 16);
      acc[g][i].y += __shfl_xor_sync(0xffffffffu, acc[g][i].y, 16);
    }
  }
  float* red = reinterpret_cast<float*>(tiles);                    // [NSET*8 warps][GT][128]
  if (half == 0) {
#pragma unroll
    for (int g = 0; g < GT; ++g) {
      float4* dst = reinterpret_cast<float4*>(red + (warp * GT + g) * 128 + l16 * 8);
      dst[0] = make_float4(acc[g][0].x, acc[g][0].y, acc[g][1].x, acc[g][1].y);
      dst[1] = make_float4(acc[g][2].x, acc[g][2].y, acc[g][3].x, acc[g][3].y);
    }
    if (l16 == 0) {
#pragma unroll
      for (int g = 0; g < GT; ++g) lred[warp * GT + g] = lsum[g];
    }
  }
  __syncthreads();
  float* part = a.part + (((long long)(b * a.H_kv + h) * a.n_split + split) * a.G) * kDecPartFloats;
  for (int i = tid; i < a.G * 128; i += NT) {
    const int head = i >> 7, d = i & 127;
    const float* src = red + ((head / GT) * 8 * GT + head % GT) * 128 + d;   // warp 0 of the head's set
    float sum = 0.f;
#pragma unroll
    for (int wi = 0; wi < 8; ++wi) sum += src[wi * GT * 128];
    part[head * kDecPartFloats + d] = sum;
  }
  if (tid < a.G) {
    const float* src = lred + (tid / GT) * 8 * GT + tid % GT;
    float l = 0.f;
#pragma unroll
    for (int wi = 0; wi < 8; ++wi) l += src[wi * GT];
    part[tid * kDecPartFloats + 128] = m_ref[tid];
    part[tid * kDecPartFloats + 129] = l;
  }
}

// One CTA of 128 threads per (query head, sequence): thread d merges dim d over the splits.
__global__ void __launch_bounds__(128) decode_combine_kernel(const DecodeArgs a) {
  __shared__ float wgt[kDecMaxSplit];
  __shared__ float red_m[4], red_l[4];
  const int hq = blockIdx.x, b = blockIdx.y;
  const int h = hq / a.G, g = hq % a.G;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float* part = a.part + (((long long)(b * a.H_kv + h) * a.n_split) * a.G + g) * kDecPartFloats;
  const int cstride = a.G * kDecPartFloats;

  float m = -INFINITY;
  for (int c = threadIdx.x; c < a.n_split; c += 128) m = fmaxf(m, part[c * cstride + 128]);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
  if (lane == 0) red_m[warp] = m;
  __syncthreads();
  m = fmaxf(fmaxf(red_m[0], red_m[1]), fmaxf(red_m[2], red_m[3]));
  float l = 0.f;
  for (int c = threadIdx.x; c < a.n_split; c += 128) {
    const float wc = exp2f(part[c * cstride + 128] - m);
    wgt[c] = wc;
    l += wc * part[c * cstride + 129];
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
  if (lane == 0) red_l[warp] = l;
  __syncthreads();
  l = (red_l[0] + red_l[1]) + (red_l[2] + red_l[3]);

  const int d = threadIdx.x;
  float o[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) o[j] = 0.f;
  for (int c0 = 0; c0 < a.n_split; c0 += 8) {
    float x[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) x[j] = c0 + j < a.n_split ? part[(c0 + j) * cstride + d] : 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) o[j] = fmaf(c0 + j < a.n_split ? wgt[c0 + j] : 0.f, x[j], o[j]);
  }
  a.out[((long long)b * a.H_kv * a.G + hq) * 128 + d] =
      (((o[0] + o[1]) + (o[2] + o[3])) + ((o[4] + o[5]) + (o[6] + o[7]))) / l;
}

}  // namespace lkv
