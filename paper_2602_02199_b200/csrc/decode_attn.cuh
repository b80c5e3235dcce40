// Decode-phase attention over the compacted cache (Section 3: only the selected tokens are kept
// in the KV cache and are used for the decoding phase): for every sequence and query head,
//   out = sum_i softmax_i(<q, k_i> * scale) * v_i     over the cache entries i in [0, len)
// of the query head's KV head. The cache is read once (K and V rows, 256 bytes each): the op is
// bound by HBM bandwidth, so the kernels are plain CUDA-core code shaped for coalesced 16-byte
// loads, with all query heads of a GQA group sharing every row that is read.
//
//   decode_chunk_kernel   - one CTA per (chunk of cache entries, KV head, sequence): scores of the
//                           chunk for the G query heads of the group, softmax numerators relative
//                           to the chunk's own maximum, weighted sum of the chunk's V rows ->
//                           partial (max, sum, G x 128 accumulator) per chunk.
//   decode_combine_kernel - merges the chunks' partials per query head (fixed order).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace lkv {

constexpr int kDecThreads = 256;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int kDecChunk = 512;          // cache entries per CTA
constexpr int kDecMaxGroup = 8;         // query heads per KV head, at most
constexpr int kDecPartFloats = 128 + 2; // per (chunk, query head): accumulator, max, sum
constexpr int kDecMaxChunks = 2048;     // 1 Mi cache entries per head
constexpr int kDecRowsInFlight = 4;     // rows a half-warp requests before it starts computing

struct DecodeArgs {
  const uint16_t* Kc;     // cache keys   [batch][H_kv][cap][128]
  const uint16_t* Vc;     // cache values [batch][H_kv][cap][128]
  long long seg_stride;   // elements between (sequence, KV head) slabs
  const uint16_t* Q;      // decode queries [batch][H_q][128] via strides
  long long qs_b, qs_h;
  float* part;            // [batch][H_kv][n_chunks][G][130]
  float* out;             // [batch][H_q][128]
  int H_kv, G, len, n_chunks;
  float scale_log2e;
};

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ void unpack8(const uint4& w, float* x) {
  x[0] = bf16_lo(w.x); x[1] = bf16_hi(w.x); x[2] = bf16_lo(w.y); x[3] = bf16_hi(w.y);
  x[4] = bf16_lo(w.z); x[5] = bf16_hi(w.z); x[6] = bf16_lo(w.w); x[7] = bf16_hi(w.w);
}

// GT = query heads per KV head rounded up to a power of two (register arrays are sized by it).
template <int GT>
__global__ void __launch_bounds__(kDecThreads, GT <= 4 ? 4 : 2) decode_chunk_kernel(const DecodeArgs a) {
  __shared__ float sc[GT][kDecChunk];                              // scores, then softmax numerators
  __shared__ float red[kDecWarps / 2][GT][128];                    // output accumulators of warp pairs
  __shared__ float stat[GT][2];                                    // chunk max and sum per query head
  const int chunk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int l16 = lane & 15, half = lane >> 4;                     // 16 lanes share one cache row
  const int e0 = chunk * kDecChunk;
  const int n_e = min(kDecChunk, a.len - e0);
  const uint16_t* Kb = a.Kc + (long long)(b * a.H_kv + h) * a.seg_stride + (long long)e0 * 128 + l16 * 8;
  const uint16_t* Vb = a.Vc + (long long)(b * a.H_kv + h) * a.seg_stride + (long long)e0 * 128 + l16 * 8;
  constexpr int kStep = 2 * kDecWarps;                             // rows per pass of the CTA

  // this lane's 8 dims of every query of the group
  float q[GT][8];
#pragma unroll
  for (int g = 0; g < GT; ++g) {
    if (g < a.G) {
      unpack8(*reinterpret_cast<const uint4*>(a.Q + b * a.qs_b + (long long)(h * a.G + g) * a.qs_h + l16 * 8), q[g]);
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) q[g][i] = 0.f;
    }
  }

  // ---- scores: a half-warp per row; several rows are requested before the first is used ----------
  for (int eb = warp * 2 + half; eb < kDecChunk; eb += kStep * kDecRowsInFlight) {
    uint4 w[kDecRowsInFlight];
#pragma unroll
    for (int r = 0; r < kDecRowsInFlight; ++r) {
      const int e = eb + r * kStep;
      w[r] = (e < n_e) ? *reinterpret_cast<const uint4*>(Kb + (long long)e * 128) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int r = 0; r < kDecRowsInFlight; ++r) {
      const int e = eb + r * kStep;
      float k[8];
      unpack8(w[r], k);
      float s[GT];
#pragma unroll
      for (int g = 0; g < GT; ++g) {
        float2 t = make_float2(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 8; i += 2)
          t = __ffma2_rn(make_float2(k[i], k[i + 1]), make_float2(q[g][i], q[g][i + 1]), t);
        s[g] = t.x + t.y;
      }
      // sum over the row's 16 lanes; while more than one head is left, each step also halves the
      // heads a lane keeps, so that the lane ends up with the full sum of one head
      int mine = 0;                                 // the head this lane will hold
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
      constexpr int kDup = GT >= 16 ? 1 : 16 / GT;  // lanes per head after the reduction
      if ((l16 & (kDup - 1)) == 0 && mine < a.G) sc[mine][e] = (e < n_e) ? s[0] * a.scale_log2e : -INFINITY;
    }
  }
  __syncthreads();

  // ---- softmax numerators relative to the chunk's maximum: warp g takes query head g ---------------
  for (int g = warp; g < a.G; g += kDecWarps) {
    float m = -INFINITY;
    for (int e = lane; e < kDecChunk; e += 32) m = fmaxf(m, sc[g][e]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    float l = 0.f;
    for (int e = lane; e < kDecChunk; e += 32) {
      const float p = exp2f(sc[g][e] - m);          // n_e >= 1, so m is finite
      sc[g][e] = p;
      l += p;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
    if (lane == 0) { stat[g][0] = m; stat[g][1] = l; }
  }
  __syncthreads();

  // ---- weighted sum of the chunk's V rows: the lane keeps 8 dims for each head of the group --------
  float2 acc[GT][4];
#pragma unroll
  for (int g = 0; g < GT; ++g)
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[g][i] = make_float2(0.f, 0.f);
  for (int eb = warp * 2 + half; eb < kDecChunk; eb += kStep * kDecRowsInFlight) {
    uint4 w[kDecRowsInFlight];
#pragma unroll
    for (int r = 0; r < kDecRowsInFlight; ++r) {
      const int e = eb + r * kStep;
      w[r] = (e < n_e) ? *reinterpret_cast<const uint4*>(Vb + (long long)e * 128) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int r = 0; r < kDecRowsInFlight; ++r) {
      const int e = eb + r * kStep;                 // e < kDecChunk always; rows past n_e have p = 0
      float v[8];
      unpack8(w[r], v);
#pragma unroll
      for (int g = 0; g < GT; ++g) {
        if (g < a.G) {
          const float p = sc[g][e];
          const float2 pp = make_float2(p, p);
#pragma unroll
          for (int i = 0; i < 4; ++i) acc[g][i] = __ffma2_rn(pp, make_float2(v[2 * i], v[2 * i + 1]), acc[g][i]);
        }
      }
    }
  }
  // the two half-warps of a warp hold different rows of the same dims
#pragma unroll
  for (int g = 0; g < GT; ++g)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      acc[g][i].x += __shfl_xor_sync(0xffffffffu, acc[g][i].x, 16);
      acc[g][i].y += __shfl_xor_sync(0xffffffffu, acc[g][i].y, 16);
    }
  // across warps in two rounds (odd warps write, even warps add; then the four sums are added)
  if ((warp & 1) && half == 0) {
#pragma unroll
    for (int g = 0; g < GT; ++g)
#pragma unroll
      for (int i = 0; i < 4; ++i)
        *reinterpret_cast<float2*>(&red[warp >> 1][g][l16 * 8 + 2 * i]) = acc[g][i];
  }
  __syncthreads();
  if (!(warp & 1) && half == 0) {
#pragma unroll
    for (int g = 0; g < GT; ++g)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float2* slot = reinterpret_cast<float2*>(&red[warp >> 1][g][l16 * 8 + 2 * i]);
        const float2 o = *slot;
        *slot = make_float2(acc[g][i].x + o.x, acc[g][i].y + o.y);
      }
  }
  __syncthreads();
  float* part = a.part + (((long long)(b * a.H_kv + h) * a.n_chunks + chunk) * a.G) * kDecPartFloats;
  for (int i = threadIdx.x; i < a.G * 128; i += kDecThreads) {
    const int g = i >> 7, d = i & 127;
    part[g * kDecPartFloats + d] = (red[0][g][d] + red[1][g][d]) + (red[2][g][d] + red[3][g][d]);
  }
  if (threadIdx.x < a.G * 2) part[(threadIdx.x >> 1) * kDecPartFloats + 128 + (threadIdx.x & 1)] = stat[threadIdx.x >> 1][threadIdx.x & 1];
}

// One CTA of 128 threads per (query head, sequence): thread d merges dim d over the chunks.
__global__ void __launch_bounds__(128) decode_combine_kernel(const DecodeArgs a) {
  __shared__ float wgt[kDecMaxChunks];
  __shared__ float red_m[4], red_l[4];
  const int hq = blockIdx.x, b = blockIdx.y;
  const int h = hq / a.G, g = hq % a.G;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float* part = a.part + (((long long)(b * a.H_kv + h) * a.n_chunks) * a.G + g) * kDecPartFloats;
  const long long cstride = (long long)a.G * kDecPartFloats;

  float m = -INFINITY;
  for (int c = threadIdx.x; c < a.n_chunks; c += 128) m = fmaxf(m, part[c * cstride + 128]);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
  if (lane == 0) red_m[warp] = m;
  __syncthreads();
  m = fmaxf(fmaxf(red_m[0], red_m[1]), fmaxf(red_m[2], red_m[3]));
  float l = 0.f;
  for (int c = threadIdx.x; c < a.n_chunks; c += 128) {
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
  float o0 = 0.f, o1 = 0.f, o2 = 0.f, o3 = 0.f;
  int c = 0;
  for (; c + 4 <= a.n_chunks; c += 4) {
    o0 = fmaf(wgt[c], part[c * cstride + d], o0);
    o1 = fmaf(wgt[c + 1], part[(c + 1) * cstride + d], o1);
    o2 = fmaf(wgt[c + 2], part[(c + 2) * cstride + d], o2);
    o3 = fmaf(wgt[c + 3], part[(c + 3) * cstride + d], o3);
  }
  for (; c < a.n_chunks; ++c) o0 = fmaf(wgt[c], part[c * cstride + d], o0);
  a.out[((long long)b * a.H_kv * a.G + hq) * 128 + d] = ((o0 + o1) + (o2 + o3)) / l;
}

}  // namespace lkv
