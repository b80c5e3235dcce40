// Recall score in closed form (Section 3.3 "Recall": tokens are ranked by their theoretical hash
// collision probability with the query): for every key of a block and KV head,
//   S_theory[j] = (1 / (G*W)) * sum_q (1 - theta(q, k_j) / pi)^K,
// theta the angle between window query q and key k_j, K the sign bits per SimHash table. It is the
// expectation over the hyperplane draw of the collision fraction that the hashing path counts, so
// it needs no hyperplanes and no tables: one pass over the keys.
//
//   theory_kernel - one CTA per (run of eight 64-key tiles of a block, KV head, block, sequence).
//                   A producer warp brings the head's query group (once) and the key tiles (ring
//                   of two stages) with TMA, 128-byte swizzle. Two groups of four consumer warps
//                   take alternate tiles, each warp 16 keys of its tile: key norms from the tile, <q, k> for all G*W queries as
//                   m16n8k16 bf16 MMAs (keys on M, eight queries per N), then per element
//                   cos = <q,k> / (|q| |k|), u = acos(-cos) / pi = 1 - theta / pi, u^K, summed
//                   over the queries. The element-wise chain (a degree-7 polynomial and a square
//                   root for acos, then u^K by repeated squaring for the usual K, by log2/exp2
//                   otherwise; under 20 instructions) bounds the kernel, not the contraction and
//                   not HBM.
#pragma once
#include "decode_attn.cuh"

namespace lkv {

constexpr int kThTile = 64;             // keys per stage
constexpr int kThTileBytes = kThTile * 256;
constexpr int kThStages = 2;
constexpr int kThWarps = 8;             // consumer warps: two groups of four take alternate tiles, 16 keys each
constexpr int kThThreads = (kThWarps + 1) * 32;
constexpr int kThTilesPerCta = 8;
constexpr int kThMaxQueries = 256;

struct TheoryArgs {
  float* out;             // [batch][H_kv][nb][S]
  int S, nb, H_kv, G, GW, kbits, tiles_in_block;
  int* status;
};

__host__ __device__ constexpr uint32_t theory_smem_bytes(int gw) {
  return 2u * gw * 128u + kThStages * kThTileBytes + kThMaxQueries * 4u + (1u + 2u * kThStages) * 8u + 1024u;
}

// Byte offset of the 16-byte chunk (0..15) of a row in a tile of two 128-byte-swizzled boxes of
// `box_bytes` each.
__device__ __forceinline__ uint32_t swz128(uint32_t row, uint32_t chunk, uint32_t box_bytes) {
  return (chunk >> 3) * box_bytes + row * 128u + (((chunk & 7u) ^ (row & 7u)) << 4);
}
// sum of squares of eight bf16 values
__device__ __forceinline__ float sum_squares8(const uint4& w) {
  const uint32_t v[4] = {w.x, w.y, w.z, w.w};
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float lo = __uint_as_float(v[i] << 16), hi = __uint_as_float(v[i] & 0xFFFF0000u);
    s = fmaf(lo, lo, s);
    s = fmaf(hi, hi, s);
  }
  return s;
}
// acos(x) / pi ~= sqrt(1 - x) * P(x) on [0, 1], |error| < 3e-8 (degree 7, the form of Abramowitz &
// Stegun 4.4.46; the coefficients are those of the fit in acos_poly.py beside this file, divided by
// pi). LKV_ACOS_TOP is the leading coefficient, LKV_ACOS_POLY the Horner steps below it.
#define LKV_ACOS_TOP (-4.0197156638e-04f)
#define LKV_ACOS_POLY(STEP) \
  STEP(2.1235386008e-03f) STEP(-5.4398557361e-03f) STEP(9.8335642476e-03f) STEP(-1.5971107888e-02f) \
  STEP(2.8322911244e-02f) STEP(-6.8308920822e-02f) STEP(4.9999999306e-01f)
__device__ __forceinline__ float sqrt_approx(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// x^KB for two values by repeated squaring (KB a compile-time count of sign bits).
template <int KB>
__device__ __forceinline__ float2 pow_int2(float2 x) {
  float2 r = make_float2(1.f, 1.f), sq = x;
  bool first = true;
#pragma unroll
  for (int b = KB; b > 0; b >>= 1) {
    if (b & 1) { r = first ? sq : __fmul2_rn(r, sq); first = false; }
    if (b > 1) sq = __fmul2_rn(sq, sq);
  }
  return r;
}
// (1 - theta/pi)^K for two cosines: u = acos(-c) / pi = 1 - acos(c)/pi (c >= 0), acos(|c|)/pi (c < 0).
// KB > 0: u^KB by multiplication; KB == 0: any K at run time as 2^(K log2 u). u = 0 gives 0 either way.
template <int KB>
__device__ __forceinline__ float2 collide_pow2(float2 c, float kbits) {
  const float2 x = make_float2(fminf(fabsf(c.x), 1.f), fminf(fabsf(c.y), 1.f));
  float2 p = make_float2(LKV_ACOS_TOP, LKV_ACOS_TOP);            // Horner, highest coefficient first
#define LKV_HORNER(A) p = __ffma2_rn(p, x, make_float2(A, A));
  LKV_ACOS_POLY(LKV_HORNER)
#undef LKV_HORNER
  const float2 om = __ffma2_rn(x, make_float2(-1.f, -1.f), make_float2(1.f, 1.f));   // 1 - x
  const float2 a = __fmul2_rn(make_float2(sqrt_approx(om.x), sqrt_approx(om.y)), p);
  const float2 u = make_float2(c.x >= 0.f ? 1.f - a.x : a.x, c.y >= 0.f ? 1.f - a.y : a.y);
  if (KB > 0) return pow_int2<KB>(u);
  return make_float2(ex2_approx(kbits * lg2_approx(u.x)), ex2_approx(kbits * lg2_approx(u.y)));
}

template <int KB>
__global__ void __launch_bounds__(kThThreads, 2)
theory_kernel(const __grid_constant__ CUtensorMap map_k,    // K: (d, nb*S, H_kv, batch), box (64, 64, 1, 1)
              const __grid_constant__ CUtensorMap map_q,    // Q: (d, W, H_q, batch), box (64, W, G, 1)
              const TheoryArgs a) {
  extern __shared__ uint8_t tsm_raw[];
  const uint32_t base = (smem_u32(tsm_raw) + 1023u) & ~1023u;
  uint8_t* const gen = tsm_raw + (base - smem_u32(tsm_raw));
  const uint32_t q_box = (uint32_t)a.GW * 128u;
  const uint32_t sm_q = base, sm_k = base + 2u * q_box;
  float* rq = reinterpret_cast<float*>(gen + 2u * q_box + kThStages * kThTileBytes);          // [256] 1/|q|
  const uint32_t sm_bars = sm_k + kThStages * kThTileBytes + kThMaxQueries * 4u;
  const uint32_t bar_q = sm_bars;
  auto bar_full = [&](int s) { return sm_bars + 8u * (1 + s); };
  auto bar_empty = [&](int s) { return sm_bars + 8u * (1 + kThStages + s); };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, c = lane & 3;
  const int h = blockIdx.y / a.nb, t = blockIdx.y % a.nb, b = blockIdx.z;
  const int tile0 = blockIdx.x * kThTilesPerCta;
  const int n_tiles = min(kThTilesPerCta, a.tiles_in_block - tile0);

  if (tid == 0) {
    mbar_init(bar_q, 1);
    for (int s = 0; s < kThStages; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 4); }
    fence_mbar_init();
  }
  __syncthreads();

  if (warp == kThWarps) {
    // ---- producer ---------------------------------------------------------------------------------
    if (lane == 0) {
      mbar_expect_tx(bar_q, 2u * q_box);
      tma_load_4d(sm_q, &map_q, bar_q, 0, 0, h * a.G, b);
      tma_load_4d(sm_q + q_box, &map_q, bar_q, 64, 0, h * a.G, b);
      for (int j = 0; j < n_tiles; ++j) {
        const int st = j % kThStages;
        if (j >= kThStages && !mbar_wait(bar_empty(st), (uint32_t)(j / kThStages - 1) & 1u)) {
          record_status(a.status, kStatusTimeout);
          break;
        }
        const uint32_t dst = sm_k + st * kThTileBytes;
        const int row0 = t * a.S + (tile0 + j) * kThTile;
        mbar_expect_tx(bar_full(st), kThTileBytes);
        tma_load_4d(dst, &map_k, bar_full(st), 0, row0, h, b);
        tma_load_4d(dst + kThTileBytes / 2, &map_k, bar_full(st), 64, row0, h, b);
      }
    }
    return;
  }

  // ---- consumers ------------------------------------------------------------------------------------
  bool alive = __all_sync(0xffffffffu, mbar_wait(bar_q, 0));
  if (alive) {
    for (int q = tid; q < a.GW; q += kThWarps * 32) {
      float n2 = 0.f;
#pragma unroll
      for (int ch = 0; ch < 16; ++ch) n2 += sum_squares8(*reinterpret_cast<const uint4*>(gen + swz128(q, ch, q_box)));
      rq[q] = n2 > 0.f ? 1.0f / sqrtf(n2) : 0.f;
    }
  }
  asm volatile("bar.sync 1, %0;" ::"n"(kThWarps * 32) : "memory");     // the consumer warps only
  const float kbits = (float)a.kbits, inv_gw = 1.0f / (float)a.GW;
  float* out = a.out + (((long long)(b * a.H_kv + h) * a.nb + t) * a.S);

  const int rows = (warp & 3) * 16;                                  // the warp's keys within a tile
  for (int j = warp >> 2; j < n_tiles && alive; j += 2) {
    const int st = j % kThStages;
    if (!__all_sync(0xffffffffu, mbar_wait(bar_full(st), (uint32_t)(j / kThStages) & 1u))) {
      if (lane == 0) record_status(a.status, kStatusTimeout);
      alive = false;
      break;
    }
    const uint32_t k_tile = sm_k + st * kThTileBytes;
    const uint8_t* k_gen = gen + 2u * q_box + st * kThTileBytes;
    // the warp's 16 keys as A fragments for all eight 16-dim steps, and the norms of keys g, g+8
    uint32_t ak[8][4];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) ldsm_x4(k_tile + dec_swz(rows + (lane & 15), 2 * ks + (lane >> 4)), ak[ks]);
    float n_lo = 0.f, n_hi = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      n_lo += sum_squares8(*reinterpret_cast<const uint4*>(k_gen + dec_swz(rows + g, c + 4 * i)));
      n_hi += sum_squares8(*reinterpret_cast<const uint4*>(k_gen + dec_swz(rows + g + 8, c + 4 * i)));
    }
    n_lo += __shfl_xor_sync(0xffffffffu, n_lo, 1); n_lo += __shfl_xor_sync(0xffffffffu, n_lo, 2);
    n_hi += __shfl_xor_sync(0xffffffffu, n_hi, 1); n_hi += __shfl_xor_sync(0xffffffffu, n_hi, 2);
    const float rk_lo = n_lo > 0.f ? 1.0f / sqrtf(n_lo) : 0.f, rk_hi = n_hi > 0.f ? 1.0f / sqrtf(n_hi) : 0.f;
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_empty(st));                     // the tile lives in registers now

    float sum_lo = 0.f, sum_hi = 0.f;
#pragma unroll 4
    for (int nt = 0; nt < a.GW / 8; ++nt) {
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int k2 = 0; k2 < 4; ++k2) {
        uint32_t qf[4];                                             // B fragments of two 16-dim steps
        ldsm_x4(sm_q + swz128(8 * nt + (lane & 7), 4 * k2 + (lane >> 3), q_box), qf);
        mma_bf16(acc, ak[2 * k2], qf[0], qf[1]);
        mma_bf16(acc, ak[2 * k2 + 1], qf[2], qf[3]);
      }
      const float2 r = *reinterpret_cast<const float2*>(rq + 8 * nt + 2 * c);
      const float2 p_lo = collide_pow2<KB>(__fmul2_rn(make_float2(acc[0], acc[1]), __fmul2_rn(r, make_float2(rk_lo, rk_lo))), kbits);
      const float2 p_hi = collide_pow2<KB>(__fmul2_rn(make_float2(acc[2], acc[3]), __fmul2_rn(r, make_float2(rk_hi, rk_hi))), kbits);
      sum_lo += p_lo.x + p_lo.y;
      sum_hi += p_hi.x + p_hi.y;
    }
    sum_lo += __shfl_xor_sync(0xffffffffu, sum_lo, 1); sum_lo += __shfl_xor_sync(0xffffffffu, sum_lo, 2);
    sum_hi += __shfl_xor_sync(0xffffffffu, sum_hi, 1); sum_hi += __shfl_xor_sync(0xffffffffu, sum_hi, 2);
    if (c == 0) {
      const int key = (tile0 + j) * kThTile + rows + g;       // within the block
      if (key < a.S) out[key] = sum_lo * inv_gw;
      if (key + 8 < a.S) out[key + 8] = sum_hi * inv_gw;
    }
  }
}

}  // namespace lkv
