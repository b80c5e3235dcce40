// SimHash signatures of the window queries (Section 3.3 "Recall"; Algorithm 1 line 6 counts
// collisions against exactly these query buckets) in one kernel:
//
//   qsig_kernel - Q_win . P^T for one KV head's group of window queries and eight tables of
//                 hyperplanes on the tensor core (tcgen05, fp32 accumulation in TMEM); every
//                 thread owns a query row, packs the sign bits of each table into a bucket code,
//                 recomputes the bits that came from a projection too small to trust exactly
//                 (fp64 accumulation of exact bf16 products; rare), writes the codes and counts
//                 them into the tables' histograms (the number of window queries per bucket).
//                 The kernel also clears the call's collision counts and restarts the fix-up
//                 counters.
//
// Bucket code: hyperplane r*K + b0 sits at bit K-1-b0; bit = [projection >= 0].
#pragma once
#include "ptx.cuh"
#include "stream_gemm.cuh"
#include "aux_kernels.cuh"

namespace lkv {

constexpr int kQsigThreads = 128;
constexpr int kQsigTables = 8;             // tables per CTA: 8*K hyperplanes, a multiple of 16 for every K

struct QsigArgs {
  const uint16_t* Q;       // [batch][H_q][W][d] via strides (exact recomputation reads it directly)
  long long qs_b, qs_h, qs_w;
  const uint16_t* P;       // [L*K][128]
  uint16_t* hist;          // [batch][H_kv][L][2^K]
  uint16_t* qbuckets;      // [batch][H_kv][GW][L]
  int H_kv, G, W, GW;
  int q_rows_alloc;        // rows reserved per 64-column half for the query group (multiple of 128)
  int lsh_tables;
  uint4* zero_begin;       // the call's collision counts, cleared here (16-byte units)
  long long zero_n;
  int* counters;           // fix-up and changed counters, restarted here
  int* seg_counters;       // per-segment fix-up list lengths, restarted here
  int n_seg_counters;
  int* status;
  int n_real_tables;       // tables from this index on are padding: their histograms stay empty
  int q_w0;                // first window position of this pass; W and GW describe the pass
  int q_row0, q_rows_total;   // qbuckets rows: [bh][q_rows_total][L], this pass starts at row q_row0
  int first_part;          // nonzero: clear the counts, restart the counters, store the histogram;
                           // zero: a later part of a wide window: add to the histogram
  int release_next;        // nonzero: the next kernel in the stream was launched to start beside this one
  int* done_counter;       // every CTA adds one when its results are written: the projection pass, which may
                           // start while later kernels still run, is held back until all of them have
};

// <x, y> over 128 bf16 elements in fp64 (every product is exact); 16-byte loads, all in flight at once.
__device__ __noinline__ double exact_dot128(const uint16_t* x, const uint16_t* y) {
  uint4 xv[16], yv[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    xv[i] = *reinterpret_cast<const uint4*>(x + 8 * i);
    yv[i] = *reinterpret_cast<const uint4*>(y + 8 * i);
  }
  double acc0 = 0.0, acc1 = 0.0;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const uint32_t xw[4] = {xv[i].x, xv[i].y, xv[i].z, xv[i].w};
    const uint32_t yw[4] = {yv[i].x, yv[i].y, yv[i].z, yv[i].w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      acc0 = fma(bf16_to_f64((uint16_t)(xw[e] & 0xFFFF)), bf16_to_f64((uint16_t)(yw[e] & 0xFFFF)), acc0);
      acc1 = fma(bf16_to_f64((uint16_t)(xw[e] >> 16)), bf16_to_f64((uint16_t)(yw[e] >> 16)), acc1);
    }
  }
  return acc0 + acc1;
}

__host__ __device__ inline uint32_t qsig_smem_bytes(int q_rows_alloc, int kbits) {
  return 2u * q_rows_alloc * 128u + 2u * (kQsigTables * kbits) * 128u + kQsigTables * (4u << kbits) + 64u + 1024u;
}

// One CTA per (group of eight tables, KV head, sequence). A = the group's queries (row blocks of
// 128), B = the 8*K hyperplanes of the tables, D[query][hyperplane] in TMEM (one 128-column slot
// per row block).
template <int KBITS>
__global__ void __launch_bounds__(kQsigThreads, 1)
qsig_kernel(const __grid_constant__ CUtensorMap map_q,    // Q: (d, W, H_q, batch), box (64, W, G, 1)
            const __grid_constant__ CUtensorMap map_p,    // P: (d, L*K), box (64, 8*K)
            const QsigArgs a) {
  extern __shared__ uint8_t smem_raw[];
  constexpr int N = kQsigTables * KBITS;           // hyperplanes of the CTA
  constexpr int LD = (N & -N) < 32 ? (N & -N) : 32;
  constexpr uint32_t nbins = 1u << KBITS;
  constexpr uint32_t bucket_mask = nbins - 1u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tg = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  // the log-sum-exp pass that follows needs nothing from this kernel: it may take the SMs this
  // small grid leaves free (it waits for this kernel only before it ends)
  if (a.release_next) allow_dependents();
  const int nmb = (a.GW + 127) / 128;
  const size_t bh = (size_t)b * a.H_kv + h;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t q_atom = a.q_rows_alloc * 128u;
  const uint32_t sm_q = base;
  const uint32_t sm_p = sm_q + 2u * q_atom;
  const uint32_t sm_bins = sm_p + 2u * N * 128u;
  const uint32_t sm_bars = sm_bins + kQsigTables * nbins * 4u;
  const uint32_t bar_load = sm_bars, bar_mma = sm_bars + 8, sm_slot = sm_bars + 16;
  uint8_t* const gen_base = smem_raw + (base - smem_u32(smem_raw));
  uint32_t* bins = reinterpret_cast<uint32_t*>(gen_base + (sm_bins - base));      // [8][2^K]
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen_base + (sm_slot - base));

  if (threadIdx.x == 0) {
    mbar_init(bar_load, 1);
    mbar_init(bar_mma, 1);
    fence_mbar_init();
  }
  const uint32_t tmem_cols = nmb == 2 ? 256u : 128u;   // one 128-column slot per row block
  if (warp == 0) { tmem_alloc(sm_slot, tmem_cols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0 && lane == 0) {
    mbar_expect_tx(bar_load, 2u * a.GW * 128u + 2u * N * 128u);
    tma_load_4d(sm_q, &map_q, bar_load, 0, a.q_w0, h * a.G, b);
    tma_load_4d(sm_q + q_atom, &map_q, bar_load, kAtomCols, a.q_w0, h * a.G, b);
    tma_load_2d(sm_p, &map_p, bar_load, 0, tg * N);
    tma_load_2d(sm_p + N * 128u, &map_p, bar_load, kAtomCols, tg * N);
  }
  // while the operands fly: this CTA's share of the count array, and empty histograms
  {
    const long long cta = ((long long)b * gridDim.y + h) * gridDim.x + tg;
    const long long nctas = (long long)gridDim.x * gridDim.y * gridDim.z;
    const long long per = (a.zero_n + nctas - 1) / nctas;
    const long long z0 = cta * per, z1 = min(a.zero_n, z0 + per);
    if (a.first_part) {
      for (long long i = z0 + threadIdx.x; i < z1; i += kQsigThreads) a.zero_begin[i] = make_uint4(0u, 0u, 0u, 0u);
      if (cta == 0 && threadIdx.x < 2) a.counters[threadIdx.x] = 0;
      if (cta == nctas - 1)
        for (int i = threadIdx.x; i < a.n_seg_counters; i += kQsigThreads) a.seg_counters[i] = 0;
    }
    for (uint32_t i = threadIdx.x; i < kQsigTables * nbins; i += kQsigThreads) bins[i] = 0;
  }
  __syncthreads();

  bool ok = true;
  if (warp == 0) {
    ok = mbar_wait_spin(bar_load, 0);
    tc_fence_after();
    if (ok && elect_one()) {
      const uint32_t idesc = umma_idesc_bf16(128, N);
      const uint32_t q_lo = umma_sdesc_lo(sm_q), p_lo = umma_sdesc_lo(sm_p);
#pragma unroll
      for (int mb = 0; mb < 2; ++mb) {
        if (mb < nmb) {
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint32_t qk = q_lo + (k >> 2) * (q_atom >> 4) + (k & 3) * 2 + mb * ((128 * 128) >> 4);
            const uint32_t pk = p_lo + (k >> 2) * ((N * 128) >> 4) + (k & 3) * 2;
            umma_bf16_lo(tmem_base + mb * 128, qk, pk, idesc, k > 0);
          }
        }
      }
      umma_commit(bar_mma);
    }
    __syncwarp();
  }
  // every thread: its query row of each row block
  if (ok) ok = mbar_wait(bar_mma, 0);
  if (ok) {
    tc_fence_after();
    const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
    for (int mb = 0; mb < nmb; ++mb) {
      const int q = mb * 128 + warp * 32 + lane;
      uint32_t v[N];
#pragma unroll
      for (int j = 0; j < N / LD; ++j) tmem_ld_cols<LD>(t_lane + mb * 128 + j * LD, v + j * LD);
      tmem_wait_ld();
      reg_fence<N>(v);
      if (q >= a.GW) continue;
      float amax = 0.f;
#pragma unroll
      for (int k = 0; k < 16; k += 2) amax = max3_abs(__uint_as_float(v[k]), __uint_as_float(v[k + 1]), amax);
      const float tau = amax * (1.0f / 32768.0f);
      const uint16_t* row = a.Q + b * a.qs_b + (long long)(h * a.G + q / a.W) * a.qs_h + (a.q_w0 + q % a.W) * a.qs_w;
      uint32_t codes[kQsigTables];
#pragma unroll
      for (int t = 0; t < kQsigTables; ++t) {
        uint32_t neg = 0, doubt = 0;
#pragma unroll
        for (int k = 0; k < KBITS; ++k) {
          const uint32_t x = v[t * KBITS + k];
          neg = __funnelshift_l(x, neg, 1);
          if (!(fabsf(__uint_as_float(x)) >= tau)) doubt |= 1u << (KBITS - 1 - k);
        }
        uint32_t code = (~neg) & bucket_mask;
        while (doubt) {                             // rare: the 128-term sum in fp64, exact products
          const int pos = 31 - __clz(doubt);        // code bit; hyperplane r*K + (K-1-pos)
          doubt &= ~(1u << pos);
          const uint16_t* plane = a.P + ((size_t)(tg * kQsigTables + t) * KBITS + (KBITS - 1 - pos)) * 128;
          code = (code & ~(1u << pos)) | ((exact_dot128(row, plane) >= 0.0 ? 1u : 0u) << pos);
        }
        codes[t] = code;
        if (tg * kQsigTables + t < a.n_real_tables) atomicAdd(&bins[t * nbins + code], 1u);
      }
      // eight consecutive tables: one 16-byte store (L is a multiple of 8)
      uint4 packed;
      packed.x = codes[0] | (codes[1] << 16);
      packed.y = codes[2] | (codes[3] << 16);
      packed.z = codes[4] | (codes[5] << 16);
      packed.w = codes[6] | (codes[7] << 16);
      *reinterpret_cast<uint4*>(a.qbuckets + (bh * a.q_rows_total + a.q_row0 + q) * a.lsh_tables + tg * kQsigTables) = packed;
    }
  }
  if (!ok) record_status(a.status, kStatusTimeout);
  tc_fence_before();
  __syncthreads();
  if (ok) {
    uint16_t* out = a.hist + (bh * a.lsh_tables + (size_t)tg * kQsigTables) * nbins;
    for (uint32_t i = threadIdx.x; i < kQsigTables * nbins; i += kQsigThreads)
      out[i] = (uint16_t)(a.first_part ? bins[i] : bins[i] + out[i]);
  }
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, tmem_cols);
  }
  if (a.done_counter) {
    __syncthreads();                                   // the CTA's histograms, codes and zeros are written ...
    if (threadIdx.x == 0) {
      __threadfence();                                 // ... and visible before the count goes up
      atomicAdd(a.done_counter, 1);
    }
  }
}

}  // namespace lkv
