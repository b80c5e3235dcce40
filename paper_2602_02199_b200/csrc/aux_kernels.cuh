// The non-GEMM kernels of the selection path:
//   signfix_kernel - exact recomputation of key sign bits whose tensor-core projection was too
//                    close to zero to trust, with the matching correction of the counts.
//   select_kernel  - Algorithm 1 lines 4-8: two-stage top-k per (sequence, KV head, block) by
//                    shared-memory radix selection, ties to the lower index, ascending output.
//   append_kernel  - gather of the kept K/V rows into the append-only cache (16-byte vectors).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace lkv {

__device__ __forceinline__ double bf16_to_f64(uint16_t b) {
  return static_cast<double>(__uint_as_float(static_cast<uint32_t>(b) << 16));
}

// ------------------------------------------------------------------------------------------------
// Exact recomputation of flagged key signs. An item names a key, a table, the provisional bucket
// code and a mask of the code bits whose projection was too small to trust. Every segment has its
// own list. Eight lanes per item: for every masked bit the 128-term dot product is formed in fp64
// (exact bf16 products, sixteen terms per lane, reduction over the eight lanes) and the bit is
// replaced by its exact sign. If the bucket code changes, the key's count is corrected by
// hist[new] - hist[old]. The selection kernel runs this for its own segment before it reads the
// counts; the kernel below serves callers that want the counts alone.
// ------------------------------------------------------------------------------------------------
struct SignfixArgs {
  const uint16_t* Kp;     // keys via strides
  long long ks_b, ks_h, ks_t;
  const uint16_t* P;
  const uint16_t* hist;
  uint32_t* counts;
  uint16_t* key_buckets;  // or nullptr
  const int4* items;      // [seg][cap]: (segment, key, table, code | mask << 16)
  const int* n_items;     // [seg]
  int cap;
  int H_kv, nb, S, K, L;
  int* n_changed;
  int S_stride;           // tokens between the first keys of consecutive segments
  int* n_total;           // sum of the list lengths (reporting)
};

// The items of segment `seg`, taken by lane group `gid` of `ngroups` (a group = eight consecutive
// lanes of a warp; all 32 lanes of the warp must call). `smem_counts`, when given, is the calling
// CTA's copy of the segment's counts and receives the corrections as well.
__device__ __forceinline__ void signfix_segment(const SignfixArgs& a, int seg, int gid, int ngroups, uint32_t* smem_counts) {
  const int lane = threadIdx.x & 31;
  const int sl = lane & 7;                              // lane within the group of eight that shares an item
  const uint32_t gmask = 0xFFu << (lane & 24);          // the group's lanes
  const int n = min(a.n_items[seg], a.cap);
  const int4* items = a.items + (size_t)seg * a.cap;
  const int t = seg % a.nb;
  const int h = (seg / a.nb) % a.H_kv;
  const int b = seg / (a.nb * a.H_kv);
  for (int it = gid; it < n; it += ngroups) {
    const int4 item = items[it];
    const int key = item.y, r = item.z;
    const uint32_t old_code = (uint32_t)item.w & 0xFFFFu;
    uint32_t mask = (uint32_t)item.w >> 16;
    // sixteen key elements per lane
    const uint16_t* krow = a.Kp + b * a.ks_b + h * a.ks_h + ((long long)t * a.S_stride + key) * a.ks_t + sl * 16;
    const uint4 ka = *reinterpret_cast<const uint4*>(krow), kb = *reinterpret_cast<const uint4*>(krow + 8);
    const uint32_t kw[8] = {ka.x, ka.y, ka.z, ka.w, kb.x, kb.y, kb.z, kb.w};
    uint32_t code = old_code;
    while (mask) {
      const int pos = 31 - __clz(mask);          // code bit; hyperplane r*K + (K-1-pos)
      mask &= ~(1u << pos);
      const uint16_t* prow = a.P + ((size_t)r * a.K + (a.K - 1 - pos)) * 128 + sl * 16;
      const uint4 pa = *reinterpret_cast<const uint4*>(prow), pb = *reinterpret_cast<const uint4*>(prow + 8);
      const uint32_t pw[8] = {pa.x, pa.y, pa.z, pa.w, pb.x, pb.y, pb.z, pb.w};
      double acc0 = 0.0, acc1 = 0.0;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        acc0 = fma(bf16_to_f64((uint16_t)(kw[e] & 0xFFFF)), bf16_to_f64((uint16_t)(pw[e] & 0xFFFF)), acc0);
        acc1 = fma(bf16_to_f64((uint16_t)(kw[e] >> 16)), bf16_to_f64((uint16_t)(pw[e] >> 16)), acc1);
      }
      double acc = acc0 + acc1;
#pragma unroll
      for (int off = 4; off > 0; off >>= 1) acc += __shfl_xor_sync(gmask, acc, off);
      code = (code & ~(1u << pos)) | ((acc >= 0.0 ? 1u : 0u) << pos);
    }
    if (sl == 0 && code != old_code) {
      const uint16_t* hr = a.hist + ((size_t)(b * a.H_kv + h) * a.L + r) * ((size_t)1 << a.K);
      const uint32_t delta = (uint32_t)hr[code] - (uint32_t)hr[old_code];
      atomicAdd(a.counts + (size_t)seg * a.S + key, delta);
      if (smem_counts) atomicAdd(smem_counts + key, delta);
      if (a.key_buckets) a.key_buckets[((size_t)seg * a.S + key) * a.L + r] = (uint16_t)code;
      atomicAdd(a.n_changed, 1);
    }
  }
  if (gid == 0 && sl == 0) atomicAdd(a.n_total, a.n_items[seg]);
}

constexpr int kSignfixCtasPerSeg = 2;   // CTAs of 256 threads (32 lane groups each) per segment

__global__ void __launch_bounds__(256) signfix_kernel(const SignfixArgs a) {
  signfix_segment(a, blockIdx.y, (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 3), (int)((gridDim.x * blockDim.x) >> 3), nullptr);
}

// ------------------------------------------------------------------------------------------------
// Two-stage top-k. One CTA of 1024 threads per segment; scores and counts live in shared memory.
// ------------------------------------------------------------------------------------------------
constexpr int kSelThreads = 1024;

__device__ __forceinline__ uint32_t orderable_f32(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Exclusive scan of one int per thread over the whole CTA; `total` receives the sum.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += n;
  }
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int s = warp_sums[lane];
    int si = s;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, si, off);
      if (lane >= off) si += n;
    }
    warp_sums[lane] = si - s;          // exclusive warp offsets
    if (lane == 31) warp_sums[32] = si;
  }
  __syncthreads();
  const int res = warp_sums[warp] + incl - v;
  total = warp_sums[32];
  __syncthreads();
  return res;
}

// Among the participating elements j in [lo, hi) (flag[j] == 0) finds the k-th largest value T
// (k >= 1, k <= number of participants) and how many elements equal to T belong to the top k.
// `top_shift` is the position of the highest byte that can differ between values (24 for arbitrary
// 32-bit keys); the bytes above it must be zero in every value.
__device__ void radix_select_kth(const uint32_t* vals, const uint8_t* flag, int lo, int hi, int k, int top_shift,
                                 int* hist, int* misc, uint32_t& T, int& need) {
  uint32_t prefix = 0, mask = ~((top_shift >= 24) ? 0xFFFFFFFFu : ((1u << (top_shift + 8)) - 1u));
  int remaining = k;
  for (int shift = top_shift; shift >= 0; shift -= 8) {
    for (int i = threadIdx.x; i < 256; i += kSelThreads) hist[i] = 0;
    __syncthreads();
    for (int j = lo + threadIdx.x; j < hi; j += kSelThreads) {
      if (!flag[j]) {
        const uint32_t u = vals[j];
        if ((u & mask) == prefix) atomicAdd(&hist[(u >> shift) & 255], 1);
      }
    }
    __syncthreads();
    if (threadIdx.x < 32) {
      const int lane = threadIdx.x;
      int c[8], tot = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { c[i] = hist[255 - 8 * lane - i]; tot += c[i]; }
      int incl = tot;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += n;
      }
      const int excl = incl - tot;       // elements with a larger digit than this lane's range
      if (excl < remaining && remaining <= incl) {
        int run = excl;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (run < remaining && remaining <= run + c[i]) { misc[0] = 255 - 8 * lane - i; misc[1] = remaining - run; }
          run += c[i];
        }
      }
    }
    __syncthreads();
    prefix |= (uint32_t)misc[0] << shift;
    mask |= 0xFFu << shift;
    remaining = misc[1];
    __syncthreads();
  }
  T = prefix;
  need = remaining;
}

// Marks (flag = 1) the k largest participating elements of [lo, hi); equal values: lower index.
__device__ void mark_topk(const uint32_t* vals, uint8_t* flag, int lo, int hi, int k, int top_shift, int* hist,
                          int* misc, int* warp_sums) {
  if (k <= 0) return;                    // uniform across the CTA
  uint32_t T;
  int need;
  radix_select_kth(vals, flag, lo, hi, k, top_shift, hist, misc, T, need);
  const int n = hi - lo;
  const int per = (n + kSelThreads - 1) / kSelThreads;
  const int j0 = lo + threadIdx.x * per;
  const int j1 = min(hi, j0 + per);
  int eq = 0;
  for (int j = j0; j < j1; ++j) eq += (!flag[j] && vals[j] == T) ? 1 : 0;
  int total;
  int rank = block_exclusive_scan(eq, warp_sums, total);
  for (int j = j0; j < j1; ++j) {
    if (flag[j]) continue;
    const uint32_t u = vals[j];
    if (u > T) flag[j] = 1;
    else if (u == T) { if (rank < need) flag[j] = 1; ++rank; }
  }
  __syncthreads();
}

// The S scored keys of a segment fall into three classes: kept whatever their scores (two index
// ranges: Section 3.1's anchors and local window), excluded (one range: a tail that is held back
// for the next block under look-back, Section 3.2), and candidates (everything else).
struct SelectArgs {
  const float* s_exact;     // [n_seg][S]
  const uint32_t* counts;   // [n_seg][S]
  int32_t* idx;             // [n_seg][B], B = kept + k_exact + k_lsh
  int S, k_exact, k_lsh;
  int keep_a_lo, keep_a_hi, keep_b_lo, keep_b_hi;   // kept ranges [lo, hi); empty when lo >= hi
  int excl_lo, excl_hi;                             // excluded range
  int cand_lo, cand_hi;                             // a range that contains every candidate
  int count_top_shift;      // highest byte position (0, 8, 16 or 24) in which two counts can differ
  int has_fix;              // nonzero: `fix` names the segment lists of doubtful key signs to settle first
  SignfixArgs fix;
};

__global__ void __launch_bounds__(kSelThreads, 1) select_kernel(const SelectArgs a) {
  extern __shared__ uint8_t smem_sel[];
  uint32_t* ukey = reinterpret_cast<uint32_t*>(smem_sel);
  uint32_t* ucnt = ukey + a.S;
  uint8_t* flag = reinterpret_cast<uint8_t*>(ucnt + a.S);
  __shared__ int hist[256];
  __shared__ int misc[2];
  __shared__ int warp_sums[33];
  const int seg = blockIdx.x;
  const int S = a.S, lo = a.cand_lo, hi = a.cand_hi;
  const int B = max(0, a.keep_a_hi - a.keep_a_lo) + max(0, a.keep_b_hi - a.keep_b_lo) + a.k_exact + a.k_lsh;
  // flag: 0 candidate, 1 kept, 2 excluded
  for (int j = threadIdx.x; j < S; j += kSelThreads) {
    ukey[j] = orderable_f32(a.s_exact[(size_t)seg * S + j]);
    ucnt[j] = a.counts[(size_t)seg * S + j];
    const bool kept = (j >= a.keep_a_lo && j < a.keep_a_hi) || (j >= a.keep_b_lo && j < a.keep_b_hi);
    flag[j] = kept ? 1 : ((j >= a.excl_lo && j < a.excl_hi) ? 2 : 0);
  }
  __syncthreads();
  if (a.has_fix) {          // exact signs first: the corrections reach the shared-memory counts as well
    signfix_segment(a.fix, seg, (int)(threadIdx.x >> 3), kSelThreads >> 3, ucnt);
    __syncthreads();
  }
  mark_topk(ukey, flag, lo, hi, a.k_exact, 24, hist, misc, warp_sums);            // K_exact
  mark_topk(ucnt, flag, lo, hi, a.k_lsh, a.count_top_shift, hist, misc, warp_sums);  // K_lsh from the residual
  // ordered compaction of all kept indices
  const int per = (S + kSelThreads - 1) / kSelThreads;
  const int j0 = threadIdx.x * per, j1 = min(S, j0 + per);
  int cnt = 0;
  for (int j = j0; j < j1; ++j) cnt += flag[j] == 1;
  int total;
  int out = block_exclusive_scan(cnt, warp_sums, total);
  for (int j = j0; j < j1; ++j)
    if (flag[j] == 1) { if (out < B) a.idx[(size_t)seg * B + out] = j; ++out; }
}

// ------------------------------------------------------------------------------------------------
// Gather + append. 16 threads move one 256-byte row of K and of V as 16-byte vectors.
// ------------------------------------------------------------------------------------------------
struct AppendArgs {
  const uint16_t* K;
  const uint16_t* V;
  long long ks_b, ks_h, ks_t;   // source strides (elements): batch, head, token
  int H_kv, nb;
  int S_stride;                 // source rows between the first rows of consecutive blocks
  int B;                        // entries per segment
  const int32_t* idx;           // [batch][H_kv][nb][B]; NULL: entry i is source row i
  uint16_t* Kc;
  uint16_t* Vc;
  int32_t* pos;
  long long c_seg_stride;       // elements between (batch, head) cache slabs
  long long pos_seg_stride;
  long long dst_off0;           // first destination entry of block t = 0
  int pos_base0;                // absolute position of token 0 of block t = 0
  int n_src_rows;               // rows of a source segment: an index outside [0, n_src_rows) is not read
  int* status;                  // receives kAppendBadIndex when an index was out of range
};

constexpr int kAppendRowsPerCta = 64;
constexpr int kAppendBadIndex = 1;   // LASER_KV_ERR_INVALID_ARG

__device__ __forceinline__ uint4 ld_nc_v4(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__global__ void __launch_bounds__(256, 8) append_kernel(const AppendArgs a) {
  const int seg = blockIdx.y;                      // (b*H_kv + h)*nb + t
  const int t = seg % a.nb;
  const int bh = seg / a.nb;
  const int h = bh % a.H_kv, b = bh / a.H_kv;
  const int part = threadIdx.x & 15;
  const int i_end = min(a.B, (int)(blockIdx.x + 1) * kAppendRowsPerCta);
  const long long src_base = b * a.ks_b + h * a.ks_h + (long long)t * a.S_stride * a.ks_t;
  const long long dst_base = bh * a.c_seg_stride + (a.dst_off0 + (long long)t * a.B) * 128;
  int32_t* pos = a.pos + bh * a.pos_seg_stride + a.dst_off0 + (long long)t * a.B;
  const int32_t* idx = a.idx ? a.idx + (size_t)seg * a.B : nullptr;
  for (int i = blockIdx.x * kAppendRowsPerCta + (threadIdx.x >> 4); i < i_end; i += 16) {
    const int src = idx ? idx[i] : i;
    if ((unsigned)src >= (unsigned)a.n_src_rows) {          // never read outside the segment
      if (part == 0) atomicCAS(a.status, 0, kAppendBadIndex);
      continue;
    }
    const long long so = src_base + (long long)src * a.ks_t + part * 8;
    const long long dof = dst_base + (long long)i * 128 + part * 8;
    const uint4 kv = ld_nc_v4(a.K + so);
    const uint4 vv = ld_nc_v4(a.V + so);
    *reinterpret_cast<uint4*>(a.Kc + dof) = kv;
    *reinterpret_cast<uint4*>(a.Vc + dof) = vv;
    if (part == 0) pos[i] = a.pos_base0 + t * a.S_stride + src;
  }
}

// ------------------------------------------------------------------------------------------------
// Consensus aggregation: the paper's Algorithm 1 line 3 scores a candidate with the attention it
// receives from all heads (and layers). For every sequence b and position i of the call's blocks,
// adds the scores and the collision counts of the H KV heads and either stores the sums or adds
// them to sums carried over from other layers.
// ------------------------------------------------------------------------------------------------
struct ConsensusArgs {
  const float4* s;        // [batch][H][n4]  (n4 = n_blocks * S / 4)
  const uint4* c;         // [batch][H][n4]
  float4* s_acc;          // [batch][n4]
  uint4* c_acc;           // [batch][n4]
  long long n4;
  int batch, H;
  int carry;              // 0: overwrite the sums, 1: add to them
};

__global__ void __launch_bounds__(256) consensus_kernel(const ConsensusArgs a) {
  const long long total = (long long)a.batch * a.n4;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long b = i / a.n4, j = i - b * a.n4;
    float4 fs = a.carry ? a.s_acc[i] : make_float4(0.f, 0.f, 0.f, 0.f);
    uint4 cs = a.carry ? a.c_acc[i] : make_uint4(0u, 0u, 0u, 0u);
    for (int h = 0; h < a.H; ++h) {              // fixed order: deterministic sums
      const float4 x = a.s[(b * a.H + h) * a.n4 + j];
      const uint4 y = a.c[(b * a.H + h) * a.n4 + j];
      fs.x += x.x; fs.y += x.y; fs.z += x.z; fs.w += x.w;
      cs.x += y.x; cs.y += y.y; cs.z += y.z; cs.w += y.w;
    }
    a.s_acc[i] = fs;
    a.c_acc[i] = cs;
  }
}

}  // namespace lkv
