// Key-streaming tensor-core kernels for the two dense contractions of the selection path:
//   * the window-score contraction Q_win . K^T  (Section 3.3 "Precision", Algorithm 1 line 3)
//   * the hyperplane projection K . P^T         (Section 3.3 "Recall", hash functions h_r)
// One persistent, warp-specialised skeleton serves three passes. The 128-key tiles of a launch
// form one sequence (hyperplane chunk, sequence, KV head, block, tile); every CTA owns a
// contiguous, equally long slice of it. A CTA keeps one small operand stationary in shared
// memory (the window queries of the current KV head, or a chunk of hyperplanes with the matching
// slice of the query-bucket histogram), reloads it only when its slice crosses into another
// head or chunk, and streams key tiles through a TMA -> tcgen05.mma -> TMEM -> register pipeline:
//
//   kLse   : D[query][key]; a thread owns one query row and a range of key columns and keeps an
//            online (max, sum-exp2) pair; at the end of each block's run of tiles the column
//            groups are merged and one partial per (block segment, CTA) goes to global memory.
//   kScore : D[key][query]; a thread owns one key and a range of query columns and sums
//            exp2(s - lse_q); the four column groups are added in a fixed order -> S_exact[key].
//   kProj  : D[key][hyperplane]; a thread owns one key and a range of tables, packs sign bits
//            into K-bit bucket ids, looks the buckets up in the query-bucket histogram (count of
//            window queries per bucket) and adds the collisions to count[key]. Signs decided by
//            a projection that is tiny relative to the key's other projections are queued for
//            an exact recomputation.
//   kTheory: D[key][query] as kScore; instead of softmax weights the epilogue turns every inner
//            product into the cosine of the angle between query and key (key norms from the tile
//            in shared memory, query norms from the stationary operand) and sums the closed-form
//            collision probability (1 - theta/pi)^K over the queries.
//
// Warp roles (608 threads): warp 0 = TMA producer, warps 1 and 2 = MMA issuers (warp 1 also owns
// the TMEM allocation), warps 3..18 = four epilogue groups of four warps (TMEM lane quarter =
// warp_id % 4) that split the accumulator columns of every tile. The tensor pipe runs only while
// an issuing thread feeds it (it queues next to nothing), so the two MMA warps take alternate
// tiles: the waits, fences and commits of one overlap the MMAs of the other. An epilogue thread copies its columns to registers,
// hands the accumulator buffer back to the MMA warp and only then does its arithmetic.
// All cross-warp hand-offs are mbarriers with bounded waits; there is no CTA-wide barrier
// inside the tile loop.
#pragma once
#include "ptx.cuh"
#include "theory_math.cuh"

namespace lkv {

constexpr int kTileKeys = 128;                 // keys per streamed tile (UMMA M or N)
constexpr int kAtomCols = 64;                  // bf16 elements per 128-byte swizzle row
constexpr int kTileAtomBytes = kTileKeys * 128;  // one 64-column half of a key tile
constexpr int kTileBytes = 2 * kTileAtomBytes;   // 128 keys x 128 dims bf16
constexpr int kStages = 4;
constexpr int kEpiGroups = 4;
constexpr int kEpilogueThreads = kEpiGroups * 128;
constexpr int kMmaWarps = 2;
constexpr int kStreamThreads = 32 * (1 + kMmaWarps) + kEpilogueThreads;
constexpr int kEpiCols = 64;                   // accumulator columns an epilogue thread holds at most
constexpr int kXchBytes = 8192;                // exchange area between epilogue warps
constexpr int kXchTheoryBytes = 12288;         // kTheory adds the key-norm partials [2][4 groups][128 keys]
constexpr int kTmemCols = 512;
constexpr int kAccStride = 256;                // TMEM columns per accumulator buffer (kLse, kScore: two buffers)
constexpr int kMaxAcc = 4;                     // most accumulator buffers of any mode

// kProj accumulators are TC*K columns wide: as many buffers as fit the 512 TMEM columns, at most 4.
__host__ __device__ constexpr int proj_acc_stride(int kbits, int tc) { return (kbits * tc + 31) / 32 * 32; }
__host__ __device__ constexpr int proj_num_acc(int kbits, int tc) {
  return 512 / proj_acc_stride(kbits, tc) < kMaxAcc ? 512 / proj_acc_stride(kbits, tc) : kMaxAcc;
}
constexpr int kMaxStreamCtas = 256;            // upper bound of the persistent grid (slot arithmetic)
constexpr int kPolyPairsOf32 = 10;             // of every 32 column pairs, this many take 2^x on the FMA pipe

enum StreamMode { kLse = 0, kScore = 1, kProj = 2, kTheory = 3 };

enum : int { kStatusOk = 0, kStatusCapacity = 3, kStatusTimeout = 6 };

struct StreamArgs {
  // problem geometry
  int S;               // keys per segment (a block; with look-back, the held-back tail of the previous block + the block)
  int S_stride;        // tokens between the first keys of consecutive segments (the block size)
  int nb;              // blocks in this call
  int H_kv, batch;
  int G, W, GW;        // GQA group size, window queries per head in this pass, G*W
  int q_w0;            // first window position of this pass (a window wider than 256/G queries is scored in parts)
  int accumulate;      // kScore: add to s_exact instead of storing (second and later parts)
  int lse2_stride, lse2_off;   // lse2[seg * lse2_stride + lse2_off + query of this pass]
  int tiles_in_block;  // ceil(S / 128)
  int nseg;            // batch * H_kv * nb
  long long n_tiles;   // tiles of this launch: nseg * tiles_in_block (* n_chunks for kProj)
  int lse_ctas;        // grid of the kLse launch over the same segments (slot arithmetic)
  int n_slot;          // log-sum-exp partial slots per segment
  int stat_rows;       // rows of the stationary operand (GW, or tables_per_chunk * lsh_bits)
  int stat_rows_alloc; // rows reserved per 64-column half in shared memory (multiple of 8)
  int n_chunks, tables_per_chunk, lsh_bits, lsh_tables;
  float scale_log2e;   // softmax scale * log2(e), positive
  // buffers (device)
  float2* lse_part;        // [seg][n_slot][GW]  (max, sum) in the log2 domain
  float* lse2;             // [seg][GW]
  float* s_exact;          // [seg][S]
  uint32_t* counts;        // [seg][S]
  const uint16_t* hist;    // [batch][H_kv][L][2^K]
  uint16_t* key_buckets;   // [seg][S][L] or nullptr
  int4* fix_items;         // [seg][fix_cap]: (seg, key, table, provisional bucket | doubtful bits << 16)
  int* fix_count;          // [seg]: items queued for the segment
  int fix_cap;             // items a segment's list can hold
  int* status;
  uint32_t polls, poll_ns;     // budget of the hand-off waits: polls, and nanoseconds a poll may suspend
  int overlap_prev;    // launched (with the programmatic-serialization attribute) to start beside the kernel ahead
  int release_next;    // the kernel after this one was launched that way: let it take the SMs as they fall free
  int end_wait;        // wait for the grid ahead before this kernel ends, so that what follows in the stream follows both
  // Words in global memory that order kernels running beside each other without waiting for a whole
  // grid (which, besides coupling every CTA to the slowest one, takes microseconds after the grid's
  // last CTA has gone):
  int* lse_flags;             // [seg][n_slot]: kLse writes lse_epoch when a segment's partial of a CTA is in place,
  int lse_epoch;              //   kScore waits for the flags of the partials it is about to read (null: ordinary order)
  const int* gate_counter;    // kScore: the count the query-signature kernel's CTAs add to (or null) ...
  int gate_target;            // ... and its value when all are done: only then is the projection pass released
};

__device__ __forceinline__ void record_status(int* status, int code) {
  atomicCAS(status, kStatusOk, code);
}

// The CTA whose slice [c*T/G, (c+1)*T/G) of a T-tile sequence split over G CTAs holds tile x.
__host__ __device__ inline int cta_of_tile(long long x, long long T, int G) {
  return (int)(((x + 1) * G - 1) / T);
}

// Position in the tile sequence: hyperplane chunk, (sequence, KV head) pair, block, tile in block.
struct TileCursor {
  int chunk, bh, t, tib;
  int seg;             // bh * nb + t
};
__device__ __forceinline__ TileCursor cursor_at(long long x, const StreamArgs& a) {
  const long long per_chunk = (long long)a.nseg * a.tiles_in_block;
  TileCursor c;
  c.chunk = (int)(x / per_chunk);
  const long long r = x - (long long)c.chunk * per_chunk;
  c.seg = (int)(r / a.tiles_in_block);
  c.tib = (int)(r - (long long)c.seg * a.tiles_in_block);
  c.bh = c.seg / a.nb;
  c.t = c.seg - c.bh * a.nb;
  return c;
}
__device__ __forceinline__ void cursor_advance(TileCursor& c, const StreamArgs& a) {
  if (++c.tib == a.tiles_in_block) {
    c.tib = 0;
    ++c.seg;
    if (++c.t == a.nb) {
      c.t = 0;
      if (++c.bh == a.batch * a.H_kv) { c.bh = 0; c.seg = 0; ++c.chunk; }
    }
  }
}
// The tile after c belongs to another segment / needs another stationary operand.
__device__ __forceinline__ bool cursor_last_of_segment(const TileCursor& c, const StreamArgs& a) {
  return c.tib == a.tiles_in_block - 1;
}
__device__ __forceinline__ bool cursor_last_of_group(const TileCursor& c, const StreamArgs& a) {
  return c.tib == a.tiles_in_block - 1 && c.t == a.nb - 1;
}

// Reads NC (a multiple of 16) columns starting at taddr into v.
template <int NC>
__device__ __forceinline__ void load_epi_cols(uint32_t taddr, uint32_t* v) {
#pragma unroll
  for (int j = 0; j < NC / 16; ++j) tmem_ld_x16(taddr + 16 * j, v + 16 * j);
  tmem_wait_ld();
  reg_fence<NC>(v);
}

// sum over k < N of 2^(v[k] * c2 + addend[k]); addend is per column (kScore: -lse of the query,
// read from shared memory) or one value for all columns (kLse: -running max). Pairs of columns
// go through packed fp32 arithmetic; a fixed subset of the pairs evaluates 2^x with the
// polynomial on the FMA pipe, the others use the special-function unit.
template <int N, bool PER_COLUMN>
__device__ __forceinline__ float sum_exp2(const uint32_t* v, float c2, const float* addend_s, float addend_all) {
  const float2 c22 = make_float2(c2, c2);
  float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll
  for (int k = 0; k < N; k += 4) {
    float2 ad0, ad1;
    if constexpr (PER_COLUMN) {
      const float4 ls = *reinterpret_cast<const float4*>(addend_s + k);
      ad0 = make_float2(ls.x, ls.y);
      ad1 = make_float2(ls.z, ls.w);
    } else {
      ad0 = make_float2(addend_all, addend_all);
      ad1 = ad0;
    }
    const float2 x0 = fma2(make_float2(__uint_as_float(v[k]), __uint_as_float(v[k + 1])), c22, ad0);
    const float2 x1 = fma2(make_float2(__uint_as_float(v[k + 2]), __uint_as_float(v[k + 3])), c22, ad1);
    const int p0 = k / 2, p1 = k / 2 + 1;     // pair indices, compile-time after unrolling
    const float2 e0 = ((p0 * kPolyPairsOf32) % 32 < kPolyPairsOf32) ? ex2_poly2(x0)
                                                                     : make_float2(ex2_approx(x0.x), ex2_approx(x0.y));
    const float2 e1 = ((p1 * kPolyPairsOf32) % 32 < kPolyPairsOf32) ? ex2_poly2(x1)
                                                                     : make_float2(ex2_approx(x1.x), ex2_approx(x1.y));
    acc0 = add2(acc0, e0);
    acc1 = add2(acc1, e1);
  }
  return (acc0.x + acc0.y) + (acc1.x + acc1.y);
}

// NT consecutive tables of the chunk, starting at table `t_begin` (a multiple of NT), for the
// calling thread's key: packs the sign bits of each table's K projections into a bucket code,
// looks the code up in the histogram slice and returns the summed collisions. A table whose
// smallest |projection| is below 2^-15 of the largest |projection| among the key's first 16
// hyperplanes of the chunk is queued for an exact recomputation of its signs. All of the thread's
// columns are read into registers first and the accumulator buffer is handed back to the MMA warp
// (arrive on `bar_release`) before the arithmetic starts; the per-table work is branch-free so
// that the tables interleave. `t_begin` is a run-time value so that the four epilogue groups
// share one copy of this code.
template <int KBITS, int NT>
__device__ __forceinline__ uint32_t proj_tables(uint32_t t_acc, uint32_t bar_release, const uint16_t* hist_s,
                                                const StreamArgs& a, int seg, int key, int table0, int t_begin,
                                                bool valid) {
  constexpr int NC = NT * KBITS;                               // columns of this thread
  constexpr uint32_t bucket_mask = (1u << KBITS) - 1u;
  uint32_t v[NC];
  uint32_t v16[16];
  const uint32_t t_col = t_acc + t_begin * KBITS;
#pragma unroll
  for (int j = 0; j < NC / 32; ++j) tmem_ld_x32(t_col + 32 * j, v + 32 * j);
  if constexpr (NC % 32 != 0) tmem_ld_cols<NC % 32>(t_col + (NC / 32) * 32, v + (NC / 32) * 32);
  tmem_ld_x16(t_acc, v16);
  tmem_wait_ld();
  reg_fence<NC>(v);
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
  const uint16_t* hist_g = hist_s + ((uint32_t)t_begin << KBITS);
  uint32_t partial = 0;
  float lowest = INFINITY;
#pragma unroll
  for (int t = 0; t < NT; ++t) {
    partial += hist_g[((uint32_t)t << KBITS) + code[t]];
    lowest = fminf(lowest, amin[t]);
  }
  if (valid && (a.key_buckets != nullptr || !(lowest >= tau))) {
#pragma unroll
    for (int t = 0; t < NT; ++t) {
      const int r = table0 + t_begin + t;
      if (a.key_buckets) a.key_buckets[((size_t)seg * a.S + key) * a.lsh_tables + r] = (uint16_t)code[t];
      if (!(amin[t] >= tau)) {
        uint32_t doubt = 0;                                // code bits whose projection is below tau
#pragma unroll
        for (int k = 0; k < KBITS; ++k)
          if (!(fabsf(__uint_as_float(v[t * KBITS + k])) >= tau)) doubt |= 1u << (KBITS - 1 - k);
        const int slot = atomicAdd(a.fix_count + seg, 1);
        if (slot < a.fix_cap) a.fix_items[(size_t)seg * a.fix_cap + slot] = make_int4(seg, key, r, (int)(code[t] | (doubt << 16)));
        else record_status(a.status, kStatusCapacity);
      }
    }
  }
  return partial;
}

// What an epilogue thread knows about its place in the CTA.
struct EpiCtx {
  int quarter, lane, row;      // TMEM lane quarter of the warp, lane in the warp, TMEM lane of the thread
  int ewarp, wg;               // epilogue warp 0..15, epilogue group 0..3
  uint32_t t_lane;             // TMEM address of the thread's lane, column 0
  long long x_begin, x_end;    // the CTA's slice of the tile sequence
  uint32_t bar_tfull, bar_tempty, bar_stat, bar_stat_free, bar_xa, bar_xb;
  uint8_t* xch_s;              // exchange area
  const uint16_t* hist_s;      // histogram slice (kProj)
  uint32_t bar_full, bar_empty, bar_kn;   // kTheory: the epilogue reads the key tile itself
  const uint8_t* stat_s;       // stationary operand, generic pointer (kTheory: query norms)
  const uint8_t* stages_s;     // key-tile ring, generic pointer
  uint32_t stat_atom_bytes;
};

// A run: the tiles of one block segment that fall inside the CTA's slice. The epilogue loops walk
// the slice run by run, so that the per-tile work carries no segment or group bookkeeping.
struct TileRun {
  TileCursor c;        // first tile of the run
  int ntiles;
  bool ends_group;     // the tile after the run (if any) needs another stationary operand
};
__device__ __forceinline__ TileRun run_at(long long x, long long x_end, const StreamArgs& a) {
  TileRun r;
  r.c = cursor_at(x, a);
  const long long left = x_end - x;
  const int in_block = a.tiles_in_block - r.c.tib;
  r.ntiles = left < in_block ? (int)left : in_block;
  r.ends_group = (r.c.tib + r.ntiles == a.tiles_in_block) && (r.c.t == a.nb - 1);
  return r;
}

// kLse: CW key columns per thread (64 when G*W > 128: two query row blocks x two column groups;
// 32 otherwise: one row block x four column groups).
template <int CW>
__device__ __forceinline__ bool lse_epilogue(const StreamArgs& a, const EpiCtx& e, int nmb) {
  constexpr int ncg = kTileKeys / CW;                  // column groups
  const int mb = e.wg % nmb, cg = e.wg / nmb;
  const int c0 = cg * CW;
  const int q = mb * 128 + e.row;                      // this thread's query
  const int nq = nmb * 128;
  float2* xch = reinterpret_cast<float2*>(e.xch_s);    // [ncg - 1][nq]
  const float c2 = a.scale_log2e;
  const uint32_t t_col = e.t_lane + mb * 128 + c0;
  int flushes = 0;
  uint32_t it = 0;
  for (long long x = e.x_begin; x < e.x_end;) {
    const TileRun r = run_at(x, e.x_end, a);
    float m = -INFINITY, l = 0.f;
    int nvalid = a.S - r.c.tib * kTileKeys - c0;       // key columns of this thread's range that hold a key
    for (int j = 0; j < r.ntiles; ++j, ++it, nvalid -= kTileKeys) {
      const uint32_t acc = it & 1;
      if (!mbar_wait(e.bar_tfull + 8 * acc, (it >> 1) & 1, a.polls, a.poll_ns)) return false;
      tc_fence_after();
      uint32_t v[CW];
      load_epi_cols<CW>(t_col + acc * kAccStride, v);
      tc_fence_before();
      mbar_arrive(e.bar_tempty + 8 * acc);
      if (nvalid < CW) {
        asm volatile("" ::: "memory");                 // keeps this rare path a real branch
#pragma unroll
        for (int k = 0; k < CW; ++k) if (k >= nvalid) v[k] = 0xff800000u;
      }
      float cmax = -INFINITY;
#pragma unroll
      for (int k = 0; k < CW; k += 2) cmax = max3(__uint_as_float(v[k]), __uint_as_float(v[k + 1]), cmax);
      const float m_new = fmaxf(m, cmax * c2);
      const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
      const float add = sum_exp2<CW, false>(v, c2, nullptr, -m_use);
      l = l * ex2_approx(m - m_use) + add;
      m = m_new;
    }
    // end of this segment's run of tiles: merge the column groups, write one partial
    if (cg > 0) {
      if (flushes > 0 && !mbar_wait(e.bar_xb, (uint32_t)(flushes - 1) & 1, a.polls, a.poll_ns)) return false;
      xch[(cg - 1) * nq + q] = make_float2(m, l);
      mbar_arrive(e.bar_xa);
    } else {
      if (!mbar_wait(e.bar_xa, (uint32_t)flushes & 1, a.polls, a.poll_ns)) return false;
      float mx = m;
#pragma unroll
      for (int g2 = 1; g2 < ncg; ++g2) mx = fmaxf(mx, xch[(g2 - 1) * nq + q].x);
      float lt = (mx == -INFINITY) ? 0.f : l * ex2_approx(m - mx);
#pragma unroll
      for (int g2 = 1; g2 < ncg; ++g2) {
        const float2 o = xch[(g2 - 1) * nq + q];
        if (o.x != -INFINITY) lt += o.y * ex2_approx(o.x - mx);
      }
      mbar_arrive(e.bar_xb);
      const int slot = (int)blockIdx.x - cta_of_tile((long long)r.c.seg * a.tiles_in_block, a.n_tiles, gridDim.x);
      if (q < a.GW) a.lse_part[((size_t)r.c.seg * a.n_slot + slot) * a.GW + q] = make_float2(mx, lt);
      if (a.lse_flags) {
        // the score pass may be reading already: the partial's flag goes up once every thread of this
        // column group has stored (and fenced) its entry
        __threadfence();
        mbar_arrive(e.bar_kn);
        if (q == 0) {
          if (!mbar_wait(e.bar_kn, (uint32_t)flushes & 1, a.polls, a.poll_ns)) return false;
          __threadfence();
          st_release_gpu(a.lse_flags + (size_t)r.c.seg * a.n_slot + slot, a.lse_epoch);
        }
      }
    }
    ++flushes;
    x += r.ntiles;
    if (r.ends_group && x < e.x_end) mbar_arrive(e.bar_stat_free);
  }
  return true;
}

// kScore: NC query columns [c0, c0 + NC) per thread; the groups' sums meet in group 0.
template <int NC>
__device__ __forceinline__ bool score_epilogue(const StreamArgs& a, const EpiCtx& e, int c0) {
  float* lw = reinterpret_cast<float*>(e.xch_s) + e.ewarp * kEpiCols;       // this warp's -lse values
  float* part = reinterpret_cast<float*>(e.xch_s + 16 * kEpiCols * 4);      // [2 acc][3 groups][128 keys]
  const float c2 = a.scale_log2e;
  uint32_t it = 0;
  for (long long x = e.x_begin; x < e.x_end;) {
    const TileRun r = run_at(x, e.x_end, a);
    if constexpr (NC > 0) {
      // log2-sum-exp2 of this warp's queries from the partials of the CTAs that covered the segment
      const long long first = (long long)r.c.seg * a.tiles_in_block;
      const int cf = cta_of_tile(first, a.n_tiles, a.lse_ctas);
      const int n_used = cta_of_tile(first + a.tiles_in_block - 1, a.n_tiles, a.lse_ctas) - cf + 1;
      if (a.lse_flags) {
        // the log-sum-exp pass may still be running: wait for the flags of this segment's partials
        bool ready = true;
        if (e.lane < n_used)
          ready = wait_flag_equals(a.lse_flags + (size_t)r.c.seg * a.n_slot + e.lane, a.lse_epoch,
                                   a.poll_ns == 0 ? a.polls : kMaxFlagPolls);
        if (!__all_sync(0xffffffffu, ready)) return false;
      }
      __syncwarp();
#pragma unroll
      for (int half = 0; half < (NC + 31) / 32; ++half) {
        const int j = e.lane + 32 * half;
        if (j < NC) {
          const int qq = c0 + j;
          const float2* p = a.lse_part + (size_t)r.c.seg * a.n_slot * a.GW + qq;
          float mx = -INFINITY;
          for (int s2 = 0; s2 < n_used; ++s2) mx = fmaxf(mx, __ldcg(p + (size_t)s2 * a.GW).x);
          float sum = 0.f;
          for (int s2 = 0; s2 < n_used; ++s2) {
            const float2 pe = __ldcg(p + (size_t)s2 * a.GW);
            if (pe.x != -INFINITY) sum += pe.y * exp2f(pe.x - mx);
          }
          const float lse = mx + log2f(sum);
          if (r.c.tib == 0 && e.quarter == 0) a.lse2[(size_t)r.c.seg * a.lse2_stride + a.lse2_off + qq] = lse;
          lw[j] = -lse;
        }
      }
      __syncwarp();
    }
    float* out = a.s_exact + (size_t)r.c.seg * a.S;
    int key = r.c.tib * kTileKeys + e.row;
    for (int j = 0; j < r.ntiles; ++j, ++it, key += kTileKeys) {
      const uint32_t acc = it & 1;
      if (!mbar_wait(e.bar_tfull + 8 * acc, (it >> 1) & 1, a.polls, a.poll_ns)) return false;
      tc_fence_after();
      float sum = 0.f;
      if constexpr (NC > 0) {
        uint32_t v[NC];
        load_epi_cols<NC>(e.t_lane + acc * kAccStride + c0, v);
        tc_fence_before();
        mbar_arrive(e.bar_tempty + 8 * acc);
        sum = sum_exp2<NC, true>(v, c2, lw, 0.f);
      } else {
        tc_fence_before();
        mbar_arrive(e.bar_tempty + 8 * acc);
      }
      // groups 1..3 hand their sums to group 0, which adds them in a fixed order
      if (e.wg > 0) {
        if (it >= 2 && !mbar_wait(e.bar_xb + 8 * acc, ((it >> 1) - 1) & 1, a.polls, a.poll_ns)) return false;
        part[(acc * 3 + (e.wg - 1)) * 128 + e.row] = sum;
        mbar_arrive(e.bar_xa + 8 * acc);
      } else {
        if (!mbar_wait(e.bar_xa + 8 * acc, (it >> 1) & 1, a.polls, a.poll_ns)) return false;
        const float tot = ((sum + part[(acc * 3 + 0) * 128 + e.row]) + part[(acc * 3 + 1) * 128 + e.row]) +
                          part[(acc * 3 + 2) * 128 + e.row];
        mbar_arrive(e.bar_xb + 8 * acc);
        if (key < a.S) out[key] = a.accumulate ? out[key] + tot : tot;
      }
    }
    x += r.ntiles;
    if (r.ends_group && x < e.x_end) mbar_arrive(e.bar_stat_free);
  }
  return true;
}

// kProj: sign bits -> bucket codes -> histogram lookups.
// Bucket code of a table: bit b of the table (hyperplane r*K + b) sits at position K-1-b, i.e.
// the first hyperplane is the most significant bit; bit = [projection >= 0].
// Group g handles tables [g*TC/4, (g+1)*TC/4) of the chunk.
template <int KBITS, int TC>
__device__ __forceinline__ bool proj_epilogue(const StreamArgs& a, const EpiCtx& e) {
  constexpr int TQ = TC / kEpiGroups;
  constexpr uint32_t NACC = proj_num_acc(KBITS, TC), STRIDE = proj_acc_stride(KBITS, TC);
  bool new_group = true;
  uint32_t gen = 0, acc = 0, acc_phase = 0;
  for (long long x = e.x_begin; x < e.x_end;) {
    const TileRun r = run_at(x, e.x_end, a);
    if (new_group) {
      // histogram slice landed (async-proxy writes are visible after the wait)
      if (!mbar_wait(e.bar_stat, gen & 1, a.polls, a.poll_ns)) return false;
      ++gen;
    }
    uint32_t* cnt = a.counts + (size_t)r.c.seg * a.S;
    const int table0 = r.c.chunk * TC;
    int key = r.c.tib * kTileKeys + e.row;
    for (int j = 0; j < r.ntiles; ++j, key += kTileKeys) {
      if (!mbar_wait_spin(e.bar_tfull + 8 * acc, acc_phase, a.polls, a.poll_ns)) return false;
      tc_fence_after();
      const bool valid = key < a.S;
      const uint32_t partial = proj_tables<KBITS, TQ>(e.t_lane + acc * STRIDE, e.bar_tempty + 8 * acc, e.hist_s, a,
                                                      r.c.seg, key, table0, e.wg * TQ, valid);
      if (valid) atomicAdd(cnt + key, partial);
      if (++acc == NACC) { acc = 0; acc_phase ^= 1; }
    }
    x += r.ntiles;
    new_group = r.ends_group;
    if (new_group && x < e.x_end) mbar_arrive(e.bar_stat_free);
  }
  return true;
}

// Sum of squares of the bf16 elements of 16-byte chunks [c_begin, c_begin + n) of row `row` of an
// operand stored as two 64-column halves (`half_bytes` apart) of 128-byte rows with the 128-byte
// swizzle (8-row groups 1024 bytes apart).
__device__ __forceinline__ float row_sum_squares(const uint8_t* op, uint32_t half_bytes, int row, int c_begin, int n) {
  float s2 = 0.f;
  const uint8_t* r = op + (uint32_t)(row >> 3) * 1024u + (uint32_t)(row & 7) * 128u;
  for (int c16 = c_begin; c16 < c_begin + n; ++c16) {
    const uint4 w = *reinterpret_cast<const uint4*>(r + (uint32_t)(c16 >> 3) * half_bytes + (uint32_t)(((c16 & 7) ^ (row & 7)) << 4));
    const uint32_t v[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float lo = __uint_as_float(v[i] << 16), hi = __uint_as_float(v[i] & 0xFFFF0000u);
      s2 = fmaf(lo, lo, s2);
      s2 = fmaf(hi, hi, s2);
    }
  }
  return s2;
}

// kTheory: NC query columns [c0, c0 + NC) per thread; KB sign bits per table (0: any number, taken
// from the arguments at run time). The four groups each square-sum a quarter of every key row of
// the tile (the stage is released by the MMAs' commit and by the sixteen epilogue warps), the
// groups' sums of the collision probabilities meet in group 0 as in the score pass.
template <int NC, int KB>
__device__ __forceinline__ bool theory_epilogue(const StreamArgs& a, const EpiCtx& e, int c0) {
  float* rqw = reinterpret_cast<float*>(e.xch_s) + e.ewarp * kEpiCols;       // this warp's 1/|q| values
  float* part = reinterpret_cast<float*>(e.xch_s + 16 * kEpiCols * 4);       // [2 acc][3 groups][128 keys]
  float* kn = reinterpret_cast<float*>(e.xch_s + 16 * kEpiCols * 4 + 2 * 3 * 128 * 4);   // [2][4 groups][128 keys]
  const float kbits = (float)a.lsh_bits, inv_gw = 1.0f / (float)a.GW;
  bool new_group = true;
  uint32_t gen = 0, it = 0;
  for (long long x = e.x_begin; x < e.x_end;) {
    const TileRun r = run_at(x, e.x_end, a);
    if (new_group) {
      // the head's window queries landed: 1 / |q| of this warp's columns
      if (!mbar_wait(e.bar_stat, gen & 1, a.polls, a.poll_ns)) return false;
      ++gen;
      __syncwarp();
      if constexpr (NC > 0) {
#pragma unroll
        for (int half = 0; half < (NC + 31) / 32; ++half) {
          const int j = e.lane + 32 * half;
          if (j < NC) {
            const float n2 = row_sum_squares(e.stat_s, e.stat_atom_bytes, c0 + j, 0, 16);
            rqw[j] = n2 > 0.f ? 1.0f / sqrtf(n2) : 0.f;      // correctly rounded: acos is ill-conditioned at |cos| = 1
          }
        }
      }
      __syncwarp();
    }
    float* out = a.s_exact + (size_t)r.c.seg * a.S;
    int key = r.c.tib * kTileKeys + e.row;
    for (int j = 0; j < r.ntiles; ++j, ++it, key += kTileKeys) {
      // this group's quarter of the key norms, straight from the tile in shared memory
      const uint32_t st = it % kStages;
      if (!mbar_wait(e.bar_full + 8 * st, (it / kStages) & 1, a.polls, a.poll_ns)) return false;
      const float q2 = row_sum_squares(e.stages_s + st * kTileBytes, kTileAtomBytes, e.row, 4 * e.wg, 4);
      float* knb = kn + (it & 1) * (kEpiGroups * 128);
      knb[e.wg * 128 + e.row] = q2;
      __syncwarp();
      if (e.lane == 0) { mbar_arrive(e.bar_empty + 8 * st); mbar_arrive(e.bar_kn + 8 * (it & 1)); }
      if (!mbar_wait(e.bar_kn + 8 * (it & 1), (it >> 1) & 1, a.polls, a.poll_ns)) return false;
      const float n2 = (knb[e.row] + knb[128 + e.row]) + (knb[256 + e.row] + knb[384 + e.row]);
      const float rk = n2 > 0.f ? 1.0f / sqrtf(n2) : 0.f;

      const uint32_t acc = it & 1;
      if (!mbar_wait(e.bar_tfull + 8 * acc, (it >> 1) & 1, a.polls, a.poll_ns)) return false;
      tc_fence_after();
      float sum = 0.f;
      if constexpr (NC > 0) {
        uint32_t v[NC];
        load_epi_cols<NC>(e.t_lane + acc * kAccStride + c0, v);
        tc_fence_before();
        mbar_arrive(e.bar_tempty + 8 * acc);
        const float2 rk2 = make_float2(rk, rk);
        float2 s0 = make_float2(0.f, 0.f), s1 = make_float2(0.f, 0.f);
#pragma unroll
        for (int k = 0; k < NC; k += 4) {
          const float4 rq = *reinterpret_cast<const float4*>(rqw + k);
          const float2 c0v = __fmul2_rn(make_float2(__uint_as_float(v[k]), __uint_as_float(v[k + 1])),
                                        __fmul2_rn(make_float2(rq.x, rq.y), rk2));
          const float2 c1v = __fmul2_rn(make_float2(__uint_as_float(v[k + 2]), __uint_as_float(v[k + 3])),
                                        __fmul2_rn(make_float2(rq.z, rq.w), rk2));
          s0 = add2(s0, collide_pow2<KB>(c0v, kbits));
          s1 = add2(s1, collide_pow2<KB>(c1v, kbits));
        }
        sum = (s0.x + s0.y) + (s1.x + s1.y);
      } else {
        tc_fence_before();
        mbar_arrive(e.bar_tempty + 8 * acc);
      }
      // groups 1..3 hand their sums to group 0, which adds them in a fixed order
      if (e.wg > 0) {
        if (it >= 2 && !mbar_wait(e.bar_xb + 8 * acc, ((it >> 1) - 1) & 1, a.polls, a.poll_ns)) return false;
        part[(acc * 3 + (e.wg - 1)) * 128 + e.row] = sum;
        mbar_arrive(e.bar_xa + 8 * acc);
      } else {
        if (!mbar_wait(e.bar_xa + 8 * acc, (it >> 1) & 1, a.polls, a.poll_ns)) return false;
        const float tot = ((sum + part[(acc * 3 + 0) * 128 + e.row]) + part[(acc * 3 + 1) * 128 + e.row]) +
                          part[(acc * 3 + 2) * 128 + e.row];
        mbar_arrive(e.bar_xb + 8 * acc);
        if (key < a.S) out[key] = tot * inv_gw;
      }
    }
    x += r.ntiles;
    new_group = r.ends_group;
    if (new_group && x < e.x_end) mbar_arrive(e.bar_stat_free);
  }
  return true;
}

// Shared memory carve-up, identical on host (sizes) and device (addresses).
__host__ __device__ inline uint32_t stream_smem_bytes(int mode, int stat_rows_alloc, int hist_bytes) {
  uint32_t b = 2u * stat_rows_alloc * 128u + kStages * kTileBytes;
  if (mode == kProj) b += (hist_bytes + 127u) & ~127u;
  b += (mode == kTheory) ? kXchTheoryBytes : kXchBytes;    // exchange area: per-warp values, cross-group partials
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

  // ---- this CTA's slice of the tile sequence ------------------------------------------------
  const long long x_begin = (long long)blockIdx.x * a.n_tiles / gridDim.x;
  const long long x_end = (long long)(blockIdx.x + 1) * a.n_tiles / gridDim.x;

  // ---- shared memory ---------------------------------------------------------------------
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t stat_atom_bytes = a.stat_rows_alloc * 128u;
  const uint32_t sm_stat = base;
  const uint32_t sm_stages = sm_stat + 2u * stat_atom_bytes;
  uint32_t cur = sm_stages + kStages * kTileBytes;
  const uint32_t hist_bytes = (MODE == kProj) ? (uint32_t)TC * (2u << KBITS) : 0u;
  const uint32_t sm_hist = cur;
  if (MODE == kProj) cur += (hist_bytes + 127u) & ~127u;
  const uint32_t sm_xch = cur;
  cur += (MODE == kTheory) ? kXchTheoryBytes : kXchBytes;
  const uint32_t sm_bars = cur;
  const uint32_t sm_tmem_slot = cur + 192;
  const uint32_t bar_full = sm_bars;                   // kStages barriers: tile landed
  const uint32_t bar_empty = sm_bars + 8 * kStages;    // kStages barriers: tile consumed by the MMAs
  const uint32_t bar_tfull = sm_bars + 16 * kStages;   // kMaxAcc: accumulator complete
  const uint32_t bar_tempty = bar_tfull + 8 * kMaxAcc; // kMaxAcc: accumulator copied out by all epilogue threads
  const uint32_t bar_stat = bar_tempty + 8 * kMaxAcc;  // stationary operand landed
  const uint32_t bar_stat_free = bar_stat + 8;         // stationary operand no longer in use
  const uint32_t bar_xa = bar_stat_free + 8;           // 2: mode-specific hand-off, "data written"
  const uint32_t bar_xb = bar_xa + 16;                 // 2: mode-specific hand-off, "data consumed"
  const uint32_t bar_kn = bar_xb + 16;                 // 2: kTheory, key-norm partials of a tile written
  uint8_t* const gen_base = smem_raw + (base - smem_u32(smem_raw));
  const uint16_t* hist_s = reinterpret_cast<const uint16_t*>(gen_base + (sm_hist - base));
  uint8_t* const xch_s = gen_base + (sm_xch - base);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen_base + (sm_tmem_slot - base));

  const int nmb = (MODE == kLse) ? (a.GW + 127) / 128 : 1;   // query row blocks of 128

  if (threadIdx.x == 0) {
    // a stage is free once the MMAs have read it; under kTheory the epilogue warps read it too
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, MODE == kTheory ? 1 + kEpilogueThreads / 32 : 1);
    }
    if (MODE == kTheory) { mbar_init(bar_kn, kEpilogueThreads / 32); mbar_init(bar_kn + 8, kEpilogueThreads / 32); }
    for (int s = 0; s < kMaxAcc; ++s) { mbar_init(bar_tfull + 8 * s, 1); mbar_init(bar_tempty + 8 * s, kEpilogueThreads); }
    mbar_init(bar_stat, 1);
    mbar_init(bar_stat_free, kEpilogueThreads);
    if (MODE == kLse) {
      mbar_init(bar_kn, nmb * 128);                      // column group 0 stored a segment's partial (flag hand-off)
      mbar_init(bar_xa, kEpilogueThreads - nmb * 128);   // column groups 1.. wrote their (max, sum)
      mbar_init(bar_xb, nmb * 128);                      // column group 0 merged them
    } else {
      for (int s = 0; s < 2; ++s) { mbar_init(bar_xa + 8 * s, kEpilogueThreads - 128); mbar_init(bar_xb + 8 * s, 128); }
    }
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(sm_tmem_slot, kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // (a score pass that itself started early releases its successor only once it has waited: see below)
  if (a.release_next) {
    if (a.gate_counter == nullptr) {
      allow_dependents();
    } else if (threadIdx.x == 0) {
      // the kernel to be released needs what the query-signature kernel wrote: its CTAs count themselves done
      if (!wait_counter_reached(a.gate_counter, a.gate_target, a.poll_ns == 0 ? a.polls : kMaxFlagPolls))
        record_status(a.status, kStatusTimeout);
      allow_dependents();
    }
  }

  if (warp == 0) {
    // ================= TMA producer =================
    if (lane == 0 && x_begin < x_end) {
      bool ok = true;
      tma_prefetch_desc(&map_keys);
      tma_prefetch_desc(&map_stat);
      TileCursor c = cursor_at(x_begin, a);
      bool new_group = true;
      int gen = 0, h = 0, b = 0;
      long long it = 0;
      for (long long x = x_begin; x < x_end; ++x, ++it) {
        if (new_group) {
          // stationary operand (+ histogram slice) of the new head / chunk
          if (gen > 0) ok = mbar_wait(bar_stat_free, (uint32_t)(gen - 1) & 1, a.polls, a.poll_ns);
          if (!ok) break;
          b = c.bh / a.H_kv;
          h = c.bh - b * a.H_kv;
          const uint32_t stat_bytes = 2u * a.stat_rows * 128u;
          mbar_expect_tx(bar_stat, stat_bytes + hist_bytes);
          if (MODE == kProj) {
            const int row0 = c.chunk * a.stat_rows;
            tma_load_2d(sm_stat, &map_stat, bar_stat, 0, row0);
            tma_load_2d(sm_stat + stat_atom_bytes, &map_stat, bar_stat, kAtomCols, row0);
            const uint16_t* hsrc = a.hist + ((size_t)c.bh * a.lsh_tables + (size_t)c.chunk * TC) * ((size_t)1 << KBITS);
            bulk_load(sm_hist, hsrc, hist_bytes, bar_stat);
          } else {
            tma_load_4d(sm_stat, &map_stat, bar_stat, 0, a.q_w0, h * a.G, b);
            tma_load_4d(sm_stat + stat_atom_bytes, &map_stat, bar_stat, kAtomCols, a.q_w0, h * a.G, b);
          }
          ++gen;
        }
        const int s = (int)(it % kStages);
        if (it >= kStages) ok = mbar_wait(bar_empty + 8 * s, (uint32_t)((it / kStages) - 1) & 1, a.polls, a.poll_ns);
        if (!ok) break;
        const uint32_t dst = sm_stages + s * kTileBytes;
        const int token = c.t * a.S_stride + c.tib * kTileKeys;
        mbar_expect_tx(bar_full + 8 * s, kTileBytes);
        tma_load_4d(dst, &map_keys, bar_full + 8 * s, 0, token, h, b);
        tma_load_4d(dst + kTileAtomBytes, &map_keys, bar_full + 8 * s, kAtomCols, token, h, b);
        new_group = cursor_last_of_group(c, a);
        cursor_advance(c, a);
      }
      if (!ok) {
        record_status(a.status, kStatusTimeout);
        // let copies already in flight land before the CTA may exit (full budget, whatever the
        // hand-off budget is: shared memory must not be written after the CTA has gone)
        for (long long i = (it > kStages ? it - kStages : 0); i < it; ++i)
          mbar_wait(bar_full + 8 * (int)(i % kStages), (uint32_t)(i / kStages) & 1);
        if (gen > 0) mbar_wait(bar_stat, (uint32_t)(gen - 1) & 1);
      }
    }
    __syncwarp();
  } else if (warp <= kMmaWarps) {
    // ================= MMA issuers =================
    // Both warps walk the whole slice (uniform waits and address arithmetic) and issue alternate
    // tiles; within a warp one elected lane issues the MMAs and their commits.
    if (x_begin < x_end) {
      bool ok = true;
      const uint32_t mine = (uint32_t)(warp - 1);
      const uint32_t idesc = (MODE == kLse) ? umma_idesc_bf16(128, kTileKeys)
                                            : umma_idesc_bf16(128, a.stat_rows);
      constexpr uint32_t NACC = (MODE == kProj) ? proj_num_acc(KBITS, TC) : 2;
      constexpr uint32_t ACC_STRIDE = (MODE == kProj) ? proj_acc_stride(KBITS, TC) : kAccStride;
      const uint32_t stat_lo = umma_sdesc_lo(sm_stat);
      const uint32_t stat_atom_lo = stat_atom_bytes >> 4;
      TileCursor c = cursor_at(x_begin, a);
      bool new_group = true, need_stat = false;
      uint32_t gen = 0, it = 0, last_use = 0;
      int last_acc = -1;
      for (long long x = x_begin; x < x_end; ++x, ++it) {
        if (new_group) { ++gen; need_stat = true; }   // stationary operand number `gen` serves this tile
        if (it % kMmaWarps == mine) {
          if (need_stat) {
            ok = mbar_wait_spin(bar_stat, (gen - 1) & 1, a.polls, a.poll_ns);
            if (!ok) break;
            need_stat = false;
          }
          const uint32_t s = it % kStages;
          const uint32_t acc = it % NACC, use = it / NACC;
          if (use > 0) ok = mbar_wait_spin(bar_tempty + 8 * acc, (use - 1) & 1, a.polls, a.poll_ns);
          if (ok) ok = mbar_wait_spin(bar_full + 8 * s, (it / kStages) & 1, a.polls, a.poll_ns);
          if (!ok) break;
          tc_fence_after();
          const uint32_t tile_lo = umma_sdesc_lo(sm_stages + s * kTileBytes);
          const uint32_t d0 = tmem_base + acc * ACC_STRIDE;
          if (elect_one()) {
#pragma unroll
            for (int mb = 0; mb < 2; ++mb) {
              if (mb < nmb) {
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                  const uint32_t tile_k = tile_lo + (k >> 2) * (kTileAtomBytes >> 4) + (k & 3) * 2;
                  const uint32_t stat_k = stat_lo + (k >> 2) * stat_atom_lo + (k & 3) * 2 + mb * ((128 * 128) >> 4);
                  if (MODE == kLse) umma_bf16_lo(d0 + mb * 128, stat_k, tile_k, idesc, k > 0);
                  else umma_bf16_lo(d0, tile_k, stat_k, idesc, k > 0);
                }
              }
            }
            umma_commit(bar_empty + 8 * s);     // stage reusable once these MMAs have read it
            umma_commit(bar_tfull + 8 * acc);   // accumulator ready for the epilogue
          }
          __syncwarp();
          last_acc = (int)acc;
          last_use = use;
        }
        new_group = cursor_last_of_group(c, a);
        cursor_advance(c, a);
      }
      if (!ok) {
        if (lane == 0) record_status(a.status, kStatusTimeout);
        // the MMAs this warp issued last must have completed before the TMEM they write is freed
        // (full budget; the completion of their commit is the accumulator-ready barrier's phase)
        if (last_acc >= 0) mbar_wait(bar_tfull + 8 * last_acc, last_use & 1);
      }
    }
    __syncwarp();
  } else if (x_begin < x_end) {
    // ================= epilogue warps: four groups of four =================
    // Every group covers all 128 TMEM lanes (lane quarter = warp_id % 4); the groups split the
    // accumulator columns of every tile between them.
    EpiCtx e;
    e.quarter = warp & 3;
    e.lane = lane;
    e.row = e.quarter * 32 + lane;
    e.t_lane = tmem_base + ((uint32_t)(e.quarter * 32) << 16);
    e.ewarp = warp - 1 - kMmaWarps;
    e.wg = e.ewarp >> 2;
    e.x_begin = x_begin;
    e.x_end = x_end;
    e.bar_tfull = bar_tfull; e.bar_tempty = bar_tempty; e.bar_stat = bar_stat; e.bar_stat_free = bar_stat_free;
    e.bar_xa = bar_xa; e.bar_xb = bar_xb;
    e.xch_s = xch_s;
    e.hist_s = hist_s;
    e.bar_full = bar_full; e.bar_empty = bar_empty; e.bar_kn = bar_kn;
    e.stat_s = gen_base + (sm_stat - base);
    e.stages_s = gen_base + (sm_stages - base);
    e.stat_atom_bytes = stat_atom_bytes;
    bool ok;
    if constexpr (MODE == kLse) {
      ok = (nmb == 2) ? lse_epilogue<64>(a, e, nmb) : lse_epilogue<32>(a, e, nmb);
    } else if constexpr (MODE == kScore) {
      // started beside the log-sum-exp pass: tiles are loaded and multiplied meanwhile; the normalisers
      // of a segment are read once their flags are up (or, without flags, once that grid has completed)
      if (a.overlap_prev && a.lse_flags == nullptr) grid_dependency_wait();
      // group g sums the query columns [c0, c1); widths are multiples of 16, at most 64
      const int cw = ((a.GW + kEpiGroups - 1) / kEpiGroups + 15) & ~15;
      const int c0 = e.wg * cw;
      const int ncols = max(0, min(a.GW, c0 + cw) - c0);
      switch (ncols) {
        case 64: ok = score_epilogue<64>(a, e, c0); break;
        case 48: ok = score_epilogue<48>(a, e, c0); break;
        case 32: ok = score_epilogue<32>(a, e, c0); break;
        case 16: ok = score_epilogue<16>(a, e, c0); break;
        default: ok = score_epilogue<0>(a, e, c0); break;
      }
    } else if constexpr (MODE == kTheory) {
      const int cw = ((a.GW + kEpiGroups - 1) / kEpiGroups + 15) & ~15;
      const int c0 = e.wg * cw;
      const int ncols = max(0, min(a.GW, c0 + cw) - c0);
      switch (ncols) {
        case 64: ok = theory_epilogue<64, KBITS>(a, e, c0); break;
        case 48: ok = theory_epilogue<48, KBITS>(a, e, c0); break;
        case 32: ok = theory_epilogue<32, KBITS>(a, e, c0); break;
        case 16: ok = theory_epilogue<16, KBITS>(a, e, c0); break;
        default: ok = theory_epilogue<0, KBITS>(a, e, c0); break;
      }
    } else {
      ok = proj_epilogue<KBITS, TC>(a, e);
    }
    if (!ok) record_status(a.status, kStatusTimeout);
  }

  // ---- teardown ----------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (a.end_wait) grid_dependency_wait();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace lkv
