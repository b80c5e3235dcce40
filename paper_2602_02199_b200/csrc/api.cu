// Host runtime and C ABI of the LASER-KV selection library: configuration checks, budget
// arithmetic (Appendix B Eq. 1, Section 3.1), workspace carving, TMA descriptors and the launch
// sequence of one select call. Every step of the path runs in the CUDA kernels included below;
// there is no CPU path.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <string>
#include <vector>

#include "../../include/laser_kv.h"
#include "aux_kernels.cuh"
#include "stream_gemm.cuh"
#include "query_proj.cuh"
#include "decode_attn.cuh"

namespace {

using namespace lkv;

constexpr int kHeadDim = 128;
constexpr size_t kAlign = 256;
constexpr int kMaxSmem = 227 * 1024;

constexpr int kProfKernels = 6;
const char* const kProfNames[kProfKernels] = {"qsig_kernel", "stream_kernel<lse>", "stream_kernel<score>",
                                              "stream_kernel<proj>", "select_kernel", "append_kernel"};

std::atomic<long long> g_launches{0};
thread_local std::string g_last_error;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct Derived {
  int B, anchors, k_exact, k_lsh, G, GW;
  int n_qparts, Wp, GWp;   // parts a wide window is scored in; window positions and queries per part
  int tiles_in_block;
  int TC, n_chunks;
  int Kp, Lp;          // bits per table and tables as the kernels see them (padded, see derive)
  double alpha, ratio;
  float scale;
  int fix_cap;
  int S_ws;            // largest number of scored keys per segment (sizes the workspace)
  long long cap;       // cache entries per (sequence, KV head)
  int nseg_max;
};

struct Carve {
  size_t ctrl, dec_count, hist, qbuckets, lse_part, lse_flags, lse2, s_exact, counts, idx, fix_counts, fix_items, key_buckets, padP, total;
};

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

}  // namespace

struct laser_kv_ctx {
  laser_kv_config_t cfg;
  Derived d;
  Carve carve;
  uint8_t* ws = nullptr;
  uint16_t* cacheK = nullptr;
  uint16_t* cacheV = nullptr;
  int32_t* cachePos = nullptr;
  const uint16_t* P = nullptr;
  CUtensorMap mapP;    // hyperplanes, box = one chunk of the projection pass
  CUtensorMap mapPq;   // hyperplanes, box = the eight tables of one query-signature CTA
  EncodeTiledFn encode = nullptr;
  int num_sms = 1;
  std::vector<long long> blocks_done;   // per layer: blocks processed
  std::vector<long long> entries_done;  // per layer: cache entries final per (sequence, KV head)
  std::vector<long long> tokens_done;   // per layer: tokens of the blocks processed
  std::vector<int> held_back;           // per layer: tokens the last block holds back (look-back), 0 once appended
  std::vector<char> sealed;             // per layer: a short last block or the look-back close ended the sequence
  std::vector<char> lookback_done;      // per layer: laser_kv_lookback_close has run
  struct LayerBudget { int B, anchors, k_exact, k_lsh; };
  std::vector<LayerBudget> budget;      // per layer; the configured budget unless laser_kv_set_layer_budget changed it
  int last_B = 0;                       // budget of the last select call (debug view)
  std::string last_error;
  bool have_call = false;
  int last_nb = 0;
  int last_S_len = 0, last_shift = 0;   // scored keys per segment of the last pass, rows of them before the block
  int last_fixups = 0;
  // host-buffer path: copies run on a stream of their own, chunk by chunk
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_join = nullptr;
  std::vector<cudaEvent_t> ev_chunk;
  // staging buffers of recent host-path calls with the event that marks the end of their last use
  struct StageUse { const void* k; const void* v; const void* q; cudaEvent_t done; };
  std::vector<StageUse> stage_use;
  uint32_t handoff_polls = 0;           // 0: built-in wait budgets (laser_kv_set_wait_budget)
  laser_kv_counters_t counters = {0, 0, 0, 0, 0};
  bool log = false;                     // LASER_KV_LOG: one stderr line per call
  // optional per-kernel timing (events only; no device memory)
  bool profiling = false;
  // ordering words of kernels that run beside each other: how far the query-signature kernel's
  // completion counter (ctrl word 8, only grows) will have got once everything launched so far has
  // run, and the value the next log-sum-exp pass writes into its flags (never 0, the flags' initial state)
  uint32_t qsig_done_total = 0, lse_epoch = 0;
  std::vector<cudaEvent_t> ev_pool;
  std::vector<std::vector<cudaEvent_t>> ev_pending;
  float prof_ms[kProfKernels] = {0};
  int prof_launches[kProfKernels] = {0};
};

namespace {

laser_kv_status_t fail(laser_kv_ctx* h, laser_kv_status_t s, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (h) h->last_error = buf;
  g_last_error = buf;
  return s;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Kernels launch on the calling thread's current device: it must be the one the handle lives on.
laser_kv_status_t check_device(laser_kv_ctx* h, const char* who) {
  int dev = -1;
  const cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(h, LASER_KV_ERR_CUDA, "%s: cudaGetDevice: %s", who, cudaGetErrorString(e));
  if (dev != h->cfg.device)
    return fail(h, LASER_KV_ERR_STATE, "%s: the current device is %d, the handle was created on device %d", who, dev, h->cfg.device);
  return LASER_KV_OK;
}

// Persistent grid of a streaming launch: one CTA per SM, never more CTAs than tiles.
int stream_grid(long long n_tiles, int num_sms) {
  long long g = num_sms < kMaxStreamCtas ? num_sms : kMaxStreamCtas;
  if (g < 1) g = 1;
  return (int)(n_tiles < g ? n_tiles : g);
}

// Log-sum-exp partial slots per segment when `grid` CTAs split the tiles of `nseg` equally long
// segments into equal contiguous slices: a segment meets at most ceil(grid / nseg) + 1 slices.
int lse_slots(int grid, int nseg) { return (grid + nseg - 1) / nseg + 1; }

// Bytes that hold the partials of any launch over at most `nseg_max` segments, whatever the grid:
// nseg * lse_slots(grid, nseg) <= grid + 2 * nseg.
size_t lse_part_bytes_bound(size_t nseg_max, int GW) {
  return ((size_t)kMaxStreamCtas + 2 * nseg_max) * (size_t)GW * sizeof(float2);
}

// Largest supported tables-per-chunk for the projection pass: K*TC a multiple of 16 and at
// most 256 columns, L divisible by TC, histogram slice + operands within shared memory.
int pick_tc(int K, int L) {
  const int cands[3] = {32, 16, 8};
  for (int tc : cands) {
    if (L % tc) continue;
    const int n = K * tc;
    if (n > 256 || (n % 16)) continue;
    const uint32_t smem = stream_smem_bytes(kProj, n, tc * (2 << K));
    if (smem > (uint32_t)kMaxSmem) continue;
    return tc;
  }
  return 0;
}

laser_kv_status_t derive(const laser_kv_config_t* c, Derived* d) {
  if (!c) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "config is NULL");
  if (c->n_layers < 1 || c->batch < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 ||
      c->block_size < 1 || c->window < 1 || c->max_blocks < 1 || c->max_blocks_per_call < 1 ||
      c->lsh_bits < 1 || c->lsh_tables < 1)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "config: counts must be positive");
  if (c->n_q_heads % c->n_kv_heads)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "config: n_q_heads must be a multiple of n_kv_heads");
  if (c->protection_divisor < 2)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "config: protection_divisor must be >= 2");
  if (c->head_dim != kHeadDim)
    return fail(nullptr, LASER_KV_ERR_UNSUPPORTED, "config: head_dim must be 128");
  if (c->block_size % 8 || c->block_size > 16384)
    return fail(nullptr, LASER_KV_ERR_UNSUPPORTED, "config: block_size must be a multiple of 8, at most 16384");
  d->alpha = c->alpha < 0 ? 0.75 : c->alpha;
  if (d->alpha > 1.0) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "config: alpha must be in [0,1]");
  d->ratio = c->ratio == 0 ? 0.25 : c->ratio;
  if (d->ratio < 0) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "config: ratio must be positive");
  d->B = c->budget_per_block;
  if (d->B == 0) {
    if (c->context_len <= 0)
      return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "config: budget_per_block == 0 needs context_len");
    d->B = laser_kv_budget(c->context_len, c->block_size, d->ratio);
  }
  if (d->B < 0 || d->B > c->block_size)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "config: budget %d does not fit a block of %d", d->B, c->block_size);
  int loc;
  laser_kv_partition(d->B, c->protection_divisor, d->alpha, &d->anchors, &loc, &d->k_exact, &d->k_lsh);
  d->G = c->n_q_heads / c->n_kv_heads;
  d->GW = d->G * c->window;
  // A pass of the scoring kernels holds at most 256 window queries of a KV head's group; a wider
  // window is scored in parts (equal ranges of window positions, all heads of the group each):
  // the probabilities and the collision histograms of the parts simply add up.
  d->n_qparts = (d->GW + 255) / 256;
  if (d->G > 256 || d->n_qparts > 4 || c->window % d->n_qparts || (d->GW / d->n_qparts) % 16)
    return fail(nullptr, LASER_KV_ERR_UNSUPPORTED,
                "config: G*W = %d must split into at most 4 equal parts of window positions, each a multiple of 16 "
                "queries and at most 256", d->GW);
  d->Wp = c->window / d->n_qparts;
  d->GWp = d->G * d->Wp;
  if (c->lsh_bits > 12)
    return fail(nullptr, LASER_KV_ERR_UNSUPPORTED, "config: lsh_bits must be at most 12");
  // The kernels take an even number (>= 4) of bits per table and tables in groups of eight. Other
  // shapes run on a padded copy of the hyperplanes: a missing bit repeats the table's first
  // hyperplane (both sides of a comparison get the same extra bit, so bucket equality is unchanged)
  // and a missing table repeats table 0 with an all-zero query histogram (no collisions).
  d->Kp = c->lsh_bits < 4 ? 4 : (c->lsh_bits + 1) / 2 * 2;
  d->Lp = (c->lsh_tables + 7) / 8 * 8;
  d->TC = pick_tc(d->Kp, d->Lp);
  if (!d->TC)
    return fail(nullptr, LASER_KV_ERR_UNSUPPORTED, "config: no table chunking for %d bits x %d tables", c->lsh_bits, c->lsh_tables);
  if ((long long)d->GW * d->Lp > 0x7fffffffLL)
    return fail(nullptr, LASER_KV_ERR_UNSUPPORTED, "config: G*W*lsh_tables too large");
  d->n_chunks = d->Lp / d->TC;
  d->tiles_in_block = (c->block_size + kTileKeys - 1) / kTileKeys;
  if (c->softmax_scale < 0.f || c->softmax_scale != c->softmax_scale)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "config: softmax_scale must be positive (0 selects 1/sqrt(head_dim))");
  d->scale = c->softmax_scale == 0.f ? 1.0f / std::sqrt((float)c->head_dim) : c->softmax_scale;
  d->cap = (long long)c->max_blocks * d->B;
  const long long nseg = (long long)c->batch * c->n_kv_heads * c->max_blocks_per_call;
  if (nseg > (1 << 22)) return fail(nullptr, LASER_KV_ERR_UNSUPPORTED, "config: too many segments per call");
  d->nseg_max = (int)nseg;
  if (c->lookback != 0 && c->lookback != 1)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "config: lookback must be 0 or 1");
  // with look-back a segment is the previous block's held-back tail followed by the block
  d->S_ws = c->block_size + (c->lookback ? d->anchors : 0);
  // exact-sign work list of a segment: about 5e-4 of its (key, table) pairs are expected
  long long fc = d->S_ws * (long long)d->Lp / 256;
  if (fc < 256) fc = 256;
  if (fc > (1 << 22)) fc = 1 << 22;
  d->fix_cap = (int)fc;
  return LASER_KV_OK;
}

void carve_ws(const laser_kv_config_t* c, const Derived& d, Carve* v) {
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  const size_t nseg = d.nseg_max, S = d.S_ws;
  const size_t bh = (size_t)c->batch * c->n_kv_heads;
  v->ctrl = take(256);
  v->dec_count = take(bh * 4);        // finished decode splits per (sequence, KV head)
  v->hist = take(bh * d.Lp * ((size_t)2 << d.Kp));
  v->qbuckets = take(bh * d.GW * d.Lp * 2);
  v->lse_part = take(lse_part_bytes_bound(nseg, d.GWp));
  v->lse_flags = take(lse_part_bytes_bound(nseg, 1) / sizeof(float2) * sizeof(int));   // one word per (segment, slot)
  v->lse2 = take(nseg * d.GW * 4);
  v->s_exact = take(nseg * S * 4);
  v->counts = take(nseg * S * 4 + 16);     // cleared in 16-byte units
  v->idx = take(nseg * (size_t)(d.B > 0 ? d.B : 1) * 4);
  v->fix_counts = take(nseg * sizeof(int));
  v->fix_items = take(nseg * (size_t)d.fix_cap * sizeof(int4));
  v->key_buckets = take(c->debug ? nseg * S * d.Lp * 2 : 0);
  v->padP = take((d.Kp != c->lsh_bits || d.Lp != c->lsh_tables) ? (size_t)d.Kp * d.Lp * kHeadDim * 2 : 0);
  v->total = off;
}

size_t cache_bytes_of(const laser_kv_config_t* c, const Derived& d) {
  const size_t per = (size_t)c->n_layers * c->batch * c->n_kv_heads * (size_t)d.cap;
  return align_up(per * kHeadDim * 2) * 2 + align_up(per * 4);
}

bool encode_map(laser_kv_ctx* h, CUtensorMap* m, const void* ptr, int rank, const uint64_t* dims,
                const uint64_t* strides_bytes, const uint32_t* box) {
  cuuint64_t gd[4];
  cuuint64_t gs[3];
  cuuint32_t bx[4], es[4];
  for (int i = 0; i < rank; ++i) { gd[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) gs[i] = strides_bytes[i];
  const CUresult r = h->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank,
                               const_cast<void*>(ptr), gd, gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    fail(h, LASER_KV_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
    return false;
  }
  return true;
}

// The dynamic shared-memory limit is an attribute of (kernel, device): set it once per device that
// the process launches the kernel on. `done` holds one bit per device ordinal below 64.
template <typename Fn>
cudaError_t ensure_smem_limit(std::atomic<unsigned long long>& done, Fn* fn, int bytes) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const unsigned long long bit = (dev >= 0 && dev < 64) ? 1ull << dev : 0ull;
  if (bit && (done.load(std::memory_order_relaxed) & bit)) return cudaSuccess;
  e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && bit) done.fetch_or(bit);
  return e;
}

template <int MODE, int KB, int TCv>
cudaError_t launch_stream(const CUtensorMap& mk, const CUtensorMap& ms, const StreamArgs& a, int grid,
                          uint32_t smem, cudaStream_t st) {
  static std::atomic<unsigned long long> limit_set{0};   // per instantiation
  const cudaError_t e = ensure_smem_limit(limit_set, stream_kernel<MODE, KB, TCv>, kMaxSmem);
  if (e != cudaSuccess) return e;
  if (a.overlap_prev) {
    // may start while the kernel before it in the stream, whose results it does not read, still runs
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kStreamThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t le = cudaLaunchKernelEx(&cfg, stream_kernel<MODE, KB, TCv>, mk, ms, a);
    g_launches.fetch_add(1);
    return le != cudaSuccess ? le : cudaGetLastError();
  }
  stream_kernel<MODE, KB, TCv><<<grid, kStreamThreads, smem, st>>>(mk, ms, a);
  g_launches.fetch_add(1);
  return cudaGetLastError();
}

cudaError_t launch_proj(int K, int TCv, const CUtensorMap& mk, const CUtensorMap& ms, const StreamArgs& a,
                        int grid, uint32_t smem, cudaStream_t st) {
#define LKV_CASE(KB, T) if (K == KB && TCv == T) return launch_stream<kProj, KB, T>(mk, ms, a, grid, smem, st)
  LKV_CASE(4, 8);  LKV_CASE(4, 16);  LKV_CASE(4, 32);
  LKV_CASE(6, 8);  LKV_CASE(6, 16);  LKV_CASE(6, 32);
  LKV_CASE(8, 8);  LKV_CASE(8, 16);  LKV_CASE(8, 32);
  LKV_CASE(10, 8); LKV_CASE(10, 16);
  LKV_CASE(12, 8); LKV_CASE(12, 16);
#undef LKV_CASE
  return cudaErrorInvalidValue;
}

template <int KB>
cudaError_t launch_qsig_t(const CUtensorMap& mq, const CUtensorMap& mp, const QsigArgs& a, dim3 grid, uint32_t smem,
                          cudaStream_t st) {
  static std::atomic<unsigned long long> limit_set{0};   // per instantiation
  const cudaError_t e = ensure_smem_limit(limit_set, qsig_kernel<KB>, kMaxSmem);
  if (e != cudaSuccess) return e;
  qsig_kernel<KB><<<grid, kQsigThreads, smem, st>>>(mq, mp, a);
  g_launches.fetch_add(1);
  return cudaGetLastError();
}

cudaError_t launch_qsig(int K, const CUtensorMap& mq, const CUtensorMap& mp, const QsigArgs& a, dim3 grid, uint32_t smem,
                        cudaStream_t st) {
  switch (K) {
    case 4: return launch_qsig_t<4>(mq, mp, a, grid, smem, st);
    case 6: return launch_qsig_t<6>(mq, mp, a, grid, smem, st);
    case 8: return launch_qsig_t<8>(mq, mp, a, grid, smem, st);
    case 10: return launch_qsig_t<10>(mq, mp, a, grid, smem, st);
    case 12: return launch_qsig_t<12>(mq, mp, a, grid, smem, st);
  }
  return cudaErrorInvalidValue;
}

// `count_max` bounds every count (0 = no bound known): it lets the count stage skip radix passes
// over bytes that are zero everywhere.
laser_kv_status_t launch_select(SelectArgs a, int n_seg, uint32_t count_max, cudaStream_t st) {
  static std::atomic<unsigned long long> limit_set{0};
  const size_t smem = (size_t)a.S * 9;
  if (ensure_smem_limit(limit_set, select_kernel, kMaxSmem - 2048) != cudaSuccess)
    return fail(nullptr, LASER_KV_ERR_CUDA, "cudaFuncSetAttribute(select_kernel) failed");
  int top_shift = 24;
  if (count_max != 0) {
    top_shift = 0;
    while (top_shift < 24 && (count_max >> (top_shift + 8)) != 0) top_shift += 8;
  }
  a.count_top_shift = top_shift;
  select_kernel<<<n_seg, kSelThreads, smem, st>>>(a);
  g_launches.fetch_add(1);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(nullptr, LASER_KV_ERR_CUDA, "select_kernel launch: %s", cudaGetErrorString(e));
  return LASER_KV_OK;
}

laser_kv_status_t launch_append(const AppendArgs& a, int n_seg, cudaStream_t st) {
  if (a.B <= 0 || n_seg <= 0) return LASER_KV_OK;
  dim3 grid((a.B + kAppendRowsPerCta - 1) / kAppendRowsPerCta, n_seg);
  append_kernel<<<grid, 256, 0, st>>>(a);
  g_launches.fetch_add(1);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(nullptr, LASER_KV_ERR_CUDA, "append_kernel launch: %s", cudaGetErrorString(e));
  return LASER_KV_OK;
}


// Splits per (sequence, KV head) of a decode call: as many as fill the GPU's resident CTAs once,
// never more than tiles in the cache.
int decode_splits(const laser_kv_ctx* h, long long len) {
  const laser_kv_config_t& c = h->cfg;
  long long n = (long long)h->num_sms * kDecCtasPerSm / ((long long)c.batch * c.n_kv_heads);
  const long long tiles = (len + kDecTile - 1) / kDecTile;
  if (n > tiles) n = tiles;
  if (n > kDecMaxSplit) n = kDecMaxSplit;
  return n < 1 ? 1 : (int)n;
}

}  // namespace

extern "C" {

int32_t laser_kv_budget(int64_t context_len, int32_t block_size, double ratio) {
  if (context_len <= 0 || block_size <= 0 || !(ratio > 0.0)) return -1;
  const double num = 2.0 * ratio * (double)block_size * (double)context_len;
  const double q = std::floor(num / ((double)block_size + (double)context_len));
  return q > 2147483647.0 ? -1 : (int32_t)q;
}

laser_kv_status_t laser_kv_partition(int32_t B, int32_t n, double alpha, int32_t* anchors, int32_t* local,
                                     int32_t* k_exact, int32_t* k_lsh) {
  if (B < 0 || n < 2 || !(alpha >= 0.0 && alpha <= 1.0))
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "partition: need B >= 0, n >= 2, 0 <= alpha <= 1");
  const int32_t a = B / n;
  const int32_t b_long = B - 2 * a;
  int32_t ke = (int32_t)std::floor(alpha * (double)b_long);
  if (ke < 0) ke = 0;
  if (ke > b_long) ke = b_long;
  if (anchors) *anchors = a;
  if (local) *local = a;
  if (k_exact) *k_exact = ke;
  if (k_lsh) *k_lsh = b_long - ke;
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_query_sizes(const laser_kv_config_t* cfg, size_t* cache_bytes, size_t* workspace_bytes) {
  Derived d;
  const laser_kv_status_t s = derive(cfg, &d);
  if (s != LASER_KV_OK) return s;
  Carve v;
  carve_ws(cfg, d, &v);
  if (cache_bytes) *cache_bytes = cache_bytes_of(cfg, d);
  if (workspace_bytes) *workspace_bytes = v.total;
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_init(const laser_kv_config_t* cfg, const void* hyperplanes, void* cache_mem,
                                size_t cache_bytes, void* workspace, size_t workspace_bytes,
                                laser_kv_handle_t* out) {
  if (!out) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "init: out is NULL");
  *out = nullptr;
  Derived d;
  laser_kv_status_t s = derive(cfg, &d);
  if (s != LASER_KV_OK) return s;
  if (!hyperplanes || !cache_mem || !workspace)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "init: NULL device buffer");
  if ((reinterpret_cast<uintptr_t>(cache_mem) | reinterpret_cast<uintptr_t>(workspace)) & (kAlign - 1))
    return fail(nullptr, LASER_KV_ERR_ALIGNMENT, "init: cache and workspace must be 256-byte aligned");
  if (!aligned16(hyperplanes)) return fail(nullptr, LASER_KV_ERR_ALIGNMENT, "init: hyperplanes must be 16-byte aligned");
  Carve v;
  carve_ws(cfg, d, &v);
  if (cache_bytes < cache_bytes_of(cfg, d) || workspace_bytes < v.total)
    return fail(nullptr, LASER_KV_ERR_CAPACITY, "init: cache needs %zu bytes, workspace %zu bytes",
                cache_bytes_of(cfg, d), v.total);
  int ndev = 0;
  cudaError_t e = cudaGetDeviceCount(&ndev);
  if (e != cudaSuccess || ndev <= cfg->device)
    return fail(nullptr, LASER_KV_ERR_CUDA, "init: no usable CUDA device %d (%s); this library has no CPU path",
                cfg->device, cudaGetErrorString(e));
  if ((e = cudaSetDevice(cfg->device)) != cudaSuccess)
    return fail(nullptr, LASER_KV_ERR_CUDA, "init: cudaSetDevice: %s", cudaGetErrorString(e));
  cudaDeviceProp prop;
  if ((e = cudaGetDeviceProperties(&prop, cfg->device)) != cudaSuccess)
    return fail(nullptr, LASER_KV_ERR_CUDA, "init: cudaGetDeviceProperties: %s", cudaGetErrorString(e));
  if (prop.major != 10)
    return fail(nullptr, LASER_KV_ERR_UNSUPPORTED, "init: device is sm_%d%d; the kernels are built for sm_100a only",
                prop.major, prop.minor);
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn)
    return fail(nullptr, LASER_KV_ERR_CUDA, "init: cuTensorMapEncodeTiled not available from the driver");

  laser_kv_ctx* h = new laser_kv_ctx();
  h->cfg = *cfg;
  h->d = d;
  h->carve = v;
  h->ws = static_cast<uint8_t*>(workspace);
  h->encode = reinterpret_cast<EncodeTiledFn>(fn);
  h->num_sms = prop.multiProcessorCount;
  const size_t per = (size_t)cfg->n_layers * cfg->batch * cfg->n_kv_heads * (size_t)d.cap;
  uint8_t* cm = static_cast<uint8_t*>(cache_mem);
  h->cacheK = reinterpret_cast<uint16_t*>(cm);
  h->cacheV = reinterpret_cast<uint16_t*>(cm + align_up(per * kHeadDim * 2));
  h->cachePos = reinterpret_cast<int32_t*>(cm + 2 * align_up(per * kHeadDim * 2));
  h->P = static_cast<const uint16_t*>(hyperplanes);
  {
    const char* lg = getenv("LASER_KV_LOG");
    h->log = lg && lg[0] && strcmp(lg, "0") != 0;
  }
  h->blocks_done.assign(cfg->n_layers, 0);
  h->entries_done.assign(cfg->n_layers, 0);
  h->tokens_done.assign(cfg->n_layers, 0);
  h->held_back.assign(cfg->n_layers, 0);
  h->sealed.assign(cfg->n_layers, 0);
  h->lookback_done.assign(cfg->n_layers, 0);
  h->budget.assign(cfg->n_layers, laser_kv_ctx::LayerBudget{d.B, d.anchors, d.k_exact, d.k_lsh});
  h->last_B = d.B;
  if ((d.Kp != cfg->lsh_bits || d.Lp != cfg->lsh_tables)) {
    // padded copy of the hyperplanes in the workspace (see derive): real bits, then repeats of the
    // table's first hyperplane, then repeats of (padded) table 0
    const size_t row = (size_t)kHeadDim * 2;
    uint8_t* dst = h->ws + v.padP;
    const uint8_t* src = static_cast<const uint8_t*>(hyperplanes);
    const int K = cfg->lsh_bits, L = cfg->lsh_tables;
    e = cudaMemcpy2D(dst, (size_t)d.Kp * row, src, (size_t)K * row, (size_t)K * row, (size_t)L, cudaMemcpyDeviceToDevice);
    for (int b = K; b < d.Kp && e == cudaSuccess; ++b)
      e = cudaMemcpy2D(dst + (size_t)b * row, (size_t)d.Kp * row, src, (size_t)K * row, row, (size_t)L, cudaMemcpyDeviceToDevice);
    for (int r = L; r < d.Lp && e == cudaSuccess; ++r)
      e = cudaMemcpy(dst + (size_t)r * d.Kp * row, dst, (size_t)d.Kp * row, cudaMemcpyDeviceToDevice);
    if (e != cudaSuccess) {
      delete h;
      return fail(nullptr, LASER_KV_ERR_CUDA, "init: padded hyperplane copy: %s", cudaGetErrorString(e));
    }
    h->P = reinterpret_cast<const uint16_t*>(dst);
  }
  {
    const uint64_t dims[2] = {(uint64_t)kHeadDim, (uint64_t)d.Lp * d.Kp};
    const uint64_t strides[1] = {(uint64_t)kHeadDim * 2};
    const uint32_t box[2] = {(uint32_t)kAtomCols, (uint32_t)(d.TC * d.Kp)};
    const uint32_t boxq[2] = {(uint32_t)kAtomCols, (uint32_t)(kQsigTables * d.Kp)};
    if (!encode_map(h, &h->mapP, h->P, 2, dims, strides, box) || !encode_map(h, &h->mapPq, h->P, 2, dims, strides, boxq)) {
      const std::string msg = h->last_error;
      delete h;
      return fail(nullptr, LASER_KV_ERR_CUDA, "%s", msg.c_str());
    }
  }
  if ((e = cudaMemset(h->ws + v.ctrl, 0, v.hist - v.ctrl)) != cudaSuccess ||   // status words and decode counters
      (e = cudaMemset(h->ws + v.lse_flags, 0, v.lse2 - v.lse_flags)) != cudaSuccess) {   // no partial is flagged yet
    delete h;
    return fail(nullptr, LASER_KV_ERR_CUDA, "init: cudaMemset: %s", cudaGetErrorString(e));
  }
  *out = h;
  return LASER_KV_OK;
}

}  // extern "C"

namespace {

// Geometry of one group of launches of the select path: which keys a segment scores and what
// becomes of them (Section 3.1's partition; Section 3.2's look-back shifts it by one local window).
struct CallGeom {
  int S_len;                 // scored keys per segment
  int shift;                 // rows before the block's first token that belong to the segment (0 or anchors)
  int keep_a_lo, keep_a_hi, keep_b_lo, keep_b_hi, excl_lo, excl_hi, cand_lo, cand_hi;   // scored-key index ranges
  int k_exact, k_lsh;
  int B_out;                 // cache entries per block and head
  int S_tok;                 // tokens per block of this pass (the block size; fewer for a short last block)
  int held_back;             // tokens of each block that stay undecided after the pass (look-back)
};

// Geometry of a pass over blocks of `S_tok` tokens with budget `B` per block (Section 3.1: anchors
// and local window a = floor(B/n) each, recall budget B - 2a split by alpha, Algorithm 1 lines 4/7).
// Plain rule: anchors and local window kept, Algorithm 1 on what lies between.
// Look-back (Section 3.2): the block's local window is held back instead and the `released`
// held-back tokens of the previous block (0 for the first block of a sequence) are scored with it:
// the segment is those tokens followed by the block, the block's anchors are kept, the released
// tokens and the block's middle are the candidates, and the recall budget grows by the entries the
// previous window no longer occupies.
CallGeom make_geom(int S_tok, int B, int n, double alpha, bool lookback, int released) {
  const int a = B / n;
  CallGeom g;
  g.S_tok = S_tok;
  const int b_long = B - 2 * a + (lookback ? released : 0);
  int ke = (int)std::floor(alpha * (double)b_long);
  if (ke < 0) ke = 0;
  if (ke > b_long) ke = b_long;
  g.k_exact = ke; g.k_lsh = b_long - ke;
  g.held_back = lookback ? a : 0;
  if (!lookback) {
    g.S_len = S_tok; g.shift = 0;
    g.keep_a_lo = 0; g.keep_a_hi = a; g.keep_b_lo = S_tok - a; g.keep_b_hi = S_tok;
    g.excl_lo = g.excl_hi = 0;
    g.cand_lo = a; g.cand_hi = S_tok - a;
    g.B_out = B;
  } else {
    g.S_len = S_tok + released; g.shift = released;
    g.keep_a_lo = released; g.keep_a_hi = released + a; g.keep_b_lo = g.keep_b_hi = 0;
    g.excl_lo = released + S_tok - a; g.excl_hi = released + S_tok;
    g.cand_lo = 0; g.cand_hi = released + S_tok - a;
    g.B_out = a + b_long;
  }
  return g;
}

// One pass of the path over nb consecutive blocks with the same geometry. K_blk / V_blk point at
// the first token of the first block; with g.shift > 0 the g.shift rows before it (the tail of the
// previous block) are read as well. `first_token` is the position of the first block's first token,
// `entries_done` the cache entries already final per head.
laser_kv_status_t run_select(laser_kv_ctx* h, int layer, const void* K_blk, const void* V_blk, const void* Q_win,
                             const int64_t kv_strides[3], const int64_t q_strides[3], int nb, const CallGeom& g,
                             long long first_token, long long entries_done, cudaStream_t st) {
  const laser_kv_config_t& c = h->cfg;
  const Derived& d = h->d;
  const int S = g.S_tok, S_len = g.S_len, B = g.B_out;
  const int nseg = c.batch * c.n_kv_heads * nb;
  const int tiles_in_block = (S_len + kTileKeys - 1) / kTileKeys;
  uint8_t* ws = h->ws;
  int* ctrl = reinterpret_cast<int*>(ws + h->carve.ctrl);
  uint16_t* hist = reinterpret_cast<uint16_t*>(ws + h->carve.hist);
  uint16_t* qb = reinterpret_cast<uint16_t*>(ws + h->carve.qbuckets);
  float2* lse_part = reinterpret_cast<float2*>(ws + h->carve.lse_part);
  int* lse_flags = reinterpret_cast<int*>(ws + h->carve.lse_flags);
  float* lse2 = reinterpret_cast<float*>(ws + h->carve.lse2);
  float* s_exact = reinterpret_cast<float*>(ws + h->carve.s_exact);
  uint32_t* counts = reinterpret_cast<uint32_t*>(ws + h->carve.counts);
  int32_t* idx = reinterpret_cast<int32_t*>(ws + h->carve.idx);
  int4* fix_items = reinterpret_cast<int4*>(ws + h->carve.fix_items);
  int* fix_counts = reinterpret_cast<int*>(ws + h->carve.fix_counts);
  uint16_t* key_buckets = c.debug ? reinterpret_cast<uint16_t*>(ws + h->carve.key_buckets) : nullptr;
  // the segment's first key: g.shift rows before the block
  const uint16_t* K0 = static_cast<const uint16_t*>(K_blk) - (long long)g.shift * kv_strides[2];
  const uint16_t* V0 = static_cast<const uint16_t*>(V_blk) - (long long)g.shift * kv_strides[2];

  // TMA descriptors for this call's K and Q_win
  CUtensorMap mapK, mapQ;
  {
    const uint64_t tokens = (uint64_t)nb * S + g.shift;
    const uint64_t dims[4] = {(uint64_t)kHeadDim, tokens, (uint64_t)c.n_kv_heads, (uint64_t)c.batch};
    // a dimension of extent 1 never advances; give it a dense stride if the caller passed 0
    const uint64_t s_tok = (uint64_t)kv_strides[2];
    const uint64_t s_head = kv_strides[1] > 0 ? (uint64_t)kv_strides[1] : s_tok * tokens;
    const uint64_t s_batch = kv_strides[0] > 0 ? (uint64_t)kv_strides[0] : s_head * (uint64_t)c.n_kv_heads;
    if ((c.n_kv_heads > 1 && kv_strides[1] == 0) || (c.batch > 1 && kv_strides[0] == 0))
      return fail(h, LASER_KV_ERR_INVALID_ARG, "select_block: zero stride on a dimension of extent > 1");
    const uint64_t strides[3] = {s_tok * 2, s_head * 2, s_batch * 2};
    const uint32_t box[4] = {(uint32_t)kAtomCols, (uint32_t)kTileKeys, 1, 1};
    if (!encode_map(h, &mapK, K0, 4, dims, strides, box)) return LASER_KV_ERR_CUDA;
  }
  {
    const uint64_t dims[4] = {(uint64_t)kHeadDim, (uint64_t)c.window, (uint64_t)c.n_q_heads, (uint64_t)c.batch};
    const uint64_t s_w = (uint64_t)q_strides[2];
    const uint64_t s_head = q_strides[1] > 0 ? (uint64_t)q_strides[1] : s_w * (uint64_t)c.window;
    const uint64_t s_batch = q_strides[0] > 0 ? (uint64_t)q_strides[0] : s_head * (uint64_t)c.n_q_heads;
    if ((c.n_q_heads > 1 && q_strides[1] == 0) || (c.batch > 1 && q_strides[0] == 0))
      return fail(h, LASER_KV_ERR_INVALID_ARG, "select_block: zero stride on a dimension of extent > 1");
    const uint64_t strides[3] = {s_w * 2, s_head * 2, s_batch * 2};
    const uint32_t box[4] = {(uint32_t)kAtomCols, (uint32_t)d.Wp, (uint32_t)d.G, 1};
    if (!encode_map(h, &mapQ, Q_win, 4, dims, strides, box)) return LASER_KV_ERR_CUDA;
  }

  cudaError_t e;
#define LKV_CUDA(call, what)                                                                   \
  if ((e = (call)) != cudaSuccess) return fail(h, LASER_KV_ERR_CUDA, "select_block: %s: %s", what, cudaGetErrorString(e))

  std::vector<cudaEvent_t> marks;
  auto mark = [&]() {
    if (!h->profiling) return;
    cudaEvent_t ev;
    if (!h->ev_pool.empty()) { ev = h->ev_pool.back(); h->ev_pool.pop_back(); }
    else if (cudaEventCreate(&ev) != cudaSuccess) return;
    cudaEventRecord(ev, st);
    marks.push_back(ev);
  };
  mark();
  // A stage whose share of the recall budget is empty (alpha = 1: no LSH picks; alpha = 0 or n = 2:
  // no exact picks) is not computed, unless the debug view was asked for, which shows every
  // intermediate result.
  const bool need_lsh = g.k_lsh > 0 || c.debug;
  const bool need_exact = g.k_exact > 0 || c.debug;
  // 1. query signatures and bucket histograms; the kernel also clears the counts and restarts the
  //    fix-up counter (ctrl[1]) and the changed counter (ctrl[2]); the status word (ctrl[0]) is kept
  if (need_lsh) {
    const int q_alloc = ((d.GWp + 127) / 128) * 128;
    for (int part = 0; part < d.n_qparts; ++part) {      // a window wider than a pass: its parts add up in the histogram
      QsigArgs qa{static_cast<const uint16_t*>(Q_win), q_strides[0], q_strides[1], q_strides[2], h->P, hist, qb,
                  c.n_kv_heads, d.G, d.Wp, d.GWp, q_alloc, d.Lp,
                  reinterpret_cast<uint4*>(counts), ((long long)nseg * S_len + 3) / 4, ctrl + 1, fix_counts, nseg, ctrl,
                  c.lsh_tables, part * d.Wp, part * d.GWp, d.GW, part == 0 ? 1 : 0,
                  (need_exact && !h->profiling) ? 1 : 0, ctrl + 8};
      dim3 grid(d.Lp / kQsigTables, c.n_kv_heads, c.batch);
      LKV_CUDA(launch_qsig(d.Kp, mapQ, h->mapPq, qa, grid, qsig_smem_bytes(q_alloc, d.Kp), st), "qsig_kernel");
      h->qsig_done_total += grid.x * grid.y * grid.z;
    }
  }

  StreamArgs sa;
  memset(&sa, 0, sizeof sa);
  sa.S = S_len; sa.S_stride = S; sa.nb = nb; sa.H_kv = c.n_kv_heads; sa.batch = c.batch;
  sa.G = d.G; sa.W = d.Wp; sa.GW = d.GWp; sa.lse2_stride = d.GW;
  sa.tiles_in_block = tiles_in_block; sa.nseg = nseg;
  const long long seg_tiles = (long long)nseg * tiles_in_block;
  const int base_ctas = stream_grid(seg_tiles, h->num_sms);
  sa.n_tiles = seg_tiles; sa.lse_ctas = base_ctas; sa.n_slot = lse_slots(base_ctas, nseg);
  sa.n_chunks = d.n_chunks; sa.tables_per_chunk = d.TC; sa.lsh_bits = d.Kp; sa.lsh_tables = d.Lp;
  sa.scale_log2e = d.scale * 1.4426950408889634f;
  sa.lse_part = lse_part; sa.lse2 = lse2; sa.s_exact = s_exact; sa.counts = counts; sa.hist = hist;
  sa.key_buckets = key_buckets; sa.fix_items = fix_items; sa.fix_count = fix_counts; sa.fix_cap = d.fix_cap;
  sa.status = ctrl;
  sa.polls = h->handoff_polls ? h->handoff_polls : kMaxPolls;
  sa.poll_ns = h->handoff_polls ? 0u : kPollHintNs;

  mark();
  // 2. per-query log-sum-exp over each segment's keys
  if (need_exact) {
    StreamArgs a1 = sa;
    a1.stat_rows = d.GWp;
    a1.stat_rows_alloc = ((d.GWp + 127) / 128) * 128;
    const uint32_t smem = stream_smem_bytes(kLse, a1.stat_rows_alloc, 0);
    a1.overlap_prev = (need_lsh && !h->profiling) ? 1 : 0;      // beside the query-signature kernel
    a1.release_next = h->profiling ? 0 : 1;                       // the score pass starts as SMs fall free
    if (!h->profiling) {
      if (++h->lse_epoch == 0) h->lse_epoch = 1;
      a1.lse_flags = lse_flags;
      a1.lse_epoch = (int)h->lse_epoch;
    }
    LKV_CUDA((launch_stream<kLse, 0, 0>(mapK, mapQ, a1, base_ctas, smem, st)), "lse pass");
  }
  mark();
  // 3. summed attention probabilities per key
  if (need_exact) {
    StreamArgs a2 = sa;
    a2.stat_rows = d.GWp;
    a2.stat_rows_alloc = d.GWp;
    const uint32_t smem = stream_smem_bytes(kScore, a2.stat_rows_alloc, 0);
    // the projection pass reads nothing the score pass writes: it takes each SM as the score pass leaves it
    const bool proj_beside = need_lsh && !h->profiling;
    a2.release_next = (proj_beside && d.n_qparts == 1) ? 1 : 0;
    a2.overlap_prev = h->profiling ? 0 : 1;
    if (!h->profiling) { a2.lse_flags = lse_flags; a2.lse_epoch = (int)h->lse_epoch; }
    if (a2.release_next) { a2.gate_counter = ctrl + 8; a2.gate_target = (int)h->qsig_done_total; }
    LKV_CUDA((launch_stream<kScore, 0, 0>(mapK, mapQ, a2, base_ctas, smem, st)), "score pass");
    // the remaining parts of a window wider than a pass: their probabilities add to the first part's
    for (int part = 1; part < d.n_qparts; ++part) {
      StreamArgs b1 = sa, b2 = sa;
      b1.q_w0 = b2.q_w0 = part * d.Wp;
      b1.lse2_off = b2.lse2_off = part * d.GWp;
      b1.stat_rows = b2.stat_rows = d.GWp;
      b1.stat_rows_alloc = ((d.GWp + 127) / 128) * 128;
      b2.stat_rows_alloc = d.GWp;
      b2.accumulate = 1;
      b2.release_next = (proj_beside && part == d.n_qparts - 1) ? 1 : 0;
      b1.overlap_prev = 0;                                        // follows a score pass: launched the ordinary way
      b1.release_next = h->profiling ? 0 : 1;
      b2.overlap_prev = h->profiling ? 0 : 1;
      if (!h->profiling) {
        if (++h->lse_epoch == 0) h->lse_epoch = 1;
        b1.lse_flags = b2.lse_flags = lse_flags;
        b1.lse_epoch = b2.lse_epoch = (int)h->lse_epoch;
      }
      if (b2.release_next) { b2.gate_counter = ctrl + 8; b2.gate_target = (int)h->qsig_done_total; }
      LKV_CUDA((launch_stream<kLse, 0, 0>(mapK, mapQ, b1, base_ctas, stream_smem_bytes(kLse, b1.stat_rows_alloc, 0), st)), "lse pass");
      LKV_CUDA((launch_stream<kScore, 0, 0>(mapK, mapQ, b2, base_ctas, smem, st)), "score pass");
    }
  }
  mark();
  // 4. key signatures and collision counts
  if (need_lsh) {
    StreamArgs a3 = sa;
    a3.stat_rows = d.TC * d.Kp;
    a3.stat_rows_alloc = a3.stat_rows;
    a3.n_tiles = seg_tiles * d.n_chunks;
    const uint32_t smem = stream_smem_bytes(kProj, a3.stat_rows_alloc, d.TC * (2 << d.Kp));
    a3.overlap_prev = (need_exact && !h->profiling) ? 1 : 0;     // beside the tail of the score pass
    a3.end_wait = a3.overlap_prev;                                // the selection kernel follows both
    LKV_CUDA(launch_proj(d.Kp, d.TC, mapK, h->mapP, a3, stream_grid(a3.n_tiles, h->num_sms), smem, st),
             "projection pass");
  }
  mark();
  // 5. exact signs where the tensor-core projection was too close to zero (every segment's CTA
  //    settles its own list first), then the two-stage top-k
  {
    SelectArgs sel{s_exact, counts, idx, S_len, g.k_exact, g.k_lsh, g.keep_a_lo, g.keep_a_hi, g.keep_b_lo, g.keep_b_hi,
                   g.excl_lo, g.excl_hi, g.cand_lo, g.cand_hi, 0, need_lsh ? 1 : 0,
                   SignfixArgs{K0, kv_strides[0], kv_strides[1], kv_strides[2], h->P, hist, counts, key_buckets, fix_items,
                               fix_counts, d.fix_cap, c.n_kv_heads, nb, S_len, d.Kp, d.Lp, ctrl + 2, S, ctrl + 1}};
    const laser_kv_status_t s = launch_select(sel, nseg, (uint32_t)d.GW * (uint32_t)d.Lp, st);
    if (s != LASER_KV_OK) { h->last_error = g_last_error; return s; }
  }
  mark();
  // 6. gather + append
  {
    const size_t layer_off = (size_t)layer * c.batch * c.n_kv_heads * (size_t)d.cap;
    AppendArgs aa{K0, V0, kv_strides[0], kv_strides[1], kv_strides[2], c.n_kv_heads, nb, S, B, idx,
                  h->cacheK + layer_off * kHeadDim, h->cacheV + layer_off * kHeadDim, h->cachePos + layer_off,
                  d.cap * kHeadDim, d.cap, entries_done, (int)first_token - g.shift, S_len, ctrl};
    const laser_kv_status_t s = launch_append(aa, nseg, st);
    if (s != LASER_KV_OK) { h->last_error = g_last_error; return s; }
  }
  mark();
#undef LKV_CUDA
  if (h->profiling && marks.size() == kProfKernels + 1) h->ev_pending.push_back(marks);
  else for (cudaEvent_t ev : marks) h->ev_pool.push_back(ev);
  h->have_call = true;
  h->last_nb = nb;
  h->last_B = B;
  h->last_S_len = S_len;
  h->last_shift = g.shift;
  {
    laser_kv_counters_t& k = h->counters;
    const long long rows = (long long)c.batch * c.n_kv_heads * nb;
    k.blocks += nb;
    k.tokens += (long long)c.batch * nb * S;
    k.entries_appended += rows * B;
    k.algorithmic_bytes += rows * S * kHeadDim * 2                               // keys, once
                           + (long long)c.batch * c.n_q_heads * c.window * kHeadDim * 2
                           + (long long)c.lsh_tables * c.lsh_bits * kHeadDim * 2
                           + rows * B * (4LL * kHeadDim * 2 + 4);                   // kept K and V rows in and out, positions
    if (h->log)
      fprintf(stderr, "[laser_kv] layer %d: %d block(s) of %d tokens (segment %d keys, %d before the block), "
                      "%d entries per block and head, k_exact %d, k_lsh %d, first token %lld\n",
              layer, nb, S, S_len, g.shift, B, g.k_exact, g.k_lsh, first_token);
  }
  return LASER_KV_OK;
}

}  // namespace

extern "C" {

// Argument checks shared by the block and the short-block entry points.
static laser_kv_status_t check_select_args(laser_kv_ctx* h, int layer, const void* K_blk, const void* V_blk, const void* Q_win,
                                           const int64_t kv_strides[3], const int64_t q_strides[3], const char* who) {
  const laser_kv_config_t& c = h->cfg;
  if (layer < 0 || layer >= c.n_layers) return fail(h, LASER_KV_ERR_INVALID_ARG, "%s: layer %d out of range", who, layer);
  if (!K_blk || !V_blk || !Q_win || !kv_strides || !q_strides) return fail(h, LASER_KV_ERR_INVALID_ARG, "%s: NULL argument", who);
  if (h->sealed[layer])
    return fail(h, LASER_KV_ERR_STATE, "%s: layer %d has had its last block (a short block or laser_kv_lookback_close); reset it first", who, layer);
  if (!aligned16(K_blk) || !aligned16(V_blk) || !aligned16(Q_win))
    return fail(h, LASER_KV_ERR_ALIGNMENT, "%s: device pointers must be 16-byte aligned", who);
  for (int i = 0; i < 3; ++i)
    if (kv_strides[i] < 0 || q_strides[i] < 0 || (kv_strides[i] % 8) || (q_strides[i] % 8))
      return fail(h, LASER_KV_ERR_ALIGNMENT, "%s: strides must be non-negative multiples of 8 elements", who);
  if (kv_strides[2] < kHeadDim || q_strides[2] < kHeadDim)
    return fail(h, LASER_KV_ERR_INVALID_ARG, "%s: row stride smaller than head_dim", who);
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_select_block(laser_kv_handle_t h, int32_t layer, const void* K_blk, const void* V_blk,
                                        const void* Q_win, const int64_t kv_strides[3], const int64_t q_strides[3],
                                        int32_t n_blocks, void* stream) {
  if (!h) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "select_block: NULL handle");
  if (const laser_kv_status_t ds = check_device(h, "select_block")) return ds;
  const laser_kv_config_t& c = h->cfg;
  if (const laser_kv_status_t as = check_select_args(h, layer, K_blk, V_blk, Q_win, kv_strides, q_strides, "select_block")) return as;
  if (n_blocks < 1) return fail(h, LASER_KV_ERR_INVALID_ARG, "select_block: n_blocks must be >= 1");
  if (n_blocks > c.max_blocks_per_call)
    return fail(h, LASER_KV_ERR_CAPACITY, "select_block: n_blocks %d exceeds max_blocks_per_call %d", n_blocks, c.max_blocks_per_call);
  if (h->blocks_done[layer] + n_blocks > c.max_blocks)
    return fail(h, LASER_KV_ERR_CAPACITY, "select_block: layer %d cache holds %lld of %d blocks; cannot append %d",
                layer, h->blocks_done[layer], c.max_blocks, n_blocks);
  if (h->tokens_done[layer] + (long long)n_blocks * c.block_size > 0x7fffffffLL)
    return fail(h, LASER_KV_ERR_UNSUPPORTED, "select_block: absolute positions exceed int32");

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  h->counters.select_calls += 1;
  const laser_kv_ctx::LayerBudget lb = h->budget[layer];
  const int S = c.block_size, n = c.protection_divisor;
  const bool lookback = c.lookback && lb.anchors > 0;
  laser_kv_status_t s = LASER_KV_OK;
  int first_n = 0;
  if (lookback && h->blocks_done[layer] == 0) {
    // the first block of a sequence has no held-back tokens before it: it goes alone
    const CallGeom g0 = make_geom(S, lb.B, n, h->d.alpha, true, 0);
    s = run_select(h, layer, K_blk, V_blk, Q_win, kv_strides, q_strides, 1, g0, 0, 0, st);
    if (s != LASER_KV_OK) return s;
    h->entries_done[layer] = g0.B_out;
    h->blocks_done[layer] = 1;
    h->tokens_done[layer] = S;
    h->held_back[layer] = g0.held_back;
    first_n = 1;
  }
  if (n_blocks > first_n) {
    const CallGeom g1 = make_geom(S, lb.B, n, h->d.alpha, lookback, lookback ? h->held_back[layer] : 0);
    const long long off = (long long)first_n * S * kv_strides[2];
    const int nb = n_blocks - first_n;
    s = run_select(h, layer, static_cast<const uint16_t*>(K_blk) + off, static_cast<const uint16_t*>(V_blk) + off, Q_win,
                   kv_strides, q_strides, nb, g1, h->tokens_done[layer], h->entries_done[layer], st);
    if (s != LASER_KV_OK) return s;
    h->entries_done[layer] += (long long)nb * g1.B_out;
    h->blocks_done[layer] += nb;
    h->tokens_done[layer] += (long long)nb * S;
    h->held_back[layer] = g1.held_back;
  }
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_select_tail(laser_kv_handle_t h, int32_t layer, const void* K_blk, const void* V_blk,
                                       const void* Q_win, const int64_t kv_strides[3], const int64_t q_strides[3],
                                       int32_t n_tokens, void* stream) {
  if (!h) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "select_tail: NULL handle");
  if (const laser_kv_status_t ds = check_device(h, "select_tail")) return ds;
  const laser_kv_config_t& c = h->cfg;
  if (const laser_kv_status_t as = check_select_args(h, layer, K_blk, V_blk, Q_win, kv_strides, q_strides, "select_tail")) return as;
  if (n_tokens < 1 || n_tokens >= c.block_size)
    return fail(h, LASER_KV_ERR_INVALID_ARG, "select_tail: n_tokens must be in [1, block_size); whole blocks go through laser_kv_select_block");
  if (h->blocks_done[layer] + 1 > c.max_blocks)
    return fail(h, LASER_KV_ERR_CAPACITY, "select_tail: layer %d cache holds %lld of %d blocks", layer, h->blocks_done[layer], c.max_blocks);
  if (h->tokens_done[layer] + n_tokens > 0x7fffffffLL)
    return fail(h, LASER_KV_ERR_UNSUPPORTED, "select_tail: absolute positions exceed int32");
  h->counters.select_calls += 1;
  const laser_kv_ctx::LayerBudget lb = h->budget[layer];
  const int B_t = lb.B < n_tokens ? lb.B : n_tokens;           // the same rule on the tokens there are
  const bool lookback = c.lookback != 0;
  const CallGeom g = make_geom(n_tokens, B_t, c.protection_divisor, h->d.alpha, lookback, lookback ? h->held_back[layer] : 0);
  if (g.B_out > 0) {
    const laser_kv_status_t s = run_select(h, layer, K_blk, V_blk, Q_win, kv_strides, q_strides, 1, g, h->tokens_done[layer],
                                           h->entries_done[layer], static_cast<cudaStream_t>(stream));
    if (s != LASER_KV_OK) return s;
  }
  h->entries_done[layer] += g.B_out;
  h->blocks_done[layer] += 1;
  h->tokens_done[layer] += n_tokens;
  h->held_back[layer] = g.held_back;
  h->sealed[layer] = 1;
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_lookback_close(laser_kv_handle_t h, int32_t layer, const void* K_tail, const void* V_tail,
                                          const int64_t kv_strides[3], void* stream) {
  if (!h) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "lookback_close: NULL handle");
  if (const laser_kv_status_t ds = check_device(h, "lookback_close")) return ds;
  const laser_kv_config_t& c = h->cfg;
  const Derived& d = h->d;
  if (layer < 0 || layer >= c.n_layers) return fail(h, LASER_KV_ERR_INVALID_ARG, "lookback_close: layer %d out of range", layer);
  if (!c.lookback) return fail(h, LASER_KV_ERR_STATE, "lookback_close: the handle was created without look-back");
  if (h->blocks_done[layer] == 0) return fail(h, LASER_KV_ERR_STATE, "lookback_close: layer %d holds no block", layer);
  if (h->lookback_done[layer]) return fail(h, LASER_KV_ERR_STATE, "lookback_close: layer %d is already closed", layer);
  const int a = h->held_back[layer];
  if (a > 0) {
    if (!K_tail || !V_tail || !kv_strides) return fail(h, LASER_KV_ERR_INVALID_ARG, "lookback_close: NULL argument");
    if (!aligned16(K_tail) || !aligned16(V_tail))
      return fail(h, LASER_KV_ERR_ALIGNMENT, "lookback_close: device pointers must be 16-byte aligned");
    for (int i = 0; i < 3; ++i)
      if (kv_strides[i] < 0 || (kv_strides[i] % 8))
        return fail(h, LASER_KV_ERR_ALIGNMENT, "lookback_close: strides must be non-negative multiples of 8 elements");
    if (kv_strides[2] < kHeadDim || (c.n_kv_heads > 1 && !kv_strides[1]) || (c.batch > 1 && !kv_strides[0]))
      return fail(h, LASER_KV_ERR_INVALID_ARG, "lookback_close: bad strides");
    const size_t layer_off = (size_t)layer * c.batch * c.n_kv_heads * (size_t)d.cap;
    int* ctrl = reinterpret_cast<int*>(h->ws + h->carve.ctrl);
    const long long first_pos = h->tokens_done[layer] - a;
    AppendArgs aa{static_cast<const uint16_t*>(K_tail), static_cast<const uint16_t*>(V_tail), kv_strides[0], kv_strides[1],
                  kv_strides[2], c.n_kv_heads, 1, 0, a, nullptr, h->cacheK + layer_off * kHeadDim,
                  h->cacheV + layer_off * kHeadDim, h->cachePos + layer_off, d.cap * kHeadDim, d.cap,
                  h->entries_done[layer], (int)first_pos, a, ctrl};
    const laser_kv_status_t s = launch_append(aa, c.batch * c.n_kv_heads, static_cast<cudaStream_t>(stream));
    if (s != LASER_KV_OK) { h->last_error = g_last_error; return s; }
    h->entries_done[layer] += a;
    h->held_back[layer] = 0;
  }
  h->lookback_done[layer] = 1;
  h->sealed[layer] = 1;
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_select_block_host(laser_kv_handle_t h, int32_t layer, const void* K_host, const void* V_host,
                                             const void* Q_host, void* K_stage, void* V_stage, void* Q_stage,
                                             int32_t n_blocks, int32_t* pos_out_host, void* stream) {
  if (!h) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "select_block_host: NULL handle");
  if (!K_host || !V_host || !Q_host || !K_stage || !V_stage || !Q_stage)
    return fail(h, LASER_KV_ERR_INVALID_ARG, "select_block_host: NULL argument");
  if (layer < 0 || layer >= h->cfg.n_layers) return fail(h, LASER_KV_ERR_INVALID_ARG, "select_block_host: layer out of range");
  if (n_blocks < 1 || n_blocks > h->cfg.max_blocks_per_call)
    return fail(h, LASER_KV_ERR_CAPACITY, "select_block_host: n_blocks out of range");
  const laser_kv_config_t& c = h->cfg;
  if (c.lookback)
    return fail(h, LASER_KV_ERR_UNSUPPORTED, "select_block_host: look-back needs the previous block's tail in device memory; "
                                             "use laser_kv_select_block on a contiguous device copy of the context");
  if (const laser_kv_status_t ds = check_device(h, "select_block_host")) return ds;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t T = (size_t)n_blocks * c.block_size;
  const size_t q_bytes = (size_t)c.batch * c.n_q_heads * c.window * kHeadDim * 2;
  // The blocks travel in up to four chunks on the handle's copy stream; the selection of a chunk
  // starts on `stream` as soon as its keys and values have landed, while the next chunk is copied.
  constexpr int kHostChunks = 4;
  const int n_chunks = n_blocks < kHostChunks ? n_blocks : kHostChunks;
  cudaError_t e = cudaSuccess;
  if (!h->copy_stream) e = cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking);
  if (e == cudaSuccess && !h->ev_join) e = cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming);
  while (e == cudaSuccess && (int)h->ev_chunk.size() < kHostChunks) {
    cudaEvent_t ev;
    if ((e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming)) == cudaSuccess) h->ev_chunk.push_back(ev);
  }
  if (e != cudaSuccess) return fail(h, LASER_KV_ERR_CUDA, "select_block_host: stream or event: %s", cudaGetErrorString(e));
  // The copies must not overtake earlier readers of the staging buffers. Buffers that an earlier
  // host-path call of this handle used are released by that call's own event, so that a caller who
  // alternates between two sets of staging buffers gets the next call's copies running under the
  // tail of the previous call; buffers not seen before wait for everything already on `stream`.
  constexpr size_t kStageSlots = 4;
  bool k_known = false, v_known = false, q_known = false;
  for (auto& u : h->stage_use) {
    if (u.k == K_stage || u.v == V_stage || u.q == Q_stage) {
      k_known |= u.k == K_stage; v_known |= u.v == V_stage; q_known |= u.q == Q_stage;
      if ((e = cudaStreamWaitEvent(h->copy_stream, u.done, 0)) != cudaSuccess)
        return fail(h, LASER_KV_ERR_CUDA, "select_block_host: wait: %s", cudaGetErrorString(e));
    }
  }
  // any buffer the handle has not seen may still be in use by work already on `stream`
  if (!(k_known && v_known && q_known) && ((e = cudaEventRecord(h->ev_join, st)) != cudaSuccess ||
                                           (e = cudaStreamWaitEvent(h->copy_stream, h->ev_join, 0)) != cudaSuccess))
    return fail(h, LASER_KV_ERR_CUDA, "select_block_host: wait: %s", cudaGetErrorString(e));
  if ((e = cudaMemcpyAsync(Q_stage, Q_host, q_bytes, cudaMemcpyHostToDevice, h->copy_stream)) != cudaSuccess)
    return fail(h, LASER_KV_ERR_CUDA, "select_block_host: H2D copy: %s", cudaGetErrorString(e));
  const int64_t kvs[3] = {(int64_t)c.n_kv_heads * (int64_t)T * kHeadDim, (int64_t)T * kHeadDim, kHeadDim};
  const int64_t qs[3] = {(int64_t)c.n_q_heads * c.window * kHeadDim, (int64_t)c.window * kHeadDim, kHeadDim};
  const long long before = h->entries_done[layer];
  const size_t pitch = T * kHeadDim * 2, rows = (size_t)c.batch * c.n_kv_heads;
  // Only the kept rows of V are ever read (by the append kernel). When the host V buffer is pinned
  // and mapped into the device's address space the kernel reads those rows in place over the bus
  // and V is not staged at all; pageable memory takes the copy.
  const uint8_t* v_mapped = nullptr;
  {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, V_host) == cudaSuccess && at.type == cudaMemoryTypeHost && at.devicePointer &&
        aligned16(at.devicePointer))
      v_mapped = static_cast<const uint8_t*>(at.devicePointer);
    else
      cudaGetLastError();   // an unregistered pointer is not an error here
  }
  // Remembers when the last reader of the staging buffers (so far) is done. Also called when the call
  // fails between chunks: the chunks already launched still read the buffers, and the blocks they
  // appended stay appended.
  auto remember_use = [&]() -> cudaError_t {
    laser_kv_ctx::StageUse* slot = nullptr;
    for (auto& u : h->stage_use)
      if (u.k == K_stage && u.v == V_stage && u.q == Q_stage) slot = &u;
    if (!slot) {
      // drop every entry that shares a buffer with this call, then take a free or the oldest slot
      for (size_t i = 0; i < h->stage_use.size();) {
        auto& u = h->stage_use[i];
        if (u.k == K_stage || u.v == V_stage || u.q == Q_stage) { cudaEventDestroy(u.done); h->stage_use.erase(h->stage_use.begin() + i); }
        else ++i;
      }
      if (h->stage_use.size() >= kStageSlots) { cudaEventDestroy(h->stage_use.front().done); h->stage_use.erase(h->stage_use.begin()); }
      cudaEvent_t ev;
      const cudaError_t ce = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
      if (ce != cudaSuccess) return ce;
      h->stage_use.push_back(laser_kv_ctx::StageUse{K_stage, V_stage, Q_stage, ev});
      slot = &h->stage_use.back();
    }
    return cudaEventRecord(slot->done, st);
  };
  for (int ch = 0; ch < n_chunks; ++ch) {
    const int b0 = (int)((long long)ch * n_blocks / n_chunks), b1 = (int)((long long)(ch + 1) * n_blocks / n_chunks);
    const size_t off = (size_t)b0 * c.block_size * kHeadDim * 2;           // bytes into every (sequence, head) slab
    const size_t width = (size_t)(b1 - b0) * c.block_size * kHeadDim * 2;
    uint8_t* kd = static_cast<uint8_t*>(K_stage) + off;
    uint8_t* vd = static_cast<uint8_t*>(V_stage) + off;
    if ((e = cudaMemcpy2DAsync(kd, pitch, static_cast<const uint8_t*>(K_host) + off, pitch, width, rows,
                               cudaMemcpyHostToDevice, h->copy_stream)) != cudaSuccess ||
        (!v_mapped && (e = cudaMemcpy2DAsync(vd, pitch, static_cast<const uint8_t*>(V_host) + off, pitch, width, rows,
                                             cudaMemcpyHostToDevice, h->copy_stream)) != cudaSuccess) ||
        (e = cudaEventRecord(h->ev_chunk[ch], h->copy_stream)) != cudaSuccess ||
        (e = cudaStreamWaitEvent(st, h->ev_chunk[ch], 0)) != cudaSuccess) {
      remember_use();
      return fail(h, LASER_KV_ERR_CUDA, "select_block_host: H2D copy: %s", cudaGetErrorString(e));
    }
    const laser_kv_status_t s = laser_kv_select_block(h, layer, kd, v_mapped ? static_cast<const void*>(v_mapped + off) : vd,
                                                      Q_stage, kvs, qs, b1 - b0, stream);
    if (s != LASER_KV_OK) { remember_use(); return s; }
  }
  if (pos_out_host) {
    const Derived& d = h->d;
    const size_t layer_off = (size_t)layer * c.batch * c.n_kv_heads * (size_t)d.cap;
    const size_t n_new = (size_t)(h->entries_done[layer] - before);
    const int32_t* src = h->cachePos + layer_off + before;
    e = cudaMemcpy2DAsync(pos_out_host, n_new * 4, src, (size_t)d.cap * 4, n_new * 4,
                          (size_t)c.batch * c.n_kv_heads, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return fail(h, LASER_KV_ERR_CUDA, "select_block_host: D2H copy: %s", cudaGetErrorString(e));
  }
  if ((e = remember_use()) != cudaSuccess)
    return fail(h, LASER_KV_ERR_CUDA, "select_block_host: event: %s", cudaGetErrorString(e));
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_cache_view(laser_kv_handle_t h, int32_t layer, laser_kv_view_t* out) {
  if (!h || !out) return fail(h, LASER_KV_ERR_INVALID_ARG, "cache_view: NULL argument");
  if (layer < 0 || layer >= h->cfg.n_layers) return fail(h, LASER_KV_ERR_INVALID_ARG, "cache_view: layer out of range");
  const laser_kv_config_t& c = h->cfg;
  const Derived& d = h->d;
  const size_t layer_off = (size_t)layer * c.batch * c.n_kv_heads * (size_t)d.cap;
  out->K = h->cacheK + layer_off * kHeadDim;
  out->V = h->cacheV + layer_off * kHeadDim;
  out->pos = h->cachePos + layer_off;
  out->len = h->entries_done[layer];
  out->cap = d.cap;
  out->kv_strides[0] = (int64_t)c.n_kv_heads * d.cap * kHeadDim;
  out->kv_strides[1] = d.cap * kHeadDim;
  out->kv_strides[2] = kHeadDim;
  out->pos_strides[0] = (int64_t)c.n_kv_heads * d.cap;
  out->pos_strides[1] = d.cap;
  return LASER_KV_OK;
}


size_t laser_kv_decode_attention_scratch_bytes(laser_kv_handle_t h) {
  if (!h) return 0;
  const laser_kv_config_t& c = h->cfg;
  return (size_t)c.batch * c.n_q_heads * decode_splits(h, h->d.cap) * kDecPartFloats * sizeof(float);
}

laser_kv_status_t laser_kv_decode_attention(laser_kv_handle_t h, int32_t layer, const void* Q_dec,
                                            const int64_t q_strides[2], float softmax_scale, float* out,
                                            void* scratch, size_t scratch_bytes, void* stream) {
  if (!h) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "decode_attention: NULL handle");
  if (!Q_dec || !q_strides || !out || !scratch) return fail(h, LASER_KV_ERR_INVALID_ARG, "decode_attention: NULL argument");
  const laser_kv_config_t& c = h->cfg;
  const Derived& d = h->d;
  if (layer < 0 || layer >= c.n_layers) return fail(h, LASER_KV_ERR_INVALID_ARG, "decode_attention: layer %d out of range", layer);
  if (!aligned16(Q_dec) || !aligned16(out) || !aligned16(scratch))
    return fail(h, LASER_KV_ERR_ALIGNMENT, "decode_attention: device pointers must be 16-byte aligned");
  if (q_strides[0] < 0 || q_strides[1] < 0 || (q_strides[0] % 8) || (q_strides[1] % 8))
    return fail(h, LASER_KV_ERR_ALIGNMENT, "decode_attention: strides must be non-negative multiples of 8 elements");
  if (softmax_scale < 0.f || softmax_scale != softmax_scale)
    return fail(h, LASER_KV_ERR_INVALID_ARG, "decode_attention: softmax_scale must be positive (0 selects the configured scale)");
  const int G = c.n_q_heads / c.n_kv_heads;
  if (G > kDecMaxGroup) return fail(h, LASER_KV_ERR_UNSUPPORTED, "decode_attention: more than %d query heads per KV head", kDecMaxGroup);
  const long long len = h->entries_done[layer];
  if (len < 1) return fail(h, LASER_KV_ERR_STATE, "decode_attention: layer %d cache is empty", layer);
  if (len > 0x7fffffffLL) return fail(h, LASER_KV_ERR_UNSUPPORTED, "decode_attention: cache longer than 2^31 entries");
  if (const laser_kv_status_t ds = check_device(h, "decode_attention")) return ds;
  const int n_split = decode_splits(h, len);
  const size_t need = (size_t)c.batch * c.n_q_heads * n_split * kDecPartFloats * sizeof(float);
  if (scratch_bytes < need) return fail(h, LASER_KV_ERR_CAPACITY, "decode_attention: scratch needs %zu bytes, got %zu", need, scratch_bytes);

  const size_t layer_off = (size_t)layer * c.batch * c.n_kv_heads * (size_t)d.cap * kHeadDim;
  // the layer's cache as (d, len, H_kv, batch): rows past len read as zeros
  CUtensorMap mapK, mapV;
  {
    const uint64_t dims[4] = {(uint64_t)kHeadDim, (uint64_t)len, (uint64_t)c.n_kv_heads, (uint64_t)c.batch};
    const uint64_t strides[3] = {(uint64_t)kHeadDim * 2, (uint64_t)d.cap * kHeadDim * 2,
                                 (uint64_t)c.n_kv_heads * d.cap * kHeadDim * 2};
    const uint32_t box[4] = {64, (uint32_t)kDecTile, 1, 1};
    if (!encode_map(h, &mapK, h->cacheK + layer_off, 4, dims, strides, box)) return LASER_KV_ERR_CUDA;
    if (!encode_map(h, &mapV, h->cacheV + layer_off, 4, dims, strides, box)) return LASER_KV_ERR_CUDA;
  }
  DecodeArgs a;
  a.Q = static_cast<const uint16_t*>(Q_dec);
  a.qs_b = q_strides[0];
  a.qs_h = q_strides[1];
  a.part = static_cast<float*>(scratch);
  a.out = out;
  a.H_kv = c.n_kv_heads;
  a.G = G;
  a.len = (int)len;
  a.n_split = n_split;
  a.scale_log2e = (softmax_scale == 0.f ? d.scale : softmax_scale) * 1.4426950408889634f;
  a.status = reinterpret_cast<int*>(h->ws + h->carve.ctrl);
  a.counters = reinterpret_cast<int*>(h->ws + h->carve.dec_count);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const dim3 grid((unsigned)n_split, (unsigned)c.n_kv_heads, (unsigned)c.batch);
  static std::atomic<unsigned long long> limit_set{0};
  cudaError_t e = ensure_smem_limit(limit_set, decode_split_kernel, (int)dec_smem_bytes());
  if (e != cudaSuccess) return fail(h, LASER_KV_ERR_CUDA, "decode_split_kernel attribute: %s", cudaGetErrorString(e));
  decode_split_kernel<<<grid, kDecThreads, dec_smem_bytes(), st>>>(mapK, mapV, a);
  g_launches.fetch_add(1);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(h, LASER_KV_ERR_CUDA, "decode_split_kernel launch: %s", cudaGetErrorString(e));
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_debug_view(laser_kv_handle_t h, laser_kv_debug_t* out) {
  if (!h || !out) return fail(h, LASER_KV_ERR_INVALID_ARG, "debug_view: NULL argument");
  if (!h->have_call) return fail(h, LASER_KV_ERR_STATE, "debug_view: no select call yet");
  const laser_kv_config_t& c = h->cfg;
  uint8_t* ws = h->ws;
  out->s_exact = reinterpret_cast<const float*>(ws + h->carve.s_exact);
  out->counts = reinterpret_cast<const uint32_t*>(ws + h->carve.counts);
  out->lse2 = reinterpret_cast<const float*>(ws + h->carve.lse2);
  out->query_buckets = reinterpret_cast<const uint16_t*>(ws + h->carve.qbuckets);
  out->key_buckets = c.debug ? reinterpret_cast<const uint16_t*>(ws + h->carve.key_buckets) : nullptr;
  out->hist = reinterpret_cast<const uint16_t*>(ws + h->carve.hist);
  out->idx = reinterpret_cast<const int32_t*>(ws + h->carve.idx);
  out->n_blocks = h->last_nb;
  out->batch = c.batch;
  out->n_kv_heads = c.n_kv_heads;
  out->block_size = c.block_size;
  out->segment_keys = h->last_S_len;
  out->segment_shift = h->last_shift;
  out->budget = h->last_B;
  out->gw = h->d.GW;
  out->window_part = h->d.Wp;
  out->lsh_tables = h->d.Lp;
  out->lsh_bits = h->d.Kp;
  out->n_sign_fixups = h->last_fixups;
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_poll_status(laser_kv_handle_t h, void* stream) {
  if (!h) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "poll_status: NULL handle");
  if (const laser_kv_status_t ds = check_device(h, "poll_status")) return ds;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int host[4] = {0, 0, 0, 0};
  cudaError_t e = cudaMemcpyAsync(host, h->ws + h->carve.ctrl, sizeof host, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return fail(h, LASER_KV_ERR_CUDA, "poll_status: %s", cudaGetErrorString(e));
  h->last_fixups = host[1];
  if (host[0] != 0) {
    cudaMemsetAsync(h->ws + h->carve.ctrl, 0, 4, st);
    cudaMemsetAsync(h->ws + h->carve.dec_count, 0, h->carve.hist - h->carve.dec_count, st);   // a failed decode call may leave counts
    cudaStreamSynchronize(st);
    if (host[0] == LASER_KV_ERR_TIMEOUT) return fail(h, LASER_KV_ERR_TIMEOUT, "a bounded device-side wait gave up");
    if (host[0] == LASER_KV_ERR_CAPACITY)
      return fail(h, LASER_KV_ERR_CAPACITY, "an exact-sign recompute list overflowed (%d items in all, capacity %d per segment)", host[1], h->d.fix_cap);
    return fail(h, (laser_kv_status_t)host[0], "device status word %d", host[0]);
  }
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_reset(laser_kv_handle_t h, int32_t layer) {
  if (!h) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "reset: NULL handle");
  if (layer < -1 || layer >= h->cfg.n_layers) return fail(h, LASER_KV_ERR_INVALID_ARG, "reset: layer out of range");
  if (h->log) fprintf(stderr, "[laser_kv] reset layer %d\n", layer);
  for (int l = 0; l < h->cfg.n_layers; ++l) {
    if (layer != -1 && l != layer) continue;
    h->blocks_done[l] = 0;
    h->entries_done[l] = 0;
    h->tokens_done[l] = 0;
    h->held_back[l] = 0;
    h->sealed[l] = 0;
    h->lookback_done[l] = 0;
  }
  return LASER_KV_OK;
}

void laser_kv_destroy(laser_kv_handle_t h) {
  if (!h) return;
  if (h->log)
    fprintf(stderr, "[laser_kv] destroy: %lld select call(s), %lld block(s), %lld tokens, %lld entries appended\n",
            (long long)h->counters.select_calls, (long long)h->counters.blocks, (long long)h->counters.tokens,
            (long long)h->counters.entries_appended);
  for (auto& set : h->ev_pending) for (cudaEvent_t ev : set) cudaEventDestroy(ev);
  for (cudaEvent_t ev : h->ev_pool) cudaEventDestroy(ev);
  for (cudaEvent_t ev : h->ev_chunk) cudaEventDestroy(ev);
  for (auto& u : h->stage_use) cudaEventDestroy(u.done);
  if (h->ev_join) cudaEventDestroy(h->ev_join);
  if (h->copy_stream) cudaStreamDestroy(h->copy_stream);
  delete h;
}

laser_kv_status_t laser_kv_set_layer_budget(laser_kv_handle_t h, int32_t layer, int32_t budget_per_block) {
  if (!h) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "set_layer_budget: NULL handle");
  if (layer < 0 || layer >= h->cfg.n_layers) return fail(h, LASER_KV_ERR_INVALID_ARG, "set_layer_budget: layer out of range");
  if (budget_per_block < 0 || budget_per_block > h->d.B)
    return fail(h, LASER_KV_ERR_INVALID_ARG, "set_layer_budget: budget %d outside [0, %d] (the configured budget sizes the cache)",
                budget_per_block, h->d.B);
  if (h->blocks_done[layer] != 0)
    return fail(h, LASER_KV_ERR_STATE, "set_layer_budget: layer %d already holds %lld blocks", layer, h->blocks_done[layer]);
  laser_kv_ctx::LayerBudget lb;
  lb.B = budget_per_block;
  int loc;
  laser_kv_partition(lb.B, h->cfg.protection_divisor, h->d.alpha, &lb.anchors, &loc, &lb.k_exact, &lb.k_lsh);
  h->budget[layer] = lb;
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_get_counters(laser_kv_handle_t h, laser_kv_counters_t* out) {
  if (!h || !out) return fail(h, LASER_KV_ERR_INVALID_ARG, "get_counters: NULL argument");
  *out = h->counters;
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_set_wait_budget(laser_kv_handle_t h, uint32_t max_polls) {
  if (!h) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "set_wait_budget: NULL handle");
  h->handoff_polls = max_polls;
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_profile_enable(laser_kv_handle_t h, int32_t on) {
  if (!h) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "profile_enable: NULL handle");
  for (auto& set : h->ev_pending) for (cudaEvent_t ev : set) h->ev_pool.push_back(ev);
  h->ev_pending.clear();
  for (int i = 0; i < kProfKernels; ++i) { h->prof_ms[i] = 0.f; h->prof_launches[i] = 0; }
  h->profiling = on != 0;
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_profile_read(laser_kv_handle_t h, int32_t* n_kernels, const char** names, float* total_ms,
                                        int32_t* launches) {
  if (!h || !n_kernels || !names || !total_ms || !launches)
    return fail(h, LASER_KV_ERR_INVALID_ARG, "profile_read: NULL argument");
  for (auto& set : h->ev_pending) {
    cudaError_t e = cudaEventSynchronize(set.back());
    if (e != cudaSuccess) return fail(h, LASER_KV_ERR_CUDA, "profile_read: %s", cudaGetErrorString(e));
    for (int i = 0; i < kProfKernels; ++i) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, set[i], set[i + 1]) == cudaSuccess) { h->prof_ms[i] += ms; h->prof_launches[i] += 1; }
    }
    for (cudaEvent_t ev : set) h->ev_pool.push_back(ev);
  }
  h->ev_pending.clear();
  *n_kernels = kProfKernels;
  for (int i = 0; i < kProfKernels; ++i) { names[i] = kProfNames[i]; total_ms[i] = h->prof_ms[i]; launches[i] = h->prof_launches[i]; }
  return LASER_KV_OK;
}

const char* laser_kv_status_string(laser_kv_status_t s) {
  switch (s) {
    case LASER_KV_OK: return "ok";
    case LASER_KV_ERR_INVALID_ARG: return "invalid argument";
    case LASER_KV_ERR_UNSUPPORTED: return "unsupported configuration";
    case LASER_KV_ERR_CAPACITY: return "capacity exceeded";
    case LASER_KV_ERR_ALIGNMENT: return "misaligned pointer or stride";
    case LASER_KV_ERR_CUDA: return "CUDA error";
    case LASER_KV_ERR_TIMEOUT: return "device-side wait timed out";
    case LASER_KV_ERR_STATE: return "call sequence error";
  }
  return "unknown status";
}

const char* laser_kv_last_error(laser_kv_handle_t h) { return h ? h->last_error.c_str() : g_last_error.c_str(); }

int64_t laser_kv_launch_count(void) { return g_launches.load(); }

laser_kv_status_t laser_kv_two_stage_topk(const float* s_exact, const uint32_t* counts, int32_t n_segments, int32_t S,
                                          int32_t anchors, int32_t k_exact, int32_t k_lsh, int32_t* idx_out,
                                          void* stream) {
  if (!s_exact || !counts || !idx_out) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "two_stage_topk: NULL argument");
  if (n_segments < 1 || S < 1 || anchors < 0 || k_exact < 0 || k_lsh < 0)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "two_stage_topk: negative or zero size");
  if (2LL * anchors + k_exact + k_lsh > S)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "two_stage_topk: keep count exceeds the segment");
  if (S > 16384) return fail(nullptr, LASER_KV_ERR_UNSUPPORTED, "two_stage_topk: S > 16384");
  if (2 * anchors + k_exact + k_lsh == 0) return LASER_KV_OK;
  const SelectArgs sel{s_exact, counts, idx_out, S, k_exact, k_lsh, 0, anchors, S - anchors, S, 0, 0, anchors, S - anchors, 0};
  return launch_select(sel, n_segments, 0u, static_cast<cudaStream_t>(stream));
}

// ---- window scores on caller-fed inputs ----------------------------------------------------------
namespace {

struct ScoreGeom {
  int batch, H_q, H_kv, S, W, nb, G, GW, tiles_in_block, nseg;
  float scale;
  size_t off_part, off_lse2, total;   // scratch layout: [0,256) status word, partials, lse2
};

laser_kv_status_t score_geometry(int32_t batch, int32_t n_q_heads, int32_t n_kv_heads, int32_t block_size,
                                 int32_t window, int32_t n_blocks, float softmax_scale, ScoreGeom* g) {
  if (batch < 1 || n_q_heads < 1 || n_kv_heads < 1 || block_size < 1 || window < 1 || n_blocks < 1)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "window_scores: sizes must be positive");
  if (n_q_heads % n_kv_heads) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "window_scores: n_q_heads %% n_kv_heads != 0");
  g->batch = batch; g->H_q = n_q_heads; g->H_kv = n_kv_heads; g->S = block_size; g->W = window; g->nb = n_blocks;
  g->G = n_q_heads / n_kv_heads;
  g->GW = g->G * window;
  if (g->GW % 16 || g->GW > 256 || window > 256 || block_size % 8)
    return fail(nullptr, LASER_KV_ERR_UNSUPPORTED, "window_scores: G*W must be a multiple of 16, at most 256; block_size a multiple of 8");
  const long long nseg = (long long)batch * n_kv_heads * n_blocks;
  if (nseg > (1 << 22) || (long long)n_blocks * block_size > 0x7fffffffLL)
    return fail(nullptr, LASER_KV_ERR_UNSUPPORTED, "window_scores: too many segments");
  g->nseg = (int)nseg;
  g->tiles_in_block = (block_size + kTileKeys - 1) / kTileKeys;
  if (softmax_scale < 0.f || softmax_scale != softmax_scale)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "window_scores: softmax_scale must be positive (0 selects 1/sqrt(128))");
  g->scale = softmax_scale == 0.f ? 1.0f / std::sqrt((float)kHeadDim) : softmax_scale;
  g->off_part = 256;
  g->off_lse2 = align_up(g->off_part + lse_part_bytes_bound((size_t)g->nseg, g->GW));
  g->total = align_up(g->off_lse2 + (size_t)g->nseg * g->GW * 4);
  return LASER_KV_OK;
}

EncodeTiledFn driver_encode_fn() {
  static EncodeTiledFn cached = nullptr;
  if (cached) return cached;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  cached = reinterpret_cast<EncodeTiledFn>(fn);
  return cached;
}

// Log-sum-exp pass then score pass, with the partials in `scratch` (device, g.total bytes).
laser_kv_status_t run_window_scores(const ScoreGeom& g, const void* K_blk, const void* Q_win, const int64_t kv_strides[3],
                                    const int64_t q_strides[3], uint8_t* scratch, bool clear_status, float* s_exact_out,
                                    cudaStream_t st) {
  if (!K_blk || !Q_win || !kv_strides || !q_strides || !s_exact_out)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "window_scores: NULL argument");
  if (!aligned16(K_blk) || !aligned16(Q_win) || !aligned16(s_exact_out))
    return fail(nullptr, LASER_KV_ERR_ALIGNMENT, "window_scores: device pointers must be 16-byte aligned");
  for (int i = 0; i < 3; ++i)
    if (kv_strides[i] < 0 || q_strides[i] < 0 || (kv_strides[i] % 8) || (q_strides[i] % 8))
      return fail(nullptr, LASER_KV_ERR_ALIGNMENT, "window_scores: strides must be non-negative multiples of 8 elements");
  if (kv_strides[2] < kHeadDim || q_strides[2] < kHeadDim || (g.H_kv > 1 && !kv_strides[1]) || (g.batch > 1 && !kv_strides[0]) ||
      (g.H_q > 1 && !q_strides[1]) || (g.batch > 1 && !q_strides[0]))
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "window_scores: bad strides");
  EncodeTiledFn enc = driver_encode_fn();
  if (!enc) return fail(nullptr, LASER_KV_ERR_CUDA, "window_scores: cuTensorMapEncodeTiled not available (no CUDA driver?)");
  CUtensorMap mapK, mapQ;
  const cuuint32_t ones[4] = {1, 1, 1, 1};
  {
    const cuuint64_t s_tok = (cuuint64_t)kv_strides[2];
    const cuuint64_t s_head = kv_strides[1] > 0 ? (cuuint64_t)kv_strides[1] : s_tok * (cuuint64_t)g.nb * g.S;
    const cuuint64_t s_batch = kv_strides[0] > 0 ? (cuuint64_t)kv_strides[0] : s_head * (cuuint64_t)g.H_kv;
    const cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)g.nb * g.S, (cuuint64_t)g.H_kv, (cuuint64_t)g.batch};
    const cuuint64_t strides[3] = {s_tok * 2, s_head * 2, s_batch * 2};
    const cuuint32_t box[4] = {(cuuint32_t)kAtomCols, (cuuint32_t)kTileKeys, 1, 1};
    const CUresult r = enc(&mapK, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(K_blk), dims, strides, box, ones,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(nullptr, LASER_KV_ERR_CUDA, "window_scores: tensor map of K failed (CUresult %d)", (int)r);
  }
  {
    const cuuint64_t s_w = (cuuint64_t)q_strides[2];
    const cuuint64_t s_head = q_strides[1] > 0 ? (cuuint64_t)q_strides[1] : s_w * (cuuint64_t)g.W;
    const cuuint64_t s_batch = q_strides[0] > 0 ? (cuuint64_t)q_strides[0] : s_head * (cuuint64_t)g.H_q;
    const cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)g.W, (cuuint64_t)g.H_q, (cuuint64_t)g.batch};
    const cuuint64_t strides[3] = {s_w * 2, s_head * 2, s_batch * 2};
    const cuuint32_t box[4] = {(cuuint32_t)kAtomCols, (cuuint32_t)g.W, (cuuint32_t)g.G, 1};
    const CUresult r = enc(&mapQ, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(Q_win), dims, strides, box, ones,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(nullptr, LASER_KV_ERR_CUDA, "window_scores: tensor map of Q failed (CUresult %d)", (int)r);
  }
  cudaError_t e;
  // caller scratch: the status word must start at zero (the built-in array starts at zero and keeps
  // the first error until it is read); the partials are fully overwritten before they are read
  if (clear_status && (e = cudaMemsetAsync(scratch, 0, 256, st)) != cudaSuccess)
    return fail(nullptr, LASER_KV_ERR_CUDA, "window_scores: memset: %s", cudaGetErrorString(e));
  StreamArgs sa;
  memset(&sa, 0, sizeof sa);
  int dev = 0, num_sms = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess ||
      (e = cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
    return fail(nullptr, LASER_KV_ERR_CUDA, "window_scores: device query: %s", cudaGetErrorString(e));
  sa.S = g.S; sa.S_stride = g.S; sa.nb = g.nb; sa.H_kv = g.H_kv; sa.batch = g.batch;
  sa.G = g.G; sa.W = g.W; sa.GW = g.GW; sa.lse2_stride = g.GW; sa.tiles_in_block = g.tiles_in_block; sa.nseg = g.nseg;
  sa.n_tiles = (long long)g.nseg * g.tiles_in_block;
  const int ctas = stream_grid(sa.n_tiles, num_sms);
  sa.lse_ctas = ctas; sa.n_slot = lse_slots(ctas, g.nseg);
  sa.scale_log2e = g.scale * 1.4426950408889634f;
  sa.lse_part = reinterpret_cast<float2*>(scratch + g.off_part);
  sa.lse2 = reinterpret_cast<float*>(scratch + g.off_lse2);
  sa.s_exact = s_exact_out;
  sa.status = reinterpret_cast<int*>(scratch);
  sa.polls = kMaxPolls; sa.poll_ns = kPollHintNs;
  StreamArgs a1 = sa;
  a1.stat_rows = g.GW;
  a1.stat_rows_alloc = ((g.GW + 127) / 128) * 128;
  if ((e = launch_stream<kLse, 0, 0>(mapK, mapQ, a1, ctas, stream_smem_bytes(kLse, a1.stat_rows_alloc, 0), st)) != cudaSuccess)
    return fail(nullptr, LASER_KV_ERR_CUDA, "window_scores: lse pass: %s", cudaGetErrorString(e));
  StreamArgs a2 = sa;
  a2.stat_rows = g.GW;
  a2.stat_rows_alloc = g.GW;
  if ((e = launch_stream<kScore, 0, 0>(mapK, mapQ, a2, ctas, stream_smem_bytes(kScore, a2.stat_rows_alloc, 0), st)) != cudaSuccess)
    return fail(nullptr, LASER_KV_ERR_CUDA, "window_scores: score pass: %s", cudaGetErrorString(e));
  return LASER_KV_OK;
}

}  // namespace

size_t laser_kv_window_scores_scratch_bytes(int32_t batch, int32_t n_q_heads, int32_t n_kv_heads, int32_t block_size,
                                            int32_t window, int32_t n_blocks) {
  ScoreGeom g;
  if (score_geometry(batch, n_q_heads, n_kv_heads, block_size, window, n_blocks, 0.f, &g) != LASER_KV_OK) return 0;
  return g.total;
}

laser_kv_status_t laser_kv_window_scores(const void* K_blk, const void* Q_win, const int64_t kv_strides[3],
                                         const int64_t q_strides[3], int32_t batch, int32_t n_q_heads, int32_t n_kv_heads,
                                         int32_t block_size, int32_t window, int32_t n_blocks, float softmax_scale,
                                         void* scratch, size_t scratch_bytes, float* s_exact_out, void* stream) {
  ScoreGeom g;
  const laser_kv_status_t s = score_geometry(batch, n_q_heads, n_kv_heads, block_size, window, n_blocks, softmax_scale, &g);
  if (s != LASER_KV_OK) return s;
  if (!scratch) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "window_scores: scratch is NULL");
  if (reinterpret_cast<uintptr_t>(scratch) & (kAlign - 1))
    return fail(nullptr, LASER_KV_ERR_ALIGNMENT, "window_scores: scratch must be 256-byte aligned");
  if (scratch_bytes < g.total)
    return fail(nullptr, LASER_KV_ERR_CAPACITY, "window_scores: scratch needs %zu bytes, got %zu", g.total, scratch_bytes);
  return run_window_scores(g, K_blk, Q_win, kv_strides, q_strides, static_cast<uint8_t*>(scratch), true, s_exact_out,
                           static_cast<cudaStream_t>(stream));
}

// ---- window scores without any allocation ---------------------------------------------------------
// Scratch for laser_kv_window_scores_static: lives in the library's device image, so every GPU
// that loads the library holds these bytes until the process exits.
#define LASER_KV_STATIC_SCRATCH_BYTES (2u << 20)
static __device__ __align__(256) unsigned char g_static_scratch[LASER_KV_STATIC_SCRATCH_BYTES];

namespace {

// In host code the symbol above is only a stand-in; the device address has to be asked for, per
// device, with that device current. Cached after the first successful lookup.
laser_kv_status_t static_scratch_address(uint8_t** out) {
  constexpr int kMaxDevices = 64;
  static std::mutex mu;
  static uint8_t* cached[kMaxDevices] = {nullptr};
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices)
    return fail(nullptr, LASER_KV_ERR_CUDA, "window_scores_static: cudaGetDevice: %s", cudaGetErrorString(e));
  std::lock_guard<std::mutex> lock(mu);
  if (!cached[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p)
      return fail(nullptr, LASER_KV_ERR_CUDA, "window_scores_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
    cached[dev] = static_cast<uint8_t*>(p);
  }
  *out = cached[dev];
  return LASER_KV_OK;
}

}  // namespace

size_t laser_kv_window_scores_static_max_bytes(void) { return LASER_KV_STATIC_SCRATCH_BYTES; }

laser_kv_status_t laser_kv_window_scores_static(const void* K_blk, const void* Q_win, const int64_t kv_strides[3],
                                                const int64_t q_strides[3], int32_t batch, int32_t n_q_heads,
                                                int32_t n_kv_heads, int32_t block_size, int32_t window, int32_t n_blocks,
                                                float softmax_scale, float* s_exact_out, void* stream) {
  ScoreGeom g;
  laser_kv_status_t s = score_geometry(batch, n_q_heads, n_kv_heads, block_size, window, n_blocks, softmax_scale, &g);
  if (s != LASER_KV_OK) return s;
  if (g.total > LASER_KV_STATIC_SCRATCH_BYTES)
    return fail(nullptr, LASER_KV_ERR_CAPACITY,
                "window_scores_static: this problem needs %zu bytes of scratch but the built-in array holds %u; "
                "use laser_kv_window_scores with caller scratch or pass fewer blocks per call",
                g.total, (unsigned)LASER_KV_STATIC_SCRATCH_BYTES);
  uint8_t* scratch = nullptr;
  if ((s = static_scratch_address(&scratch)) != LASER_KV_OK) return s;
  return run_window_scores(g, K_blk, Q_win, kv_strides, q_strides, scratch, false, s_exact_out, static_cast<cudaStream_t>(stream));
}

laser_kv_status_t laser_kv_window_scores_static_status(void* stream) {
  uint8_t* scratch = nullptr;
  const laser_kv_status_t s = static_scratch_address(&scratch);
  if (s != LASER_KV_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int word = 0;
  cudaError_t e = cudaMemcpyAsync(&word, scratch, sizeof word, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return fail(nullptr, LASER_KV_ERR_CUDA, "window_scores_static_status: %s", cudaGetErrorString(e));
  if (word == 0) return LASER_KV_OK;
  e = cudaMemsetAsync(scratch, 0, sizeof word, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return fail(nullptr, LASER_KV_ERR_CUDA, "window_scores_static_status: %s", cudaGetErrorString(e));
  if (word == LASER_KV_ERR_TIMEOUT)
    return fail(nullptr, LASER_KV_ERR_TIMEOUT, "window_scores_static: a bounded device-side wait gave up; the scores of that call are incomplete");
  return fail(nullptr, (laser_kv_status_t)word, "window_scores_static: device status word %d", word);
}

// ---- collision counts on caller-fed inputs ---------------------------------------------------------
namespace {

struct CountGeom {
  ScoreGeom g;
  int K, L, TC, n_chunks, fix_cap;
  size_t off_hist, off_qb, off_fixcnt, off_fix, total;   // scratch layout after the 256-byte control block
};

laser_kv_status_t count_geometry(int32_t batch, int32_t n_q_heads, int32_t n_kv_heads, int32_t block_size, int32_t window,
                                 int32_t n_blocks, int32_t lsh_bits, int32_t lsh_tables, CountGeom* cg) {
  const laser_kv_status_t s = score_geometry(batch, n_q_heads, n_kv_heads, block_size, window, n_blocks, 0.f, &cg->g);
  if (s != LASER_KV_OK) return s;
  if (!(lsh_bits == 4 || lsh_bits == 6 || lsh_bits == 8 || lsh_bits == 10 || lsh_bits == 12) || lsh_tables < 1)
    return fail(nullptr, LASER_KV_ERR_UNSUPPORTED, "collision_counts: lsh_bits must be one of 4, 6, 8, 10, 12");
  cg->K = lsh_bits;
  cg->L = lsh_tables;
  cg->TC = pick_tc(lsh_bits, lsh_tables);
  if (!cg->TC) return fail(nullptr, LASER_KV_ERR_UNSUPPORTED, "collision_counts: lsh_tables must be a multiple of 8");
  if ((long long)cg->g.GW * lsh_tables > 0x7fffffffLL)
    return fail(nullptr, LASER_KV_ERR_UNSUPPORTED, "collision_counts: G*W*lsh_tables too large");
  cg->n_chunks = lsh_tables / cg->TC;
  long long fc = (long long)block_size * lsh_tables / 256;
  if (fc < 256) fc = 256;
  if (fc > (1 << 22)) fc = 1 << 22;
  cg->fix_cap = (int)fc;
  const size_t bh = (size_t)batch * n_kv_heads;
  size_t off = 256;
  cg->off_hist = off; off = align_up(off + bh * lsh_tables * ((size_t)2 << lsh_bits));
  cg->off_qb = off;   off = align_up(off + bh * cg->g.GW * lsh_tables * 2);
  cg->off_fixcnt = off; off = align_up(off + (size_t)cg->g.nseg * sizeof(int));
  cg->off_fix = off;  off = align_up(off + (size_t)cg->g.nseg * cg->fix_cap * sizeof(int4));
  cg->total = off;
  return LASER_KV_OK;
}

bool encode_bf16_map(EncodeTiledFn enc, CUtensorMap* m, const void* ptr, int rank, const cuuint64_t* dims,
                     const cuuint64_t* strides_bytes, const cuuint32_t* box) {
  const cuuint32_t ones[4] = {1, 1, 1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(ptr), dims, strides_bytes, box, ones,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

size_t laser_kv_collision_counts_scratch_bytes(int32_t batch, int32_t n_q_heads, int32_t n_kv_heads, int32_t block_size,
                                               int32_t window, int32_t n_blocks, int32_t lsh_bits, int32_t lsh_tables) {
  CountGeom cg;
  if (count_geometry(batch, n_q_heads, n_kv_heads, block_size, window, n_blocks, lsh_bits, lsh_tables, &cg) != LASER_KV_OK)
    return 0;
  return cg.total;
}

laser_kv_status_t laser_kv_collision_counts(const void* K_blk, const void* Q_win, const void* hyperplanes,
                                            const int64_t kv_strides[3], const int64_t q_strides[3], int32_t batch,
                                            int32_t n_q_heads, int32_t n_kv_heads, int32_t block_size, int32_t window,
                                            int32_t n_blocks, int32_t lsh_bits, int32_t lsh_tables, void* scratch,
                                            size_t scratch_bytes, uint32_t* counts_out, void* stream) {
  CountGeom cg;
  const laser_kv_status_t gs = count_geometry(batch, n_q_heads, n_kv_heads, block_size, window, n_blocks, lsh_bits,
                                              lsh_tables, &cg);
  if (gs != LASER_KV_OK) return gs;
  const ScoreGeom& g = cg.g;
  if (!K_blk || !Q_win || !hyperplanes || !kv_strides || !q_strides || !scratch || !counts_out)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "collision_counts: NULL argument");
  if (!aligned16(K_blk) || !aligned16(Q_win) || !aligned16(hyperplanes) || !aligned16(counts_out) ||
      (reinterpret_cast<uintptr_t>(scratch) & (kAlign - 1)))
    return fail(nullptr, LASER_KV_ERR_ALIGNMENT, "collision_counts: pointers must be 16-byte aligned, scratch 256-byte aligned");
  if (scratch_bytes < cg.total)
    return fail(nullptr, LASER_KV_ERR_CAPACITY, "collision_counts: scratch needs %zu bytes, got %zu", cg.total, scratch_bytes);
  for (int i = 0; i < 3; ++i)
    if (kv_strides[i] < 0 || q_strides[i] < 0 || (kv_strides[i] % 8) || (q_strides[i] % 8))
      return fail(nullptr, LASER_KV_ERR_ALIGNMENT, "collision_counts: strides must be non-negative multiples of 8 elements");
  if (kv_strides[2] < kHeadDim || q_strides[2] < kHeadDim || (g.H_kv > 1 && !kv_strides[1]) || (g.batch > 1 && !kv_strides[0]) ||
      (g.H_q > 1 && !q_strides[1]) || (g.batch > 1 && !q_strides[0]))
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "collision_counts: bad strides");
  EncodeTiledFn enc = driver_encode_fn();
  if (!enc) return fail(nullptr, LASER_KV_ERR_CUDA, "collision_counts: cuTensorMapEncodeTiled not available (no CUDA driver?)");
  CUtensorMap mapK, mapQ, mapP, mapPq;
  {
    const cuuint64_t s_tok = (cuuint64_t)kv_strides[2];
    const cuuint64_t s_head = kv_strides[1] > 0 ? (cuuint64_t)kv_strides[1] : s_tok * (cuuint64_t)g.nb * g.S;
    const cuuint64_t s_batch = kv_strides[0] > 0 ? (cuuint64_t)kv_strides[0] : s_head * (cuuint64_t)g.H_kv;
    const cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)g.nb * g.S, (cuuint64_t)g.H_kv, (cuuint64_t)g.batch};
    const cuuint64_t strides[3] = {s_tok * 2, s_head * 2, s_batch * 2};
    const cuuint32_t box[4] = {(cuuint32_t)kAtomCols, (cuuint32_t)kTileKeys, 1, 1};
    const cuuint64_t s_w = (cuuint64_t)q_strides[2];
    const cuuint64_t q_head = q_strides[1] > 0 ? (cuuint64_t)q_strides[1] : s_w * (cuuint64_t)g.W;
    const cuuint64_t q_batch = q_strides[0] > 0 ? (cuuint64_t)q_strides[0] : q_head * (cuuint64_t)g.H_q;
    const cuuint64_t qdims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)g.W, (cuuint64_t)g.H_q, (cuuint64_t)g.batch};
    const cuuint64_t qstrides[3] = {s_w * 2, q_head * 2, q_batch * 2};
    const cuuint32_t qbox[4] = {(cuuint32_t)kAtomCols, (cuuint32_t)g.W, (cuuint32_t)g.G, 1};
    const cuuint64_t pdims[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)lsh_tables * lsh_bits};
    const cuuint64_t pstrides[1] = {(cuuint64_t)kHeadDim * 2};
    const cuuint32_t pbox[2] = {(cuuint32_t)kAtomCols, (cuuint32_t)(cg.TC * lsh_bits)};
    const cuuint32_t pqbox[2] = {(cuuint32_t)kAtomCols, (cuuint32_t)(kQsigTables * lsh_bits)};
    if (!encode_bf16_map(enc, &mapK, K_blk, 4, dims, strides, box) || !encode_bf16_map(enc, &mapQ, Q_win, 4, qdims, qstrides, qbox) ||
        !encode_bf16_map(enc, &mapP, hyperplanes, 2, pdims, pstrides, pbox) ||
        !encode_bf16_map(enc, &mapPq, hyperplanes, 2, pdims, pstrides, pqbox))
      return fail(nullptr, LASER_KV_ERR_CUDA, "collision_counts: cuTensorMapEncodeTiled failed");
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e;
  int dev = 0, num_sms = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess ||
      (e = cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
    return fail(nullptr, LASER_KV_ERR_CUDA, "collision_counts: device query: %s", cudaGetErrorString(e));
  uint8_t* sc = static_cast<uint8_t*>(scratch);
  int* ctrl = reinterpret_cast<int*>(sc);
  uint16_t* hist = reinterpret_cast<uint16_t*>(sc + cg.off_hist);
  uint16_t* qb = reinterpret_cast<uint16_t*>(sc + cg.off_qb);
  int4* fix_items = reinterpret_cast<int4*>(sc + cg.off_fix);
  int* fix_counts = reinterpret_cast<int*>(sc + cg.off_fixcnt);
  // the status word must start at zero; the query-signature kernel restarts the other counters
  if ((e = cudaMemsetAsync(sc, 0, 256, st)) != cudaSuccess)
    return fail(nullptr, LASER_KV_ERR_CUDA, "collision_counts: memset: %s", cudaGetErrorString(e));
  const uint16_t* P = static_cast<const uint16_t*>(hyperplanes);
  {
    const int q_alloc = ((g.GW + 127) / 128) * 128;
    QsigArgs qa{static_cast<const uint16_t*>(Q_win), q_strides[0], q_strides[1], q_strides[2], P, hist, qb,
                g.H_kv, g.G, g.W, g.GW, q_alloc, lsh_tables,
                reinterpret_cast<uint4*>(counts_out), (long long)g.nseg * g.S / 4, ctrl + 1, fix_counts, g.nseg, ctrl,
                lsh_tables, 0, 0, g.GW, 1};
    dim3 grid(lsh_tables / kQsigTables, g.H_kv, g.batch);
    if ((e = launch_qsig(lsh_bits, mapQ, mapPq, qa, grid, qsig_smem_bytes(q_alloc, lsh_bits), st)) != cudaSuccess)
      return fail(nullptr, LASER_KV_ERR_CUDA, "collision_counts: qsig_kernel: %s", cudaGetErrorString(e));
  }
  {
    StreamArgs sa;
    memset(&sa, 0, sizeof sa);
    sa.S = g.S; sa.S_stride = g.S; sa.nb = g.nb; sa.H_kv = g.H_kv; sa.batch = g.batch;
    sa.G = g.G; sa.W = g.W; sa.GW = g.GW; sa.tiles_in_block = g.tiles_in_block; sa.nseg = g.nseg;
    sa.n_chunks = cg.n_chunks; sa.tables_per_chunk = cg.TC; sa.lsh_bits = lsh_bits; sa.lsh_tables = lsh_tables;
    sa.n_tiles = (long long)g.nseg * g.tiles_in_block * cg.n_chunks;
    sa.stat_rows = cg.TC * lsh_bits; sa.stat_rows_alloc = sa.stat_rows;
    sa.counts = counts_out; sa.hist = hist; sa.fix_items = fix_items; sa.fix_count = fix_counts; sa.fix_cap = cg.fix_cap;
    sa.status = ctrl;
    sa.polls = kMaxPolls; sa.poll_ns = kPollHintNs;
    const uint32_t smem = stream_smem_bytes(kProj, sa.stat_rows_alloc, cg.TC * (2 << lsh_bits));
    if ((e = launch_proj(lsh_bits, cg.TC, mapK, mapP, sa, stream_grid(sa.n_tiles, num_sms), smem, st)) != cudaSuccess)
      return fail(nullptr, LASER_KV_ERR_CUDA, "collision_counts: projection pass: %s", cudaGetErrorString(e));
  }
  {
    SignfixArgs fa{static_cast<const uint16_t*>(K_blk), kv_strides[0], kv_strides[1], kv_strides[2], P, hist, counts_out,
                   nullptr, fix_items, fix_counts, cg.fix_cap, g.H_kv, g.nb, g.S, lsh_bits, lsh_tables, ctrl + 2, g.S, ctrl + 1};
    signfix_kernel<<<dim3(kSignfixCtasPerSeg, g.nseg), 256, 0, st>>>(fa);
    g_launches.fetch_add(1);
    if ((e = cudaGetLastError()) != cudaSuccess)
      return fail(nullptr, LASER_KV_ERR_CUDA, "collision_counts: signfix_kernel: %s", cudaGetErrorString(e));
  }
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_collision_probability(const void* K_blk, const void* Q_win, const int64_t kv_strides[3],
                                                 const int64_t q_strides[3], int32_t batch, int32_t n_q_heads,
                                                 int32_t n_kv_heads, int32_t block_size, int32_t window, int32_t n_blocks,
                                                 int32_t lsh_bits, void* scratch, size_t scratch_bytes, float* p_out,
                                                 void* stream) {
  if (!K_blk || !Q_win || !kv_strides || !q_strides || !p_out || !scratch)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "collision_probability: NULL argument");
  if (batch < 1 || n_q_heads < 1 || n_kv_heads < 1 || block_size < 1 || window < 1 || n_blocks < 1)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "collision_probability: sizes must be positive");
  if (n_q_heads % n_kv_heads) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "collision_probability: n_q_heads %% n_kv_heads != 0");
  if (lsh_bits < 1 || lsh_bits > 64) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "collision_probability: lsh_bits must be in [1, 64]");
  const int G = n_q_heads / n_kv_heads, GW = G * window;
  if (GW % 16 || GW > 256 || window > 256 || G > 256 || block_size % 8)
    return fail(nullptr, LASER_KV_ERR_UNSUPPORTED,
                "collision_probability: G*W must be a multiple of 16, at most 256; block_size a multiple of 8");
  if ((long long)n_blocks * block_size > 0x7fffffffLL || (long long)n_kv_heads * n_blocks > 65535 || batch > 65535)
    return fail(nullptr, LASER_KV_ERR_UNSUPPORTED, "collision_probability: too many segments");
  if (!aligned16(K_blk) || !aligned16(Q_win) || !aligned16(p_out) || !aligned16(scratch))
    return fail(nullptr, LASER_KV_ERR_ALIGNMENT, "collision_probability: device pointers must be 16-byte aligned");
  if (scratch_bytes < 256) return fail(nullptr, LASER_KV_ERR_CAPACITY, "collision_probability: scratch needs 256 bytes");
  for (int i = 0; i < 3; ++i)
    if (kv_strides[i] < 0 || q_strides[i] < 0 || (kv_strides[i] % 8) || (q_strides[i] % 8))
      return fail(nullptr, LASER_KV_ERR_ALIGNMENT, "collision_probability: strides must be non-negative multiples of 8 elements");
  if (kv_strides[2] < kHeadDim || q_strides[2] < kHeadDim || (n_kv_heads > 1 && !kv_strides[1]) || (batch > 1 && !kv_strides[0]) ||
      (n_q_heads > 1 && !q_strides[1]) || (batch > 1 && !q_strides[0]))
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "collision_probability: bad strides");
  EncodeTiledFn enc = driver_encode_fn();
  if (!enc) return fail(nullptr, LASER_KV_ERR_CUDA, "collision_probability: cuTensorMapEncodeTiled not available (no CUDA driver?)");
  CUtensorMap mapK, mapQ;
  {
    const cuuint64_t s_tok = (cuuint64_t)kv_strides[2];
    const cuuint64_t s_head = kv_strides[1] > 0 ? (cuuint64_t)kv_strides[1] : s_tok * (cuuint64_t)n_blocks * block_size;
    const cuuint64_t s_batch = kv_strides[0] > 0 ? (cuuint64_t)kv_strides[0] : s_head * (cuuint64_t)n_kv_heads;
    const cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)n_blocks * block_size, (cuuint64_t)n_kv_heads, (cuuint64_t)batch};
    const cuuint64_t strides[3] = {s_tok * 2, s_head * 2, s_batch * 2};
    const cuuint32_t box[4] = {(cuuint32_t)kAtomCols, (cuuint32_t)kTileKeys, 1, 1};
    const cuuint64_t s_w = (cuuint64_t)q_strides[2];
    const cuuint64_t q_head = q_strides[1] > 0 ? (cuuint64_t)q_strides[1] : s_w * (cuuint64_t)window;
    const cuuint64_t q_batch = q_strides[0] > 0 ? (cuuint64_t)q_strides[0] : q_head * (cuuint64_t)n_q_heads;
    const cuuint64_t qdims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)window, (cuuint64_t)n_q_heads, (cuuint64_t)batch};
    const cuuint64_t qstrides[3] = {s_w * 2, q_head * 2, q_batch * 2};
    const cuuint32_t qbox[4] = {(cuuint32_t)kAtomCols, (cuuint32_t)window, (cuuint32_t)G, 1};
    if (!encode_bf16_map(enc, &mapK, K_blk, 4, dims, strides, box) || !encode_bf16_map(enc, &mapQ, Q_win, 4, qdims, qstrides, qbox))
      return fail(nullptr, LASER_KV_ERR_CUDA, "collision_probability: cuTensorMapEncodeTiled failed");
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e;
  if ((e = cudaMemsetAsync(scratch, 0, 256, st)) != cudaSuccess)
    return fail(nullptr, LASER_KV_ERR_CUDA, "collision_probability: memset: %s", cudaGetErrorString(e));
  int dev = 0, num_sms = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess ||
      (e = cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
    return fail(nullptr, LASER_KV_ERR_CUDA, "collision_probability: device query: %s", cudaGetErrorString(e));
  StreamArgs sa;
  memset(&sa, 0, sizeof sa);
  sa.S = block_size; sa.S_stride = block_size; sa.nb = n_blocks; sa.H_kv = n_kv_heads; sa.batch = batch;
  sa.G = G; sa.W = window; sa.GW = GW;
  sa.tiles_in_block = (block_size + kTileKeys - 1) / kTileKeys;
  sa.nseg = batch * n_kv_heads * n_blocks;
  sa.n_tiles = (long long)sa.nseg * sa.tiles_in_block;
  sa.stat_rows = GW; sa.stat_rows_alloc = GW;
  sa.lsh_bits = lsh_bits;
  sa.s_exact = p_out;
  sa.status = static_cast<int*>(scratch);
  sa.polls = kMaxPolls; sa.poll_ns = kPollHintNs;
  const int ctas = stream_grid(sa.n_tiles, num_sms);
  const uint32_t smem = stream_smem_bytes(kTheory, sa.stat_rows_alloc, 0);
  switch (lsh_bits) {                    // the usual table widths get the multiplication form of u^K
    case 4: e = launch_stream<kTheory, 4, 0>(mapK, mapQ, sa, ctas, smem, st); break;
    case 6: e = launch_stream<kTheory, 6, 0>(mapK, mapQ, sa, ctas, smem, st); break;
    case 8: e = launch_stream<kTheory, 8, 0>(mapK, mapQ, sa, ctas, smem, st); break;
    case 10: e = launch_stream<kTheory, 10, 0>(mapK, mapQ, sa, ctas, smem, st); break;
    case 12: e = launch_stream<kTheory, 12, 0>(mapK, mapQ, sa, ctas, smem, st); break;
    default: e = launch_stream<kTheory, 0, 0>(mapK, mapQ, sa, ctas, smem, st); break;
  }
  if (e != cudaSuccess) return fail(nullptr, LASER_KV_ERR_CUDA, "collision_probability: launch: %s", cudaGetErrorString(e));
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_consensus_accumulate(const float* s_exact, const uint32_t* counts, int32_t batch,
                                                int32_t n_heads, int32_t n_blocks, int32_t block_size, int32_t carry,
                                                float* s_acc, uint32_t* c_acc, void* stream) {
  if (!s_exact || !counts || !s_acc || !c_acc) return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "consensus_accumulate: NULL argument");
  if (batch < 1 || n_heads < 1 || n_blocks < 1 || block_size < 1 || (block_size % 4))
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "consensus_accumulate: sizes must be positive, block_size a multiple of 4");
  if (!aligned16(s_exact) || !aligned16(counts) || !aligned16(s_acc) || !aligned16(c_acc))
    return fail(nullptr, LASER_KV_ERR_ALIGNMENT, "consensus_accumulate: pointers must be 16-byte aligned");
  const long long n4 = (long long)n_blocks * block_size / 4;
  ConsensusArgs a{reinterpret_cast<const float4*>(s_exact), reinterpret_cast<const uint4*>(counts),
                  reinterpret_cast<float4*>(s_acc), reinterpret_cast<uint4*>(c_acc), n4, batch, n_heads, carry ? 1 : 0};
  const long long total = (long long)batch * n4;
  long long blocks = (total + 255) / 256;
  if (blocks > 148 * 8) blocks = 148 * 8;
  consensus_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(a);
  g_launches.fetch_add(1);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(nullptr, LASER_KV_ERR_CUDA, "consensus_kernel launch: %s", cudaGetErrorString(e));
  return LASER_KV_OK;
}

laser_kv_status_t laser_kv_gather_append(const void* K_src, const void* V_src, int64_t src_seg_stride,
                                         int64_t src_row_stride, int32_t n_src_rows, const int32_t* idx,
                                         int32_t n_segments, int32_t n_keep, void* K_dst, void* V_dst,
                                         int64_t dst_seg_stride, int64_t dst_capacity, int32_t* pos_out,
                                         int64_t pos_seg_stride, int64_t dst_offset, int32_t pos_base, int32_t* status,
                                         void* stream) {
  if (!K_src || !V_src || !idx || !K_dst || !V_dst || !pos_out || !status)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "gather_append: NULL argument");
  if (n_segments < 1 || n_keep < 0 || dst_offset < 0 || n_src_rows < 0 || dst_capacity < 0)
    return fail(nullptr, LASER_KV_ERR_INVALID_ARG, "gather_append: bad size");
  if (dst_offset + (int64_t)n_keep > dst_capacity)
    return fail(nullptr, LASER_KV_ERR_CAPACITY, "gather_append: entries [%lld, %lld) do not fit a destination of %lld entries",
                (long long)dst_offset, (long long)dst_offset + n_keep, (long long)dst_capacity);
  if (!aligned16(K_src) || !aligned16(V_src) || !aligned16(K_dst) || !aligned16(V_dst) || (src_seg_stride % 8) ||
      (src_row_stride % 8) || (dst_seg_stride % 8) || (reinterpret_cast<uintptr_t>(status) & 3u))
    return fail(nullptr, LASER_KV_ERR_ALIGNMENT, "gather_append: pointers 16-byte aligned, strides multiples of 8");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const cudaError_t e = cudaMemsetAsync(status, 0, sizeof(int32_t), st);
  if (e != cudaSuccess) return fail(nullptr, LASER_KV_ERR_CUDA, "gather_append: memset: %s", cudaGetErrorString(e));
  AppendArgs aa{static_cast<const uint16_t*>(K_src), static_cast<const uint16_t*>(V_src), src_seg_stride, 0,
                src_row_stride, 1, 1, 0, n_keep, idx, static_cast<uint16_t*>(K_dst), static_cast<uint16_t*>(V_dst),
                pos_out, dst_seg_stride, pos_seg_stride, dst_offset, pos_base, n_src_rows, status};
  return launch_append(aa, n_segments, st);
}

}  // extern "C"
