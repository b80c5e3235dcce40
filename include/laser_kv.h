/*
 * laser_kv.h - C ABI of the B200 (sm_100a) implementation of LASER-KV's prefill-time token
 * selection: for every block of a long context, score the block's keys against the
 * observation-window queries, hash keys and queries with SimHash and count collisions, run the
 * paper's two-stage Exact-LSH top-k per KV head with the keep count fixed by the protection
 * divisor n, and append the selected K/V rows to an append-only per-layer cache.
 *
 * Conventions for every entry point
 *   - Returns a laser_kv_status_t (0 = success) unless stated otherwise; never throws or aborts.
 *   - "dev" pointers are CUDA device pointers on the handle's device; "host" pointers are
 *     ordinary host memory. All tensors are bfloat16 bit patterns (uint16) unless stated.
 *   - The caller owns every device buffer (inputs, hyperplanes, cache, workspace). The library
 *     owns only the host-side handle. No entry point in this header's main section allocates
 *     device memory.
 *   - Device pointers must be 16-byte aligned, strides multiples of 8 elements
 *     (LASER_KV_ERR_ALIGNMENT otherwise).
 *   - Kernel launches are asynchronous on the caller's stream; nothing is copied back to the
 *     host unless the entry point says so.
 *   - Kernels launch on the calling thread's current device. laser_kv_init makes the handle's device
 *     current; a later handle call made while another device is current fails with
 *     LASER_KV_ERR_STATE. The handle-free step-level entry points run on the current device.
 *   - There is no CPU fallback: without a CUDA device laser_kv_init fails with LASER_KV_ERR_CUDA.
 */
#ifndef LASER_KV_H_
#define LASER_KV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct laser_kv_ctx* laser_kv_handle_t;

typedef enum {
  LASER_KV_OK = 0,
  LASER_KV_ERR_INVALID_ARG = 1,   /* null pointer, out-of-range value, inconsistent config    */
  LASER_KV_ERR_UNSUPPORTED = 2,   /* valid by the paper but outside what the kernels handle   */
  LASER_KV_ERR_CAPACITY = 3,      /* cache or workspace too small; nothing was written        */
  LASER_KV_ERR_ALIGNMENT = 4,     /* pointer or stride alignment                              */
  LASER_KV_ERR_CUDA = 5,          /* a CUDA runtime/driver call failed (see last_error)       */
  LASER_KV_ERR_TIMEOUT = 6,       /* a bounded device-side wait gave up (status word)         */
  LASER_KV_ERR_STATE = 7          /* call sequence error (e.g. debug view before any call)    */
} laser_kv_status_t;

/* One configuration per handle. Zero-initialise, then fill. */
typedef struct {
  int32_t n_layers;            /* independent per-layer caches                                   */
  int32_t batch;               /* independent sequences processed together by each call          */
  int32_t n_q_heads;           /* H_q                                                            */
  int32_t n_kv_heads;          /* H_kv; H_q % H_kv == 0; G = H_q / H_kv (GQA group)              */
  int32_t head_dim;            /* d; must be 128                                                 */
  int32_t block_size;          /* S: tokens per block (Section 3.2); multiple of 8               */
  int32_t window;              /* W: observation-window queries per query head; G*W a multiple of
                                  16; above 256 the group's queries are scored in 2..4 equal parts of
                                  window positions (W divisible by the number of parts, every part a
                                  multiple of 16 queries), up to G*W = 1024                       */
  int32_t max_blocks;          /* cache capacity per (layer, sequence, KV head) = max_blocks * B */
  int32_t max_blocks_per_call; /* upper bound on n_blocks of one select call (sizes workspace)   */
  int32_t lsh_bits;            /* K: sign bits per SimHash table, 1..12                           */
  int32_t lsh_tables;          /* L: tables (the paper's R hash rounds), any positive number      */
  int32_t protection_divisor;  /* n >= 2 (Section 3.1)                                           */
  int32_t budget_per_block;    /* B; 0 => Eq. 1 from ratio, block_size and context_len           */
  int32_t debug;               /* nonzero: also keep per-key bucket ids for laser_kv_debug_view,
                                  and compute both stages even when one has no picks to make
                                  (alpha = 1, alpha = 0, n = 2); zero: a stage without picks is
                                  skipped and its debug arrays are not refreshed               */
  int64_t context_len;         /* L of Eq. 1 (only read when budget_per_block == 0)              */
  double  ratio;               /* r of Eq. 1; 0 => 0.25                                          */
  double  alpha;               /* exact share of the recall budget; negative => 0.75             */
  float   softmax_scale;       /* 0 => 1/sqrt(head_dim)                                          */
  int32_t device;              /* CUDA device ordinal                                            */
  int32_t lookback;            /* 0: every block keeps its own local window (Section 3.1 alone);
                                  1: look-back boundary smoothing (Section 3.2), see
                                  laser_kv_select_block                                           */
} laser_kv_config_t;

/* Views returned by laser_kv_cache_view: entries [0, len) of every (sequence, KV head) are
 * final and never change again (append-only memory, Sections 1 and 3). Strides in elements. */
typedef struct {
  void*    K;                  /* dev bf16 [batch][H_kv][cap][d]                                 */
  void*    V;                  /* dev bf16 [batch][H_kv][cap][d]                                 */
  int32_t* pos;                /* dev int32 [batch][H_kv][cap]: absolute token positions         */
  int64_t  len;                /* entries valid per (sequence, KV head); the same for all        */
  int64_t  cap;                /* capacity per (sequence, KV head)                               */
  int64_t  kv_strides[3];      /* batch, head, entry strides of K and V (last dim contiguous)    */
  int64_t  pos_strides[2];     /* batch, head strides of pos                                     */
} laser_kv_view_t;

/* Intermediate results of the most recent select call (pointers into the workspace, valid
 * until the next select call). nb = that call's n_blocks; GW = G*W. A bucket code packs a table's
 * K sign bits with the table's first hyperplane as the most significant bit:
 * code = sum_b [<p_{r*K+b}, x> >= 0] << (K-1-b). hist is indexed by that code.
 * The kernels work on an even number (>= 4) of bits per table and on tables in groups of eight;
 * other shapes run on a padded copy of the hyperplanes kept in the workspace (a missing bit repeats
 * the table's first hyperplane, so bucket equality is unchanged; a missing table repeats table 0
 * with an empty query histogram, so it adds no collision). The arrays below have the padded shape:
 * lsh_bits / lsh_tables of this struct are K' = even(max(K, 4)) and L' = 8*ceil(L/8), the first K
 * bits (from the top) of a K'-bit code and the first L tables are the configured ones. */
typedef struct {
  const float*    s_exact;       /* dev fp32  [batch][H_kv][nb][S]   summed window attention     */
  const uint32_t* counts;        /* dev u32   [batch][H_kv][nb][S]   collision counts            */
  const float*    lse2;          /* dev fp32  [batch][H_kv][nb][GW]  log2-sum-exp2 per query     */
  const uint16_t* query_buckets; /* dev u16   [batch][H_kv][GW][L]                               */
  const uint16_t* key_buckets;   /* dev u16   [batch][H_kv][nb][S][L]; NULL unless config.debug  */
  const uint16_t* hist;          /* dev u16   [batch][H_kv][L][2^K]  query-bucket histogram      */
  const int32_t*  idx;           /* dev int32 [batch][H_kv][nb][B]   kept block-local indices    */
  int32_t n_blocks, batch, n_kv_heads, block_size, budget, gw, lsh_tables, lsh_bits;
  int32_t n_sign_fixups;         /* host: near-zero projections recomputed exactly (last poll)   */
  int32_t segment_keys;          /* scored keys per segment: the "S" of the arrays above; block_size,
                                    or block_size + floor(B/n) for the later blocks under look-back */
  int32_t segment_shift;         /* scored key 0 is this many tokens before the block's first token
                                    (0, or floor(B/n) for the later blocks under look-back)        */
  int32_t window_part;           /* W' = W / parts: a group of more than 256 window queries is scored
                                    in up to four parts of W' window positions each; the GW rows of
                                    lse2 and query_buckets are ordered (part, head of the group,
                                    position within the part), which is (head, position) when W' = W */
} laser_kv_debug_t;

/* Appendix B, Eq. 1: B = floor(2 r S_block L / (S_block + L)) evaluated in IEEE double.
 * Returns B, or -1 for non-positive arguments. Host only. */
int32_t laser_kv_budget(int64_t context_len, int32_t block_size, double ratio);

/* Section 3.1 and Algorithm 1 lines 4/7: anchors = local = floor(B/n); recall budget
 * B_long = B - 2*floor(B/n); k_exact = floor(alpha * B_long) (double); k_lsh = B_long - k_exact.
 * Any output pointer may be NULL. n < 2, B < 0 or alpha outside [0,1] => INVALID_ARG. Host only. */
laser_kv_status_t laser_kv_partition(int32_t B, int32_t n, double alpha, int32_t* anchors,
                                     int32_t* local, int32_t* k_exact, int32_t* k_lsh);

/* Bytes the caller must provide for the cache and the workspace of a configuration.
 * Host only; validates the configuration. */
laser_kv_status_t laser_kv_query_sizes(const laser_kv_config_t* cfg, size_t* cache_bytes,
                                       size_t* workspace_bytes);

/* Creates a handle. hyperplanes: dev bf16 [L*K][d], row r*K + b = bit b of table r (Section 3.3,
 * the hash functions h_r taken as K-bit SimHash); read by every later call, owned by the caller.
 * cache_mem / workspace: dev buffers of at least the sizes laser_kv_query_sizes reports, 256-byte
 * aligned, owned by the caller and used until laser_kv_destroy. The cache need not be cleared. */
laser_kv_status_t laser_kv_init(const laser_kv_config_t* cfg, const void* hyperplanes,
                                void* cache_mem, size_t cache_bytes, void* workspace,
                                size_t workspace_bytes, laser_kv_handle_t* out);

/* The hot path (Algorithm 1 on each block, then append): processes n_blocks consecutive blocks
 * of one layer for all `batch` sequences.
 *   K_blk, V_blk : dev bf16 [batch][H_kv][n_blocks*S][d] addressed through kv_strides =
 *                  {batch, head, token} strides in elements (last dim contiguous); block i of
 *                  this call occupies tokens [i*S, (i+1)*S).
 *   Q_win        : dev bf16 [batch][H_q][W][d] through q_strides = {batch, head, query}; the
 *                  same window scores every block of the call; query head h*G+g belongs to KV
 *                  head h.
 * Per block and KV head it keeps exactly B tokens: the first and last floor(B/n) of the block,
 * the k_exact candidates with the largest summed attention probability, and the k_lsh remaining
 * candidates with the most SimHash collisions (ties: lower index). Rows are appended in
 * ascending position at [len, len + n_blocks*B); len advances on the host. The blocks' absolute
 * positions continue from the blocks already appended to this layer.
 * With config.lookback = 1 (Section 3.2: the scoring window of block t is expanded to include the
 * tail of block t-1, so that tokens at a block's edge are judged with the context that follows them)
 * the local window slides instead of being kept block by block. With a = floor(B/n):
 *   - the first block of a sequence keeps its a anchors and Algorithm 1's picks from [a, S - a) with
 *     the recall budget B - 2a; its last a tokens are held back (B - a entries appended);
 *   - every later block scores the held-back a tokens of the previous block together with its own S
 *     keys (one softmax over a + S keys, one collision count each), keeps its a anchors, and runs
 *     Algorithm 1 on the held-back tokens plus [a, S - a) of the block with recall budget B - a
 *     (k_exact = floor(alpha * (B - a))); its own last a tokens are held back in turn (B entries
 *     appended, ascending positions);
 *   - laser_kv_lookback_close appends the tail of the last block. The cache then holds B entries per
 *     block, as without look-back.
 * The held-back tokens are not stored by the library: for every block but the first of the sequence
 * the a rows before K_blk / V_blk (same strides) must be the previous block's last a tokens, i.e. the
 * pointers must point into a buffer that holds the context contiguously. laser_kv_select_block_host
 * does not support look-back. laser_kv_debug_view then describes the last pass only (the first block
 * of a sequence is a pass of its own).
 * A handle's workspace serves one call at a time: calls on the same handle must be issued to one
 * stream (or be ordered by the caller); concurrent streams need one handle each.
 * Inside a call some kernels are launched so that they may start before the kernel ahead of them
 * has drained (programmatic stream serialization, where a kernel does not read that kernel's
 * results). Towards everything else on the stream the call behaves as ordinary launches do: its
 * first kernel starts after all earlier work, and work queued after the call starts after all of it.
 * Errors: CAPACITY if the cache cannot take n_blocks more blocks or n_blocks exceeds
 * max_blocks_per_call (nothing is launched). */
laser_kv_status_t laser_kv_select_block(laser_kv_handle_t h, int32_t layer, const void* K_blk,
                                        const void* V_blk, const void* Q_win,
                                        const int64_t kv_strides[3], const int64_t q_strides[3],
                                        int32_t n_blocks, void* stream);

/* A last block that has fewer tokens than block_size (the paper's contexts are whole numbers of
 * blocks; reading taken here: the same rule on the tokens there are). n_tokens in [1, block_size)
 * tokens at K_blk / V_blk (same layout and strides as laser_kv_select_block, one block) are scored
 * against Q_win and selected with the budget B_t = min(B, n_tokens): anchors and local window
 * floor(B_t/n) each, recall budget B_t - 2*floor(B_t/n) split by alpha; a block with no more tokens
 * than B keeps all of them. B_t entries are appended (under look-back the block's last floor(B_t/n)
 * tokens are held back for laser_kv_lookback_close like any block's, and the previous block's
 * held-back tokens are decided here). Afterwards the layer accepts no further block until
 * laser_kv_reset (positions would no longer be those of whole blocks). */
laser_kv_status_t laser_kv_select_tail(laser_kv_handle_t h, int32_t layer, const void* K_blk,
                                       const void* V_blk, const void* Q_win,
                                       const int64_t kv_strides[3], const int64_t q_strides[3],
                                       int32_t n_tokens, void* stream);

/* Closes a look-back sequence (config.lookback = 1): appends the a = floor(B/n) tokens that the last
 * block held back - nothing follows them, so nothing can prune them. K_tail / V_tail: dev bf16
 * [batch][H_kv][a][d] through kv_strides, the last a rows of the last block (same strides as the
 * block; a = floor(B_t/n) of that block's own budget when it was a short one). Afterwards the layer accepts no block until laser_kv_reset. STATE if the
 * handle has no look-back, the layer holds no block or is closed already. */
laser_kv_status_t laser_kv_lookback_close(laser_kv_handle_t h, int32_t layer, const void* K_tail,
                                          const void* V_tail, const int64_t kv_strides[3], void* stream);

/* Same path driven from HOST memory: copies the (contiguous) host tensors K_host, V_host
 * [batch][H_kv][n_blocks*S][d] and Q_host [batch][H_q][W][d] into the caller's device staging
 * buffers K_stage, V_stage, Q_stage (same shapes), runs laser_kv_select_block on them, and
 * copies the appended positions (int32 [batch][H_kv][n_blocks*B]) to pos_out_host. The blocks
 * travel in up to four chunks on a copy stream that the handle owns, ordered after the work
 * already on `stream`; the selection of a chunk runs on `stream` once the chunk has landed, while
 * the next chunk is copied. Only the kept rows of V are ever read: when V_host is page-locked
 * memory that the device can address (cudaHostAlloc / cudaHostRegister), the append kernel reads
 * those rows in place over the bus and V_stage stays untouched; pageable V_host is copied like
 * K_host. Everything the call does is complete when `stream` is (pin the host buffers, or the
 * copies serialise); the host buffers must stay valid until then; the call does not synchronise.
 * The copies of a call wait for the previous host-path call of this handle that used the same
 * staging buffers (and, for buffers the handle has not seen, for everything already on `stream`):
 * a caller who alternates between two sets of staging buffers gets the next call's copies running
 * under the tail of the previous call. The staging buffers belong to the call until `stream` has
 * passed it; any other work of the caller that touches them must be ordered against the host-path
 * calls by the caller. pos_out_host may be NULL. If the call fails after some chunks were launched,
 * those chunks' blocks stay appended (laser_kv_cache_view's len tells how many) and the rest are
 * not. */
laser_kv_status_t laser_kv_select_block_host(laser_kv_handle_t h, int32_t layer,
                                             const void* K_host, const void* V_host,
                                             const void* Q_host, void* K_stage, void* V_stage,
                                             void* Q_stage, int32_t n_blocks,
                                             int32_t* pos_out_host, void* stream);

/* Current view of one layer's cache. Host only (no synchronisation: pending kernels on the
 * caller's stream may still be writing entries counted in len). */
laser_kv_status_t laser_kv_cache_view(laser_kv_handle_t h, int32_t layer, laser_kv_view_t* out);

/* Pointers to the last call's intermediates; STATE before the first select call. */
laser_kv_status_t laser_kv_debug_view(laser_kv_handle_t h, laser_kv_debug_t* out);

/* Synchronises `stream`, reads the device status word and returns OK or the first error a
 * kernel recorded (TIMEOUT for a bounded wait that gave up, CAPACITY if the exact-sign
 * recompute list overflowed). Clears the word. */
laser_kv_status_t laser_kv_poll_status(laser_kv_handle_t h, void* stream);

/* Per-layer budgets: an alternative allocation policy on the same kernels (Section 2 discusses
 * methods that give layers different cache sizes; LASER-KV itself uses one B for every layer,
 * Appendix B). Sets the number of tokens kept per block in `layer` to budget_per_block, split
 * by the handle's protection divisor and alpha as in laser_kv_partition. The configured budget
 * stays the maximum (it sizes the cache and the workspace): 0 <= budget_per_block <= it, else
 * INVALID_ARG; the layer's cache must be empty (STATE otherwise; laser_kv_reset empties it).
 * Later calls for the layer keep budget_per_block tokens per block; cache_view's len and decode
 * attention follow. Host only. */
laser_kv_status_t laser_kv_set_layer_budget(laser_kv_handle_t h, int32_t layer, int32_t budget_per_block);

/* Diagnostics: poll budget of the hand-off waits inside the streaming kernels (tile landed, stage
 * free, accumulator ready / drained, exchange areas). Every such wait is bounded: when its budget
 * runs out the waiting role records LASER_KV_ERR_TIMEOUT in the status word that
 * laser_kv_poll_status reads, the kernel lets copies and tensor-core work already in flight finish
 * (those waits always keep the built-in budget), frees its tensor memory and returns; the results of
 * that call are then incomplete. max_polls = 0 restores the built-in budgets (a second or more,
 * never reached by a working pipeline); a small value makes the give-up path reachable on purpose,
 * which is what the tests use it for. Host only; applies to later calls on this handle. */
laser_kv_status_t laser_kv_set_wait_budget(laser_kv_handle_t h, uint32_t max_polls);

/* Forgets the contents of one layer's cache (layer = -1: all layers). Host only. */
laser_kv_status_t laser_kv_reset(laser_kv_handle_t h, int32_t layer);

void laser_kv_destroy(laser_kv_handle_t h);

const char* laser_kv_status_string(laser_kv_status_t s);

/* Text of the most recent error on this handle ("" if none). NULL handle: the most recent
 * error of a call that had no handle (init, query_sizes, step entry points). */
const char* laser_kv_last_error(laser_kv_handle_t h);

/* Per-handle counters since laser_kv_init (host only, no synchronisation): calls of the select
 * entry points, blocks and tokens they covered (tokens per sequence, summed over the batch), cache
 * entries appended per (sequence, KV head) summed over sequences and heads, and the bytes the method
 * itself has to move for that work (keys read once, window queries and hyperplanes per call, every
 * kept K and V row read once and written once, positions). With the environment variable
 * LASER_KV_LOG set to a non-empty value other than 0 when the handle is created, every select call,
 * reset and destroy also writes one line to stderr (host side only; nothing changes on the device). */
typedef struct {
  int64_t select_calls, blocks, tokens, entries_appended, algorithmic_bytes;
} laser_kv_counters_t;
laser_kv_status_t laser_kv_get_counters(laser_kv_handle_t h, laser_kv_counters_t* out);

/* Number of this library's kernels launched by the calling process so far (all handles). */
int64_t laser_kv_launch_count(void);

/* Optional per-kernel timing. When enabled, every select call records CUDA events on the caller's
 * stream between its kernels (no synchronisation, no device memory). laser_kv_profile_read waits
 * for the recorded events, adds the elapsed times to per-kernel totals and reports them:
 * names[i] is a static string, total_ms[i] the accumulated device time and launches[i] the number
 * of launches of kernel i since profiling was enabled; *n_kernels is set to the number of entries
 * (at most 16; pass arrays of 16). Enabling resets the totals. */
laser_kv_status_t laser_kv_profile_enable(laser_kv_handle_t h, int32_t on);
laser_kv_status_t laser_kv_profile_read(laser_kv_handle_t h, int32_t* n_kernels, const char** names,
                                        float* total_ms, int32_t* launches);

/* ---- step-level entry points (same kernels as the hot path, caller-fed inputs) ------------- */

/* Algorithm 1 lines 4-8 on given scores: for each of n_segments independent segments of S
 * tokens, pick k_exact of the candidates [anchors, S - anchors) by s_exact (fp32, larger first),
 * then k_lsh of the remaining candidates by counts (u32, larger first), ties to the lower index,
 * and write the kept indices [0, anchors) + picks + [S - anchors, S) in ascending order.
 *   s_exact dev fp32 [n_segments][S]; counts dev u32 [n_segments][S];
 *   idx_out dev int32 [n_segments][2*anchors + k_exact + k_lsh].
 * Needs 2*anchors + k_exact + k_lsh <= S. */
laser_kv_status_t laser_kv_two_stage_topk(const float* s_exact, const uint32_t* counts,
                                          int32_t n_segments, int32_t S, int32_t anchors,
                                          int32_t k_exact, int32_t k_lsh, int32_t* idx_out,
                                          void* stream);

/* Step 1 of the path alone (Section 3.3 "Precision", Algorithm 1 line 3, per layer and KV head):
 * S_exact[b][h][t][j] = sum over the window queries (g, w) of KV head h's group of
 * softmax_j(<q_{g,w}, k_j> * scale), the softmax taken over the S keys of block t.
 *   K_blk, Q_win, kv_strides, q_strides, n_blocks : as for laser_kv_select_block.
 *   softmax_scale : 0 => 1/sqrt(128).
 *   scratch       : dev, 256-byte aligned, at least laser_kv_window_scores_scratch_bytes(...) bytes,
 *                   owned by the caller; holds the per-query log-sum-exp partials between the two
 *                   kernels. Its first int is a status word (0, or LASER_KV_ERR_TIMEOUT if a bounded
 *                   device-side wait gave up).
 *   s_exact_out   : dev fp32 [batch][H_kv][n_blocks][S].
 * head_dim is 128; G*W must be a multiple of 16 and at most 256. */
size_t laser_kv_window_scores_scratch_bytes(int32_t batch, int32_t n_q_heads, int32_t n_kv_heads,
                                            int32_t block_size, int32_t window, int32_t n_blocks);
laser_kv_status_t laser_kv_window_scores(const void* K_blk, const void* Q_win,
                                         const int64_t kv_strides[3], const int64_t q_strides[3],
                                         int32_t batch, int32_t n_q_heads, int32_t n_kv_heads,
                                         int32_t block_size, int32_t window, int32_t n_blocks,
                                         float softmax_scale, void* scratch, size_t scratch_bytes,
                                         float* s_exact_out, void* stream);

/* laser_kv_window_scores for callers that cannot hand over scratch memory. (The paper has no
 * counterpart to this entry point; it exists for integration only.)
 *
 * Who needs it: code that runs where device allocation is off the table - a plugin inside a
 * serving engine whose memory pool already owns the whole GPU, so a cudaMalloc would fail or eat
 * into a reservation it must not touch; a hook in a latency-critical decode loop where the
 * implicit device synchronisation of cudaMalloc/cudaFree is unacceptable; a sandboxed extension
 * that is simply not allowed to call the allocator. Such a caller still passes its inputs and
 * its output buffer, but the log-sum-exp partials that laser_kv_window_scores keeps in `scratch`
 * go to an array built into the library image instead:
 *   - size LASER_KV_STATIC_SCRATCH_BYTES = 2 MiB (laser_kv_window_scores_static_max_bytes()),
 *     resident on every GPU that loads the library, until the process exits;
 *   - a problem whose laser_kv_window_scores_scratch_bytes(...) exceeds it is rejected with
 *     LASER_KV_ERR_CAPACITY and nothing is launched (a 128k-token layer of 16 blocks x 8 KV
 *     heads x 256 window queries needs about 1.2 MiB and fits);
 *   - this function never calls cudaMalloc, cudaFree or any allocating library routine.
 * The first call on each device looks up the array's device address (with the CUDA device of
 * the inputs current, as for every call); make that first call before starting any stream
 * capture. All calls on a device share the one array: it still holds the previous call's
 * partials (everything but the status word at its start is overwritten before it is read), and
 * two calls whose kernels overlap on the GPU - different
 * streams, or different host threads - race on it. Serialise them.
 * Arguments and results are those of laser_kv_window_scores without scratch/scratch_bytes.
 * The status word of these calls lives at the start of the built-in array, where the caller cannot
 * look: laser_kv_window_scores_static_status(stream) synchronises `stream`, copies the word to the
 * host (a plain 4-byte copy, no allocation), and returns LASER_KV_OK or the first error a kernel of
 * any earlier static call on this device recorded (LASER_KV_ERR_TIMEOUT: a bounded device-side wait
 * gave up and that call's scores are incomplete), clearing it. The word is sticky: it is not reset
 * by later calls, only by reading it. */
size_t laser_kv_window_scores_static_max_bytes(void);
laser_kv_status_t laser_kv_window_scores_static_status(void* stream);
laser_kv_status_t laser_kv_window_scores_static(const void* K_blk, const void* Q_win,
                                                const int64_t kv_strides[3], const int64_t q_strides[3],
                                                int32_t batch, int32_t n_q_heads, int32_t n_kv_heads,
                                                int32_t block_size, int32_t window, int32_t n_blocks,
                                                float softmax_scale, float* s_exact_out, void* stream);

/* Steps 2 and 3 of the path alone (Section 3.3 "Recall", Algorithm 1 line 6, per layer and KV head):
 * count[b][h][t][j] = number of (window query of KV head h's group, table r) pairs whose K-bit
 * SimHash bucket h_r(q) equals h_r(k_j), k_j the j-th key of block t; S_lsh = count / (L * G * W).
 *   K_blk, Q_win, kv_strides, q_strides, n_blocks : as for laser_kv_select_block.
 *   hyperplanes : dev bf16 [lsh_tables * lsh_bits][128], table-major (row r*K + b = bit b of table r).
 *   scratch     : dev, 256-byte aligned, at least laser_kv_collision_counts_scratch_bytes(...) bytes,
 *                 owned by the caller (query histogram, query codes, exact-sign work list). Its first
 *                 int is a status word (0, LASER_KV_ERR_TIMEOUT, or LASER_KV_ERR_CAPACITY if the
 *                 exact-sign list overflowed).
 *   counts_out  : dev u32 [batch][H_kv][n_blocks][S].
 * head_dim is 128; lsh_bits in {4,6,8,10,12}; lsh_tables a multiple of 8. */
size_t laser_kv_collision_counts_scratch_bytes(int32_t batch, int32_t n_q_heads, int32_t n_kv_heads,
                                               int32_t block_size, int32_t window, int32_t n_blocks,
                                               int32_t lsh_bits, int32_t lsh_tables);
laser_kv_status_t laser_kv_collision_counts(const void* K_blk, const void* Q_win, const void* hyperplanes,
                                            const int64_t kv_strides[3], const int64_t q_strides[3],
                                            int32_t batch, int32_t n_q_heads, int32_t n_kv_heads,
                                            int32_t block_size, int32_t window, int32_t n_blocks,
                                            int32_t lsh_bits, int32_t lsh_tables, void* scratch,
                                            size_t scratch_bytes, uint32_t* counts_out, void* stream);

/* Recall score in closed form (Section 3.3 "Recall" as worded: tokens are ranked by their
 * theoretical hash collision probability with the query; Algorithm 1 line 6 prints the empirical
 * fraction, whose expectation over the hyperplane draw this is):
 *   p[b][h][t][j] = (1 / (G*W)) * sum over the window queries q of KV head h's group of
 *                   (1 - theta(q, k_j) / pi)^lsh_bits,   theta = angle between q and key j of block t
 * (a zero vector counts as orthogonal to everything). No hyperplanes, no tables. The values are
 * non-negative floats, so their bit patterns order like unsigned integers: cast p_out to
 * uint32_t* and pass it as `counts` to laser_kv_two_stage_topk to rank the recall stage by it.
 *   K_blk, Q_win, kv_strides, q_strides, n_blocks : as for laser_kv_select_block.
 *   scratch : dev, 16-byte aligned, at least 256 bytes; its first int is a status word (0 or
 *             LASER_KV_ERR_TIMEOUT), cleared by the call.
 *   p_out   : dev fp32 [batch][H_kv][n_blocks][S].
 * head_dim is 128; G*W a multiple of 16, at most 256; lsh_bits in [1, 64]. fp32 arithmetic on exact
 * bf16 products. */
laser_kv_status_t laser_kv_collision_probability(const void* K_blk, const void* Q_win, const int64_t kv_strides[3],
                                                 const int64_t q_strides[3], int32_t batch, int32_t n_q_heads,
                                                 int32_t n_kv_heads, int32_t block_size, int32_t window,
                                                 int32_t n_blocks, int32_t lsh_bits, void* scratch,
                                                 size_t scratch_bytes, float* p_out, void* stream);

/* Consensus aggregation (Section 3.3 "Precision" as printed: a candidate's score is the attention
 * it receives summed over all layers and heads, so that one index set serves every head): adds the
 * per-head outputs of laser_kv_window_scores and laser_kv_collision_counts over the n_heads heads,
 *   s_acc[b][t][j] (+)= sum_h s_exact[b][h][t][j],   c_acc[b][t][j] (+)= sum_h counts[b][h][t][j],
 * overwriting the sums when carry == 0 and adding to them when carry != 0 (further layers).
 * Heads are added in ascending order, so the fp32 sums are reproducible. Feed the sums to
 * laser_kv_two_stage_topk (n_segments = batch * n_blocks) and the resulting index lists to
 * laser_kv_gather_append once per head.
 *   s_exact dev fp32, counts dev u32 [batch][n_heads][n_blocks][S]; s_acc dev fp32, c_acc dev u32
 *   [batch][n_blocks][S]; all 16-byte aligned; S a multiple of 4. */
laser_kv_status_t laser_kv_consensus_accumulate(const float* s_exact, const uint32_t* counts, int32_t batch,
                                                int32_t n_heads, int32_t n_blocks, int32_t block_size,
                                                int32_t carry, float* s_acc, uint32_t* c_acc, void* stream);

/* Append step (Sections 1 and 3): for each of n_segments segments copies rows idx[seg][i] of the
 * segment's K and V (dev bf16, row length d = 128, consecutive rows `src_row_stride` elements
 * apart, n_src_rows rows per segment, segment s starting at src + s*src_seg_stride) to dst rows
 * [dst_offset + i] of the segment's cache (segments dst_seg_stride elements apart, rows d apart,
 * dst_capacity rows per segment) and writes pos_base + idx[seg][i] to
 * pos_out[s*pos_seg_stride + dst_offset + i].
 *   idx    : dev int32 [n_segments][n_keep], values in [0, n_src_rows). An index outside that range
 *            is never dereferenced: its row and position are skipped and *status becomes
 *            LASER_KV_ERR_INVALID_ARG.
 *   status : dev int32, 4-byte aligned, owned by the caller; cleared by the call (on `stream`) and
 *            set by the kernel as described; read it after `stream` has passed the call.
 * Errors on the host: CAPACITY when dst_offset + n_keep exceeds dst_capacity (nothing is launched). */
laser_kv_status_t laser_kv_gather_append(const void* K_src, const void* V_src,
                                         int64_t src_seg_stride, int64_t src_row_stride,
                                         int32_t n_src_rows, const int32_t* idx, int32_t n_segments,
                                         int32_t n_keep, void* K_dst, void* V_dst,
                                         int64_t dst_seg_stride, int64_t dst_capacity,
                                         int32_t* pos_out, int64_t pos_seg_stride,
                                         int64_t dst_offset, int32_t pos_base, int32_t* status,
                                         void* stream);

/* Decode-phase attention over a layer's compacted cache (Section 3: once a block is processed only
 * the selected tokens stay in the KV cache and serve the decoding phase; Section 4.1 evaluates the
 * answers generated from that cache). For every sequence b and query head hq of KV head
 * h = hq / G it computes, over the len = blocks appended so far * B cache entries of (b, h),
 *   out[b][hq][:] = sum_i softmax_i(<Q_dec[b][hq], K_cache[b][h][i]> * scale) * V_cache[b][h][i].
 * bf16 inputs, products and sums in fp32, output fp32.
 *   Q_dec         : dev bf16, element (b, hq, :) at Q_dec + b*q_strides[0] + hq*q_strides[1], row of
 *                   128 contiguous elements; 16-byte aligned, strides multiples of 8 elements.
 *   softmax_scale : 0 selects the handle's configured scale.
 *   out           : dev fp32 [batch][n_q_heads][128], 16-byte aligned.
 *   scratch       : dev, 16-byte aligned, at least laser_kv_decode_attention_scratch_bytes(h) bytes
 *                   (per-chunk partial sums), owned by the caller, reusable after the stream has
 *                   passed the call.
 * Asynchronous on `stream`, ordered after earlier select calls on the same stream. Errors:
 * LASER_KV_ERR_STATE when the layer's cache is empty, LASER_KV_ERR_UNSUPPORTED for more than 8 query
 * heads per KV head or more than 1 Mi entries per head, LASER_KV_ERR_CAPACITY for a short scratch. */
size_t laser_kv_decode_attention_scratch_bytes(laser_kv_handle_t h);
laser_kv_status_t laser_kv_decode_attention(laser_kv_handle_t h, int32_t layer, const void* Q_dec,
                                            const int64_t q_strides[2], float softmax_scale, float* out,
                                            void* scratch, size_t scratch_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LASER_KV_H_ */
