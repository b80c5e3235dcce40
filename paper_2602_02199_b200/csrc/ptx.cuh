// Thin inline-PTX wrappers for the sm_100a features the kernels use: mbarriers, TMA tiled and
// bulk copies, tcgen05 (5th-generation tensor core) MMA with TMEM accumulators.
// Every wait is bounded by a poll budget; a wait that gives up returns false and the caller
// records LASER_KV_ERR_TIMEOUT in the status word and unwinds (no trap, no endless loop).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace lkv {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}

// ---- programmatic dependent launch ----------------------------------------------------------
// A kernel launched with the programmatic-serialization attribute may start as soon as every CTA of
// the kernel before it in the stream has called allow_dependents() (or has exited); it must not
// rely on that kernel's results before grid_dependency_wait() has returned, which waits for that
// kernel's completion and the visibility of its writes. Without the attribute both are no-ops.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void allow_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Bounded waits on words in global memory that another kernel of the same stream writes: a counter
// that only grows has reached `target` (signed difference, so it may wrap), or a flag equals `value`.
// They order kernels that run beside each other. The kernel that writes has always started, and
// never waits for the reader, before the reader is launched, so the waits end; the poll limit is a
// backstop after which the caller records a timeout.
__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_gpu(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ bool wait_counter_reached(const int* counter, int target, uint32_t max_polls) {
  for (uint32_t n = 0; n < max_polls; ++n) {
    if (ld_acquire_gpu(counter) - target >= 0) return true;
    __nanosleep(100);
  }
  return false;
}
__device__ __forceinline__ bool wait_flag_equals(const int* flag, int value, uint32_t max_polls) {
  for (uint32_t n = 0; n < max_polls; ++n) {
    if (ld_acquire_gpu(flag) == value) return true;
    __nanosleep(100);
  }
  return false;
}
constexpr uint32_t kMaxFlagPolls = 1u << 23;     // x 100 ns and more: about a second

// ---- mbarrier -------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// Orders global-memory accesses of ordinary loads and stores (already ordered before this thread
// by fences and barriers) before later reads of the same memory by bulk copies.
__device__ __forceinline__ void fence_proxy_async_global() {
  asm volatile("fence.proxy.async.global;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded waits for the phase with the given parity. One poll is a try_wait that may suspend the
// thread for up to `hint_ns` nanoseconds (the hardware may cut that short; it returns as soon as
// the phase completes), so the longest wait is max_polls * hint_ns: the built-in budgets give about
// two seconds, far beyond any legitimate wait of these kernels. A wait that runs out returns false;
// the caller records LASER_KV_ERR_TIMEOUT and unwinds. hint_ns = 0 is the diagnostic form: every
// poll is a non-suspending test_wait, so that a handful of polls really is a short time and a test
// can make a healthy pipeline's waits run out.
constexpr uint32_t kMaxPolls = 200;
constexpr uint32_t kPollHintNs = 10u * 1000u * 1000u;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t max_polls = kMaxPolls,
                                          uint32_t hint_ns = kPollHintNs) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t.reg .u32 n;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"      // fast path: already complete
      "@p bra LKV_WAIT_DONE;\n\t"
      "mov.u32 n, 0;\n\t"
      "setp.eq.u32 q, %4, 0;\n"
      "LKV_WAIT_TRY:\n\t"
      "@!q mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %4;\n\t"
      "@q mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "@p bra LKV_WAIT_DONE;\n\t"
      "add.u32 n, n, 1;\n\t"
      "setp.lt.u32 p, n, %3;\n\t"
      "@p bra LKV_WAIT_TRY;\n\t"
      "setp.ne.u32 p, n, n;\n"
      "LKV_WAIT_DONE:\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(max_polls), "r"(hint_ns)
      : "memory");
  return ok != 0;
}
// The same wait under the name the critical-path roles (MMA issuer, projection epilogue) use.
constexpr uint32_t kMaxSpinPolls = kMaxPolls;
__device__ __forceinline__ bool mbar_wait_spin(uint32_t bar, uint32_t parity, uint32_t max_polls = kMaxPolls,
                                               uint32_t hint_ns = kPollHintNs) {
  return mbar_wait(bar, parity, max_polls, hint_ns);
}

// ---- TMA -------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* m, uint32_t bar,
                                            int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* m, uint32_t bar,
                                            int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
// Untiled bulk copy global -> shared; both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes,
                                          uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
          "r"(dst),
      "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
      : "memory");
}

// ---- tcgen05 / TMEM ---------------------------------------------------------------------------
// Whole-warp calls (".sync.aligned"): every lane of the calling warp must execute them.
__device__ __forceinline__ void tmem_alloc(uint32_t smem_result, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                   smem_result),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// D[tmem] (+)= A[smem] * B[smem]; bf16 inputs, fp32 accumulate; issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives (count 1) on the mbarrier once all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                   bar)
               : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Each thread of the warp reads 32-bit columns [col, col+N) of its own TMEM lane
// (lane = 32 * (warp_id % 4) + lane_id, encoded in the upper half of taddr by the caller).
#define LKV_TMEM_LD_DECL(N)                                                                    \
  __device__ __forceinline__ void tmem_ld_x##N(uint32_t taddr, uint32_t* r)

LKV_TMEM_LD_DECL(32) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]),
        "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]),
        "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
LKV_TMEM_LD_DECL(16) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
LKV_TMEM_LD_DECL(8) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7])
      : "r"(taddr)
      : "memory");
}
LKV_TMEM_LD_DECL(4) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(taddr)
               : "memory");
}
LKV_TMEM_LD_DECL(2) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0, %1}, [%2];"
               : "=r"(r[0]), "=r"(r[1])
               : "r"(taddr)
               : "memory");
}
LKV_TMEM_LD_DECL(1) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r[0]) : "r"(taddr)
               : "memory");
}
#undef LKV_TMEM_LD_DECL

// Loads N consecutive columns (any N in 1..32) as a sum of power-of-two loads.
template <int N>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t* r) {
  static_assert(N >= 1 && N <= 32, "1..32 columns");
  int done = 0;
  if constexpr (N & 32) { tmem_ld_x32(taddr + done, r + done); done += 32; }
  if constexpr (N & 16) { tmem_ld_x16(taddr + done, r + done); done += 16; }
  if constexpr (N & 8)  { tmem_ld_x8(taddr + done, r + done);  done += 8; }
  if constexpr (N & 4)  { tmem_ld_x4(taddr + done, r + done);  done += 4; }
  if constexpr (N & 2)  { tmem_ld_x2(taddr + done, r + done);  done += 2; }
  if constexpr (N & 1)  { tmem_ld_x1(taddr + done, r + done);  done += 1; }
}

// ---- descriptors ------------------------------------------------------------------------------
// Instruction descriptor of tcgen05.mma kind::f16: bf16 x bf16 -> fp32, both operands K-major.
// Fields: [4,6) accumulator format (1 = f32); [7,10) A format (1 = bf16); [10,13) B format;
// bit 15 / 16 A / B major (0 = K-major); [17,23) N >> 3; [24,29) M >> 4.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(N >> 3) << 17) |
         (static_cast<uint32_t>(M >> 4) << 24);
}

// Shared-memory matrix descriptor for a K-major bf16 tile stored as rows of 128 bytes
// (64 elements) with the 128-byte swizzle, 8-row groups 1024 bytes apart - the layout a TMA
// load with CU_TENSOR_MAP_SWIZZLE_128B and a 64-element inner box produces at a 1024-byte
// aligned address. Fields: [0,14) address >> 4; [16,30) leading byte offset >> 4 (unused for
// swizzled K-major, set to 1); [32,46) stride byte offset >> 4 (1024 B between 8-row groups);
// [46,48) descriptor version 1; [61,64) layout 2 = 128-byte swizzle.
__device__ __forceinline__ uint64_t umma_sdesc_sw128(uint32_t saddr) {
  return static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4) | (1ull << 16) |
         (static_cast<uint64_t>(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

// The same descriptor split in two words: the high word is one constant for every operand of
// these kernels, the low word is (address >> 4) plus the version bit, so stepping through an
// operand is a 32-bit add of (byte offset >> 4).
constexpr uint32_t kSdescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t umma_sdesc_lo(uint32_t saddr) {
  return ((saddr & 0x3FFFFu) >> 4) | (1u << 16);
}
// tcgen05.mma with both shared-memory descriptors given by their low words.
__device__ __forceinline__ void umma_bf16_lo(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "mov.b64 da, {%1, %5};\n\t"
      "mov.b64 db, {%2, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kSdescHi)
      : "memory");
}

// tcgen05.wait::ld that also names the loaded registers as in/out operands, so that no use of
// them can be scheduled before the wait (the loads are asynchronous until then).
__device__ __forceinline__ void tmem_wait_ld_dep32(uint32_t* r) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]),
                 "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]),
                 "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]),
                 "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]),
                 "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]),
                 "+r"(r[31])
               :
               : "memory");
}
__device__ __forceinline__ void tmem_wait_ld_dep16(uint32_t* r) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]),
                 "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]),
                 "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
               :
               : "memory");
}

// Orders every later use of r[0..N) after the preceding volatile asm statements (in particular a
// tcgen05.wait::ld) without emitting an instruction: the registers are named as read-write
// operands of an empty volatile asm. N must be a multiple of 2.
template <int N>
__device__ __forceinline__ void reg_fence(uint32_t* r) {
  static_assert(N % 2 == 0, "even register count");
  if constexpr (N >= 8) {
    asm volatile("" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7])
                 :: "memory");
    reg_fence<N - 8>(r + 8);
  } else if constexpr (N >= 2) {
    asm volatile("" : "+r"(r[0]), "+r"(r[1]) :: "memory");
    reg_fence<N - 2>(r + 2);
  }
}

// 2^x on the FMA pipe (no MUFU): round-to-nearest split x = n + f, f in [-0.5, 0.5], degree-4
// minimax polynomial for 2^f (max relative error 2.7e-6), exponent patched in with one integer
// multiply-add. Valid for x >= -126 after the clamp; larger negatives return 2^-126.
__device__ __forceinline__ float ex2_poly(float x) {
  x = fmaxf(x, -126.0f);
  const float t = x + 12582912.0f;            // 1.5 * 2^23: low mantissa bits now hold round(x)
  const float f = x - (t - 12582912.0f);
  float p = 0.009570101276040077f;
  p = fmaf(p, f, 0.05591785907745361f);
  p = fmaf(p, f, 0.240247443318367f);
  p = fmaf(p, f, 0.6931217908859253f);
  p = fmaf(p, f, 0.9999992847442627f);
  return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
}

// Three-input minimum / maximum of magnitudes, one instruction each.
__device__ __forceinline__ float min3_abs(float a, float b, float c) {
  float d;
  asm("min.abs.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float max3_abs(float a, float b, float c) {
  float d;
  asm("max.abs.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Packed fp32 arithmetic: one instruction works on two values held in a register pair.
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ float2 add2(float2 a, float2 b) { return __fadd2_rn(a, b); }

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2_approx(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ex2_poly for a pair of values with the packed instructions (same polynomial, same result).
__device__ __forceinline__ float2 ex2_poly2(float2 x) {
  x.x = fmaxf(x.x, -126.0f);
  x.y = fmaxf(x.y, -126.0f);
  const float2 magic = make_float2(12582912.0f, 12582912.0f);
  const float2 t = add2(x, magic);
  const float2 r = add2(t, make_float2(-12582912.0f, -12582912.0f));
  const float2 f = fma2(r, make_float2(-1.0f, -1.0f), x);
  float2 p = fma2(make_float2(0.009570101276040077f, 0.009570101276040077f), f,
                  make_float2(0.05591785907745361f, 0.05591785907745361f));
  p = fma2(p, f, make_float2(0.240247443318367f, 0.240247443318367f));
  p = fma2(p, f, make_float2(0.6931217908859253f, 0.6931217908859253f));
  p = fma2(p, f, make_float2(0.9999992847442627f, 0.9999992847442627f));
  float2 e;
  e.x = __int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23));
  e.y = __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23));
  return e;
}

}  // namespace lkv
