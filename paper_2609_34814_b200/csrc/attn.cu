// Block-sparse FlashAttention-style forward for sm_100a, scheduled by a row order.
//
// What it computes (Sections 2.1-2.3 of the WaveAlign paper): for query block i of head h,
//   O_i = softmax(scale * Q_i K_sel^T) V_sel  over the tokens of the K/V blocks listed for
// (h, i), visited in the listed order, with the online-softmax state and the partial output
// kept on chip and written once.  The order in which query blocks are started is the
// head-major concatenation of row_order (Algorithm 2's output): persistent CTAs, one per
// SM, take tickets from a global counter, so a freed SM starts the next row of the list at
// once - the streaming "wave" behaviour of Section 2.3 that the schedule is built for.
//
// Structure of one CTA (320 threads):
//   warp 0      producer: takes tickets, publishes tasks, issues TMA loads of the Q tile and
//               of the K/V tiles (128-byte-swizzled slabs) into a shared-memory ring
//   warp 1      MMA issuer: S = Q K^T (operands in shared memory) and O += P V (P read from
//               tensor memory) as tcgen05.mma with fp32 accumulators in tensor memory; three
//               S buffers, so Q K_{j+1}^T and Q K_{j+2}^T are done while the softmax of S_j runs
//   warps 2-9   softmax: thread (row, half) reads half a row of S from tensor memory, the two
//               halves exchange their maxima through shared memory, then the thread writes P
//               (bf16) over the columns S came from; the running max / sum stay in registers;
//               O in tensor memory is rescaled only when the max grew by more than 2^8; the
//               epilogue normalises and stores O at the ORIGINAL row (no inverse permutation)
// Every wait on an mbarrier is bounded; when one runs out the CTA records
// {WAVEAL_ERR_TIMEOUT, site} and all roles leave through the common teardown.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cmath>
#include "host_common.h"

namespace {

constexpr int kThreads = 320;
constexpr int kSoftmaxWarp0 = 2;
constexpr long long kTimeoutCycles = 4000000000ll;   // ~2 s at boost clock
#ifndef WAVEAL_POLY_EVERY
#define WAVEAL_POLY_EVERY 0
#endif
constexpr int kPolyEvery = WAVEAL_POLY_EVERY;          // n > 0: 1 pair in n computes 2^x on the FMA pipe (0 = off: measured slower, the softmax is issue-bound)

// ------------------------------------------------------------------ PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// One lane of a converged warp gets true.  tcgen05.mma / tcgen05.commit are issued under
// this predicate, one instruction at a time, with their operands computed by the whole warp:
// the operands then stay in uniform registers (a branch on the lane index instead makes the
// compiler move every operand from vector registers, which halves the MMA issue rate).
__device__ __forceinline__ uint32_t elect_one() {
  uint32_t pred = 0;
  asm volatile(
      "{\n\t.reg .b32 rx;\n\t.reg .pred px;\n\t"
      "elect.sync rx|px, 0xFFFFFFFF;\n\t"
      "@px mov.s32 %0, 1;\n\t}"
      : "+r"(pred));
  return pred;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// non-blocking probe (try_wait may suspend the thread for a while when the phase is not complete)
__device__ __forceinline__ uint32_t mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, int c2, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tm)) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {   // whole warp calls; one lane issues
  if (elect_one())
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulate, one CTA
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  if (elect_one())
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// D[tmem] (+)= A[tmem] * B[smem]: A is 128 lanes x K bf16, two K elements per 32-bit column
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  if (elect_one())
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

#define WAVEAL_R32(v, o) \
  "=r"(v[o+0]), "=r"(v[o+1]), "=r"(v[o+2]), "=r"(v[o+3]), "=r"(v[o+4]), "=r"(v[o+5]), "=r"(v[o+6]), "=r"(v[o+7]), \
  "=r"(v[o+8]), "=r"(v[o+9]), "=r"(v[o+10]), "=r"(v[o+11]), "=r"(v[o+12]), "=r"(v[o+13]), "=r"(v[o+14]), "=r"(v[o+15]), \
  "=r"(v[o+16]), "=r"(v[o+17]), "=r"(v[o+18]), "=r"(v[o+19]), "=r"(v[o+20]), "=r"(v[o+21]), "=r"(v[o+22]), "=r"(v[o+23]), \
  "=r"(v[o+24]), "=r"(v[o+25]), "=r"(v[o+26]), "=r"(v[o+27]), "=r"(v[o+28]), "=r"(v[o+29]), "=r"(v[o+30]), "=r"(v[o+31])
#define WAVEAL_RW32(v, o) \
  "+r"(v[o+0]), "+r"(v[o+1]), "+r"(v[o+2]), "+r"(v[o+3]), "+r"(v[o+4]), "+r"(v[o+5]), "+r"(v[o+6]), "+r"(v[o+7]), \
  "+r"(v[o+8]), "+r"(v[o+9]), "+r"(v[o+10]), "+r"(v[o+11]), "+r"(v[o+12]), "+r"(v[o+13]), "+r"(v[o+14]), "+r"(v[o+15]), \
  "+r"(v[o+16]), "+r"(v[o+17]), "+r"(v[o+18]), "+r"(v[o+19]), "+r"(v[o+20]), "+r"(v[o+21]), "+r"(v[o+22]), "+r"(v[o+23]), \
  "+r"(v[o+24]), "+r"(v[o+25]), "+r"(v[o+26]), "+r"(v[o+27]), "+r"(v[o+28]), "+r"(v[o+29]), "+r"(v[o+30]), "+r"(v[o+31])
#define WAVEAL_IN32(v, o) \
  "r"(v[o+0]), "r"(v[o+1]), "r"(v[o+2]), "r"(v[o+3]), "r"(v[o+4]), "r"(v[o+5]), "r"(v[o+6]), "r"(v[o+7]), \
  "r"(v[o+8]), "r"(v[o+9]), "r"(v[o+10]), "r"(v[o+11]), "r"(v[o+12]), "r"(v[o+13]), "r"(v[o+14]), "r"(v[o+15]), \
  "r"(v[o+16]), "r"(v[o+17]), "r"(v[o+18]), "r"(v[o+19]), "r"(v[o+20]), "r"(v[o+21]), "r"(v[o+22]), "r"(v[o+23]), \
  "r"(v[o+24]), "r"(v[o+25]), "r"(v[o+26]), "r"(v[o+27]), "r"(v[o+28]), "r"(v[o+29]), "r"(v[o+30]), "r"(v[o+31])

// 32 consecutive fp32 columns of this thread's tensor-memory lane -> registers v[o..o+31]
#define WAVEAL_TMEM_LD32(taddr, v, o)                                                            \
  asm volatile(                                                                                  \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                  \
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "                  \
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"  \
      : WAVEAL_R32(v, o)                                                                         \
      : "r"(taddr)                                                                               \
      : "memory")
// wait for outstanding tensor-memory loads; the registers are operands so that no use of
// them can be moved above the wait
#define WAVEAL_TMEM_WAIT_LD32(v, o) asm volatile("tcgen05.wait::ld.sync.aligned;" : WAVEAL_RW32(v, o)::"memory")
#define WAVEAL_TMEM_ST32(taddr, v, o)                                                            \
  asm volatile(                                                                                  \
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "                                           \
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "                  \
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"         \
      ::WAVEAL_IN32(v, o), "r"(taddr)                                                            \
      : "memory")

#define WAVEAL_TMEM_ST16(taddr, v, o)                                                            \
  asm volatile(                                                                                  \
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "                                           \
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};"                  \
      ::"r"(v[o+0]), "r"(v[o+1]), "r"(v[o+2]), "r"(v[o+3]), "r"(v[o+4]), "r"(v[o+5]), "r"(v[o+6]), "r"(v[o+7]), \
        "r"(v[o+8]), "r"(v[o+9]), "r"(v[o+10]), "r"(v[o+11]), "r"(v[o+12]), "r"(v[o+13]), "r"(v[o+14]), "r"(v[o+15]), \
        "r"(taddr)                                                                               \
      : "memory")

__device__ __forceinline__ float ex2(float x) {
#ifdef WAVEAL_DBG_NOEXP
  return x * 0.001f + 0.5f;
#else
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
#endif
}
// 2^x on the FMA and integer pipes (for a share of the elements, to take load off the
// transcendental pipe, which would otherwise be as busy as the tensor cores): round x to the
// nearest integer n with the 1.5*2^23 trick, degree-3 polynomial for 2^(x-n) on [-0.5, 0.5]
// (relative error 7.5e-5, far below the bf16 cut of P), n added to the exponent field.
__device__ __forceinline__ float ex2_fma(float x) {
  x = fmaxf(x, -125.0f);
  const float xi = x + 12582912.0f;
  const float f = x - (xi - 12582912.0f);
  float q = fmaf(0.05517137423157692f, f, 0.2426110953092575f);
  q = fmaf(q, f, 0.6932610273361206f);
  q = fmaf(q, f, 0.9999280571937561f);
  return __int_as_float(__float_as_int(q) + (__float_as_int(xi) << 23));
}
// Register re-allocation between warpgroups (each scheduler hosts one warp of every
// warpgroup): the producer/MMA warpgroup gives registers up, the softmax warpgroups take them.
template <int N> __device__ __forceinline__ void reg_dealloc() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_alloc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
__device__ __forceinline__ void named_bar_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// shared-memory matrix descriptor, 128-byte swizzle, Blackwell version field
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;   // descriptor version
  d |= (uint64_t)2 << 61;   // SWIZZLE_128B
  return d;
}

// instruction descriptor: bf16 x bf16 -> fp32, A K-major, B K-major or MN-major
// (A and B must have the same 16-bit format: an f16 A with a bf16 B is an illegal instruction)
__host__ __device__ constexpr uint32_t make_idesc(int m, int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(m >> 4) << 24);
}

// ------------------------------------------------------------------ kernel

struct AttnParams {
  __nv_bfloat16* O;
  float* lse;
  const int* row_ptr;
  const int* kv_idx;
  const int* row_order;
  int* ws;            // [0] ticket counter, [1] abort flag
  int* dev_status;
  long long o_stride_h, o_stride_t;
  int heads, m_b, n_b, seq_q, seq_kv, interleaved;
  long long total_tasks;
  float sl2;          // scale * log2(e)
};

struct Task { int h, row, lo, n, tail_valid, pad0, pad1, pad2; };

template <int BLOCK, int D>
struct Geo {
  static constexpr int BQ = BLOCK, BK = BLOCK;
  static constexpr int SLABS = D / 64;               // 128-byte column slabs of a Q/K/V tile
  static constexpr int Q_BYTES = SLABS * 128 * 128;  // smem reserved for the 128 MMA rows
  static constexpr int TILE_BYTES = SLABS * BK * 128;
  static constexpr int KV_SLAB_BYTES = BK * 128;
  static constexpr int NSTAGE_RAW = (200 * 1024 - Q_BYTES) / TILE_BYTES;
#ifdef WAVEAL_DBG_NSTAGE
  static constexpr int NSTAGE = WAVEAL_DBG_NSTAGE;
#else
  static constexpr int NSTAGE = NSTAGE_RAW > 8 ? 8 : NSTAGE_RAW;
#endif
  static constexpr int NSBUF = 3;                    // S/P buffers in tensor memory
  static constexpr int CS = BK / 2;                  // S columns per softmax thread (half a row)
  static constexpr int PC = BK / 4;                  // packed P columns per softmax thread
  static constexpr int CO = D / 2;                   // O columns per softmax thread
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_KV = OFF_Q + Q_BYTES;
  static constexpr int OFF_BAR = OFF_KV + NSTAGE * TILE_BYTES;
  static constexpr int N_BAR = 4 + 2 + 2 * NSTAGE + 2 * NSBUF + 1 + 3;
  static constexpr int OFF_TASK = OFF_BAR + ((N_BAR * 8 + 15) / 16) * 16;
  static constexpr int OFF_MX = OFF_TASK + 2 * (int)sizeof(Task);
  static constexpr int OFF_MISC = OFF_MX + 2 * 2 * 128 * 4;
  static constexpr int SMEM_BYTES = OFF_MISC + 16 + 1024;   // + slack for 1024-byte alignment
  // tensor memory: three S/P buffers and the output accumulator
  static constexpr uint32_t S_STRIDE = 128, O_COL = 384, TMEM_COLS = 512;
};

#ifdef WAVEAL_TRACE
// debug build only: four tracer threads of CTA 0 append (tag, block, clock) records to their own
// region after the 256-byte workspace header (plain stores, no atomics)
#define TRACE_DECL int trace_n_ = 0
#define TRACE(role, tag, j)                                                                    \
  do {                                                                                         \
    if (blockIdx.x == 0 && (threadIdx.x & 31) == 0 && trace_n_ < 4000) {                       \
      int* r_ = p.ws + 64 + (role) * 8000 + 2 * trace_n_;                                      \
      r_[0] = (tag) | ((j) << 8); r_[1] = (int)clock64(); ++trace_n_;                          \
    }                                                                                          \
  } while (0)
#else
#define TRACE_DECL
#define TRACE(role, tag, j) do {} while (0)
#endif

struct Ctx {
  uint32_t bar_base;
  volatile int* abort_smem;
  int* ws;
  int* dev_status;
};

__device__ __noinline__ void signal_abort(const Ctx& c, int site) {
  *c.abort_smem = 1;
  atomicExch(&c.ws[1], 1);
  if (c.dev_status && atomicCAS(c.dev_status, 0, WAVEAL_ERR_TIMEOUT) == 0) {
    c.dev_status[1] = site;
    c.dev_status[2] = blockIdx.x;
    c.dev_status[3] = threadIdx.x;
  }
}

// bounded wait; false = gave up (this CTA is aborting)
__device__ __forceinline__ bool mbar_wait(const Ctx& c, uint32_t bar, uint32_t parity, int site) {
  if (mbar_try_wait(bar, parity)) return true;
  long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*c.abort_smem) return false;
    if (clock64() - t0 > kTimeoutCycles) { signal_abort(c, site); return false; }
  }
}

// same, with one answer for the whole warp (the roles use warp-collective instructions)
__device__ __forceinline__ bool warp_wait(const Ctx& c, uint32_t bar, uint32_t parity, int site) {
  return __all_sync(0xffffffffu, mbar_wait(c, bar, parity, site));
}

// Second half of a split wait: `tok` is the answer of a non-blocking probe issued earlier (before the
// preceding group of MMAs, so that its latency hides behind their issue: the tensor pipe's
// queue is short, and any pause of the issuing warp between two MMAs starves it).
__device__ __forceinline__ bool finish_wait(const Ctx& c, uint32_t bar, uint32_t parity, uint32_t tok, int site) {
  if (__all_sync(0xffffffffu, tok)) return true;
  return warp_wait(c, bar, parity, site);
}

template <int BLOCK, int D>
__global__ void __launch_bounds__(kThreads, 1)
k_bsattn_fwd(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
             const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
  using G = Geo<BLOCK, D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);   // provably warp-uniform role index

  const uint32_t bar0 = sbase + G::OFF_BAR;
  auto BAR = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  constexpr int B_TASK_FULL = 0, B_TASK_EMPTY = 2, B_Q_FULL = 4, B_Q_EMPTY = 5, B_KV_FULL = 6,
                B_KV_EMPTY = 6 + G::NSTAGE, B_S_FULL = 6 + 2 * G::NSTAGE, B_P_FULL = B_S_FULL + G::NSBUF,
                B_PV_DONE = B_P_FULL + G::NSBUF, B_O_FULL = B_PV_DONE + 1, B_O_FREE = B_O_FULL + 1, B_FINAL = B_O_FREE + 1;
  static_assert(B_FINAL + 1 <= G::N_BAR, "barrier count");
  Task* tasks = reinterpret_cast<Task*>(smem + G::OFF_TASK);
  float* mx = reinterpret_cast<float*>(smem + G::OFF_MX);            // [2][2][128] row-max / row-sum exchange
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + G::OFF_MISC);
  volatile int* abort_smem = reinterpret_cast<volatile int*>(smem + G::OFF_MISC + 4);
  Ctx ctx{bar0, abort_smem, p.ws, p.dev_status};

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) { mbar_init(BAR(B_TASK_FULL + i), 1); mbar_init(BAR(B_TASK_EMPTY + i), 9); }
    mbar_init(BAR(B_Q_FULL), 1);
    mbar_init(BAR(B_Q_EMPTY), 1);
    for (int i = 0; i < G::NSTAGE; ++i) { mbar_init(BAR(B_KV_FULL + i), 1); mbar_init(BAR(B_KV_EMPTY + i), 1); }
    for (int i = 0; i < G::NSBUF; ++i) mbar_init(BAR(B_S_FULL + i), 1);
    // one P barrier per S buffer: a warp may run up to two blocks ahead of the slowest one
    for (int i = 0; i < G::NSBUF; ++i) mbar_init(BAR(B_P_FULL + i), 8);
    mbar_init(BAR(B_PV_DONE), 1);
    mbar_init(BAR(B_O_FULL), 1);
    mbar_init(BAR(B_O_FREE), 8);
    mbar_init(BAR(B_FINAL), 1);
    *abort_smem = 0;
    fence_mbar_init();
    fence_proxy_async();
  }
  // the MMA reads all 128 rows of the Q region even when a query block has 64 rows: clear it once
  for (int i = tid; i < G::Q_BYTES / 16; i += kThreads) reinterpret_cast<uint4*>(smem + G::OFF_Q)[i] = make_uint4(0, 0, 0, 0);
  fence_proxy_async();
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_holder), G::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  if (warp == 0) {
    // ============================================================== producer
    if (lane == 0) { prefetch_tmap(&tmQ); prefetch_tmap(&tmK); prefetch_tmap(&tmV); }
    uint32_t task_it = 0, q_it = 0, kv_it = 0;
    TRACE_DECL;
    bool ok = true;
    uint32_t armed_mask = 0, armed_parity = 0;   // per stage: parity of the last load armed on it
    bool q_armed = false; uint32_t q_armed_parity = 0;
    while (ok) {
      long long t = 0;
      if (lane == 0) t = (p.ws[1] != 0) ? p.total_tasks : (long long)(unsigned)atomicAdd(&p.ws[0], 1);
      t = __shfl_sync(0xffffffffu, t, 0);
      Task tk{};
      if (t >= p.total_tasks) {
        tk.n = -1;
      } else {
        int h, pos;
        if (p.interleaved) { pos = (int)(t / p.heads); h = (int)(t % p.heads); }
        else { h = (int)(t / p.m_b); pos = (int)(t % p.m_b); }
        int row = p.row_order ? p.row_order[(size_t)h * p.m_b + pos] : pos;
        if (row < 0 || row >= p.m_b) row = pos;          // never index out of range
        int lo = p.row_ptr[(size_t)h * p.m_b + row], hi = p.row_ptr[(size_t)h * p.m_b + row + 1];
        tk.h = h; tk.row = row; tk.lo = lo; tk.n = max(hi - lo, 0);
        tk.tail_valid = G::BK;
        if (tk.n > 0 && (p.seq_kv % G::BK) != 0 && p.kv_idx[hi - 1] == p.n_b - 1) tk.tail_valid = p.seq_kv % G::BK;
      }
      const uint32_t slot = task_it & 1, ph = (task_it >> 1) & 1;
      ok = warp_wait(ctx, BAR(B_TASK_EMPTY + slot), ph ^ 1, 1);
      if (!ok) break;
      if (lane == 0) {
        tasks[slot] = tk;
        mbar_arrive(BAR(B_TASK_FULL + slot));
      }
      ++task_it;
      if (tk.n < 0) break;
      if (tk.n == 0) continue;
      // Q tile
      ok = warp_wait(ctx, BAR(B_Q_EMPTY), (q_it & 1) ^ 1, 2);
      if (!ok) break;
      if (lane == 0) {
        mbar_expect_tx(BAR(B_Q_FULL), G::SLABS * G::BQ * 128);
#pragma unroll
        for (int s = 0; s < G::SLABS; ++s)
          tma_load_3d(sbase + G::OFF_Q + s * 128 * 128, &tmQ, s * 64, tk.row * G::BQ, tk.h, BAR(B_Q_FULL));
      }
      q_armed = true; q_armed_parity = q_it & 1;
      ++q_it;
      // K/V tiles in the order the MMA warp consumes them: K_0..K_2, then V_j, K_{j+3} for each j
      int chunk_base = -64, my_idx = 0;
      auto load_tile = [&](bool is_k, int j) -> bool {
        if (j < chunk_base || j >= chunk_base + 32) {
          chunk_base = j & ~31;
          const int q = chunk_base + lane;
          my_idx = q < tk.n ? p.kv_idx[tk.lo + q] : 0;
        }
        int blk = __shfl_sync(0xffffffffu, my_idx, j - chunk_base);
        if (blk < 0 || blk >= p.n_b) blk = 0;            // malformed list: stay in range
        const uint32_t st = kv_it % G::NSTAGE, sph = (kv_it / G::NSTAGE) & 1;
        if (!warp_wait(ctx, BAR(B_KV_EMPTY + st), sph ^ 1, 3)) return false;
        TRACE(3, 20 + (is_k ? 0 : 1), j);
        if (lane == 0) {
#ifdef WAVEAL_DBG_NOLOAD
          if (kv_it >= (uint32_t)G::NSTAGE) { mbar_arrive(BAR(B_KV_FULL + st)); } else
#endif
          {
          mbar_expect_tx(BAR(B_KV_FULL + st), G::TILE_BYTES);
          const CUtensorMap* tm = is_k ? &tmK : &tmV;
#pragma unroll
          for (int s = 0; s < G::SLABS; ++s)
            tma_load_3d(sbase + G::OFF_KV + st * G::TILE_BYTES + s * G::KV_SLAB_BYTES, tm, s * 64, blk * G::BK, tk.h,
                        BAR(B_KV_FULL + st));
          }
        }
        armed_mask |= 1u << st;
        armed_parity = (armed_parity & ~(1u << st)) | (sph << st);
        ++kv_it;
        return true;
      };
      for (int j = 0; j < G::NSBUF && j < tk.n && ok; ++j) ok = load_tile(true, j);
      for (int j = 0; j < tk.n && ok; ++j) {
        ok = load_tile(false, j);
        if (ok && j + G::NSBUF < tk.n) ok = load_tile(true, j + G::NSBUF);
      }
    }
    if (*abort_smem) {
      // leave no bulk copy in flight into this CTA's shared memory (bounded)
      for (int st = 0; st < G::NSTAGE; ++st)
        if (armed_mask & (1u << st)) {
          long long t0 = clock64();
          while (!mbar_try_wait(BAR(B_KV_FULL + st), (armed_parity >> st) & 1) && clock64() - t0 < kTimeoutCycles / 4) {}
        }
      if (q_armed) {
        long long t0 = clock64();
        while (!mbar_try_wait(BAR(B_Q_FULL), q_armed_parity) && clock64() - t0 < kTimeoutCycles / 4) {}
      }
    }
  } else if (warp == 1) {
    // ============================================================== MMA issuer
    // Every operand of a tcgen05 instruction (descriptors, tensor-memory addresses, barrier
    // addresses) must stay warp-uniform in the compiler's eyes, otherwise each MMA pays for
    // moves into uniform registers and the issue rate drops below the tensor pipe's: values
    // read from shared memory are broadcast with a shuffle, ring positions are advanced by
    // compare-and-reset instead of modulo.
    constexpr uint32_t IDESC_QK = make_idesc(128, G::BK, false);
    constexpr uint32_t IDESC_PV = make_idesc(128, D, true);
    uint32_t task_slot = 0, task_ph = 0, q_ph = 0, o_ph = 1, kv_st = 0, kv_ph = 0, p_phase = 0;
    TRACE_DECL;
    const uint64_t qdesc0 = make_desc(sbase + G::OFF_Q, 16, 1024);
    const uint64_t kdesc0 = make_desc(sbase + G::OFF_KV, 16, 1024);
    const uint64_t vdesc0 = make_desc(sbase + G::OFF_KV, G::KV_SLAB_BYTES, 1024);
    bool ok = true;
    while (ok) {
      ok = warp_wait(ctx, BAR(B_TASK_FULL + task_slot), task_ph, 10);
      if (!ok) break;
      const int n = __shfl_sync(0xffffffffu, tasks[task_slot].n, 0);
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_TASK_EMPTY + task_slot));
      task_slot ^= 1;
      task_ph ^= (task_slot == 0);
      if (n < 0) break;
      if (n == 0) continue;
      ok = warp_wait(ctx, BAR(B_Q_FULL), q_ph, 11);
      if (!ok) break;
      q_ph ^= 1;
      // S[sb] = Q K_j^T (sb = j mod 3); overwrites the P tile that aliases S[sb], which the
      // P V three blocks earlier (issued before by this warp, executed in order) has consumed.
      // The caller has already waited for the K tile in stage kv_st.
      auto issue_qk = [&](uint32_t sb) {
        TRACE(0, 4, (int)kv_st);
        {
          // descriptors differ from the per-kernel bases only in the 14-bit address field
          const uint64_t kd = kdesc0 + (uint64_t)(kv_st * (uint32_t)(G::TILE_BYTES >> 4));
          const uint32_t d_s = tmem_base + sb * G::S_STRIDE;
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
#ifndef WAVEAL_DBG_SKIP_QK
            umma_bf16(d_s, qdesc0 + (uint64_t)(((k / 4) * 128 * 128 + (k % 4) * 32) >> 4),
                      kd + (uint64_t)(((k / 4) * G::KV_SLAB_BYTES + (k % 4) * 32) >> 4), IDESC_QK, k > 0);
#endif
          }
          tc_commit(BAR(B_KV_EMPTY + kv_st));
          tc_commit(BAR(B_S_FULL + sb));
        }
        TRACE(0, 5, (int)kv_st);
        if (++kv_st == (uint32_t)G::NSTAGE) { kv_st = 0; kv_ph ^= 1; }
      };
      for (int j = 0; j < G::NSBUF && j < n && ok; ++j) {
        ok = warp_wait(ctx, BAR(B_KV_FULL + kv_st), kv_ph, 12);
        if (ok) issue_qk((uint32_t)j);
      }
      if (!ok) break;
      if (n <= G::NSBUF) tc_commit(BAR(B_Q_EMPTY));
      // the output accumulator of the previous task has been read by the epilogue
      ok = warp_wait(ctx, BAR(B_O_FREE), o_ph, 16);
      if (!ok) break;
      o_ph ^= 1;
      // answers for the first P V of the task
      uint32_t tok_p = mbar_test_wait(BAR(B_P_FULL + 0), p_phase & 1u);
      uint32_t tok_v = mbar_test_wait(BAR(B_KV_FULL + kv_st), kv_ph);
      uint32_t sb = 0;
      for (int j = 0; j < n && ok; ++j) {
        // O (+)= P_j V_j, P_j read from tensor memory
        ok = finish_wait(ctx, BAR(B_P_FULL + sb), (p_phase >> sb) & 1u, tok_p, 14);
        if (!ok) break;
        p_phase ^= 1u << sb;
        TRACE(0, 1, j);
        ok = finish_wait(ctx, BAR(B_KV_FULL + kv_st), kv_ph, tok_v, 15);
        if (!ok) break;
        TRACE(0, 2, j);
        const bool more_qk = j + G::NSBUF < n;
        // the K tile of block j+3 sits in the stage after this V tile: ask now, use after the MMAs
        uint32_t k_st = kv_st + 1, k_ph = kv_ph;
        if (k_st == (uint32_t)G::NSTAGE) { k_st = 0; k_ph ^= 1; }
        uint32_t tok_k = more_qk ? mbar_test_wait(BAR(B_KV_FULL + k_st), k_ph) : 1u;
        tc_fence_after();
        {
          // V tile as the N x K operand with N (head_dim) contiguous: 8 keys per 1024-byte
          // group along K (16 keys = 2048 bytes per MMA), next 64 columns of head_dim one slab further
          const uint64_t vd = vdesc0 + (uint64_t)(kv_st * (uint32_t)(G::TILE_BYTES >> 4));
          const uint32_t pbase = tmem_base + sb * G::S_STRIDE;
          const uint32_t d_o = tmem_base + G::O_COL;
          if (j > 0) {
#pragma unroll
            for (int k = 0; k < G::BK / 16; ++k) {
#ifndef WAVEAL_DBG_SKIP_PV
              umma_bf16_ts(d_o, pbase + k * 8, vd + (uint64_t)((k * 16 * 128) >> 4), IDESC_PV, 1u);
#endif
            }
          } else {
#pragma unroll
            for (int k = 0; k < G::BK / 16; ++k) {
#ifndef WAVEAL_DBG_SKIP_PV
              umma_bf16_ts(d_o, pbase + k * 8, vd + (uint64_t)((k * 16 * 128) >> 4), IDESC_PV, k > 0 ? 1u : 0u);
#endif
            }
          }
          tc_commit(BAR(B_KV_EMPTY + kv_st));
          tc_commit(BAR(B_PV_DONE));
          if (j == n - 1) tc_commit(BAR(B_O_FULL));
        }
        TRACE(0, 3, j);
        if (++kv_st == (uint32_t)G::NSTAGE) { kv_st = 0; kv_ph ^= 1; }
        if (more_qk) {
          ok = finish_wait(ctx, BAR(B_KV_FULL + kv_st), kv_ph, tok_k, 12);
          if (!ok) break;
        }
        // answers for the next P V (its V tile follows the K tile just checked)
        if (j + 1 < n) {
          uint32_t v_st = kv_st, v_ph = kv_ph;
          if (more_qk) { if (++v_st == (uint32_t)G::NSTAGE) { v_st = 0; v_ph ^= 1; } }
          const uint32_t nsb = (sb + 1 == (uint32_t)G::NSBUF) ? 0u : sb + 1;
          tok_p = mbar_test_wait(BAR(B_P_FULL + nsb), (p_phase >> nsb) & 1u);
          tok_v = mbar_test_wait(BAR(B_KV_FULL + v_st), v_ph);
        }
        if (more_qk) {
          issue_qk(sb);
          if (j + G::NSBUF == n - 1) tc_commit(BAR(B_Q_EMPTY));
        }
        if (++sb == (uint32_t)G::NSBUF) sb = 0;
      }
    }
    // every MMA issued by this warp has completed before tensor memory is released
    tc_commit(BAR(B_FINAL));
    __syncwarp();
    {
      long long t0 = clock64();
      while (!mbar_try_wait(BAR(B_FINAL), 0) && clock64() - t0 < kTimeoutCycles / 4) {}
    }
  } else {
    // ============================================================== softmax / epilogue
    // All eight warps work on every block: thread (row, half) owns half a row of S, so two
    // warps per scheduler interleave and hide each other's latencies; the two halves of a row
    // exchange their maxima through shared memory (one 64-thread named barrier per block).
    const int sw = warp - kSoftmaxWarp0;       // 0..7
    const int quad = warp & 3;                 // tensor-memory lane quadrant this warp may access
    const int half = sw >> 2;                  // which half of the S / O columns
    const int r = quad * 32 + lane;            // row of the 128-row MMA tile
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t o_addr = tmem_base + lane_addr + G::O_COL + half * G::CO;
    uint32_t task_it = 0, s_phase = 0, o_it = 0, pv_total = 0, blk_it = 0;
    TRACE_DECL;
    bool ok = true;
    while (ok) {
      const uint32_t slot = task_it & 1, ph = (task_it >> 1) & 1;
      ok = warp_wait(ctx, BAR(B_TASK_FULL + slot), ph, 20);
      if (!ok) break;
      const Task tk = tasks[slot];
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_TASK_EMPTY + slot));
      ++task_it;
      if (tk.n < 0) break;
      const long long q_tok = (long long)tk.row * G::BQ + r;
      const bool row_live = r < G::BQ && q_tok < p.seq_q;
      __nv_bfloat16* o_ptr = p.O + (size_t)tk.h * p.o_stride_h + (size_t)q_tok * p.o_stride_t + half * G::CO;
      if (tk.n == 0) {
        if (row_live) {
#pragma unroll
          for (int c = 0; c < G::CO / 8; ++c) reinterpret_cast<uint4*>(o_ptr)[c] = make_uint4(0, 0, 0, 0);
          if (p.lse && half == 0) p.lse[(size_t)tk.h * p.seq_q + q_tok] = -INFINITY;
        }
        continue;
      }
      float m_used = -INFINITY, l_run = 0.f;
      uint32_t sb = 0;
      for (int j = 0; j < tk.n && ok; ++j) {
        ok = warp_wait(ctx, BAR(B_S_FULL + sb), (s_phase >> sb) & 1u, 21);
        if (!ok) break;
        s_phase ^= 1u << sb;
        if (sw == 2 || sw == 6) TRACE(1 + half, 10 + half, j);
        tc_fence_after();
        const uint32_t s_addr = tmem_base + lane_addr + sb * G::S_STRIDE;
        uint32_t sv[G::CS];
        if constexpr (G::CS == 64) {
          WAVEAL_TMEM_LD32(s_addr + half * 64, sv, 0);
          WAVEAL_TMEM_LD32(s_addr + half * 64 + 32, sv, 32);
          WAVEAL_TMEM_WAIT_LD32(sv, 0);
          WAVEAL_TMEM_WAIT_LD32(sv, 32);
        } else {
          WAVEAL_TMEM_LD32(s_addr + half * 32, sv, 0);
          WAVEAL_TMEM_WAIT_LD32(sv, 0);
        }
        if (sw == 2 || sw == 6) TRACE(1 + half, 12 + half, j);
        // scores of keys beyond seq_kv (ragged last block) do not exist
        if (j == tk.n - 1 && tk.tail_valid < G::BK) {
#pragma unroll
          for (int c = 0; c < G::CS; ++c)
            if (half * G::CS + c >= tk.tail_valid) sv[c] = __float_as_uint(-INFINITY);
        }
        // row max: eight independent chains, then the other half of the row through smem
        float mx8[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) mx8[i] = __uint_as_float(sv[i]);
#pragma unroll
        for (int c = 8; c < G::CS; c += 8) {
#pragma unroll
          for (int i = 0; i < 8; ++i) mx8[i] = fmaxf(mx8[i], __uint_as_float(sv[c + i]));
        }
        const float mloc = fmaxf(fmaxf(fmaxf(mx8[0], mx8[1]), fmaxf(mx8[2], mx8[3])),
                                 fmaxf(fmaxf(mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])));
        float* mxb = mx + (blk_it & 1) * 256;
        ++blk_it;
        mxb[half * 128 + r] = mloc;
        named_bar_sync(1 + quad, 64);
        const float m_cand = fmaxf(m_used, fmaxf(mloc, mxb[(half ^ 1) * 128 + r]) * p.sl2);
        // keep the stale reference max unless it is exceeded by more than 2^8 (exact: the
        // final normalisation divides by a sum taken with the same reference); both halves of a
        // row see the same numbers and the two warps hold the same rows, so they decide alike
        const bool grow = __any_sync(0xffffffffu, m_cand > m_used + 8.0f);
        float alpha = 1.f;
        if (grow) {
          alpha = (m_used == -INFINITY) ? 0.f : ex2(m_used - m_cand);
          m_used = m_cand;
          l_run *= alpha;
        }
        uint32_t pk[G::PC];
        float ls4[4] = {0.f, 0.f, 0.f, 0.f};
        // p' = 2^(s*scale*log2e - m + log2(1 + 2^-9)); P is p' cut to its top 16 bits (one byte
        // permute per pair instead of a conversion on the transcendental pipe).  The extra
        // factor centres the cut's error around zero, and the row sum adds the SAME cut values
        // the tensor core multiplies with, so numerator and denominator stay consistent.
        const float neg_m = ((m_used == -INFINITY) ? 0.f : -m_used) + 0.0028150156f;
#pragma unroll
        for (int c = 0; c < G::CS; c += 2) {
          const float x0 = fmaf(__uint_as_float(sv[c]), p.sl2, neg_m);
          const float x1 = fmaf(__uint_as_float(sv[c + 1]), p.sl2, neg_m);
          // every kPolyEvery-th pair takes the polynomial path (a fixed pattern per column, so
          // the result of a row does not depend on the execution order)
          const bool poly = kPolyEvery > 0 && ((c >> 1) % (kPolyEvery > 0 ? kPolyEvery : 1)) == (kPolyEvery - 1);
          const uint32_t b0 = __float_as_uint(poly ? ex2_fma(x0) : ex2(x0));
          const uint32_t b1 = __float_as_uint(poly ? ex2_fma(x1) : ex2(x1));
          ls4[(c >> 1) & 3] += __uint_as_float(b0 & 0xFFFF0000u) + __uint_as_float(b1 & 0xFFFF0000u);
          pk[c / 2] = __byte_perm(b0, b1, 0x7632);
        }
        l_run += (ls4[0] + ls4[1]) + (ls4[2] + ls4[3]);
        if (sw == 2 || sw == 6) TRACE(1 + half, 14 + half, j);
        // rare: the reference grew, so the accumulated O is rescaled; P_{j-1} V_{j-1} (the last MMA
        // that touches O) must be complete - the barrier has seen exactly pv_total + j - 1 or
        // pv_total + j phases by now, so a parity wait is unambiguous
        if (grow && j > 0) {
          ok = warp_wait(ctx, BAR(B_PV_DONE), (pv_total + (uint32_t)j - 1u) & 1u, 22);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int c0 = 0; c0 < G::CO; c0 += 32) {
            uint32_t ov[32];
            WAVEAL_TMEM_LD32(o_addr + c0, ov, 0);
            WAVEAL_TMEM_WAIT_LD32(ov, 0);
#pragma unroll
            for (int c = 0; c < 32; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * alpha);
            WAVEAL_TMEM_ST32(o_addr + c0, ov, 0);
          }
        }
        // P_j (bf16 pairs) over the first half of the columns of S[sb]
        if constexpr (G::PC == 32) { WAVEAL_TMEM_ST32(s_addr + half * 32, pk, 0); }
        else { WAVEAL_TMEM_ST16(s_addr + half * 16, pk, 0); }
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(B_P_FULL + sb));
        if (sw == 2 || sw == 6) TRACE(1 + half, 16 + half, j);
        if (++sb == (uint32_t)G::NSBUF) sb = 0;
      }
      if (!ok) break;
      pv_total += (uint32_t)tk.n;
      // ---- epilogue: O / l at the original row position
      ok = warp_wait(ctx, BAR(B_O_FULL), o_it & 1, 23);
      if (!ok) break;
      ++o_it;
      tc_fence_after();
      if (sw == 2 || sw == 6) TRACE(1 + half, 18 + half, tk.n);
      float* lx = mx + (blk_it & 1) * 256;      // the buffer the last block did not use
      ++blk_it;
      lx[half * 128 + r] = l_run;
      named_bar_sync(1 + quad, 64);
      const float l_tot = l_run + lx[(half ^ 1) * 128 + r];
      const float inv_l = 1.0f / l_tot;
      uint32_t ov[G::CO];
#pragma unroll
      for (int c = 0; c < G::CO; c += 32) WAVEAL_TMEM_LD32(o_addr + c, ov, c);
#pragma unroll
      for (int c = 0; c < G::CO; c += 32) WAVEAL_TMEM_WAIT_LD32(ov, c);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_O_FREE));
      if (sw == 2 || sw == 6) TRACE(1 + half, 30 + half, tk.n);
      if (row_live) {
#pragma unroll
        for (int c = 0; c < G::CO; c += 8) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(ov[c + 2 * e]) * inv_l,
                                                      __uint_as_float(ov[c + 2 * e + 1]) * inv_l);
            w[e] = *reinterpret_cast<uint32_t*>(&b2);
          }
          *reinterpret_cast<uint4*>(o_ptr + c) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        if (p.lse && half == 0) p.lse[(size_t)tk.h * p.seq_q + q_tok] = (m_used + log2f(l_tot)) * 0.6931471805599453f;
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, G::TMEM_COLS);
  }
}

// ------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// bf16 tensor [heads][seq][head_dim] with element strides {head, token}; box = 64 columns x rows
waveal_status make_map(CUtensorMap* tm, const void* base, int head_dim, int seq, int heads, long long stride_h,
                       long long stride_t, int box_rows, const char* what) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return waveal::fail(WAVEAL_ERR_CUDA, "cuTensorMapEncodeTiled entry point not available");
  cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)seq, (cuuint64_t)heads};
  cuuint64_t strides[2] = {(cuuint64_t)stride_t * 2, (cuuint64_t)stride_h * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return waveal::fail(WAVEAL_ERR_CUDA, "tensor map for %s rejected (CUresult %d)", what, (int)r);
  return WAVEAL_OK;
}

waveal_status check_desc(const waveal_attn_desc* d) {
  if (!d) return waveal::fail(WAVEAL_ERR_INVALID_ARG, "desc is NULL");
  if (d->heads <= 0 || d->seq_q <= 0 || d->seq_kv <= 0)
    return waveal::fail(WAVEAL_ERR_INVALID_ARG, "heads, seq_q and seq_kv must be positive");
  if (d->head_dim != 64 && d->head_dim != 128)
    return waveal::fail(WAVEAL_ERR_UNSUPPORTED, "head_dim %d (supported: 64, 128)", d->head_dim);
  if (d->block_q != d->block_kv || (d->block_q != 64 && d->block_q != 128))
    return waveal::fail(WAVEAL_ERR_UNSUPPORTED, "block %dx%d (supported: 64x64, 128x128)", d->block_q, d->block_kv);
  const int64_t* strides[4] = {d->q_stride, d->k_stride, d->v_stride, d->o_stride};
  for (int i = 0; i < 4; ++i) {
    if (strides[i][1] < d->head_dim || strides[i][0] < 0)
      return waveal::fail(WAVEAL_ERR_INVALID_ARG, "token stride must be >= head_dim and head stride >= 0");
    if (strides[i][0] % 8 || strides[i][1] % 8)
      return waveal::fail(WAVEAL_ERR_INVALID_ARG, "strides must be multiples of 8 elements (16 bytes)");
  }
  return WAVEAL_OK;
}

template <int BLOCK, int D>
waveal_status launch(const waveal_attn_desc* d, const void* Q, const void* K, const void* V, AttnParams& p,
                     int sms, cudaStream_t st) {
  using G = Geo<BLOCK, D>;
  CUtensorMap tq, tk, tv;
  waveal_status s;
  if ((s = make_map(&tq, Q, D, d->seq_q, d->heads, d->q_stride[0], d->q_stride[1], BLOCK, "Q")) != WAVEAL_OK) return s;
  if ((s = make_map(&tk, K, D, d->seq_kv, d->heads, d->k_stride[0], d->k_stride[1], BLOCK, "K")) != WAVEAL_OK) return s;
  if ((s = make_map(&tv, V, D, d->seq_kv, d->heads, d->v_stride[0], d->v_stride[1], BLOCK, "V")) != WAVEAL_OK) return s;
  WAVEAL_CUDA_OK(cudaFuncSetAttribute(k_bsattn_fwd<BLOCK, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM_BYTES));
  WAVEAL_CUDA_OK(cudaMemsetAsync(p.ws, 0, 16, st));  // ticket counter, abort flag (and the debug trace count)
  long long grid = p.total_tasks < sms ? p.total_tasks : sms;
  k_bsattn_fwd<BLOCK, D><<<(unsigned)grid, kThreads, G::SMEM_BYTES, st>>>(tq, tk, tv, p);
  WAVEAL_CUDA_OK(cudaGetLastError());
  waveal::launch_counter() = 1;
  return WAVEAL_OK;
}

}  // namespace

extern "C" waveal_status waveal_bsattn_workspace_bytes(const waveal_attn_desc* desc, size_t* bytes) {
  waveal_status s = check_desc(desc);
  if (s != WAVEAL_OK) return s;
  if (!bytes) return waveal::fail(WAVEAL_ERR_INVALID_ARG, "bytes is NULL");
  *bytes = 256;
  return WAVEAL_OK;
}

extern "C" waveal_status waveal_bsattn_fwd(const waveal_attn_desc* d, const void* Q, const void* K, const void* V,
                                           void* O, float* lse, const int32_t* kv_row_ptr,
                                           const int32_t* kv_block_indices, const int32_t* row_order, float scale,
                                           void* ws, size_t ws_bytes, int32_t* dev_status, void* cuda_stream) {
  waveal_status s = check_desc(d);
  if (s != WAVEAL_OK) return s;
  if (!Q || !K || !V || !O) return waveal::fail(WAVEAL_ERR_INVALID_ARG, "Q, K, V and O are required");
  if (!kv_row_ptr || !kv_block_indices) return waveal::fail(WAVEAL_ERR_INVALID_ARG, "index lists are required");
  if (!waveal::aligned(Q, 16) || !waveal::aligned(K, 16) || !waveal::aligned(V, 16) || !waveal::aligned(O, 16))
    return waveal::fail(WAVEAL_ERR_INVALID_ARG, "Q, K, V and O must be 16-byte aligned");
  if (!ws || ws_bytes < 256) return waveal::fail(WAVEAL_ERR_WORKSPACE, "workspace of 256 bytes needed");
  if (!waveal::aligned(ws, 16)) return waveal::fail(WAVEAL_ERR_INVALID_ARG, "workspace must be 16-byte aligned");
  if (!(scale == scale) || std::isinf(scale)) return waveal::fail(WAVEAL_ERR_INVALID_ARG, "scale is not finite");
  int dev = 0, sms = 0, major = 0;
  WAVEAL_CUDA_OK(cudaGetDevice(&dev));
  WAVEAL_CUDA_OK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  if (major != 10) return waveal::fail(WAVEAL_ERR_UNSUPPORTED, "device compute capability %d.x; sm_100a is required", major);
  WAVEAL_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  AttnParams p{};
  p.O = static_cast<__nv_bfloat16*>(O);
  p.lse = lse;
  p.row_ptr = kv_row_ptr; p.kv_idx = kv_block_indices; p.row_order = row_order;
  p.ws = static_cast<int*>(ws); p.dev_status = dev_status;
  p.o_stride_h = d->o_stride[0]; p.o_stride_t = d->o_stride[1];
  p.heads = d->heads;
  p.m_b = (d->seq_q + d->block_q - 1) / d->block_q;
  p.n_b = (d->seq_kv + d->block_kv - 1) / d->block_kv;
  p.seq_q = d->seq_q; p.seq_kv = d->seq_kv;
  p.interleaved = d->order_heads_interleaved ? 1 : 0;
  p.total_tasks = (long long)d->heads * p.m_b;
  const float sc = scale > 0.f ? scale : 1.0f / sqrtf((float)d->head_dim);
  p.sl2 = sc * 1.4426950408889634f;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (d->block_q == 128 && d->head_dim == 128) return launch<128, 128>(d, Q, K, V, p, sms, st);
  if (d->block_q == 64 && d->head_dim == 128) return launch<64, 128>(d, Q, K, V, p, sms, st);
  if (d->block_q == 64 && d->head_dim == 64) return launch<64, 64>(d, Q, K, V, p, sms, st);
  if (d->block_q == 128 && d->head_dim == 64) return launch<128, 64>(d, Q, K, V, p, sms, st);
  return waveal::fail(WAVEAL_ERR_UNSUPPORTED, "no kernel for block %d, head_dim %d", d->block_q, d->head_dim);
}
