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
// Structure of one CTA (608 threads; 640 in the kernels of the 64-row blocks):
//   warp 0      producer: takes tickets, publishes tasks, issues TMA loads of the Q tile and
//               of the K and V tiles (128-byte-swizzled slabs) into two shared-memory rings
//   warp 19     64-row blocks only: requests the V tiles instead of warp 0 (a tile of that shape
//               takes two list entries and up to four boxes; one warp for both streams was the
//               limit of the whole kernel there)
//   warp 18     MMA issuer 1: S_j = Q K_j^T (operands in shared memory) into one of three S
//               buffers in tensor memory, up to three blocks ahead of the softmax
//   warp 1      MMA issuer 2: O += P_j V_j (P read from tensor memory, where it lies over the
//               columns S_j came from), fp32 accumulator in tensor memory.  Two issuing warps:
//               the waits and ring arithmetic of one run while the other's MMAs execute
//   warps 2-17  softmax, two teams of eight warps that take the KV blocks of a task in turn;
//               inside a team a row of S has two owners, one per half of its columns (row max
//               in the blocks that take one, then exponentials and P in a second read of S,
//               32 columns at a time in a rolled loop).  On every scheduler two warps of each
//               team are resident, the teams half a block apart, so one team's waits and loads
//               hide behind the other's arithmetic.  The teams hand each other the running
//               reference max of every row through shared memory; every thread keeps the row
//               sum of its own columns; O in tensor memory is rescaled only when the max grew
//               by more than 2^8; the epilogue adds the four partial sums of a row, normalises
//               and stores O at the ORIGINAL row (no inverse permutation)
// Two launches per call: in the first the row max is taken in blocks 0 and 1 of a task only and
// the reference stays fixed afterwards (softmax does not depend on it short of overflow); a task
// in which a block's sum of exponentials reaches 2^24 is listed in the workspace and computed
// again by the second launch, which takes the max of every block.
// Every wait on an mbarrier is bounded; when one runs out the CTA records
// {WAVEAL_ERR_TIMEOUT, site} and all roles leave through the common teardown.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cmath>
#include "host_common.h"

namespace {

// 19 warps, and a 20th (the V tile loader) in the kernels of the 64-row blocks
template <int BLOCK> constexpr int kThreadsOf = BLOCK == 64 ? 640 : 608;
constexpr int kProducerWarp = 0, kPvWarp = 1, kSoftmaxWarp0 = 2, kQkWarp = 18, kVLoadWarp = 19;
constexpr long long kTimeoutCycles = 4000000000ll;   // ~2 s at boost clock
constexpr long long kSelfTestCycles = 4000000ll;     // ~2 ms: wait limit under WAVEAL_ATTN_SELFTEST_LOST_TILE
#ifndef WAVEAL_POLY_EVERY
#define WAVEAL_POLY_EVERY 4
#endif
constexpr int kPolyEvery = WAVEAL_POLY_EVERY;          // n > 0: 1 pair of elements in n takes 2^x from the FMA pipe (0 = all from the transcendental unit)

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

// two fp32 operations per instruction (register pairs)
__device__ __forceinline__ void ffma2(float& d0, float& d1, float a0, float a1, float b0, float b1, float c0, float c1) {
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\tmov.b64 ra, {%2,%3};\n\tmov.b64 rb, {%4,%5};\n\tmov.b64 rc, {%6,%7};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0,%1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b0), "f"(b1), "f"(c0), "f"(c1));
}
__device__ __forceinline__ void fadd2(float& d0, float& d1, float a0, float a1, float b0, float b1) {
  asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2,%3};\n\tmov.b64 rb, {%4,%5};\n\t"
      "add.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0,%1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}

// 2^(x) for two values on the FMA and integer pipes (for a share of the elements, to take load
// off the transcendental unit: at 16 results per clock and SM it is as busy as the tensor
// cores).  The caller passes s and the pair (a, b) of x = a*s + b.  The argument is first
// confined to the window [kPolyLo, kPolyLo + 128] by a saturating multiply-add
// (y = sat(x/128 - kPolyLo/128) in [0, 1]; x is taken back from y with an absolute error
// below 2^-17), so that the exponent arithmetic below can neither wrap into the sign bit
// (x >= 128.5 would) nor underflow: an x above the window comes out as 2^(kPolyLo+128) = 2^28,
// far above the limit at which the fixed-reference pass hands a task to the second launch; an x
// below it (a key that does not exist, -inf) as 2^-100.  x is then rounded to the nearest integer
// n with the 1.5*2^23 trick, a degree-3 polynomial gives 2^(x-n) on [-0.5, 0.5] (relative error
// 7.5e-5, far below the bf16 cut of P), and n is added to the exponent field.
constexpr float kPolyLo = -100.0f;
constexpr float kRedoLimit = 16777216.0f;     // 2^24: block sums at or above it (or NaN) list the task
__device__ __forceinline__ float fma_sat(float a, float b, float c) {
  float d;
  asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ void ex2_fma2(float& e0, float& e1, float s0, float s1, float a128, float b128) {
  // a128 = a/128, b128 = (b - kPolyLo)/128
  const float y0 = fma_sat(s0, a128, b128), y1 = fma_sat(s1, a128, b128);
  constexpr float kMagic = 12582912.0f;                 // 1.5 * 2^23
  float xi0, xi1, n0, n1, f0, f1, q0, q1;
  ffma2(xi0, xi1, y0, y1, 128.0f, 128.0f, kMagic + kPolyLo, kMagic + kPolyLo);   // bits: 0x4B400000 + n
  fadd2(n0, n1, xi0, xi1, -(kMagic + kPolyLo), -(kMagic + kPolyLo));             // n - kPolyLo = round(128 y)
  ffma2(f0, f1, y0, y1, 128.0f, 128.0f, -n0, -n1);                               // x - n
  ffma2(q0, q1, f0, f1, 0.05517137423157692f, 0.05517137423157692f, 0.2426110953092575f, 0.2426110953092575f);
  ffma2(q0, q1, q0, q1, f0, f1, 0.6932610273361206f, 0.6932610273361206f);
  ffma2(q0, q1, q0, q1, f0, f1, 0.9999280571937561f, 0.9999280571937561f);
  e0 = __int_as_float(__float_as_int(q0) + (__float_as_int(xi0) << 23));
  e1 = __int_as_float(__float_as_int(q1) + (__float_as_int(xi1) << 23));
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

// 16 consecutive fp32 columns
#define WAVEAL_TMEM_LD16(taddr, v, o)                                                            \
  asm volatile(                                                                                  \
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "                                                  \
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"           \
      : "=r"(v[o+0]), "=r"(v[o+1]), "=r"(v[o+2]), "=r"(v[o+3]), "=r"(v[o+4]), "=r"(v[o+5]), "=r"(v[o+6]), "=r"(v[o+7]), \
        "=r"(v[o+8]), "=r"(v[o+9]), "=r"(v[o+10]), "=r"(v[o+11]), "=r"(v[o+12]), "=r"(v[o+13]), "=r"(v[o+14]), "=r"(v[o+15]) \
      : "r"(taddr)                                                                               \
      : "memory")
#define WAVEAL_TMEM_WAIT_LD16(v, o)                                                              \
  asm volatile("tcgen05.wait::ld.sync.aligned;"                                                  \
      : "+r"(v[o+0]), "+r"(v[o+1]), "+r"(v[o+2]), "+r"(v[o+3]), "+r"(v[o+4]), "+r"(v[o+5]), "+r"(v[o+6]), "+r"(v[o+7]), \
        "+r"(v[o+8]), "+r"(v[o+9]), "+r"(v[o+10]), "+r"(v[o+11]), "+r"(v[o+12]), "+r"(v[o+13]), "+r"(v[o+14]), "+r"(v[o+15]) \
      ::"memory")
#define WAVEAL_TMEM_ST16(taddr, v, o)                                                            \
  asm volatile(                                                                                  \
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "                                           \
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};"                  \
      ::"r"(v[o+0]), "r"(v[o+1]), "r"(v[o+2]), "r"(v[o+3]), "r"(v[o+4]), "r"(v[o+5]), "r"(v[o+6]), "r"(v[o+7]), \
        "r"(v[o+8]), "r"(v[o+9]), "r"(v[o+10]), "r"(v[o+11]), "r"(v[o+12]), "r"(v[o+13]), "r"(v[o+14]), "r"(v[o+15]), \
        "r"(taddr)                                                                               \
      : "memory")

// one 32-byte store (the address must be 32-byte aligned)
__device__ __forceinline__ void st_global_v8(void* ptr, const uint32_t* w) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"l"(ptr), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
               : "memory");
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
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

// n: KV tiles of the task (a tile = 128 keys = 128/block consecutive entries of the row's list),
// len: entries of the list, tail_valid: keys of the last tile that exist.
// row2 (64-row query blocks only): a second query block with the very same list, or -1; its rows
// fill the other half of the 128-row MMA tile, so the pair costs what one block costs.  The
// ticket of the second block of a pair carries n = kAbsorbed and is skipped by whoever draws it.
struct Task { int h, row, lo, n, tail_valid, len, row2, pad2; };
constexpr int kAbsorbed = -2;

// tiles, list length and valid keys of the last tile from a list of `len` blocks of `block` keys
// whose last entry is `last`
__host__ __device__ inline void fill_tiles(Task& tk, int len, int block, int last, int n_b, int seq_kv) {
  const int kb = 128 / block;
  tk.len = len;
  tk.n = (len + kb - 1) / kb;
  tk.tail_valid = 128;
  if (len > 0) {
    tk.tail_valid = (len - (tk.n - 1) * kb) * block;
    if ((seq_kv % block) != 0 && last == n_b - 1) tk.tail_valid -= block - seq_kv % block;
  }
}

struct AttnParams {
  __nv_bfloat16* O;
  float* lse;
  const int* row_ptr;
  const int* kv_idx;
  const int* row_order;
  int* ws;            // [0] ticket counter, [1] abort flag, [2] number of tasks to redo, [3] ticket counter of
                      // the redo pass, [8 + 2i], [9 + 2i] = (head, query block) of redo entry i
  int redo_pass;      // 0: all tasks by ticket; 1: only the tasks the first pass listed
  const Task* table;         // task of every ticket of the first pass (k_task_table)
  int* dev_status;
  long long o_stride_h, o_stride_t;
  int heads, m_b, n_b, seq_q, seq_kv, interleaved;
  long long total_tasks;
  long long wait_limit;   // cycles a bounded wait may take (kTimeoutCycles; far shorter under the self-test flag)
  int drop_tile;          // self-test: the producer never loads the first K tile of ticket 0
  int no_pairing;         // 64-row blocks: never put two blocks with identical lists into one tile
  float sl2;          // scale * log2(e)
};


template <int BLOCK, int D>
struct Geo {
  // A KV tile is always 128 keys wide: one 128-key block, or two 64-key blocks that follow each
  // other in the row's list (their rows land one after the other in the tile, so the MMAs, the
  // softmax and the rings see the same shapes for both block sizes; a list of odd length ends
  // in a half tile whose missing keys are treated like keys beyond the sequence end)
  static constexpr int BQ = BLOCK, BK = 128, KB = 128 / BLOCK;
  static constexpr int SLABS = D / 64;               // 128-byte column slabs of a Q/K/V tile
  static constexpr int Q_BYTES = SLABS * 128 * 128;  // smem reserved for the 128 MMA rows
  static constexpr int TILE_BYTES = SLABS * BK * 128;
  static constexpr int KV_SLAB_BYTES = BK * 128;
  static constexpr int NSTAGE_RAW = (200 * 1024 - Q_BYTES) / TILE_BYTES;
  static constexpr int NSTAGE = NSTAGE_RAW > 8 ? 8 : NSTAGE_RAW;
  static constexpr int NKS = (NSTAGE + 1) / 2;       // K tile ring
  static constexpr int NVS = NSTAGE / 2;             // V tile ring
  static constexpr int NSBUF = 3;                    // S/P buffers in tensor memory
  static constexpr bool SPLIT_LOADERS = KB == 2;     // K and V tiles requested by a warp each (else one warp, interleaved)
  static constexpr int HC = BK / 2;                  // S columns of a row one softmax thread owns (a row has two owners)
  static constexpr int CH = 32;                      // S columns a softmax thread holds at a time
  static constexpr int NCH = HC / CH;                // such chunks per thread and block
  static constexpr int CO = D / 4;                   // O columns per epilogue thread
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = OFF_Q + Q_BYTES;
  static constexpr int OFF_V = OFF_K + NKS * TILE_BYTES;
  static constexpr int OFF_BAR = OFF_V + NVS * TILE_BYTES;
  static constexpr int N_BAR = 4 + 2 + 2 * NKS + 2 * NVS + 4 * NSBUF + 2 + 2 + 8 + 4 + 8;
  static constexpr int OFF_TASK = OFF_BAR + ((N_BAR * 8 + 15) / 16) * 16;
  static constexpr int OFF_MX = OFF_TASK + 2 * (int)sizeof(Task);
  static constexpr int OFF_MISC = OFF_MX + 4 * 128 * 4 + 2 * 2 * 2 * 128 * 4 + 2 * 4 * 128 * 8;
  static constexpr int SMEM_BYTES = OFF_MISC + 32 + 1024;   // + slack for 1024-byte alignment
  // tensor memory: three S/P buffers of 128 columns, then the output accumulator
  static constexpr uint32_t S_STRIDE = 128, O_COL = 384, TMEM_COLS = 512;
};

struct Ctx {
  uint32_t bar_base;
  volatile int* abort_smem;
  int* ws;
  int* dev_status;
  long long limit;      // cycles a wait may take before the CTA gives up
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
    if (clock64() - t0 > c.limit) { signal_abort(c, site); return false; }
  }
}

// same, with one answer for the whole warp (the roles use warp-collective instructions).  All
// lanes wait: a warp suspended as a whole in try_wait takes no issue slots, which measured
// better than polling and far better than one waiting lane with the rest at the vote.
__device__ __forceinline__ bool warp_wait(const Ctx& c, uint32_t bar, uint32_t parity, int site) {
  return __all_sync(0xffffffffu, mbar_wait(c, bar, parity, site));
}

// One K or V tile of a task into its ring stage (called by a whole warp).  Tile j covers entries
// KB*j .. of the row's list (the last tile of an odd list of 64-key blocks has one block).
// State of the caller: it (tiles loaded so far), armed / parity (per stage: a load is in flight,
// and the parity its barrier completes with), chunk_base / my_idx (32 list entries at a time,
// one per lane).  dropped: self-test of the abort path, the tile is never requested.
template <class G, int BLOCK, bool IS_K>
__device__ __forceinline__ bool load_kv_tile(const Ctx& ctx, const AttnParams& p, const Task& tk, bool dropped, int j,
                                             int lane, uint32_t sbase, uint32_t bar_full0, uint32_t bar_empty0,
                                             const CUtensorMap* tm, const CUtensorMap* tm2, uint32_t& it,
                                             uint32_t& armed, uint32_t& parity, int& chunk_base, int& my_idx) {
  constexpr uint32_t NST = IS_K ? G::NKS : G::NVS;
  auto entry = [&](int q) -> int {
    if (q < chunk_base || q >= chunk_base + 32) {
      chunk_base = q & ~31;
      const int e = chunk_base + lane;
      my_idx = e < tk.len ? p.kv_idx[tk.lo + e] : 0;
    }
    int blk = __shfl_sync(0xffffffffu, my_idx, q - chunk_base);
    if (blk < 0 || blk >= p.n_b) {                   // malformed list: report it and stay in range
      if (lane == 0 && p.dev_status && atomicCAS(p.dev_status, 0, WAVEAL_ERR_BAD_MASK) == 0) {
        p.dev_status[1] = 30; p.dev_status[2] = tk.h; p.dev_status[3] = blk;
      }
      blk = 0;
    }
    return blk;
  };
  const int nblk = G::KB == 1 ? 1 : min(G::KB, tk.len - G::KB * j);
  int blk[G::KB];
#pragma unroll
  for (int e = 0; e < G::KB; ++e) blk[e] = e < nblk ? entry(G::KB * j + e) : 0;
  const uint32_t st = it % NST, sph = (it / NST) & 1;
  const uint32_t b_full = bar_full0 + 8u * st, b_empty = bar_empty0 + 8u * st;
  if (!warp_wait(ctx, b_empty, sph ^ 1, IS_K ? 3 : 4)) return false;
  ++it;
  if (dropped) return true;
  // one lane per box: lane e*SLABS + s requests slab s of block e
  if (lane == 0) mbar_expect_tx(b_full, (uint32_t)nblk * G::SLABS * BLOCK * 128);
  __syncwarp();
  const uint32_t dst = sbase + (IS_K ? G::OFF_K : G::OFF_V) + st * G::TILE_BYTES;
  const int e = lane / G::SLABS, sl = lane % G::SLABS;
  // two 64-key blocks that follow each other in memory come as one box of 128 rows per slab
  const bool joined = G::KB == 2 && nblk == 2 && blk[G::KB - 1] == blk[0] + 1;
  if (joined) {
    if (e == 0) tma_load_3d(dst + sl * G::KV_SLAB_BYTES, tm2, sl * 64, blk[0] * BLOCK, tk.h, b_full);
  } else {
    int my_blk = blk[0];
#pragma unroll
    for (int i = 1; i < G::KB; ++i) if (e == i) my_blk = blk[i];
    if (e < nblk) tma_load_3d(dst + sl * G::KV_SLAB_BYTES + e * BLOCK * 128, tm, sl * 64, my_blk * BLOCK, tk.h, b_full);
  }
  armed |= 1u << st;
  parity = (parity & ~(1u << st)) | (sph << st);
  return true;
}

template <int BLOCK, int D, bool FAST>
__global__ void __launch_bounds__(kThreadsOf<BLOCK>, 1)
k_bsattn_fwd(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
             const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmK2,
             const __grid_constant__ CUtensorMap tmV2, const AttnParams p) {
  // tmK2 / tmV2: the same K and V with boxes of 128 rows, used by the 64-key-block kernels when the
  // two blocks of a tile lie next to each other in memory (for 128-key blocks they equal tmK / tmV)
  using G = Geo<BLOCK, D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);   // provably warp-uniform role index

  // second pass with nothing listed (or after an abort): leave before anything is set up
  if (p.redo_pass && (p.ws[2] == 0 || p.ws[1] != 0)) return;

  const uint32_t bar0 = sbase + G::OFF_BAR;
  auto BAR = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  constexpr int B_TASK_FULL = 0, B_TASK_EMPTY = 2, B_Q_FULL = 4, B_Q_EMPTY = 5, B_K_FULL = 6,
                B_K_EMPTY = B_K_FULL + G::NKS, B_V_FULL = B_K_EMPTY + G::NKS, B_V_EMPTY = B_V_FULL + G::NVS,
                B_S_FULL = B_V_EMPTY + G::NVS, B_P_FULL = B_S_FULL + G::NSBUF, B_S_FREE = B_P_FULL + 2 * G::NSBUF,
                B_O_FULL = B_S_FREE + G::NSBUF, B_O_FREE = B_O_FULL + 1, B_FINAL = B_O_FREE + 1, B_MX = B_FINAL + 2,
                B_EX = B_MX + 8, B_HX = B_EX + 4;
  static_assert(B_HX + 8 <= G::N_BAR, "barrier count");
  Task* tasks = reinterpret_cast<Task*>(smem + G::OFF_TASK);
  volatile float* mpub = reinterpret_cast<volatile float*>(smem + G::OFF_MX);   // [block index mod 4][128] reference max after a block
  volatile float* mhalf = reinterpret_cast<volatile float*>(smem + G::OFF_MX + 4 * 128 * 4);   // [use parity][team][column half][128] max of a half row
  float2* ex = reinterpret_cast<float2*>(smem + G::OFF_MX + 4 * 128 * 4 + 2 * 2 * 2 * 128 * 4);    // [task parity][team*2+half][128] (reference, sum)
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + G::OFF_MISC);
  volatile int* abort_smem = reinterpret_cast<volatile int*>(smem + G::OFF_MISC + 4);
  volatile int* redo_flag = reinterpret_cast<volatile int*>(smem + G::OFF_MISC + 8);   // [task parity]
  Ctx ctx{bar0, abort_smem, p.ws, p.dev_status, p.wait_limit};
  const long long t_start = clock64();

  if (tid == 0) {
    // a task is read by the V loader, the two MMA issuers and the sixteen softmax warps
    for (int i = 0; i < 2; ++i) { mbar_init(BAR(B_TASK_FULL + i), 1); mbar_init(BAR(B_TASK_EMPTY + i), G::SPLIT_LOADERS ? 19 : 18); }
    mbar_init(BAR(B_Q_FULL), 1);
    mbar_init(BAR(B_Q_EMPTY), 1);
    for (int i = 0; i < G::NKS; ++i) { mbar_init(BAR(B_K_FULL + i), 1); mbar_init(BAR(B_K_EMPTY + i), 1); }
    for (int i = 0; i < G::NVS; ++i) { mbar_init(BAR(B_V_FULL + i), 1); mbar_init(BAR(B_V_EMPTY + i), 1); }
    for (int i = 0; i < G::NSBUF; ++i) {
      mbar_init(BAR(B_S_FULL + i), 1);
      mbar_init(BAR(B_P_FULL + 2 * i), 4);      // one per half of P (the four warps that own that half in the block's team)
      mbar_init(BAR(B_P_FULL + 2 * i + 1), 4);
      mbar_init(BAR(B_S_FREE + i), 1);
    }
    mbar_init(BAR(B_O_FULL), 1);
    mbar_init(BAR(B_O_FREE), 16);
    mbar_init(BAR(B_FINAL), 1);
    mbar_init(BAR(B_FINAL + 1), 1);
    for (int i = 0; i < 8; ++i) mbar_init(BAR(B_MX + i), 1);
    for (int i = 0; i < 4; ++i) mbar_init(BAR(B_EX + i), 4);    // the four warps of a lane quadrant, once per task
    for (int i = 0; i < 8; ++i) mbar_init(BAR(B_HX + i), 2);    // the two owners of a row (team, quadrant), once per max
    *abort_smem = 0;
    redo_flag[0] = 0;
    redo_flag[1] = 0;
    fence_mbar_init();
    fence_proxy_async();
  }
  // the MMA reads all 128 rows of the Q region even when a query block has 64 rows: clear it once
  for (int i = tid; i < G::Q_BYTES / 16; i += kThreadsOf<BLOCK>) reinterpret_cast<uint4*>(smem + G::OFF_Q)[i] = make_uint4(0, 0, 0, 0);
  fence_proxy_async();
  if (warp == kPvWarp) {
    tmem_alloc(smem_u32(tmem_holder), G::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_holder, 0);

  // Every role walks the same sequence of tasks (query blocks) and, inside a task, of KV blocks;
  // block number g (counted over the CTA's whole life) uses S buffer g mod 3, K stage g mod NKS
  // and V stage g mod NVS, so no role needs to be told where a tile or a buffer is.
  if (warp == kProducerWarp) {
    // ============================================================== producer
    if (lane == 0) { prefetch_tmap(&tmQ); prefetch_tmap(&tmK); prefetch_tmap(&tmV); prefetch_tmap(&tmK2); prefetch_tmap(&tmV2); }
    uint32_t task_it = 0, q_it = 0, k_it = 0, v_it = 0;
    bool ok = true;
    uint32_t k_armed = 0, k_parity = 0, v_armed = 0, v_parity = 0;   // per stage: parity of the last load armed on it
    bool q_armed = false; uint32_t q_armed_parity = 0;
    // the next task: a ticket from the global counter and the task it stands for (n = -1: none left)
    auto draw = [&](long long& t_out) -> Task {
      for (;;) {
        long long t = 0, n_tasks = p.total_tasks;
        if (lane == 0) {
          if (p.redo_pass) n_tasks = min((long long)p.ws[2], p.total_tasks);   // written by the first pass
          // (volatile: another SM raises the flag while this kernel runs; a cached copy would hide it)
          t = (*reinterpret_cast<volatile int*>(&p.ws[1]) != 0) ? n_tasks
                                                               : (long long)(unsigned)atomicAdd(&p.ws[p.redo_pass ? 3 : 0], 1);
        }
        t = __shfl_sync(0xffffffffu, t, 0);
        n_tasks = __shfl_sync(0xffffffffu, n_tasks, 0);
        t_out = t;
        Task tk{};
        if (t >= n_tasks) {
          tk.n = -1;
        } else if (!p.redo_pass) {
          // one 32-byte load behind the ticket instead of a chain through three lists
          const uint4* e = reinterpret_cast<const uint4*>(p.table + t);
          const uint4 a = e[0], b = e[1];
          tk.h = (int)a.x; tk.row = (int)a.y; tk.lo = (int)a.z; tk.n = (int)a.w; tk.tail_valid = (int)b.x; tk.len = (int)b.y;
          tk.row2 = (int)b.z;
          if (tk.n == kAbsorbed) continue;          // second block of a pair: computed with its partner
        } else {
          int h = p.ws[8 + 2 * t], row = p.ws[9 + 2 * t];
          if (h < 0 || h >= p.heads) h = 0;
          if (row < 0 || row >= p.m_b) row = 0;
          int lo = p.row_ptr[(size_t)h * p.m_b + row], hi = p.row_ptr[(size_t)h * p.m_b + row + 1];
          tk.h = h; tk.row = row; tk.lo = lo; tk.row2 = -1;
          fill_tiles(tk, max(hi - lo, 0), BLOCK, hi > lo ? p.kv_idx[hi - 1] : 0, p.n_b, p.seq_kv);
        }
        return tk;
      }
    };
    // The ticket of the next task is drawn a few tiles before the current task's last loads are
    // requested, while this warp would wait for a ring stage anyway: the round trips of the
    // counter and of the table entry (~2,000 cycles) then no longer stand between the end of a
    // task and the request for the next Q tile.
    constexpr int kDrawAhead = 3;
    long long t = 0, t_next = 0;
    Task tk_next = draw(t_next);
    while (ok) {
      Task tk = tk_next;
      t = t_next;
      bool drawn = false;
      const uint32_t slot = task_it & 1, ph = (task_it >> 1) & 1;
      ok = warp_wait(ctx, BAR(B_TASK_EMPTY + slot), ph ^ 1, 1);
      if (!ok) break;
      if (lane == 0) {
        tasks[slot] = tk;
        mbar_arrive(BAR(B_TASK_FULL + slot));
      }
      ++task_it;
      if (tk.n < 0) break;
      if (tk.n <= kDrawAhead) { tk_next = draw(t_next); drawn = true; }
      if (tk.n == 0) continue;
      // Q tile
      ok = warp_wait(ctx, BAR(B_Q_EMPTY), (q_it & 1) ^ 1, 2);
      if (!ok) break;
      if (lane == 0) {
        const bool two = G::KB == 2 && tk.row2 >= 0;
        mbar_expect_tx(BAR(B_Q_FULL), (two ? 2 : 1) * G::SLABS * G::BQ * 128);
#pragma unroll
        for (int s = 0; s < G::SLABS; ++s)
          tma_load_3d(sbase + G::OFF_Q + s * 128 * 128, &tmQ, s * 64, tk.row * G::BQ, tk.h, BAR(B_Q_FULL));
        if (two) {
          // the partner's 64 rows go to rows 64..127 of the tile
#pragma unroll
          for (int s = 0; s < G::SLABS; ++s)
            tma_load_3d(sbase + G::OFF_Q + s * 128 * 128 + 64 * 128, &tmQ, s * 64, tk.row2 * G::BQ, tk.h, BAR(B_Q_FULL));
        }
      }
      q_armed = true; q_armed_parity = q_it & 1;
      ++q_it;
      int chunk_base = -64, my_idx = 0;
      if constexpr (G::SPLIT_LOADERS) {
        // all K tiles of the task, as fast as the ring takes them; the V tiles come from a warp of
        // their own (64-row shapes: a tile takes twice the list entries and boxes, and one warp
        // for both streams was the limit of the whole kernel: -27 % cycles with two)
        for (int j = 0; j < tk.n && ok; ++j) {
          if (!drawn && j >= tk.n - kDrawAhead) { tk_next = draw(t_next); drawn = true; }
          ok = load_kv_tile<G, BLOCK, true>(ctx, p, tk, p.drop_tile && t == 0 && j == 0, j, lane, sbase, BAR(B_K_FULL),
                                            BAR(B_K_EMPTY), &tmK, &tmK2, k_it, k_armed, k_parity, chunk_base, my_idx);
        }
      } else {
        // K tiles run three tiles ahead of the V tiles, like the MMAs that consume them; one warp
        // for both streams paces the start of the next task (128-row shapes: an earlier start of
        // the next task's loads costs more than a second loader gains, +2 % cycles)
        int v_chunk_base = -64, v_my_idx = 0;
        for (int j = 0; j < G::NSBUF && j < tk.n && ok; ++j)
          ok = load_kv_tile<G, BLOCK, true>(ctx, p, tk, p.drop_tile && t == 0 && j == 0, j, lane, sbase, BAR(B_K_FULL),
                                            BAR(B_K_EMPTY), &tmK, &tmK2, k_it, k_armed, k_parity, chunk_base, my_idx);
        for (int j = 0; j < tk.n && ok; ++j) {
          if (!drawn && j >= tk.n - kDrawAhead) { tk_next = draw(t_next); drawn = true; }
          ok = load_kv_tile<G, BLOCK, false>(ctx, p, tk, false, j, lane, sbase, BAR(B_V_FULL), BAR(B_V_EMPTY), &tmV, &tmV2,
                                             v_it, v_armed, v_parity, v_chunk_base, v_my_idx);
          if (ok && j + G::NSBUF < tk.n)
            ok = load_kv_tile<G, BLOCK, true>(ctx, p, tk, false, j + G::NSBUF, lane, sbase, BAR(B_K_FULL), BAR(B_K_EMPTY),
                                              &tmK, &tmK2, k_it, k_armed, k_parity, chunk_base, my_idx);
        }
      }
    }
    if (*abort_smem) {
      // leave no bulk copy in flight into this CTA's shared memory (bounded)
      for (int st = 0; st < G::NKS; ++st)
        if (k_armed & (1u << st)) {
          long long t0 = clock64();
          while (!mbar_try_wait(BAR(B_K_FULL + st), (k_parity >> st) & 1) && clock64() - t0 < p.wait_limit / 4) {}
        }
      for (int st = 0; st < G::NVS; ++st)
        if (v_armed & (1u << st)) {
          long long t0 = clock64();
          while (!mbar_try_wait(BAR(B_V_FULL + st), (v_parity >> st) & 1) && clock64() - t0 < p.wait_limit / 4) {}
        }
      if (q_armed) {
        long long t0 = clock64();
        while (!mbar_try_wait(BAR(B_Q_FULL), q_armed_parity) && clock64() - t0 < p.wait_limit / 4) {}
      }
    }
  } else if (G::SPLIT_LOADERS && warp == kVLoadWarp) {
    // ============================================================== V tile loader (64-row shapes)
    uint32_t task_slot = 0, task_ph = 0, v_it = 0, v_armed = 0, v_parity = 0;
    bool ok = true;
    while (ok) {
      ok = warp_wait(ctx, BAR(B_TASK_FULL + task_slot), task_ph, 10);
      if (!ok) break;
      const Task tk = tasks[task_slot];
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_TASK_EMPTY + task_slot));
      task_slot ^= 1;
      task_ph ^= (task_slot == 0);
      if (tk.n < 0) break;
      int chunk_base = -64, my_idx = 0;
      for (int j = 0; j < tk.n && ok; ++j)
        ok = load_kv_tile<G, BLOCK, false>(ctx, p, tk, false, j, lane, sbase, BAR(B_V_FULL), BAR(B_V_EMPTY), &tmV, &tmV2,
                                           v_it, v_armed, v_parity, chunk_base, my_idx);
    }
    if (*abort_smem) {
      // leave no bulk copy in flight into this CTA's shared memory (bounded)
      for (int st = 0; st < G::NVS; ++st)
        if (v_armed & (1u << st)) {
          long long t0 = clock64();
          while (!mbar_try_wait(BAR(B_V_FULL + st), (v_parity >> st) & 1) && clock64() - t0 < p.wait_limit / 4) {}
        }
    }
  } else if (warp == kQkWarp) {
    // ============================================================== MMA issuer 1: S = Q K^T
    // Two warps issue the MMAs, one per product: the bookkeeping of each (barrier waits, ring
    // arithmetic, descriptor set-up: a few hundred cycles of dependent scalar work per block)
    // then runs while the other's MMAs execute, and the tensor pipe is not left waiting for
    // it.  MMAs of different threads are ordered through completion barriers only.
    // Every operand of a tcgen05 instruction stays warp-uniform in the compiler's eyes
    // (shuffle-broadcast values, compare-and-reset ring positions).
    constexpr uint32_t IDESC_QK = make_idesc(128, G::BK, false);
    uint32_t task_slot = 0, task_ph = 0, q_ph = 0, k_st = 0, k_ph = 0, sb = 0, free_bits = 0, first_uses = G::NSBUF;
    const uint64_t qdesc0 = make_desc(sbase + G::OFF_Q, 16, 1024);
    const uint64_t kdesc0 = make_desc(sbase + G::OFF_K, 16, 1024);
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
      for (int j = 0; j < n && ok; ++j) {
        ok = warp_wait(ctx, BAR(B_K_FULL + k_st), k_ph, 12);
        if (!ok) break;
        // S[sb] also holds the P tile of the block that used it last: wait until that block's
        // P V has completed (its commit is phase number uses-1 of the buffer's barrier)
        if (first_uses > 0) {
          --first_uses;
        } else {
          ok = warp_wait(ctx, BAR(B_S_FREE + sb), ((free_bits >> sb) & 1u) ^ 1u, 13);
          if (!ok) break;
        }
        free_bits ^= 1u << sb;
        tc_fence_after();
        {
          // descriptors differ from the per-kernel bases only in the 14-bit address field
          const uint64_t kd = kdesc0 + (uint64_t)(k_st * (uint32_t)(G::TILE_BYTES >> 4));
          const uint32_t d_s = tmem_base + sb * G::S_STRIDE;
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            umma_bf16(d_s, qdesc0 + (uint64_t)(((k / 4) * 128 * 128 + (k % 4) * 32) >> 4),
                      kd + (uint64_t)(((k / 4) * G::KV_SLAB_BYTES + (k % 4) * 32) >> 4), IDESC_QK, k > 0);
          }
          tc_commit(BAR(B_K_EMPTY + k_st));
          tc_commit(BAR(B_S_FULL + sb));
          if (j == n - 1) tc_commit(BAR(B_Q_EMPTY));
        }
        if (++k_st == (uint32_t)G::NKS) { k_st = 0; k_ph ^= 1; }
        if (++sb == (uint32_t)G::NSBUF) sb = 0;
      }
    }
    // none of this thread's MMAs is still running when tensor memory is released (in a regular
    // run the last P V already depends on all of them; after an abort nothing else orders them)
    tc_commit(BAR(B_FINAL + 1));
    __syncwarp();
    {
      long long t0 = clock64();
      while (!mbar_try_wait(BAR(B_FINAL + 1), 0) && clock64() - t0 < p.wait_limit / 4) {}
    }
  } else if (warp == kPvWarp) {
    // ============================================================== MMA issuer 2: O += P V
    constexpr uint32_t IDESC_PV = make_idesc(128, D, true);
    uint32_t task_slot = 0, task_ph = 0, o_ph = 1, v_st = 0, v_ph = 0, sb = 0, p_phase = 0;
    const uint64_t vdesc0 = make_desc(sbase + G::OFF_V, G::KV_SLAB_BYTES, 1024);
    bool ok = true;
    while (ok) {
      ok = warp_wait(ctx, BAR(B_TASK_FULL + task_slot), task_ph, 10);
      if (!ok) break;
      const int n = __shfl_sync(0xffffffffu, tasks[task_slot].n, 0);
      const bool half_tail = __shfl_sync(0xffffffffu, tasks[task_slot].tail_valid, 0) <= 64;
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_TASK_EMPTY + task_slot));
      task_slot ^= 1;
      task_ph ^= (task_slot == 0);
      if (n < 0) break;
      if (n == 0) continue;
      // the output accumulator of the previous task has been read by the epilogue
      ok = warp_wait(ctx, BAR(B_O_FREE), o_ph, 16);
      if (!ok) break;
      o_ph ^= 1;
      for (int j = 0; j < n && ok; ++j) {
        // P_j arrives in two halves (the first and the second half of the block's keys), each
        // with its own barrier: the MMAs on the first half run while the softmax team is still
        // computing the second
        const uint64_t vd = vdesc0 + (uint64_t)(v_st * (uint32_t)(G::TILE_BYTES >> 4));
        const uint32_t pbase = tmem_base + sb * G::S_STRIDE;
        const uint32_t d_o = tmem_base + G::O_COL;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const uint32_t pb = sb * 2 + h;
          ok = warp_wait(ctx, BAR(B_P_FULL + pb), (p_phase >> pb) & 1u, 14);
          if (!ok) break;
          p_phase ^= 1u << pb;
          if (h == 0) {
            ok = warp_wait(ctx, BAR(B_V_FULL + v_st), v_ph, 15);
            if (!ok) break;
          }
          tc_fence_after();
          // (the second half of a half tile has no keys: its V rows were never loaded)
          if (G::KB == 2 && h == 1 && j == n - 1 && half_tail) continue;
          // V tile as the N x K operand with N (head_dim) contiguous: 8 keys per 1024-byte
          // group along K (16 keys = 2048 bytes per MMA), next 64 columns of head_dim one slab further
#pragma unroll
          for (int kk = 0; kk < G::BK / 32; ++kk) {
            const int k = h * (G::BK / 32) + kk;
            // P of key half h lies over the first columns of that half's own S columns
            umma_bf16_ts(d_o, pbase + h * G::HC + kk * 8, vd + (uint64_t)((k * 16 * 128) >> 4), IDESC_PV, (j > 0 || k > 0) ? 1u : 0u);
          }
        }
        if (!ok) break;
        {
          tc_commit(BAR(B_V_EMPTY + v_st));
          tc_commit(BAR(B_S_FREE + sb));
          if (j == n - 1) tc_commit(BAR(B_O_FULL));
        }
        if (++v_st == (uint32_t)G::NVS) { v_st = 0; v_ph ^= 1; }
        if (++sb == (uint32_t)G::NSBUF) sb = 0;
      }
    }
    // every MMA has completed before tensor memory is released: the last P V depends on all
    // the Q K^T products through the softmax warps
    tc_commit(BAR(B_FINAL));
    __syncwarp();
    {
      long long t0 = clock64();
      while (!mbar_try_wait(BAR(B_FINAL), 0) && clock64() - t0 < p.wait_limit / 4) {}
    }
  } else {
    // ============================================================== softmax / epilogue
    // Sixteen warps: two teams take the KV blocks of a task in turn (team = block index mod 2),
    // and inside a team a row of S has two owners, one per half of its columns (a warp can reach
    // only the 32 tensor-memory lanes of its quadrant, so the two owners of a row sit in warps
    // four apart).  Four softmax warps per scheduler instead of two: the loop is bound by
    // instruction issue and latency, and twice the warps hide twice the latency.  The owners
    // of a row share its reference max (exchanged through shared memory in the blocks that
    // take one); each keeps the sum of its own columns; P of a column half is written over the
    // first columns of that half's own S columns and released with its own barrier.  The two
    // teams hand each other the running reference of each row (shared memory + one mbarrier
    // per lane quadrant and block parity), because both accumulate into the same O.  The
    // epilogue adds the four partial sums of a row.
    const int sw = warp - kSoftmaxWarp0;       // 0..15
    const int quad = warp & 3;                 // tensor-memory lane quadrant this warp may access
    const int team = (sw >> 2) & 1;            // owns blocks j with (j & 1) == team
    const int half = sw >> 3;                  // column half of S; epilogue: quarter team*2+half of the O columns
    const int r = quad * 32 + lane;            // row of the 128-row MMA tile
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t o_row = tmem_base + lane_addr + G::O_COL;
    const int part = team * 2 + half;
    uint32_t task_it = 0, s_phase = 0, o_it = 0, mx_phase = 0, hx_it = 0, sb = 0;   // s_phase bit b: parity of the uses of S[b] so far
    bool ok = true;
    while (ok) {
      const uint32_t slot = task_it & 1, ph = (task_it >> 1) & 1;
      ok = warp_wait(ctx, BAR(B_TASK_FULL + slot), ph, 20);
      if (!ok) break;
      const Task tk = tasks[slot];
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_TASK_EMPTY + slot));
      float2* exb = ex + (task_it & 1) * 512;
      const uint32_t rslot = task_it & 1;
      ++task_it;
      if (tk.n < 0) break;
      // rows 64..127 of the tile belong to the partner block of a pair (64-row blocks only)
      const bool second = G::KB == 2 && r >= G::BQ;
      const long long q_tok = second ? (long long)tk.row2 * G::BQ + (r - G::BQ) : (long long)tk.row * G::BQ + r;
      const bool row_live = (second ? tk.row2 >= 0 : r < G::BQ) && q_tok < p.seq_q;
      // rows 64..127 of a tile that no second block shares hold nothing: their warps only keep
      // the barriers of the tile going (each output row of an MMA depends on its own row of S / P alone)
      const bool idle = G::KB == 2 && quad >= 2 && tk.row2 < 0;
      __nv_bfloat16* o_ptr = p.O + (size_t)tk.h * p.o_stride_h + (size_t)q_tok * p.o_stride_t + part * G::CO;
      if (tk.n == 0) {
        if (row_live) {
#pragma unroll
          for (int c = 0; c < G::CO / 8; ++c) reinterpret_cast<uint4*>(o_ptr)[c] = make_uint4(0, 0, 0, 0);
          if (p.lse && part == 0) p.lse[(size_t)tk.h * p.seq_q + q_tok] = -INFINITY;
        }
        continue;
      }
      // l_run: sum over this thread's columns of this team's blocks, relative to the reference m_ref
      float m_ref = -INFINITY, l_run = 0.f;
      for (int j = 0; j < tk.n && ok; ++j) {
        const uint32_t par = (uint32_t)j & 1u;
        if ((int)par == team) {
          ok = warp_wait(ctx, BAR(B_S_FULL + sb), (s_phase >> sb) & 1u, 21);
          if (!ok) break;
          if (idle) {
            if (lane == 0) mbar_arrive(BAR(B_P_FULL + sb * 2 + half));
            s_phase ^= 1u << sb;
            if (++sb == (uint32_t)G::NSBUF) sb = 0;
            continue;
          }
          tc_fence_after();
          const uint32_t s_addr = tmem_base + lane_addr + sb * G::S_STRIDE + half * G::HC;
          const bool ragged = j == tk.n - 1 && tk.tail_valid < G::BK;
          const int col0 = half * G::HC;       // first key of the block this thread looks at
          // ---- pass 1: row max (the values are loaded again for the exponentials: a second
          // tensor-memory load is cheaper than keeping them in registers)
          // In the first pass over the tasks (FAST) only blocks 0 and 1 of a task take a max and
          // may move the reference; from block 2 on both teams keep the reference of block 1.
          // Any reference gives the same softmax as long as nothing overflows, so the later
          // blocks only watch the sum of the exponentials they produce: if it ever reaches 2^24 the
          // task is put on a list and computed again by the second launch, which takes the
          // max of every block (the rule of the paper's online softmax).
          const bool fixed_ref = FAST && j >= 2;
          float mloc = -INFINITY;
          if (!fixed_ref) {
#pragma unroll 1
            for (int ch = 0; ch < G::NCH; ++ch) {
              uint32_t sv[G::CH];
              WAVEAL_TMEM_LD32(s_addr + ch * G::CH, sv, 0);
              WAVEAL_TMEM_WAIT_LD32(sv, 0);
              // scores of keys beyond seq_kv (ragged last block) do not exist
              if (ragged) {
#pragma unroll
                for (int c = 0; c < G::CH; ++c)
                  if (col0 + ch * G::CH + c >= tk.tail_valid) sv[c] = __float_as_uint(-INFINITY);
              }
              float mx8[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) mx8[i] = __uint_as_float(sv[i]);
#pragma unroll
              for (int c = 8; c < G::CH; c += 8) {
#pragma unroll
                for (int i = 0; i < 8; ++i) mx8[i] = fmaxf(mx8[i], __uint_as_float(sv[c + i]));
              }
              mloc = fmaxf(mloc, fmaxf(fmaxf(fmaxf(mx8[0], mx8[1]), fmaxf(mx8[2], mx8[3])),
                                       fmaxf(fmaxf(mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7]))));
            }
            // the other owner of the row (same team and quadrant, other column half)
            // (two buffers by use parity: the partner's next value cannot land on one not yet read)
            volatile float* mh = mhalf + (hx_it & 1u) * 512;
            mh[(team * 2 + half) * 128 + r] = mloc;
            __syncwarp();
            if (lane == 0) mbar_arrive(BAR(B_HX + team * 4 + quad));
            ok = warp_wait(ctx, BAR(B_HX + team * 4 + quad), hx_it & 1u, 26);
            if (!ok) break;
            ++hx_it;
            mloc = fmaxf(mloc, mh[(team * 2 + (half ^ 1)) * 128 + r]);
          }
          // ---- the row's reference after block j-1, from the other team
          float m_prev = m_ref;
          if (j > 0 && (!fixed_ref || j == 2)) {
            // that team's arrival for block j-1 is phase number (arrivals of that parity so far) - 1
            ok = warp_wait(ctx, BAR(B_MX + quad * 2 + (par ^ 1u)), ((mx_phase >> (par ^ 1u)) & 1u) ^ 1u, 24);
            if (!ok) break;
            m_prev = mpub[((j - 1) & 3) * 128 + r];
          }
          const float m_cand = fmaxf(m_prev, mloc * p.sl2);
          // keep the stale reference unless it is exceeded by more than 2^8 (exact: the final
          // normalisation divides by a sum taken with the same reference); both owners of a row
          // see the same values and take the same decision
          const bool grow = !fixed_ref && __any_sync(0xffffffffu, m_cand > m_prev + 8.0f);
          const float m_new = grow ? m_cand : m_prev;
          if (!fixed_ref && half == 0) {
            // (slot j mod 4: the owner of block j+4 cannot get there before both owners of block
            // j+1 have read this one)
            mpub[(j & 3) * 128 + r] = m_new;
            __syncwarp();
            if (lane == 0) mbar_arrive(BAR(B_MX + quad * 2 + par));
          }
          if (m_new != m_ref) {
            l_run *= (m_ref == -INFINITY) ? 0.f : ex2(m_ref - m_new);
            m_ref = m_new;
          }
          // rare: the reference grew, so O (blocks 0..j-1) is rescaled; its last MMA (block j-1)
          // must be complete: that is the latest phase of the barrier of the S buffer before
          // this one (the next P V on that buffer needs a P this team has not produced yet).
          // Done before any part of P_j is released to the MMA warp; each owner takes half of
          // the row's output columns.
          if (grow && j > 0) {
            const uint32_t sbp = sb == 0 ? (uint32_t)G::NSBUF - 1u : sb - 1u;
            ok = warp_wait(ctx, BAR(B_S_FREE + sbp), ((s_phase >> sbp) & 1u) ^ 1u, 22);
            if (!ok) break;
            tc_fence_after();
            const float alpha = ex2(m_prev - m_new);
#pragma unroll 1
            for (int c0 = half * (D / 2); c0 < (half + 1) * (D / 2); c0 += 32) {
              uint32_t ov[32];
              WAVEAL_TMEM_LD32(o_row + c0, ov, 0);
              WAVEAL_TMEM_WAIT_LD32(ov, 0);
#pragma unroll
              for (int c = 0; c < 32; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * alpha);
              WAVEAL_TMEM_ST32(o_row + c0, ov, 0);
            }
          }
          // p' = 2^(s*scale*log2e - m + log2(1 + 2^-9)); P is p' cut to its top 16 bits (one byte
          // permute per pair instead of a conversion).  The extra factor centres the cut's error
          // around zero, like a rounding; the row sum adds the uncut p' and the epilogue takes
          // the factor out again.  Multiply-adds and sums work on register pairs (f32x2).
          const float neg_m = ((m_new == -INFINITY) ? 0.f : -m_new) + 0.0028150156f;
          const float a128 = p.sl2 * 0.0078125f, b128 = (neg_m - kPolyLo) * 0.0078125f;   // polynomial share
          float ls4[4] = {0.f, 0.f, 0.f, 0.f};
          // ---- pass 2: exponentials; P (bf16 pairs) goes over the first half of the thread's own
          // S columns, each chunk after its S values have been read.  A rolled loop over
          // 32-column chunks: the body stays small enough for the instruction cache.
#pragma unroll 1
          for (int ch = 0; ch < G::NCH; ++ch) {
            uint32_t sv[G::CH];
            WAVEAL_TMEM_LD32(s_addr + ch * G::CH, sv, 0);
            WAVEAL_TMEM_WAIT_LD32(sv, 0);
            if (ragged) {
#pragma unroll
              for (int c = 0; c < G::CH; ++c)
                if (col0 + ch * G::CH + c >= tk.tail_valid) sv[c] = __float_as_uint(-INFINITY);
            }
            uint32_t pk[G::CH / 2];
#pragma unroll
            for (int c = 0; c < G::CH; c += 2) {
              float e0, e1;
              if (kPolyEvery > 0 && ((c >> 1) % (kPolyEvery > 0 ? kPolyEvery : 1)) == (kPolyEvery > 0 ? kPolyEvery : 1) - 1) {
                ex2_fma2(e0, e1, __uint_as_float(sv[c]), __uint_as_float(sv[c + 1]), a128, b128);
              } else {
                float x0, x1;
                ffma2(x0, x1, __uint_as_float(sv[c]), __uint_as_float(sv[c + 1]), p.sl2, p.sl2, neg_m, neg_m);
                e0 = ex2(x0); e1 = ex2(x1);
              }
              fadd2(ls4[c & 2], ls4[(c & 2) + 1], ls4[c & 2], ls4[(c & 2) + 1], e0, e1);
              pk[c / 2] = __byte_perm(__float_as_uint(e0), __float_as_uint(e1), 0x7632);
            }
            WAVEAL_TMEM_ST16(s_addr + ch * 16, pk, 0);
          }
          const float l_blk = (ls4[0] + ls4[1]) + (ls4[2] + ls4[3]);
          l_run += l_blk;
          // all terms are positive (the transcendental unit returns +inf on overflow, the
          // polynomial share saturates at 2^28), so a sum below 2^24 bounds every exponent it
          // covers; at or above it (or not a number) the fixed reference is too far off:
          // redo the task
          if (fixed_ref && __any_sync(0xffffffffu, !(l_blk < kRedoLimit))) redo_flag[rslot] = 1;
          tc_wait_st();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(BAR(B_P_FULL + sb * 2 + half));
        }
        // both teams count every block
        s_phase ^= 1u << sb;
        if (!(FAST && j >= 2) && !idle) mx_phase ^= 1u << par;   // one flip per arrival on that parity's barrier
        if (++sb == (uint32_t)G::NSBUF) sb = 0;
      }
      if (!ok) break;
      // ---- epilogue: O / l at the original row position; l = the four partial sums of the row
      // brought to the final reference (the larger of the two teams', references never shrink)
      // (the partial sums are final once the thread's last tile is done: publish them before the
      // wait for the last P V, so that nothing but the load of O stands between that MMA and the
      // first one of the next task)
      exb[part * 128 + r] = make_float2(m_ref, l_run);
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_EX + quad));
      ok = warp_wait(ctx, BAR(B_O_FULL), o_it & 1, 23);
      if (!ok) break;
      ++o_it;
      tc_fence_after();
      if (FAST && sw == 0 && lane == 0 && redo_flag[rslot]) {
        // every warp's blocks of this task lie before O_FULL; the slot is used again two tasks
        // later, after this warp's O_FREE arrival below
        const int e = atomicAdd(&p.ws[2], (G::KB == 2 && tk.row2 >= 0) ? 2 : 1);
        p.ws[8 + 2 * e] = tk.h;
        p.ws[9 + 2 * e] = tk.row;
        if (G::KB == 2 && tk.row2 >= 0) { p.ws[10 + 2 * e] = tk.h; p.ws[11 + 2 * e] = tk.row2; }   // computed again one by one
        redo_flag[rslot] = 0;
      }
      uint32_t ov[G::CO];
      static_assert(G::CO == 32 || G::CO == 16, "a quarter of head_dim 128 or 64");
      if constexpr (G::CO == 32) { WAVEAL_TMEM_LD32(o_row + part * G::CO, ov, 0); WAVEAL_TMEM_WAIT_LD32(ov, 0); }
      else { WAVEAL_TMEM_LD16(o_row + part * G::CO, ov, 0); WAVEAL_TMEM_WAIT_LD16(ov, 0); }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_O_FREE));
      // the other three warps of this lane quadrant have written their parts: a bounded wait
      // like every other, so that a warp whose partners gave up does not stay behind
      ok = warp_wait(ctx, BAR(B_EX + quad), (o_it & 1) ^ 1, 25);
      if (!ok) break;
      const float2 e00 = exb[0 * 128 + r], e01 = exb[1 * 128 + r], e10 = exb[2 * 128 + r], e11 = exb[3 * 128 + r];
      const float m0 = fmaxf(e00.x, e01.x), m1 = fmaxf(e10.x, e11.x);     // the two owners of a team agree; a team
      const float m_all = fmaxf(m0, m1);                                   // without blocks (n == 1) has -inf
      const float a0 = (m0 == -INFINITY) ? 0.f : ex2(m0 - m_all);
      const float a1 = (m1 == -INFINITY) ? 0.f : ex2(m1 - m_all);
      const float l_tot = a0 * (e00.y + e01.y) + a1 * (e10.y + e11.y);
      const float inv_l = 1.0019531f / l_tot;    // the sums carry the centring factor 1 + 2^-9
      if (row_live) {
        // a thread holds a piece of one row, so a store instruction of a warp touches 32 rows:
        // its cost in the memory pipe is per row, not per byte.  32-byte stores halve the number
        // of instructions where the row piece is 32-byte aligned (else 16-byte stores)
        uint32_t w[G::CO / 2];
#pragma unroll
        for (int c = 0; c < G::CO; c += 2) {
          __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(ov[c]) * inv_l, __uint_as_float(ov[c + 1]) * inv_l);
          w[c / 2] = *reinterpret_cast<uint32_t*>(&b2);
        }
        if ((reinterpret_cast<uintptr_t>(o_ptr) & 31) == 0) {
#pragma unroll
          for (int c = 0; c < G::CO / 2; c += 8) st_global_v8(o_ptr + 2 * c, w + c);
        } else {
#pragma unroll
          for (int c = 0; c < G::CO / 2; c += 4)
            *reinterpret_cast<uint4*>(o_ptr + 2 * c) = make_uint4(w[c], w[c + 1], w[c + 2], w[c + 3]);
        }
        if (p.lse && part == 0) p.lse[(size_t)tk.h * p.seq_q + q_tok] = (m_all + log2f(l_tot) - 0.0028150156f) * 0.6931471805599453f;
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == kPvWarp) {
    tc_fence_after();
    tmem_dealloc(tmem_base, G::TMEM_COLS);
  }
  // SM cycles this CTA was alive: the largest over the grid is the launch's length in cycles,
  // a figure that does not depend on the clock the GPU happened to run at
  if (tid == 0) {
    const long long dt = clock64() - t_start;
    atomicMax(&p.ws[p.redo_pass ? 5 : 4], (int)(dt > 0x7fffffffll ? 0x7fffffffll : dt));
  }
}

// Task of every ticket (head-major or position-major over the planned order), so that the
// persistent CTAs need one load behind a ticket instead of a chain through row_order, the row
// pointers and the index list.
// The inputs are checked on the way (one thread per task, so it costs nothing): an entry of
// row_order outside [0, M_B), a row-pointer pair that is negative, decreasing or beyond the end
// of the index list, or a last index outside [0, N_B) is reported as
// {WAVEAL_ERR_BAD_MASK, site, head, offending value} and the task is given an empty list
// (its output rows become 0) instead of reading out of range.
__global__ void k_task_table(AttnParams p, int block_k, Task* table) {
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= p.total_tasks) return;
  int h, pos;
  if (p.interleaved) { pos = (int)(t / p.heads); h = (int)(t % p.heads); }
  else { h = (int)(t / p.m_b); pos = (int)(t % p.m_b); }
  auto report = [&](int site, int value) {
    if (p.dev_status && atomicCAS(p.dev_status, 0, WAVEAL_ERR_BAD_MASK) == 0) {
      p.dev_status[1] = site; p.dev_status[2] = h; p.dev_status[3] = value;
    }
  };
  int row = p.row_order ? p.row_order[(size_t)h * p.m_b + pos] : pos;
  bool bad = false;
  if (row < 0 || row >= p.m_b) { report(31, row); row = pos; bad = true; }
  const long long nnz = p.row_ptr[p.total_tasks];
  const int lo = p.row_ptr[(size_t)h * p.m_b + row], hi = p.row_ptr[(size_t)h * p.m_b + row + 1];
  if (lo < 0 || hi < lo || (long long)hi > nnz) { report(32, lo < 0 ? lo : hi); bad = true; }
  Task tk{};
  tk.h = h; tk.row = row; tk.lo = bad ? 0 : lo; tk.row2 = -1;
  int len = bad ? 0 : hi - lo, last = 0;
  if (len > 0) {
    last = p.kv_idx[hi - 1];
    if (last < 0 || last >= p.n_b) { report(33, last); len = 0; }
  }
  fill_tiles(tk, len, block_k, last, p.n_b, p.seq_kv);
  // 64-row query blocks: two blocks with the very same list share one 128-row tile.  Candidates:
  //  - rows that select every KV block (list length = N_B: rows that attend to everything), wherever
  //    they stand: the 1st and 2nd, the 3rd and 4th, ... such row of the head's order form pairs,
  //    run at the position of the first of the two;
  //  - any other two rows at positions 2i and 2i+1 of the order (Stage 2 of the plan puts rows of
  //    equal count side by side).
  // A pair is formed only if the two lists are equal entry by entry; both threads of a pair run
  // the same comparison, the first keeps the task, the second one's ticket is absorbed.
  if (block_k == 64 && len > 0 && !bad && !p.no_pairing) {
    const size_t hb = (size_t)h * p.m_b;
    auto row_at = [&](int ps) {
      const int r = p.row_order ? p.row_order[hb + ps] : ps;
      return (r < 0 || r >= p.m_b) ? -1 : r;
    };
    auto len_of = [&](int r) { return p.row_ptr[hb + r + 1] - p.row_ptr[hb + r]; };
    int mate = -1;            // the other row of the candidate pair
    bool first = true;        // this thread's row is the first of the two
    if (len == p.n_b) {
      int before = 0;
      for (int ps = 0; ps < pos; ++ps) { const int r = row_at(ps); if (r >= 0 && len_of(r) == p.n_b) ++before; }
      first = (before & 1) == 0;
      if (first) {
        for (int ps = pos + 1; ps < p.m_b && mate < 0; ++ps) { const int r = row_at(ps); if (r >= 0 && len_of(r) == p.n_b) mate = r; }
      } else {
        for (int ps = pos - 1; ps >= 0 && mate < 0; --ps) { const int r = row_at(ps); if (r >= 0 && len_of(r) == p.n_b) mate = r; }
      }
    } else if ((pos ^ 1) < p.m_b) {
      const int r = row_at(pos ^ 1);
      if (r >= 0 && len_of(r) == len) { mate = r; first = (pos & 1) == 0; }
    }
    if (mate >= 0 && mate != row) {
      const int lo2 = p.row_ptr[hb + mate], hi2 = p.row_ptr[hb + mate + 1];
      bool same = lo2 >= 0 && hi2 - lo2 == len && (long long)hi2 <= nnz;
      for (int e = 0; same && e < len; ++e) same = p.kv_idx[lo + e] == p.kv_idx[lo2 + e];
      if (same) {
        if (first) { tk.row2 = mate; atomicAdd(&p.ws[6], 1); }     // word 6: pairs formed by this call
        else tk.n = kAbsorbed;
      }
    }
  }
  if (tk.n > 0) atomicAdd(&p.ws[7], tk.n);    // word 7: KV tiles (128 rows x 128 keys) this call runs
  table[t] = tk;
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

// byte offset of the ticket table in the workspace (32-byte aligned, behind header and redo list)
long long table_offset(long long tasks) { return (32 + 8 * tasks + 31) / 32 * 32; }

template <int BLOCK, int D>
waveal_status launch(const waveal_attn_desc* d, const void* Q, const void* K, const void* V, AttnParams& p,
                     int sms, cudaStream_t st) {
  using G = Geo<BLOCK, D>;
  CUtensorMap tq, tk, tv, tk2, tv2;
  waveal_status s;
  if ((s = make_map(&tq, Q, D, d->seq_q, d->heads, d->q_stride[0], d->q_stride[1], BLOCK, "Q")) != WAVEAL_OK) return s;
  if ((s = make_map(&tk, K, D, d->seq_kv, d->heads, d->k_stride[0], d->k_stride[1], BLOCK, "K")) != WAVEAL_OK) return s;
  if ((s = make_map(&tv, V, D, d->seq_kv, d->heads, d->v_stride[0], d->v_stride[1], BLOCK, "V")) != WAVEAL_OK) return s;
  if ((s = make_map(&tk2, K, D, d->seq_kv, d->heads, d->k_stride[0], d->k_stride[1], 128, "K (128-row boxes)")) != WAVEAL_OK) return s;
  if ((s = make_map(&tv2, V, D, d->seq_kv, d->heads, d->v_stride[0], d->v_stride[1], 128, "V (128-row boxes)")) != WAVEAL_OK) return s;
  WAVEAL_CUDA_OK(cudaFuncSetAttribute(k_bsattn_fwd<BLOCK, D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM_BYTES));
  WAVEAL_CUDA_OK(cudaFuncSetAttribute(k_bsattn_fwd<BLOCK, D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM_BYTES));
  WAVEAL_CUDA_OK(cudaMemsetAsync(p.ws, 0, 32, st));  // ticket counters, abort flag, redo count
  long long grid = p.total_tasks < sms ? p.total_tasks : sms;
  Task* table = reinterpret_cast<Task*>(reinterpret_cast<char*>(p.ws) + table_offset(p.total_tasks));
  p.table = table;
  p.redo_pass = 0;
  p.wait_limit = kTimeoutCycles;
  p.drop_tile = 0;
  if (d->flags & WAVEAL_ATTN_SELFTEST_LOST_TILE) { p.wait_limit = kSelfTestCycles; p.drop_tile = 1; }
  p.no_pairing = (d->flags & WAVEAL_ATTN_NO_ROW_PAIRING) ? 1 : 0;
  k_task_table<<<(unsigned)((p.total_tasks + 255) / 256), 256, 0, st>>>(p, BLOCK, table);
  WAVEAL_CUDA_OK(cudaGetLastError());
  if (d->flags & WAVEAL_ATTN_ONLINE_MAX_ONLY) {
    p.redo_pass = 0;
    k_bsattn_fwd<BLOCK, D, false><<<(unsigned)grid, kThreadsOf<BLOCK>, G::SMEM_BYTES, st>>>(tq, tk, tv, tk2, tv2, p);
    WAVEAL_CUDA_OK(cudaGetLastError());
    waveal::launch_counter() = 2;
    return WAVEAL_OK;
  }
  // first pass: reference fixed after the first two blocks of a task; second pass: the tasks the
  // first one listed (normally none: its CTAs leave at once), max of every block
  p.redo_pass = 0;
  k_bsattn_fwd<BLOCK, D, true><<<(unsigned)grid, kThreadsOf<BLOCK>, G::SMEM_BYTES, st>>>(tq, tk, tv, tk2, tv2, p);
  WAVEAL_CUDA_OK(cudaGetLastError());
  p.redo_pass = 1;
  k_bsattn_fwd<BLOCK, D, false><<<(unsigned)grid, kThreadsOf<BLOCK>, G::SMEM_BYTES, st>>>(tq, tk, tv, tk2, tv2, p);
  WAVEAL_CUDA_OK(cudaGetLastError());
  waveal::launch_counter() = 3;
  return WAVEAL_OK;
}

}  // namespace

extern "C" waveal_status waveal_bsattn_workspace_bytes(const waveal_attn_desc* desc, size_t* bytes) {
  waveal_status s = check_desc(desc);
  if (s != WAVEAL_OK) return s;
  if (!bytes) return waveal::fail(WAVEAL_ERR_INVALID_ARG, "bytes is NULL");
  // 32 bytes of counters and flags, one (head, query block) pair per task for the redo list,
  // then the 32-byte task of every ticket
  const long long tasks = (long long)desc->heads * ((desc->seq_q + desc->block_q - 1) / desc->block_q);
  *bytes = (size_t)((table_offset(tasks) + 32 * tasks + 255) / 256 * 256);
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
  size_t ws_need = 0;
  if ((s = waveal_bsattn_workspace_bytes(d, &ws_need)) != WAVEAL_OK) return s;
  if (!ws || ws_bytes < ws_need) return waveal::fail(WAVEAL_ERR_WORKSPACE, "workspace of %zu bytes needed", ws_need);
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
