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
//   warp 1      MMA issuer: S = Q K^T and O += P V as tcgen05.mma with fp32 accumulators in
//               tensor memory; S is double-buffered so that S_{j+1} is computed while the
//               softmax of S_j runs
//   warps 2-9   softmax: thread (row, column half) reads its half row of S from tensor
//               memory, keeps the running max / sum, writes P (bf16) into shared memory in
//               the operand layout of the second MMA, rescales O in tensor memory only when
//               the max grew by more than 2^8, and finally normalises and stores O at the
//               ORIGINAL row position (no inverse permutation pass)
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

// ------------------------------------------------------------------ PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

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
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulate, one CTA
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
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

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
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
  static constexpr int PSLABS = BK / 64;             // slabs of the P tile (keys are its K dim)
  static constexpr int Q_BYTES = SLABS * 128 * 128;  // smem reserved for 128 MMA rows
  static constexpr int P_BYTES = PSLABS * 128 * 128;
  static constexpr int TILE_BYTES = SLABS * BK * 128;
  static constexpr int KV_SLAB_BYTES = BK * 128;
  static constexpr int NSTAGE = BLOCK == 128 ? 4 : 8;
  static constexpr int CS = BK / 2;                  // S columns per softmax thread
  static constexpr int CO = D / 2;                   // O columns per softmax thread
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_P = OFF_Q + Q_BYTES;
  static constexpr int OFF_KV = OFF_P + P_BYTES;
  static constexpr int OFF_BAR = OFF_KV + NSTAGE * TILE_BYTES;
  static constexpr int N_BAR = 2 + 2 + 2 + 2 * NSTAGE + 2 + 2 + 2 + 1;
  static constexpr int OFF_TASK = OFF_BAR + ((N_BAR * 8 + 15) / 16) * 16;
  static constexpr int OFF_MX = OFF_TASK + 2 * (int)sizeof(Task);
  static constexpr int OFF_MISC = OFF_MX + 2 * 2 * 128 * 4;
  static constexpr int SMEM_BYTES = OFF_MISC + 16 + 1024;   // + slack for 1024-byte alignment
  static constexpr uint32_t S_COL0 = 0, S_COL1 = 128, O_COL = 256, TMEM_COLS = 512;
};

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

template <int BLOCK, int D>
__global__ void __launch_bounds__(kThreads, 1)
k_bsattn_fwd(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
             const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
  using G = Geo<BLOCK, D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // barrier addresses
  const uint32_t bar0 = sbase + G::OFF_BAR;
  auto BAR = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  constexpr int B_TASK_FULL = 0, B_TASK_EMPTY = 2, B_Q_FULL = 4, B_Q_EMPTY = 5, B_KV_FULL = 6,
                B_KV_EMPTY = 6 + G::NSTAGE, B_S_FULL = 6 + 2 * G::NSTAGE, B_S_EMPTY = B_S_FULL + 2,
                B_P_FULL = B_S_EMPTY + 2, B_PV_DONE = B_P_FULL + 1, B_FINAL = B_PV_DONE + 1;
  static_assert(B_FINAL + 1 <= G::N_BAR, "barrier count");
  Task* tasks = reinterpret_cast<Task*>(smem + G::OFF_TASK);
  float* mx = reinterpret_cast<float*>(smem + G::OFF_MX);            // [2][2][128]
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + G::OFF_MISC);
  volatile int* abort_smem = reinterpret_cast<volatile int*>(smem + G::OFF_MISC + 4);
  Ctx ctx{bar0, abort_smem, p.ws, p.dev_status};

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) { mbar_init(BAR(B_TASK_FULL + i), 1); mbar_init(BAR(B_TASK_EMPTY + i), 9); }
    mbar_init(BAR(B_Q_FULL), 1);
    mbar_init(BAR(B_Q_EMPTY), 1);
    for (int i = 0; i < G::NSTAGE; ++i) { mbar_init(BAR(B_KV_FULL + i), 1); mbar_init(BAR(B_KV_EMPTY + i), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(BAR(B_S_FULL + i), 1); mbar_init(BAR(B_S_EMPTY + i), 8); }
    mbar_init(BAR(B_P_FULL), 8);
    mbar_init(BAR(B_PV_DONE), 1);
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
    bool ok = true;
    uint32_t armed_mask = 0, armed_parity = 0;   // per-stage: a load is (or was) in flight with this parity
    bool q_armed = false; uint32_t q_armed_parity = 0;
    while (ok) {
      long long t = 0;
      if (lane == 0) {
        t = (p.ws[1] != 0) ? p.total_tasks : (long long)(unsigned)atomicAdd(&p.ws[0], 1);
      }
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
      // K/V tiles in consumption order: K_0, then for each j: K_{j+1} (if any), V_j
      const int n_tiles = 2 * tk.n;
      int chunk_base = -32, my_idx = 0;
      for (int e = 0; e < n_tiles && ok; ++e) {
        // tile e: e == 0 -> K_0; odd e -> (e+1)/2 < n ? K_{(e+1)/2} : V_{n-1}...
        // sequence: K0, K1, V0, K2, V1, ..., K_{n-1}, V_{n-2}, V_{n-1}
        int j; bool is_k;
        if (e == 0) { j = 0; is_k = true; }
        else if (e == n_tiles - 1) { j = tk.n - 1; is_k = false; }
        else if (e & 1) { j = (e + 1) / 2; is_k = true; }
        else { j = e / 2 - 1; is_k = false; }
        if (j < chunk_base || j >= chunk_base + 32) {
          chunk_base = j & ~31;
          int q = chunk_base + lane;
          my_idx = q < tk.n ? p.kv_idx[tk.lo + q] : 0;
        }
        int blk = __shfl_sync(0xffffffffu, my_idx, j - chunk_base);
        if (blk < 0 || blk >= p.n_b) blk = 0;            // malformed list: stay in range
        const uint32_t st = kv_it % G::NSTAGE, sph = (kv_it / G::NSTAGE) & 1;
        ok = warp_wait(ctx, BAR(B_KV_EMPTY + st), sph ^ 1, 3);
        if (!ok) break;
        if (lane == 0) {
          mbar_expect_tx(BAR(B_KV_FULL + st), G::TILE_BYTES);
          const CUtensorMap* tm = is_k ? &tmK : &tmV;
#pragma unroll
          for (int s = 0; s < G::SLABS; ++s)
            tma_load_3d(sbase + G::OFF_KV + st * G::TILE_BYTES + s * G::KV_SLAB_BYTES, tm, s * 64, blk * G::BK, tk.h,
                        BAR(B_KV_FULL + st));
        }
        armed_mask |= 1u << st;
        armed_parity = (armed_parity & ~(1u << st)) | (sph << st);
        ++kv_it;
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
    constexpr uint32_t IDESC_QK = make_idesc(128, G::BK, false);
    constexpr uint32_t IDESC_PV = make_idesc(128, D, true);
    uint32_t task_it = 0, q_it = 0, kv_it = 0, s_it = 0, p_it = 0;
    bool ok = true;
    while (ok) {
      const uint32_t slot = task_it & 1, ph = (task_it >> 1) & 1;
      ok = warp_wait(ctx, BAR(B_TASK_FULL + slot), ph, 10);
      if (!ok) break;
      const int n = tasks[slot].n;
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_TASK_EMPTY + slot));
      ++task_it;
      if (n < 0) break;
      if (n == 0) continue;
      ok = warp_wait(ctx, BAR(B_Q_FULL), q_it & 1, 11);
      if (!ok) break;
      ++q_it;
      // one QK^T: S[buf] = Q K_j^T
      auto issue_qk = [&]() -> bool {
        const uint32_t st = kv_it % G::NSTAGE, sph = (kv_it / G::NSTAGE) & 1;
        const uint32_t buf = s_it & 1, bph = (s_it >> 1) & 1;
        if (!warp_wait(ctx, BAR(B_KV_FULL + st), sph, 12)) return false;
        if (!warp_wait(ctx, BAR(B_S_EMPTY + buf), bph ^ 1, 13)) return false;
        tc_fence_after();
        if (lane == 0) {
          const uint32_t kbase = sbase + G::OFF_KV + st * G::TILE_BYTES;
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            uint64_t a = make_desc(sbase + G::OFF_Q + (k / 4) * 128 * 128 + (k % 4) * 32, 16, 1024);
            uint64_t b = make_desc(kbase + (k / 4) * G::KV_SLAB_BYTES + (k % 4) * 32, 16, 1024);
            umma_bf16(tmem_base + (buf ? G::S_COL1 : G::S_COL0), a, b, IDESC_QK, k > 0);
          }
          tc_commit(BAR(B_KV_EMPTY + st));
          tc_commit(BAR(B_S_FULL + buf));
        }
        __syncwarp();
        ++kv_it; ++s_it;
        return true;
      };
      ok = issue_qk();
      // once the last QK^T of the task is issued, its completion frees the Q tile
      if (ok && n == 1) { if (lane == 0) tc_commit(BAR(B_Q_EMPTY)); __syncwarp(); }
      for (int j = 0; j < n && ok; ++j) {
        if (j + 1 < n) {
          ok = issue_qk();
          if (!ok) break;
          if (j + 2 == n) { if (lane == 0) tc_commit(BAR(B_Q_EMPTY)); __syncwarp(); }
        }
        // O (+)= P_j V_j
        const uint32_t st = kv_it % G::NSTAGE, sph = (kv_it / G::NSTAGE) & 1;
        ok = warp_wait(ctx, BAR(B_P_FULL), p_it & 1, 14);
        if (!ok) break;
        ok = warp_wait(ctx, BAR(B_KV_FULL + st), sph, 15);
        if (!ok) break;
        tc_fence_after();
        if (lane == 0) {
          const uint32_t vbase = sbase + G::OFF_KV + st * G::TILE_BYTES;
#pragma unroll
          for (int k = 0; k < G::BK / 16; ++k) {
            uint64_t a = make_desc(sbase + G::OFF_P + (k / 4) * 128 * 128 + (k % 4) * 32, 16, 1024);
            // V tile as the N x K operand with N (head_dim) contiguous: 8 keys per 1024-byte
            // group along K, next 64 columns of head_dim one slab further
            uint64_t b = make_desc(vbase + k * 16 * 128, G::KV_SLAB_BYTES, 1024);
            umma_bf16(tmem_base + G::O_COL, a, b, IDESC_PV, (j > 0 || k > 0) ? 1u : 0u);
          }
          tc_commit(BAR(B_KV_EMPTY + st));
          tc_commit(BAR(B_PV_DONE));
        }
        __syncwarp();
        ++kv_it; ++p_it;
      }
    }
    // every MMA issued by this thread has completed before tensor memory is released
    if (lane == 0) tc_commit(BAR(B_FINAL));
    __syncwarp();
    {
      long long t0 = clock64();
      while (!mbar_try_wait(BAR(B_FINAL), 0) && clock64() - t0 < kTimeoutCycles / 4) {}
    }
  } else {
    // ============================================================== softmax / epilogue
    const int sw = warp - kSoftmaxWarp0;       // 0..7
    const int quad = warp & 3;                 // tensor-memory lane quadrant this warp may access
    const int half = sw >> 2;                  // which half of the S / O columns
    const int r = quad * 32 + lane;            // row of the 128-row MMA tile
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    uint32_t task_it = 0, s_it = 0, pv_it = 0;
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
      for (int j = 0; j < tk.n && ok; ++j) {
        const uint32_t buf = s_it & 1, bph = (s_it >> 1) & 1;
        ok = warp_wait(ctx, BAR(B_S_FULL + buf), bph, 21);
        if (!ok) break;
        tc_fence_after();
        uint32_t sv[G::CS];
        const uint32_t s_addr = tmem_base + lane_addr + (buf ? G::S_COL1 : G::S_COL0) + half * G::CS;
#pragma unroll
        for (int c = 0; c < G::CS; c += 32) WAVEAL_TMEM_LD32(s_addr + c, sv, c);
#pragma unroll
        for (int c = 0; c < G::CS; c += 32) WAVEAL_TMEM_WAIT_LD32(sv, c);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(B_S_EMPTY + buf));
        ++s_it;
        // scores of keys beyond seq_kv (ragged last block) do not exist
        if (j == tk.n - 1 && tk.tail_valid < G::BK) {
#pragma unroll
          for (int c = 0; c < G::CS; ++c)
            if (half * G::CS + c >= tk.tail_valid) sv[c] = __float_as_uint(-INFINITY);
        }
        float mloc = -INFINITY;
#pragma unroll
        for (int c = 0; c < G::CS; ++c) mloc = fmaxf(mloc, __uint_as_float(sv[c]));
        float* mxb = mx + (j & 1) * 256;
        mxb[half * 128 + r] = mloc;
        named_bar_sync(1 + quad, 64);
        const float m_blk = fmaxf(mloc, mxb[(half ^ 1) * 128 + r]) * p.sl2;
        const float m_cand = fmaxf(m_used, m_blk);
        // keep the stale reference max unless it is exceeded by more than 2^8 (exact: the
        // final normalisation divides by a sum taken with the same reference)
        const bool grow = __any_sync(0xffffffffu, m_cand > m_used + 8.0f);
        float alpha = 1.f;
        if (grow) {
          alpha = (m_used == -INFINITY) ? 0.f : ex2(m_used - m_cand);
          m_used = m_cand;
          l_run *= alpha;
        }
        uint32_t pk[G::CS / 2];
        float lsum = 0.f;
        const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
#pragma unroll
        for (int c = 0; c < G::CS; c += 2) {
          float p0 = ex2(fmaf(__uint_as_float(sv[c]), p.sl2, neg_m));
          float p1 = ex2(fmaf(__uint_as_float(sv[c + 1]), p.sl2, neg_m));
          lsum += p0 + p1;
          __nv_bfloat162 b2 = __floats2bfloat162_rn(p0, p1);
          pk[c / 2] = *reinterpret_cast<uint32_t*>(&b2);
        }
        l_run += lsum;
        // P_{j-1} V_{j-1} must be complete before O is rescaled or the P tile is overwritten
        if (j > 0) {
          ok = warp_wait(ctx, BAR(B_PV_DONE), pv_it & 1, 22);
          if (!ok) break;
          ++pv_it;
          tc_fence_after();
          if (grow) {
            uint32_t ov[G::CO];
            const uint32_t o_addr = tmem_base + lane_addr + G::O_COL + half * G::CO;
#pragma unroll
            for (int c = 0; c < G::CO; c += 32) WAVEAL_TMEM_LD32(o_addr + c, ov, c);
#pragma unroll
            for (int c = 0; c < G::CO; c += 32) WAVEAL_TMEM_WAIT_LD32(ov, c);
#pragma unroll
            for (int c = 0; c < G::CO; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * alpha);
#pragma unroll
            for (int c = 0; c < G::CO; c += 32) WAVEAL_TMEM_ST32(o_addr + c, ov, c);
            tc_wait_st();
          }
        }
        // P tile, K-major with 128-byte swizzle: key k of row r lives in slab k/64 at
        // r*128 + ((k%64)/8 ^ (r%8))*16 + (k%8)*2
        {
          unsigned char* prow = smem + G::OFF_P + r * 128;
#pragma unroll
          for (int c8 = 0; c8 < G::CS / 8; ++c8) {
            const int k0 = half * G::CS + c8 * 8;
            const int slab = k0 >> 6, chunk = (k0 & 63) >> 3;
            uint4 v = make_uint4(pk[c8 * 4 + 0], pk[c8 * 4 + 1], pk[c8 * 4 + 2], pk[c8 * 4 + 3]);
            *reinterpret_cast<uint4*>(prow + slab * 128 * 128 + ((chunk ^ (r & 7)) << 4)) = v;
          }
        }
        fence_proxy_async();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(B_P_FULL));
      }
      if (!ok) break;
      // ---- epilogue: O / l at the original row position
      ok = warp_wait(ctx, BAR(B_PV_DONE), pv_it & 1, 23);
      if (!ok) break;
      ++pv_it;
      tc_fence_after();
      float* lx = mx + (tk.n & 1) * 256;      // the buffer the last block did not use
      lx[half * 128 + r] = l_run;
      named_bar_sync(1 + quad, 64);
      const float l_tot = l_run + lx[(half ^ 1) * 128 + r];
      const float inv_l = 1.0f / l_tot;
      uint32_t ov[G::CO];
      const uint32_t o_addr = tmem_base + lane_addr + G::O_COL + half * G::CO;
#pragma unroll
      for (int c = 0; c < G::CO; c += 32) WAVEAL_TMEM_LD32(o_addr + c, ov, c);
#pragma unroll
      for (int c = 0; c < G::CO; c += 32) WAVEAL_TMEM_WAIT_LD32(ov, c);
      tc_fence_before();
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
      // the exchange buffer is reused by the next task's first block: keep the pair in step
      named_bar_sync(1 + quad, 64);
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
  WAVEAL_CUDA_OK(cudaMemsetAsync(p.ws, 0, 16, st));
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
