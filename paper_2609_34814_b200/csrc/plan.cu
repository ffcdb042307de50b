// Planning kernels: block mask -> per-head execution order of the query blocks.
//
// Algorithm 2 of the WaveAlign paper with the adaptive skip of Section 4.5 in front:
//   row block counts n_i and column counts c = M^T 1, guard statistics and decision,
//   Algorithm 1 (matrix-free centred subspace iteration, T sweeps, then the Rayleigh-Ritz
//   ordering), polar angle (Eq. 4), angular sort, wave-sized buckets, descending-count sort
//   inside each bucket.
//
// Layout of the work: the mask is kept as a bitmap M and its bit transpose Mt (both stay
// resident in L2; a bitmap is smaller than index lists once density exceeds 1/32).  A
// thread-block cluster of 1 to 4 CTAs of 1024 threads (as many as the device holds at once
// for the given number of heads) owns one head and runs every step for it, with the iteration
// blocks X, Y, Z (fp64) in shared memory, so the whole plan is one launch after the transpose
// and no step needs a grid-wide barrier.  The CTAs of a cluster keep identical copies of the
// state: the cheap steps (counts, guard, QR, rotation) are done by each of them in the same
// order, the two mask sweeps of an iteration - where the time goes - are split by rows and
// each result is written into every copy through distributed shared memory; the lead CTA does
// the sorts and writes the outputs.  All floating-point reductions use a fixed thread ->
// element assignment and a fixed combination tree, and a row is summed by the same lanes in the
// same order whichever CTA takes it, so a plan is reproducible bit for bit and does not
// depend on the cluster size.
#include <cfloat>
#include <climits>
#include <cmath>
#include <mutex>
#include "host_common.h"

namespace {

using u64 = unsigned long long;
constexpr int kPlanThreads = 1024;
constexpr int kPlanWarps = kPlanThreads / 32;
constexpr int kMaxSort = 16384;          // largest padded row count the in-smem sort takes
constexpr size_t kSmemMax = 232448;      // 227 KB opt-in limit per CTA on sm_100

// ------------------------------------------------------------------ format conversion

// index lists -> bitmap (bitmap zeroed beforehand); one warp per (head, row)
__global__ void k_csr_to_bitmap(const int* __restrict__ row_ptr, const int* __restrict__ idx,
                                u64* __restrict__ bits, long long n_rows, int wq, int n_kv,
                                int m_b, int* dev_status) {
  long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  int lane = threadIdx.x & 31;
  if (row >= n_rows) return;
  int lo = row_ptr[row], hi = row_ptr[row + 1];
  for (int e = lo + lane; e < hi; e += 32) {
    int j = idx[e];
    if (j < 0 || j >= n_kv) {
      if (dev_status && atomicCAS(dev_status, 0, WAVEAL_ERR_BAD_MASK) == 0) {
        dev_status[1] = 1; dev_status[2] = (int)(row / m_b); dev_status[3] = j;
      }
      continue;
    }
    atomicOr(&bits[row * wq + (j >> 6)], 1ull << (j & 63));
  }
}

// Mt[h][j][i>>6] bit (i&63) = M[h][i][j>>6] bit (j&63); one 64x64-bit tile per CTA of 64 threads
__global__ void k_transpose_bits(const u64* __restrict__ M, u64* __restrict__ Mt, int m_b, int n_b,
                                 int wq, int wk) {
  __shared__ u64 tile[64];
  int h = blockIdx.z, jw = blockIdx.x, iw = blockIdx.y, t = threadIdx.x;
  int i = iw * 64 + t;
  tile[t] = i < m_b ? M[((size_t)h * m_b + i) * wq + jw] : 0ull;
  __syncthreads();
  int j = jw * 64 + t;
  if (j < n_b) {
    u64 o = 0;
#pragma unroll 8
    for (int r = 0; r < 64; ++r) o |= ((tile[r] >> t) & 1ull) << r;
    Mt[((size_t)h * n_b + j) * wk + iw] = o;
  }
}

// per-row popcount over all heads (used by bitmap -> index lists)
__global__ void k_row_popcount(const u64* __restrict__ bits, long long n_rows, int wq, int* __restrict__ cnt) {
  long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  int lane = threadIdx.x & 31;
  if (row >= n_rows) return;
  int c = 0;
  for (int w = lane; w < wq; w += 32) c += __popcll(bits[row * wq + w]);
#pragma unroll
  for (int o = 16; o; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
  if (lane == 0) cnt[row] = c;
}

// exclusive scan of cnt[0..n) into ptr[0..n]; single CTA
__global__ void k_exclusive_scan(const int* __restrict__ cnt, long long n, int* __restrict__ ptr) {
  __shared__ int warp_tot[32];
  __shared__ int carry_s;
  int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) carry_s = 0;
  __syncthreads();
  for (long long base = 0; base < n; base += blockDim.x) {
    long long i = base + tid;
    int v = i < n ? cnt[i] : 0;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    int carry = carry_s, pre = 0;
    for (int w = 0; w < warp; ++w) pre += warp_tot[w];
    if (i < n) ptr[i] = carry + pre + incl - v;
    __syncthreads();
    if (tid == blockDim.x - 1) carry_s = carry + pre + incl;
    __syncthreads();
  }
  if (tid == 0) ptr[n] = carry_s;
}

// bitmap -> ascending index lists; one warp per (head, row)
__global__ void k_fill_indices(const u64* __restrict__ bits, long long n_rows, int wq,
                               const int* __restrict__ ptr, int* __restrict__ idx, long long capacity) {
  long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  int lane = threadIdx.x & 31;
  if (row >= n_rows) return;
  long long out = ptr[row];
  for (int w0 = 0; w0 < wq; w0 += 32) {
    int w = w0 + lane;
    u64 word = w < wq ? bits[row * wq + w] : 0ull;
    int c = __popcll(word), incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    long long pos = out + incl - c;
    while (word) {
      int b = __ffsll((long long)word) - 1;
      word &= word - 1;
      if (pos < capacity) idx[pos] = w * 64 + b;
      ++pos;
    }
    out += __shfl_sync(0xffffffffu, incl, 31);
  }
}

// ------------------------------------------------------------------ block-wide helpers

// Sum of N doubles per thread over the CTA, same result in every thread; fixed tree
// (lanes, then warps).  fp64 adds are scarce on this part, so the second level is one more
// shuffle tree in warp 0, not a serial sum in every thread.
template <int N>
__device__ __forceinline__ void block_sum(double (&v)[N], double* scratch) {
  int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int k = 0; k < N; ++k) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v[k] += __shfl_xor_sync(0xffffffffu, v[k], o);
  }
  if (lane == 0) {
#pragma unroll
    for (int k = 0; k < N; ++k) scratch[warp * N + k] = v[k];
  }
  __syncthreads();
  if (warp == 0) {
    double t[N];
#pragma unroll
    for (int k = 0; k < N; ++k) {
      t[k] = scratch[lane * N + k];           // kPlanWarps == 32: one partial per lane
#pragma unroll
      for (int o = 16; o; o >>= 1) t[k] += __shfl_xor_sync(0xffffffffu, t[k], o);
    }
    if (lane == 0) {
#pragma unroll
      for (int k = 0; k < N; ++k) scratch[kPlanWarps * N + k] = t[k];
    }
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < N; ++k) v[k] = scratch[kPlanWarps * N + k];
  __syncthreads();
}

__device__ __forceinline__ long long block_sum_i64(long long v, long long* scratch) {
  int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  long long s = 0;
  for (int w = 0; w < kPlanWarps; ++w) s += scratch[w];
  __syncthreads();
  return s;
}

__device__ __forceinline__ double block_max(double v, double* scratch) {
  int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  double s = scratch[0];
  for (int w = 1; w < kPlanWarps; ++w) s = fmax(s, scratch[w]);
  __syncthreads();
  return s;
}

__device__ __forceinline__ int block_min_int(int v, int* scratch) {
  int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o; o >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, o));
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  int s = scratch[0];
  for (int w = 1; w < kPlanWarps; ++w) s = min(s, scratch[w]);
  __syncthreads();
  return s;
}

// ---- thread-block cluster helpers: the CTAs of a cluster split the rows of the two mask sweeps
// of a head between them and write every result into each other's shared memory
__device__ __forceinline__ unsigned cluster_rank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// store a double2 at the same shared-memory offset of CTA `rank` of this cluster
__device__ __forceinline__ void store_peer(const double2* local_ptr, unsigned rank, double2 v) {
  unsigned laddr = (unsigned)__cvta_generic_to_shared(local_ptr), raddr;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(laddr), "r"(rank));
  asm volatile("st.shared::cluster.v2.f64 [%0], {%1, %2};" ::"r"(raddr), "d"(v.x), "d"(v.y) : "memory");
}

// number of set bits with index in [lo, hi) of a bit row
__device__ __forceinline__ int popcount_range(const u64* __restrict__ words, int lo, int hi) {
  if (hi <= lo) return 0;
  int w0 = lo >> 6, w1 = (hi - 1) >> 6, c = 0;
  for (int w = w0; w <= w1; ++w) {
    u64 x = words[w];
    if (w == w0) x &= ~0ull << (lo & 63);
    if (w == w1 && (hi & 63)) x &= (1ull << (hi & 63)) - 1ull;
    c += __popcll(x);
  }
  return c;
}

// dst[r] = sum_{c : bit (r, c) set} src[c] - rowscale(r) * corr ; rowscale = cnt[r] or 1.
// L lanes share one bit row (lane q of the group takes words q, q+L, ...), 32/L rows per warp
// step; the partial sums meet in a fixed shuffle tree of width L.  Fewer lanes per row than a
// whole warp keeps more rows in flight and wastes fewer of the scarce fp64 adds on the tree.
// crank / csize: this CTA's rank in its cluster and the cluster's size; the CTAs take the warp
// steps in turn, and when `peers` is set (state in shared memory) every result is also written
// into the other CTAs' copy of dst.  A row is summed by the same lanes in the same order
// whichever CTA takes it, so the result does not depend on the cluster size.
template <int L>
__device__ __forceinline__ void gather_rows_l(const u64* __restrict__ bits, int n_rows, int wpr,
                                              const double2* src, double2* dst,
                                              const int* __restrict__ cnt, double2 corr,
                                              int crank, int csize, bool peers) {
  constexpr int RPW = 32 / L;                       // rows per warp step
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int grp = lane / L, q = lane % L;
  for (int r0 = (warp + crank * kPlanWarps) * RPW; r0 < n_rows; r0 += csize * kPlanWarps * RPW) {
    const int r = r0 + grp;
    const bool live = r < n_rows;
    double ax = 0.0, ay = 0.0;
    for (int w0 = 0; w0 < wpr; w0 += 4 * L) {
      u64 word[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int w = w0 + q + k * L;
        word[k] = (live && w < wpr) ? bits[(size_t)r * wpr + w] : 0ull;
      }
      // walk the set bits of each word as two 32-bit halves (64-bit bit tricks cost twice
      // the integer instructions, and this loop is bound by them)
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const double2* sp = src + (w0 + q + k * L) * 64;
#pragma unroll
        for (int hw = 0; hw < 2; ++hw) {
          unsigned x = hw ? (unsigned)(word[k] >> 32) : (unsigned)word[k];
          while (x) {
            const int b = __ffs((int)x) - 1;
            x &= x - 1;
            const double2 v = sp[hw * 32 + b];
            ax += v.x;
            ay += v.y;
          }
        }
      }
    }
#pragma unroll
    for (int o = L / 2; o; o >>= 1) {
      ax += __shfl_xor_sync(0xffffffffu, ax, o);
      ay += __shfl_xor_sync(0xffffffffu, ay, o);
    }
    if (live && q == 0) {
      const double sc = cnt ? (double)cnt[r] : 1.0;
      const double2 v = make_double2(ax - sc * corr.x, ay - sc * corr.y);
      dst[r] = v;
      if (peers)
        for (int c = 0; c < csize; ++c)
          if (c != crank) store_peer(dst + r, (unsigned)c, v);
    }
  }
}

__device__ __forceinline__ void gather_rows(const u64* __restrict__ bits, int n_rows, int wpr,
                                            const double2* src, double2* dst,
                                            const int* __restrict__ cnt, double2 corr,
                                            int crank, int csize, bool peers) {
  // about three words per lane
  if (wpr <= 3) gather_rows_l<1>(bits, n_rows, wpr, src, dst, cnt, corr, crank, csize, peers);
  else if (wpr <= 6) gather_rows_l<2>(bits, n_rows, wpr, src, dst, cnt, corr, crank, csize, peers);
  else if (wpr <= 12) gather_rows_l<4>(bits, n_rows, wpr, src, dst, cnt, corr, crank, csize, peers);
  else if (wpr <= 24) gather_rows_l<8>(bits, n_rows, wpr, src, dst, cnt, corr, crank, csize, peers);
  else if (wpr <= 48) gather_rows_l<16>(bits, n_rows, wpr, src, dst, cnt, corr, crank, csize, peers);
  else gather_rows_l<32>(bits, n_rows, wpr, src, dst, cnt, corr, crank, csize, peers);
}

// Q factor of the thin QR of an m x 2 block: Gram-Schmidt with one re-orthogonalisation
// pass; numerically dependent columns become zero.  Returns the column sums of Q.
__device__ __forceinline__ double2 thin_qr2(const double2* zin, double2* xout, int m, double* scratch) {
  const double tiny = 1e-30 * sqrt((double)m);
  int tid = threadIdx.x;
  double a[2] = {0, 0};
  for (int i = tid; i < m; i += kPlanThreads) { double2 z = zin[i]; a[0] += z.x * z.x; a[1] += z.y * z.y; }
  block_sum<2>(a, scratch);
  double n1 = sqrt(a[0]), n2_before = sqrt(a[1]);
  bool ok1 = n1 > tiny;
  double d[1] = {0};
  for (int i = tid; i < m; i += kPlanThreads) {
    double2 z = zin[i];
    double q1 = ok1 ? z.x / n1 : 0.0;
    xout[i] = make_double2(q1, z.y);
    d[0] += q1 * z.y;
  }
  block_sum<1>(d, scratch);
  double e[1] = {0};
  for (int i = tid; i < m; i += kPlanThreads) {
    double2 x = xout[i];
    x.y = x.y - d[0] * x.x;
    xout[i] = x;
    e[0] += x.x * x.y;
  }
  block_sum<1>(e, scratch);
  double f[1] = {0};
  for (int i = tid; i < m; i += kPlanThreads) {
    double2 x = xout[i];
    x.y = x.y - e[0] * x.x;
    xout[i] = x;
    f[0] += x.y * x.y;
  }
  block_sum<1>(f, scratch);
  double n2 = sqrt(f[0]);
  bool ok2 = n2 > tiny && n2 > 1e-9 * n2_before;
  double s[2] = {0, 0};
  for (int i = tid; i < m; i += kPlanThreads) {
    double2 x = xout[i];
    x.y = ok2 ? x.y / n2 : 0.0;
    xout[i] = x;
    s[0] += x.x;
    s[1] += x.y;
  }
  block_sum<2>(s, scratch);
  return make_double2(s[0], s[1]);
}

__device__ __forceinline__ u64 splitmix64(u64 x) {
  u64 z = x + 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// monotone map double -> u64 (no NaN expected; -0.0 is removed by the caller)
__device__ __forceinline__ u64 sortable(double v) {
  u64 b = (u64)__double_as_longlong(v);
  return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
}

// ascending bitonic sort of (key, val) pairs, ties by val; n is a power of two
__device__ __forceinline__ void bitonic_sort(u64* keys, int* vals, int n) {
  for (int k = 2; k <= n; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int t = threadIdx.x; t < n; t += kPlanThreads) {
        int p = t ^ j;
        if (p > t) {
          u64 ka = keys[t], kb = keys[p];
          int va = vals[t], vb = vals[p];
          bool a_gt_b = ka > kb || (ka == kb && va > vb);
          bool asc = (t & k) == 0;
          if (a_gt_b == asc) { keys[t] = kb; keys[p] = ka; vals[t] = vb; vals[p] = va; }
        }
      }
      __syncthreads();
    }
  }
}

struct PlanParams {
  const u64* M;
  const u64* Mt;
  int m_b, n_b, wq, wk, wave, iters, mode, n_pow2, state_in_smem;
  int ring_cut;         // open the angular ring at its largest gap instead of at -pi
  int csize;            // CTAs per head (thread-block cluster size)
  u64 seed;
  long long kv_bytes, l2_bytes, min_nnz;
  int fit_num, fit_den, min_ppm, loc_num, loc_den;
  int* ws_nnz;          // [heads][m_b]
  int* ws_cnt;          // [heads][n_b]
  double2* ws_state;    // [heads][2*m_b + n_b] when the blocks do not fit shared memory
  int* row_order; int* row_nnz; unsigned char* flags; int* col_count; int* order1;
  double* embedding; long long* stats;
};

__global__ void __launch_bounds__(kPlanThreads, 1) k_plan_head(PlanParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  double* scratch = reinterpret_cast<double*>(smem);                 // (32 + 1) * 4 doubles
  unsigned char* region = smem + 2048;
  // A head is planned by a cluster of p.csize CTAs.  Everything cheap (counts, guard, QR,
  // rotations, sorts) is done by every CTA of the cluster on its own copy of the state, in the
  // same order, so the copies stay identical bit for bit; only the two mask sweeps of an
  // iteration, where the time goes, are split, and their results exchanged.
  const int csize = p.csize, crank = csize > 1 ? (int)cluster_rank() : 0;
  const int h = blockIdx.x / csize, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool lead = crank == 0;         // writes the outputs
  const int m_b = p.m_b, n_b = p.n_b;
  const u64* M = p.M + (size_t)h * m_b * p.wq;
  const u64* Mt = p.Mt + (size_t)h * n_b * p.wk;
  int* nnz = p.ws_nnz + (size_t)h * m_b;
  int* cnt = p.ws_cnt + (size_t)h * n_b;
  int* order_out = p.row_order + (size_t)h * m_b;
  int* order1_out = p.order1 ? p.order1 + (size_t)h * m_b : nullptr;

  // ---- n_i = sum_j M_ij and c = M^T 1 (Section 2.2; Algorithm 1 step 1)
  long long my_nnz = 0;
  for (int r = warp; r < m_b; r += kPlanWarps) {
    int c = 0;
    for (int w = lane; w < p.wq; w += 32) c += __popcll(M[(size_t)r * p.wq + w]);
#pragma unroll
    for (int o = 16; o; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    if (lane == 0) { nnz[r] = c; if (p.row_nnz && lead) p.row_nnz[(size_t)h * m_b + r] = c; my_nnz += c; }
  }
  for (int j = warp; j < n_b; j += kPlanWarps) {
    int c = 0;
    for (int w = lane; w < p.wk; w += 32) c += __popcll(Mt[(size_t)j * p.wk + w]);
#pragma unroll
    for (int o = 16; o; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    if (lane == 0) { cnt[j] = c; if (p.col_count && lead) p.col_count[(size_t)h * n_b + j] = c; }
  }
  // ---- guard statistics over natural-order waves (Section 4.5)
  const int n_waves = (m_b + p.wave - 1) / p.wave;
  long long ov = 0, pair2 = 0;
  for (int j = warp; j < n_b; j += kPlanWarps) {
    const u64* col = Mt + (size_t)j * p.wk;
    for (int l = lane; l < n_waves; l += 32) {
      int lo = l * p.wave, hi = min(lo + p.wave, m_b);
      long long c = popcount_range(col, lo, hi);
      ov += c * (c - 1) / 2;
      pair2 += (long long)(hi - lo - 1) * c;
    }
  }
  long long* iscratch = reinterpret_cast<long long*>(scratch);
  long long nnz_total = block_sum_i64(my_nnz, iscratch);
  ov = block_sum_i64(ov, iscratch);
  pair2 = block_sum_i64(pair2, iscratch);
  unsigned flags = 0;
  if (p.kv_bytes > 0 && p.l2_bytes > 0 && p.kv_bytes * p.fit_den <= p.l2_bytes * p.fit_num)
    flags |= WAVEAL_FLAG_SHORT_SEQ;
  if (nnz_total < p.min_nnz || nnz_total * 1000000ll < (long long)p.min_ppm * m_b * n_b)
    flags |= WAVEAL_FLAG_TOO_SPARSE;
  if (pair2 > 0 && 2 * ov * p.loc_den >= (long long)p.loc_num * pair2) flags |= WAVEAL_FLAG_ALREADY_LOCAL;
  const bool skip = p.mode == WAVEAL_FORCE_NATURAL || (p.mode == WAVEAL_AUTO && flags != 0);
  if (skip) flags |= WAVEAL_FLAG_SKIPPED;
  if (tid == 0 && lead) {
    if (p.flags) p.flags[h] = (unsigned char)flags;
    if (p.stats) { long long* s = p.stats + (size_t)h * 4; s[0] = nnz_total; s[1] = ov; s[2] = pair2; s[3] = 0; }
  }
  if (skip) {
    if (lead)
    for (int i = tid; i < m_b; i += kPlanThreads) {
      order_out[i] = i;
      if (order1_out) order1_out[i] = i;
      if (p.embedding) { p.embedding[((size_t)h * m_b + i) * 2] = 0.0; p.embedding[((size_t)h * m_b + i) * 2 + 1] = 0.0; }
    }
    return;
  }
  __syncthreads();   // nnz[] / cnt[] (global) written by this CTA are visible to all its threads

  u64* keys = reinterpret_cast<u64*>(region);
  int* vals = reinterpret_cast<int*>(region + (size_t)p.n_pow2 * 8);

  if (p.mode != WAVEAL_STAGE2_ONLY) {
    double2* X = p.state_in_smem ? reinterpret_cast<double2*>(region)
                                 : p.ws_state + (size_t)h * (2 * (size_t)m_b + n_b);
    double2* Z = X + m_b;
    double2* Y = Z + m_b;
    const double inv_m = 1.0 / (double)m_b;
    // ---- start block (counter-based) and its orthonormalisation (Algorithm 1, step 3)
    const u64 hk = (u64)h * 0x9E3779B97F4A7C15ull;
    for (int i = tid; i < m_b; i += kPlanThreads) {
      double u0 = (double)(splitmix64(p.seed ^ hk ^ (u64)(2 * i)) >> 11) * (1.0 / 9007199254740992.0);
      double u1 = (double)(splitmix64(p.seed ^ hk ^ (u64)(2 * i + 1)) >> 11) * (1.0 / 9007199254740992.0);
      Z[i] = make_double2(2.0 * u0 - 1.0, 2.0 * u1 - 1.0);
    }
    __syncthreads();
    double2 colsum = thin_qr2(Z, X, m_b, scratch);
    // ---- T sweeps + one more for the Rayleigh-Ritz step
    for (int it = 0; it <= p.iters; ++it) {
      // Y = M^T X - c (1^T X)/m
      gather_rows(Mt, n_b, p.wk, X, Y, cnt, make_double2(colsum.x * inv_m, colsum.y * inv_m), crank, csize, csize > 1);
      if (csize > 1) cluster_sync_all(); else __syncthreads();
      double cy[2] = {0, 0};
      for (int j = tid; j < n_b; j += kPlanThreads) { double2 y = Y[j]; double c = (double)cnt[j]; cy[0] += c * y.x; cy[1] += c * y.y; }
      block_sum<2>(cy, scratch);
      // Z = M Y - 1 (c^T Y)/m
      gather_rows(M, m_b, p.wq, Y, Z, nullptr, make_double2(cy[0] * inv_m, cy[1] * inv_m), crank, csize, csize > 1);
      if (csize > 1) cluster_sync_all(); else __syncthreads();
      if (it < p.iters) colsum = thin_qr2(Z, X, m_b, scratch);
    }
    // the rest (ordering, angles, sorts, outputs) is cheap: the lead CTA finishes alone.  No CTA
    // touches another's shared memory after the last exchange above.
    if (!lead) return;
    // ---- B = X^T Z, rotate onto the eigenvectors of its symmetric part, larger Ritz value first
    double b[4] = {0, 0, 0, 0};
    for (int i = tid; i < m_b; i += kPlanThreads) {
      double2 x = X[i], z = Z[i];
      b[0] += x.x * z.x; b[1] += x.x * z.y; b[2] += x.y * z.x; b[3] += x.y * z.y;
    }
    block_sum<4>(b, scratch);
    double th = 0.5 * atan2(2.0 * (0.5 * (b[1] + b[2])), b[0] - b[3]);
    double cs = cos(th), sn = sin(th);
    double mx1 = 0, mx2 = 0;
    for (int i = tid; i < m_b; i += kPlanThreads) {
      double2 x = X[i];
      double2 u = make_double2(x.x * cs + x.y * sn, x.y * cs - x.x * sn);
      X[i] = u;
      mx1 = fmax(mx1, fabs(u.x));
      mx2 = fmax(mx2, fabs(u.y));
    }
    mx1 = block_max(mx1, scratch);
    mx2 = block_max(mx2, scratch);
    // ---- sign: the first entry reaching half of the largest magnitude is made positive
    int f1 = INT_MAX, f2 = INT_MAX;
    for (int i = tid; i < m_b; i += kPlanThreads) {
      double2 u = X[i];
      if (mx1 > 0.0 && fabs(u.x) >= 0.5 * mx1) f1 = min(f1, i);
      if (mx2 > 0.0 && fabs(u.y) >= 0.5 * mx2) f2 = min(f2, i);
    }
    int* mscratch = reinterpret_cast<int*>(scratch);
    f1 = block_min_int(f1, mscratch);
    f2 = block_min_int(f2, mscratch);
    double s1 = (f1 != INT_MAX && X[f1].x < 0.0) ? -1.0 : 1.0;
    double s2 = (f2 != INT_MAX && X[f2].y < 0.0) ? -1.0 : 1.0;
    __syncthreads();
    // ---- polar angle a_i = atan2(u_2[i], u_1[i]) (Eq. 4); kept in registers across the
    //      re-use of the shared region by the sort
    constexpr int kPer = (kMaxSort + kPlanThreads - 1) / kPlanThreads;
    double ang[kPer];
#pragma unroll
    for (int k = 0; k < kPer; ++k) {
      int i = tid + k * kPlanThreads;
      ang[k] = 0.0;
      if (i < m_b) {
        double2 u = X[i];
        double u1 = s1 * u.x + 0.0, u2 = s2 * u.y + 0.0;
        if (p.embedding) { p.embedding[((size_t)h * m_b + i) * 2] = u1; p.embedding[((size_t)h * m_b + i) * 2 + 1] = u2; }
        ang[k] = atan2(u2, u1) + 0.0;
      }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kPer; ++k) {
      int i = tid + k * kPlanThreads;
      if (i < p.n_pow2) {
        keys[i] = i < m_b ? sortable(ang[k]) : ~0ull;
        vals[i] = i < m_b ? i : INT_MAX;
      }
    }
    __syncthreads();
    bitonic_sort(keys, vals, p.n_pow2);     // Stage 1: rows by ascending angle, ties by row index
    if (p.ring_cut && m_b >= 2) {
      // Variant: the sorted rows form a ring (Section 4.3.1); open it at the largest gap between
      // neighbouring angles (the gap around the back, first + 2 pi - last, included; the first
      // of equal gaps wins) instead of at -pi, where atan2 happens to put the cut.
      auto angle_at = [&](int i) {          // inverse of sortable()
        const u64 k = keys[i];
        return __longlong_as_double((long long)((k >> 63) ? (k & 0x7FFFFFFFFFFFFFFFull) : ~k));
      };
      double best = -1.0;
      for (int i = tid; i < m_b; i += kPlanThreads) {
        const double g = i + 1 < m_b ? angle_at(i + 1) - angle_at(i)
                                     : (angle_at(0) + 2.0 * 3.14159265358979323846) - angle_at(m_b - 1);
        best = fmax(best, g);
      }
      best = block_max(best, scratch);
      int at = INT_MAX;
      for (int i = tid; i < m_b; i += kPlanThreads) {
        const double g = i + 1 < m_b ? angle_at(i + 1) - angle_at(i)
                                     : (angle_at(0) + 2.0 * 3.14159265358979323846) - angle_at(m_b - 1);
        if (g == best) at = min(at, i);
      }
      at = block_min_int(at, reinterpret_cast<int*>(scratch));
      // rotate: the row behind the gap comes first (the key array is free until Stage 2 refills it)
      int* tmp = reinterpret_cast<int*>(keys);
      __syncthreads();
      for (int i = tid; i < m_b; i += kPlanThreads) {
        int src = i + at + 1;
        if (src >= m_b) src -= m_b;
        tmp[i] = vals[src];
      }
      __syncthreads();
      for (int i = tid; i < m_b; i += kPlanThreads) vals[i] = tmp[i];
      __syncthreads();
    }
  } else {
    if (!lead) return;
    if (p.embedding)
      for (int i = tid; i < m_b; i += kPlanThreads) { p.embedding[((size_t)h * m_b + i) * 2] = 0.0; p.embedding[((size_t)h * m_b + i) * 2 + 1] = 0.0; }
    for (int i = tid; i < p.n_pow2; i += kPlanThreads) vals[i] = i < m_b ? i : INT_MAX;
    __syncthreads();
  }
  if (order1_out)
    for (int i = tid; i < m_b; i += kPlanThreads) order1_out[i] = vals[i];
  if (p.mode == WAVEAL_STAGE1_ONLY) {
    for (int i = tid; i < m_b; i += kPlanThreads) order_out[i] = vals[i];
    return;
  }
  // ---- Stage 2: inside each bucket of `wave` consecutive positions, descending n_i, ties by
  //      Stage-1 position: one sort on the key (bucket, max_count - n_i, position)
  for (int i = tid; i < p.n_pow2; i += kPlanThreads) {
    if (i < m_b) {
      u64 bucket = (u64)(i / p.wave);
      u64 inv = (u64)(0x3FFFFF - min(nnz[vals[i]], 0x3FFFFF));
      keys[i] = (bucket << 44) | (inv << 22) | (u64)i;
    } else {
      keys[i] = ~0ull;
    }
  }
  __syncthreads();
  bitonic_sort(keys, vals, p.n_pow2);
  for (int i = tid; i < m_b; i += kPlanThreads) order_out[i] = vals[i];
}

// ------------------------------------------------------------------ host side

struct PlanLayout {
  size_t off_bitmap, off_mt, off_nnz, off_cnt, off_state, total;
  int wq, wk, n_pow2, state_in_smem;
  size_t smem;
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

waveal_status plan_layout(const waveal_plan_desc* d, PlanLayout* L) {
  if (!d) return waveal::fail(WAVEAL_ERR_INVALID_ARG, "desc is NULL");
  if (d->heads <= 0 || d->n_q_blocks <= 0 || d->n_kv_blocks <= 0)
    return waveal::fail(WAVEAL_ERR_INVALID_ARG, "heads, n_q_blocks and n_kv_blocks must be positive");
  if (d->wave_size < 0 || d->svd_iters < 0 || d->svd_iters > 1000)
    return waveal::fail(WAVEAL_ERR_INVALID_ARG, "wave_size must be >= 0 and svd_iters in [0, 1000]");
  const int base_mode = d->mode & ~WAVEAL_RING_CUT_LARGEST_GAP;
  if (base_mode < WAVEAL_AUTO || base_mode > WAVEAL_STAGE2_ONLY)
    return waveal::fail(WAVEAL_ERR_INVALID_ARG, "unknown mode %d", d->mode);
  if (d->l2_fit_den <= 0 || d->local_den <= 0 || d->l2_fit_num < 0 || d->local_num < 0 || d->min_density_ppm < 0)
    return waveal::fail(WAVEAL_ERR_INVALID_ARG, "guard thresholds must be non-negative with positive denominators");
  if (d->n_q_blocks > kMaxSort)
    return waveal::fail(WAVEAL_ERR_UNSUPPORTED, "n_q_blocks %d exceeds the supported maximum %d", d->n_q_blocks, kMaxSort);
  if (d->n_kv_blocks >= (1 << 22))
    return waveal::fail(WAVEAL_ERR_UNSUPPORTED, "n_kv_blocks %d exceeds the supported maximum", d->n_kv_blocks);
  size_t H = d->heads, m = d->n_q_blocks, n = d->n_kv_blocks;
  L->wq = (int)((n + 63) / 64);
  L->wk = (int)((m + 63) / 64);
  int p2 = 1;
  while (p2 < d->n_q_blocks) p2 <<= 1;
  L->n_pow2 = p2;
  size_t sort_bytes = (size_t)p2 * 12, state_bytes = (2 * m + n) * 16;
  L->state_in_smem = 2048 + (state_bytes > sort_bytes ? state_bytes : sort_bytes) <= kSmemMax;
  L->smem = 2048 + (L->state_in_smem ? (state_bytes > sort_bytes ? state_bytes : sort_bytes) : sort_bytes);
  size_t o = 0;
  L->off_bitmap = o; o = align_up(o + H * m * L->wq * 8, 256);
  L->off_mt = o;     o = align_up(o + H * n * L->wk * 8, 256);
  L->off_nnz = o;    o = align_up(o + H * m * 4, 256);
  L->off_cnt = o;    o = align_up(o + H * n * 4, 256);
  L->off_state = o;  o = align_up(o + (L->state_in_smem ? 0 : H * (2 * m + n) * 16), 256);
  L->total = o;
  return WAVEAL_OK;
}

waveal_status plan_common(const waveal_plan_desc* d, const u64* mask_bits, const int* row_ptr, const int* idx,
                          void* ws, size_t ws_bytes, const waveal_plan_out* out, cudaStream_t st) {
  PlanLayout L;
  waveal_status s = plan_layout(d, &L);
  if (s != WAVEAL_OK) return s;
  if (!out || !out->row_order) return waveal::fail(WAVEAL_ERR_INVALID_ARG, "out->row_order is required");
  if (!ws || ws_bytes < L.total)
    return waveal::fail(WAVEAL_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", L.total, ws ? ws_bytes : (size_t)0);
  if (!waveal::aligned(ws, 256)) return waveal::fail(WAVEAL_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
  if (mask_bits && !waveal::aligned(mask_bits, 8)) return waveal::fail(WAVEAL_ERR_INVALID_ARG, "mask_bits must be 8-byte aligned");
  int dev = 0, sms = 0, l2 = 0;
  WAVEAL_CUDA_OK(cudaGetDevice(&dev));
  WAVEAL_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  WAVEAL_CUDA_OK(cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev));
  WAVEAL_CUDA_OK(cudaFuncSetAttribute(k_plan_head, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L.smem));
  unsigned char* w = static_cast<unsigned char*>(ws);
  int launches = 0;
  const size_t H = d->heads, m = d->n_q_blocks, n = d->n_kv_blocks;
  const u64* M = mask_bits;
  if (!M) {
    u64* bm = reinterpret_cast<u64*>(w + L.off_bitmap);
    WAVEAL_CUDA_OK(cudaMemsetAsync(bm, 0, H * m * L.wq * 8, st));
    long long rows = (long long)(H * m);
    k_csr_to_bitmap<<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(row_ptr, idx, bm, rows, L.wq, (int)n, (int)m, out->dev_status);
    ++launches;
    M = bm;
  }
  u64* Mt = reinterpret_cast<u64*>(w + L.off_mt);
  k_transpose_bits<<<dim3(L.wq, L.wk, (unsigned)H), 64, 0, st>>>(M, Mt, (int)m, (int)n, L.wq, L.wk);
  ++launches;
  PlanParams p{};
  p.M = M; p.Mt = Mt; p.m_b = (int)m; p.n_b = (int)n; p.wq = L.wq; p.wk = L.wk;
  p.wave = d->wave_size > 0 ? d->wave_size : sms;
  p.iters = d->svd_iters; p.mode = d->mode & ~WAVEAL_RING_CUT_LARGEST_GAP;
  p.ring_cut = (d->mode & WAVEAL_RING_CUT_LARGEST_GAP) ? 1 : 0; p.n_pow2 = L.n_pow2; p.state_in_smem = L.state_in_smem;
  p.seed = d->seed;
  p.kv_bytes = d->kv_bytes_per_head; p.l2_bytes = d->l2_bytes > 0 ? d->l2_bytes : (long long)l2;
  p.min_nnz = d->min_nnz; p.fit_num = d->l2_fit_num; p.fit_den = d->l2_fit_den; p.min_ppm = d->min_density_ppm;
  p.loc_num = d->local_num; p.loc_den = d->local_den;
  p.ws_nnz = reinterpret_cast<int*>(w + L.off_nnz);
  p.ws_cnt = reinterpret_cast<int*>(w + L.off_cnt);
  p.ws_state = reinterpret_cast<double2*>(w + L.off_state);
  p.row_order = out->row_order; p.row_nnz = out->row_nnz; p.flags = out->skip_flags; p.col_count = out->col_count;
  p.order1 = out->order1; p.embedding = out->embedding; p.stats = reinterpret_cast<long long*>(out->stats);
  // CTAs per head: as many as fit the device at once (clusters of 1 to 4 CTAs on neighbouring
  // SMs), when the iteration blocks live in shared memory and some head may be planned at all
  int csize = 1;
  if (L.state_in_smem && p.mode != WAVEAL_FORCE_NATURAL && p.mode != WAVEAL_STAGE2_ONLY) {
    csize = (int)(sms / (long long)H);
    csize = csize < 1 ? 1 : csize > 4 ? 4 : csize;
  }
  p.csize = csize;
  if (csize == 1) {
    k_plan_head<<<(unsigned)H, kPlanThreads, L.smem, st>>>(p);
  } else {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(H * csize));
    cfg.blockDim = dim3(kPlanThreads);
    cfg.dynamicSmemBytes = L.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)csize; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    WAVEAL_CUDA_OK(cudaLaunchKernelEx(&cfg, k_plan_head, p));
  }
  ++launches;
  WAVEAL_CUDA_OK(cudaGetLastError());
  waveal::launch_counter() = launches;
  return WAVEAL_OK;
}

}  // namespace

extern "C" void waveal_plan_desc_default(waveal_plan_desc* d) {
  if (!d) return;
  *d = waveal_plan_desc{};
  d->svd_iters = 5;    // low end of the paper's 5-15: the attention time did not move between 3, 5 and 10 on the measured shapes
  d->mode = WAVEAL_AUTO;
  d->l2_fit_num = 9; d->l2_fit_den = 16;   // calibrated on the B200 (calibrate_guard): no gain up to K+V = 0.57 x L2 on either mask family
  d->min_density_ppm = 10000;
  d->local_num = 1; d->local_den = 2;
  d->min_nnz = 0;
}

extern "C" waveal_status waveal_plan_workspace_bytes(const waveal_plan_desc* desc, size_t* bytes) {
  PlanLayout L;
  waveal_status s = plan_layout(desc, &L);
  if (s != WAVEAL_OK) return s;
  if (!bytes) return waveal::fail(WAVEAL_ERR_INVALID_ARG, "bytes is NULL");
  *bytes = L.total;
  return WAVEAL_OK;
}

extern "C" waveal_status waveal_plan_bitmap(const waveal_plan_desc* desc, const uint64_t* mask_bits, void* ws,
                                            size_t ws_bytes, const waveal_plan_out* out, void* cuda_stream) {
  if (!mask_bits) return waveal::fail(WAVEAL_ERR_INVALID_ARG, "mask_bits is NULL");
  return plan_common(desc, reinterpret_cast<const u64*>(mask_bits), nullptr, nullptr, ws, ws_bytes, out,
                     static_cast<cudaStream_t>(cuda_stream));
}

extern "C" waveal_status waveal_plan_csr(const waveal_plan_desc* desc, const int32_t* kv_row_ptr,
                                         const int32_t* kv_block_indices, void* ws, size_t ws_bytes,
                                         const waveal_plan_out* out, void* cuda_stream) {
  if (!kv_row_ptr || !kv_block_indices) return waveal::fail(WAVEAL_ERR_INVALID_ARG, "index lists are NULL");
  return plan_common(desc, nullptr, kv_row_ptr, kv_block_indices, ws, ws_bytes, out,
                     static_cast<cudaStream_t>(cuda_stream));
}

extern "C" waveal_status waveal_bitmap_to_csr(int32_t heads, int32_t n_q_blocks, int32_t n_kv_blocks,
                                              const uint64_t* mask_bits, int32_t* kv_row_ptr_out,
                                              int32_t* kv_block_indices_out, int64_t capacity, void* ws,
                                              size_t ws_bytes, void* cuda_stream) {
  if (heads <= 0 || n_q_blocks <= 0 || n_kv_blocks <= 0)
    return waveal::fail(WAVEAL_ERR_INVALID_ARG, "heads, n_q_blocks and n_kv_blocks must be positive");
  if (!mask_bits || !kv_row_ptr_out) return waveal::fail(WAVEAL_ERR_INVALID_ARG, "mask_bits and kv_row_ptr_out are required");
  if (kv_block_indices_out && capacity < 0) return waveal::fail(WAVEAL_ERR_INVALID_ARG, "capacity must be >= 0");
  long long rows = (long long)heads * n_q_blocks;
  if (!ws || ws_bytes < (size_t)(rows + 1) * 4)
    return waveal::fail(WAVEAL_ERR_WORKSPACE, "workspace of %zu bytes needed", (size_t)(rows + 1) * 4);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int wq = (n_kv_blocks + 63) / 64;
  int* cnt = static_cast<int*>(ws);
  int launches = 0;
  k_row_popcount<<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(reinterpret_cast<const u64*>(mask_bits), rows, wq, cnt);
  k_exclusive_scan<<<1, 1024, 0, st>>>(cnt, rows, kv_row_ptr_out);
  launches += 2;
  if (kv_block_indices_out) {
    k_fill_indices<<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(reinterpret_cast<const u64*>(mask_bits), rows, wq,
                                                              kv_row_ptr_out, kv_block_indices_out, capacity);
    ++launches;
  }
  WAVEAL_CUDA_OK(cudaGetLastError());
  waveal::launch_counter() = launches;
  return WAVEAL_OK;
}

// ------------------------------------------------------------------ entry point that allocates nothing

// Scratch for waveal_bitmap_to_csr_noalloc: lives in the library image, so every GPU that
// loads the library holds this 1 MiB until the process exits.
#define WAVEAL_NOALLOC_SCRATCH_BYTES (1u << 20)
static __device__ __align__(256) unsigned char g_noalloc_scratch[WAVEAL_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mu;
void* g_scratch_addr[kMaxDevices] = {};   // device address of g_noalloc_scratch, per device

// In host code the array's name is only a handle; the address a kernel can use has to be
// asked for, once per device, with that device current.
waveal_status noalloc_scratch(void** out) {
  int dev = 0;
  WAVEAL_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return waveal::fail(WAVEAL_ERR_UNSUPPORTED, "device ordinal %d not supported", dev);
  std::lock_guard<std::mutex> lock(g_scratch_mu);
  if (!g_scratch_addr[dev]) {
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
    if (e != cudaSuccess || !ptr)
      return waveal::fail(WAVEAL_ERR_CUDA, "cudaGetSymbolAddress(static scratch) failed: %s", cudaGetErrorString(e));
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return WAVEAL_OK;
}
}  // namespace

extern "C" size_t waveal_noalloc_max_rows(void) { return WAVEAL_NOALLOC_SCRATCH_BYTES / 4 - 1; }

extern "C" waveal_status waveal_bitmap_to_csr_noalloc(int32_t heads, int32_t n_q_blocks, int32_t n_kv_blocks,
                                                      const uint64_t* mask_bits, int32_t* kv_row_ptr_out,
                                                      int32_t* kv_block_indices_out, int64_t capacity,
                                                      void* cuda_stream) {
  if (heads <= 0 || n_q_blocks <= 0 || n_kv_blocks <= 0)
    return waveal::fail(WAVEAL_ERR_INVALID_ARG, "heads, n_q_blocks and n_kv_blocks must be positive");
  const long long rows = (long long)heads * n_q_blocks;
  if ((unsigned long long)rows > (unsigned long long)waveal_noalloc_max_rows())
    return waveal::fail(WAVEAL_ERR_UNSUPPORTED,
                        "heads*n_q_blocks = %lld exceeds the %zu rows the built-in scratch holds; "
                        "use waveal_bitmap_to_csr with a caller-owned workspace",
                        rows, waveal_noalloc_max_rows());
  void* scratch = nullptr;
  waveal_status s = noalloc_scratch(&scratch);
  if (s != WAVEAL_OK) return s;
  // the per-row counts in the scratch are fully rewritten for the rows in use before they are
  // read, so nothing of the previous call's contents has to be cleared
  return waveal_bitmap_to_csr(heads, n_q_blocks, n_kv_blocks, mask_bits, kv_row_ptr_out, kv_block_indices_out,
                              capacity, scratch, WAVEAL_NOALLOC_SCRATCH_BYTES, cuda_stream);
}
