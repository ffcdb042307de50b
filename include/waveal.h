/* waveal - WaveAlign-scheduled block-sparse attention for NVIDIA B200 (sm_100a).
 *
 * C ABI of the library.  Two groups of calls:
 *   planning   waveal_plan_bitmap / waveal_plan_csr : block mask -> per-head execution order
 *              of the query blocks (Algorithm 2 of the WaveAlign paper, with the adaptive
 *              skip of Section 4.5 in front);
 *   attention  waveal_bsattn_fwd : block-sparse FlashAttention-style forward (Sections
 *              2.2-2.3) whose persistent CTAs walk that order head by head.
 *
 * Conventions for every call
 *   - "dev" pointers are device pointers on the current CUDA device, "host" pointers are
 *     host pointers.  The caller owns every buffer and the stream.
 *   - The library allocates no device memory, never frees and never synchronises (unless a
 *     call's comment says otherwise); all work is enqueued on `cuda_stream` (a cudaStream_t
 *     passed as void*, NULL = the default stream).
 *   - A problem the host can detect returns a non-zero status BEFORE anything is enqueued
 *     and leaves the outputs untouched; waveal_last_error() then describes it.
 *   - Problems only the device can detect (a bounded wait that ran out, an index out of
 *     range) are written to the `dev_status` words; the kernel leaves cleanly, nothing traps.
 *   - heads = batch * heads flattened; every head has its own mask (Algorithm 2 input
 *     M in {0,1}^{H x M_B x N_B}).
 *   - Mask bitmap: row-major uint64 [heads][n_q_blocks][ceil(n_kv_blocks/64)]; bit (j & 63)
 *     of word (j >> 6) of row i is M[i][j]; padding bits must be zero.
 *   - Index lists (CSR over the flattened (head, query block) axis): kv_row_ptr int32
 *     [heads*n_q_blocks + 1], kv_block_indices int32 [nnz], ascending and unique inside a row.
 *   - Execution order: row_order int32 [heads][n_q_blocks]; row_order[h][p] is the query
 *     block executed at position p of head h (the index-list form of P_h in Algorithm 2).
 *
 * Shape of the interface (choices of this library, fixed here so that callers need not guess)
 *   - batch is flattened into `heads`, so strides have two entries {head, token};
 *   - bf16 is the only element type, so there is no dtype field;
 *   - a plan call's outputs are grouped in one struct, waveal_plan_out: one required, the rest optional;
 *   - workspace sizes depend on the descriptor alone, never on the number of selected blocks;
 *   - dev_status has four int32 words {code, site, head or block, value};
 *   - a workspace is state of the call that uses it: two calls that may overlap on the GPU
 *     (different streams or host threads) need a workspace each.
 */
#ifndef WAVEAL_H_
#define WAVEAL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  WAVEAL_OK = 0,
  WAVEAL_ERR_INVALID_ARG = 1,   /* NULL pointer, non-positive size, misaligned pointer/stride */
  WAVEAL_ERR_UNSUPPORTED = 2,   /* head_dim / block size / dtype / device not supported      */
  WAVEAL_ERR_WORKSPACE = 3,     /* workspace missing or too small                             */
  WAVEAL_ERR_BAD_MASK = 4,      /* device-side: index out of range / unsorted                 */
  WAVEAL_ERR_CUDA = 5,          /* a CUDA runtime/driver call failed                          */
  WAVEAL_ERR_TIMEOUT = 6        /* device-side: a bounded wait ran out                        */
} waveal_status;

/* Which stages run (Section 6.5 ablation: Original, O+S1, O+S2, O+S1+S2). */
typedef enum {
  WAVEAL_AUTO = 0,           /* guard decides per head; a skipped head keeps natural order */
  WAVEAL_FORCE_REORDER = 1,  /* Stage 1 + Stage 2 on every head                            */
  WAVEAL_FORCE_NATURAL = 2,  /* identity order on every head                               */
  WAVEAL_STAGE1_ONLY = 3,    /* angular order only                                         */
  WAVEAL_STAGE2_ONLY = 4     /* natural order cut into waves, each sorted by block count   */
} waveal_mode;

/* Optional bit, OR-ed into waveal_plan_desc.mode: open the ring of angularly sorted rows at the
 * largest gap between neighbouring angles instead of at -pi, where Eq. 4's atan2 puts the cut
 * (Section 4.3.1 calls the sorted rows a ring but does not say where it is opened).  A variant
 * for experiments, off by default: it makes Stage 1 invariant under rotations of the embedding
 * and keeps a tight group of rows that straddles +-pi in one piece. */
#define WAVEAL_RING_CUT_LARGEST_GAP 16

/* skip_flags bits */
#define WAVEAL_FLAG_SKIPPED 1u        /* this head's row_order is the identity (skip applied) */
#define WAVEAL_FLAG_SHORT_SEQ 2u      /* one head's K+V fit the L2 budget (Section 4.5, case 1) */
#define WAVEAL_FLAG_TOO_SPARSE 4u     /* too little work to amortise reordering (case 2)        */
#define WAVEAL_FLAG_ALREADY_LOCAL 8u  /* natural-order waves already overlap (case 3)           */

typedef struct waveal_plan_desc {
  int32_t heads;          /* batch*heads                                                      */
  int32_t n_q_blocks;     /* M_B (Section 4.2)                                                */
  int32_t n_kv_blocks;    /* N_B                                                              */
  int32_t wave_size;      /* W = SMs x resident CTAs (Section 6.1); 0 = this device's SM count */
  int32_t svd_iters;      /* T of Algorithm 1 (paper: 5-15; library default 5)                */
  int32_t mode;           /* waveal_mode, optionally | WAVEAL_RING_CUT_LARGEST_GAP            */
  uint64_t seed;          /* seed of the start block of Algorithm 1                           */
  /* guard thresholds, all integer comparisons (the "offline profile" of Section 4.5):       */
  int64_t kv_bytes_per_head; /* bytes of K plus V of one head; 0 disables the short-seq test */
  int64_t l2_bytes;          /* cache size the test compares with; 0 = query the device      */
  int32_t l2_fit_num, l2_fit_den;  /* short-seq: kv_bytes*den <= l2_bytes*num                */
  int32_t min_density_ppm;         /* too-sparse: nnz*1e6 < ppm*M_B*N_B ...                  */
  int32_t local_num, local_den;    /* already-local: 2*ov_nat*den >= num*pair2               */
  int64_t min_nnz;                 /* ... or nnz < min_nnz (per head)                        */
} waveal_plan_desc;

/* Optional and required outputs of a plan call (all dev pointers; NULL = not wanted,
 * except row_order). */
typedef struct waveal_plan_out {
  int32_t* row_order;   /* [heads][M_B]  required                                            */
  int32_t* row_nnz;     /* [heads][M_B]  n_i = sum_j M_ij (Section 2.2)                      */
  uint8_t* skip_flags;  /* [heads]       WAVEAL_FLAG_* bits                                  */
  int32_t* col_count;   /* [heads][N_B]  c = M^T 1 (Algorithm 1)                             */
  int32_t* order1;      /* [heads][M_B]  Stage-1 order before the per-wave sort              */
  double* embedding;    /* [heads][M_B][2]  u_1, u_2 of Algorithm 1 (zeros for skipped heads) */
  int64_t* stats;       /* [heads][4]    nnz, ov_nat, pair2, 0 (guard statistics)            */
  int32_t* dev_status;  /* [4] {code, site, head, aux}; written only on a device-side failure
                           (an index list entry out of range); the caller zeroes it          */
} waveal_plan_out;

/* Fills `desc` with the library defaults (T = 5, AUTO, guard: K+V of a head within 9/16 of
 * L2, density below 1 %, natural-order locality of at least 1/2);
 * heads / block counts stay 0 for the caller to set.  Host-only, no CUDA call. */
void waveal_plan_desc_default(waveal_plan_desc* desc /*host*/);

/* Bytes of device workspace a plan call needs (the same for the bitmap and CSR entry).
 * Host-only. */
waveal_status waveal_plan_workspace_bytes(const waveal_plan_desc* desc /*host*/, size_t* bytes /*host*/);

/* Algorithm 2 from a bitmap mask.  Steps, all on the device: row block counts and column
 * counts (Algorithm 1 step 1, Algorithm 2 Stage 2), guard statistics and decision
 * (Section 4.5), T centred subspace iterations + Rayleigh-Ritz ordering (Algorithm 1),
 * polar angle (Eq. 4), angular sort, wave-sized buckets, descending-count sort per bucket.
 * ws: dev workspace of at least waveal_plan_workspace_bytes bytes, 256-byte aligned.
 * No host synchronisation: the skip decision is consumed on the device. */
waveal_status waveal_plan_bitmap(const waveal_plan_desc* desc /*host*/, const uint64_t* mask_bits /*dev*/,
                                 void* ws /*dev*/, size_t ws_bytes, const waveal_plan_out* out /*host struct of dev ptrs*/,
                                 void* cuda_stream);

/* Same from index lists; the bitmap is built in the workspace first. */
waveal_status waveal_plan_csr(const waveal_plan_desc* desc /*host*/, const int32_t* kv_row_ptr /*dev*/,
                              const int32_t* kv_block_indices /*dev*/, void* ws /*dev*/, size_t ws_bytes,
                              const waveal_plan_out* out, void* cuda_stream);

/* Bitmap -> index lists, so that the attention kernel has one input format.
 * kv_row_ptr_out: dev int32 [heads*n_q_blocks + 1] (always written).
 * kv_block_indices_out: dev int32 [capacity] or NULL to compute only the row pointers;
 * entries beyond `capacity` are not written (the caller sizes it from kv_row_ptr_out's last
 * entry or from an upper bound).  ws: dev scratch of at least
 * (heads*n_q_blocks + 1) * 4 bytes. */
waveal_status waveal_bitmap_to_csr(int32_t heads, int32_t n_q_blocks, int32_t n_kv_blocks,
                                   const uint64_t* mask_bits /*dev*/, int32_t* kv_row_ptr_out /*dev*/,
                                   int32_t* kv_block_indices_out /*dev or NULL*/, int64_t capacity,
                                   void* ws /*dev*/, size_t ws_bytes, void* cuda_stream);

/* Same conversion for callers that have no way to provide a workspace: a plug-in that sits
 * inside a serving engine between mask construction and the attention backend is handed
 * tensors, not an allocator; the engine has planned all device memory up front, and a
 * cudaMalloc / cudaFree in the middle of a denoising loop would stall every stream of the
 * device.  This entry point therefore calls no allocation routine of CUDA or of any library:
 * its scratch (the per-row counts) is a 1 MiB array built into the library image, which every
 * GPU that loads the library holds until the process exits.
 * (The paper has no counterpart of this call; it is a convenience of this library.)
 *   - limit: heads * n_q_blocks <= waveal_noalloc_max_rows() (262,143); larger problems are
 *     refused with WAVEAL_ERR_UNSUPPORTED before anything is enqueued;
 *   - the first call on each device looks up the array's device address (with that device
 *     current); make that first call before any stream capture begins;
 *   - all calls share the one array: two calls whose kernels overlap on the GPU (different
 *     streams, or different host threads) race and corrupt each other's row pointers; calls
 *     enqueued on one stream are safe.  Nothing in the array has to be cleared between calls.
 * Inputs and outputs are as for waveal_bitmap_to_csr and stay caller-owned. */
waveal_status waveal_bitmap_to_csr_noalloc(int32_t heads, int32_t n_q_blocks, int32_t n_kv_blocks,
                                           const uint64_t* mask_bits /*dev*/, int32_t* kv_row_ptr_out /*dev*/,
                                           int32_t* kv_block_indices_out /*dev or NULL*/, int64_t capacity,
                                           void* cuda_stream);
/* Largest heads * n_q_blocks the call above accepts.  Host-only. */
size_t waveal_noalloc_max_rows(void);

/* waveal_attn_desc.flags: take the row max of every KV block (the online-softmax rule as the
 * paper's backends apply it) in a single launch.  Without the flag the kernel fixes each row's
 * reference after the first two blocks of a task - softmax does not depend on the reference as
 * long as nothing overflows - watches the size of every block's sum, lists the tasks where a
 * sum reached 2^24 and computes those again, with the max of every block, in a second launch
 * on the same stream.  Results agree to rounding; the flag exists for comparison runs. */
#define WAVEAL_ATTN_ONLINE_MAX_ONLY 1
/* Self-test of the kernel's failure handling, never set in production: the loader leaves out
 * the first K tile of the first task and every bounded wait gives up after about 2 ms instead
 * of 2 s.  The call must come back with dev_status = {WAVEAL_ERR_TIMEOUT, site, ...} - the
 * site is the first of the waits behind that tile to run out: 12 (the Q K^T issuer waiting for
 * the tile), 3 or 4 (the K or the V loader waiting for a ring slot), 14 or 21 (the P V issuer and
 * the softmax warps waiting for what the product would have fed them) - with all thread blocks leaving
 * through the common exit (no trap, no fault, the context stays usable); O is then undefined.
 * The next call on the same workspace works as usual. */
#define WAVEAL_ATTN_SELFTEST_LOST_TILE 256
/* 64-row query blocks run in a 128-row tensor-core tile.  By default two query blocks of a head
 * with the very same list of KV blocks share one tile, which halves their cost: rows that select
 * every KV block pair up wherever they stand in the execution order (1st with 2nd, 3rd with 4th
 * such row; the pair runs at the position of its first row), other rows when they stand at
 * positions 2i and 2i+1 (Stage 2 of the plan puts rows of equal count side by side).  The results
 * are the same bits as without sharing (the two blocks never interact: a row of the tile only
 * sees its own row of Q).  This flag switches the sharing off (comparison runs). */
#define WAVEAL_ATTN_NO_ROW_PAIRING 2

typedef struct waveal_attn_desc {
  int32_t heads;            /* batch*heads; K/V heads == Q heads                              */
  int32_t seq_q, seq_kv;    /* true (unpadded) lengths                                        */
  int32_t head_dim;         /* 64 or 128                                                      */
  int32_t block_q, block_kv;/* 64 or 128, equal; the mask's block size (Section 2.2)          */
  int64_t q_stride[2], k_stride[2], v_stride[2], o_stride[2]; /* elements: {head, token}; head_dim contiguous */
  int32_t order_heads_interleaved; /* 0 = heads run one after another (Section 5, sequential
                                      heads); 1 = position-major across heads (parallel heads) */
  int32_t flags;            /* 0, or WAVEAL_ATTN_* bits                                        */
} waveal_attn_desc;

/* Bytes of device workspace waveal_bsattn_fwd needs: 32 bytes of counters (int32 words: ticket
 * counter, abort flag, number of tasks computed twice, ticket counter of the second launch,
 * length of the first and of the second launch in SM cycles = the largest lifetime of a thread
 * block, number of query-block pairs that shared a tile, number of 128-row x 128-key tiles the call runs),
 * 8 bytes per (head, query block) for the list of tasks to compute again and
 * 32 bytes per (head, query block) for the table that maps a ticket to its task.  The counters
 * are live state of the call (tickets are drawn from them): calls that may overlap on the GPU
 * must not share a workspace.  Host-only. */
waveal_status waveal_bsattn_workspace_bytes(const waveal_attn_desc* desc /*host*/, size_t* bytes /*host*/);

/* Block-sparse attention forward, bf16 in / fp32 accumulate / bf16 out (Sections 2.1-2.3):
 * for query block i of head h, O = softmax(scale * Q_i K_sel^T) V_sel over the tokens of
 * the K/V blocks listed for (h, i), visited in the listed (ascending) order.
 * Persistent CTAs take (head, position) tickets in head-major order and process query
 * block row_order[h][position] (Algorithm 2 output; NULL = natural order); each output
 * tile is written at its original rows, so no inverse permutation pass exists.
 * Q, K, V, O: dev bf16, 16-byte aligned, strides multiples of 8 elements, head_dim
 * contiguous; query tokens >= seq_q are not written; keys >= seq_kv are ignored.
 * lse: dev float [heads][seq_q] or NULL (natural-log sum-exp per query token; -inf for a
 * query block with an empty list, whose O is 0).
 * scale <= 0 means 1/sqrt(head_dim).
 * ws: dev workspace (waveal_bsattn_workspace_bytes), 16-byte aligned, not shared with a call
 * that may run at the same time; after the call its int32 word 2 holds the number of tasks the
 * second launch computed again (normally 0) and word 4 the launch's length in SM cycles.
 * dev_status: dev int32 [4] or NULL, zeroed by the caller; written only on a device-side
 * failure: {WAVEAL_ERR_TIMEOUT, site of the wait, thread block, thread} when a bounded wait ran
 * out, {WAVEAL_ERR_BAD_MASK, site, head, value} for an entry of row_order outside [0, M_B)
 * (site 31), a row-pointer pair that is negative, decreasing or beyond kv_row_ptr's last
 * entry (32), or an index outside [0, N_B) (33: last of a list, 30: any other, met while
 * loading).  A task with a bad row pointer or last index gets an empty list (its rows of O
 * become 0); a bad index inside a list is replaced by block 0; the kernel never reads out of
 * range.  row_order is not checked for being a permutation: a query block named twice is
 * computed twice, one never named keeps its old contents.
 * The first call in a process also looks up a driver entry point (no allocation). */
waveal_status waveal_bsattn_fwd(const waveal_attn_desc* desc /*host*/, const void* Q, const void* K, const void* V,
                                void* O, float* lse, const int32_t* kv_row_ptr /*dev*/,
                                const int32_t* kv_block_indices /*dev*/, const int32_t* row_order /*dev or NULL*/,
                                float scale, void* ws /*dev*/, size_t ws_bytes, int32_t* dev_status /*dev or NULL*/,
                                void* cuda_stream);

/* The two reorder operators of the paper's deployment (Section 5), for driving a backend
 * that cannot follow an index list: gather moves block row_order[h][p] of `src` to position p
 * of `dst` (query blocks, or mask rows with block = 1 and row_bytes = bytes of a bitmap row
 * padded to 16); scatter is the inverse (output block at position p goes back to block
 * row_order[h][p]).  Tensors are [heads][n_blocks*block rows][row_bytes] with byte strides
 * {head, row} (multiples of 16); src and dst must not overlap.  Pure copies: out-of-range
 * entries of row_order move nothing.  waveal_bsattn_fwd itself needs neither pass. */
waveal_status waveal_gather_rows(int32_t heads, int32_t n_blocks, int32_t block, int32_t row_bytes,
                                 const void* src /*dev*/, const int64_t* src_stride_bytes /*host [2]*/,
                                 void* dst /*dev*/, const int64_t* dst_stride_bytes /*host [2]*/,
                                 const int32_t* row_order /*dev [heads][n_blocks]*/, void* cuda_stream);
waveal_status waveal_scatter_rows(int32_t heads, int32_t n_blocks, int32_t block, int32_t row_bytes,
                                  const void* src /*dev*/, const int64_t* src_stride_bytes /*host [2]*/,
                                  void* dst /*dev*/, const int64_t* dst_stride_bytes /*host [2]*/,
                                  const int32_t* row_order /*dev [heads][n_blocks]*/, void* cuda_stream);

/* Number of query-block tasks the attention kernel keeps in flight on the current device
 * (SM count x CTAs per SM): the W to plan with (Section 6.1).  Returns <= 0 on failure. */
int32_t waveal_default_wave_size(void);

/* Number of kernel launches the last successful call on this thread enqueued. */
int32_t waveal_last_launch_count(void);

const char* waveal_status_string(waveal_status s);
/* Thread-local description of the last failure on this thread ("" if none). */
const char* waveal_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* WAVEAL_H_ */
