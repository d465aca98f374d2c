/*
 * psattn.h - C ABI of the prob-sparse multi-head self-attention forward library for
 * NVIDIA B200 (sm_100a).
 *
 * The operation is the attention rule of arXiv 2106.09236, Sec. 3 ("Prob-Sparse
 * Self-Attention"), applied independently to every (batch, head) unit:
 *
 *   (a) s_ij = q_i . k_j / sqrt(d) for the U sampled keys j of query i        (Eq. 11)
 *   (b) M~_i = max_j s_ij - (1/U) sum_j s_ij                                   (Eq. 11)
 *   (c) I_sparse = the u queries with the largest M~_i                         (Sec. 3.2)
 *   (d) o_i = sum_j softmax_j(s_ij) v_j over all valid keys, for i in I_sparse (Eq. 7-8, Eq. 12)
 *   (e) o_i = mean_j v_j over valid keys (or v_i, Eq. 12 as printed) otherwise (Sec. 3.1, Eq. 12)
 *
 * with U = u = n(c, len) = clamp(ceil(c ln len), 1, len) per sequence (the sample-size rule of
 * Sec. 3.2 with r_sample = c), natural logarithm, evaluated on the host in double.
 *
 * Conventions common to every call
 *   - All functions return an int status (PSATTN_OK == 0); none throws, aborts or
 *     synchronises the device, except where stated.  All device work is ordered on
 *     the caller's stream (a cudaStream_t passed as void*; NULL = the legacy default stream):
 *     it is enqueued there, except that psattn_forward may run the part of step (e) that does
 *     not depend on steps (a)-(c) on a stream owned by the plan, forked from and joined back
 *     into the caller's stream with events inside the call (which a stream capture follows).
 *     Calls on one plan must therefore be stream-ordered with each other.
 *   - "device" pointers must be device memory of the GPU that was current when the
 *     plan was created; "host" pointers are ordinary host memory.  The caller owns every
 *     buffer.  After psattn_plan_create the library allocates nothing (exception:
 *     psattn_plan_enable_host_io, which allocates staging buffers once).
 *   - Q, K, V, O are [B][H][T_max][d_head] with d_head contiguous; the element strides of
 *     the b, h and t axes are given in the descriptor (all zero = dense row-major).  Base
 *     pointers must be 16-byte aligned and the strides multiples of 8 elements.
 *     Element type: bf16 (PSATTN_BF16) or float (PSATTN_FP32); O has the input type.
 *     Accumulation is always fp32.
 *   - lengths: device int32 [B], valid length of each sequence (key-padding mask), or NULL
 *     (every sequence has length T_max).  Values are clamped to [0, T_max] (status bit 1).
 *     Rows of O at positions >= lengths[b] are written as zeros; Q, K, V there are never read.
 *   - sample_idx: device int32, row (b, i) (or (b, h, i) with idx_per_head) holds the sampled
 *     key positions of query i in its first U_b entries; row stride idx_cols elements.  Entries
 *     must lie in [0, lengths[b]); others are clamped into range and status bit 0 is set.
 *     A key that occurs twice counts twice in the mean of Eq. 11.  With idx_shared the array has
 *     one row per sequence (or per unit) instead of one per query.
 *   - sel_idx: device int32 [B][H][u_max], the selected query positions of each unit in
 *     ascending order, padded with -1.  Equal M~ values are ordered by position (lower first).
 *   - workspace: device scratch of at least psattn_workspace_bytes() bytes, 256-byte aligned.
 *     Its first 256 bytes hold the status word and must be zero before the first call that
 *     uses the buffer (psattn_read_status clears them again); the rest needs no initialisation.
 *     Calls that share a workspace must be stream-ordered.
 */
#ifndef PSATTN_H_
#define PSATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    PSATTN_OK = 0,
    PSATTN_ERR_NULL = 1,                /* a required pointer is NULL */
    PSATTN_ERR_BAD_DESC = 2,            /* a size, stride or enum in the descriptor is invalid */
    PSATTN_ERR_UNSUPPORTED = 3,         /* valid request this build cannot run (e.g. d_head != 64) */
    PSATTN_ERR_WORKSPACE_TOO_SMALL = 4,
    PSATTN_ERR_MISALIGNED = 5,          /* a base pointer is not 16-byte aligned */
    PSATTN_ERR_CUDA = 6,                /* a CUDA runtime call failed; see psattn_last_cuda_error */
    PSATTN_ERR_NO_DEVICE = 7,           /* no usable sm_100 device */
    PSATTN_ERR_TOO_LARGE = 8            /* problem exceeds a fixed built-in capacity */
};

enum { PSATTN_BF16 = 0, PSATTN_FP32 = 1 };
enum { PSATTN_FILL_MEAN_V = 0, PSATTN_FILL_OWN_V = 1 };
enum { PSATTN_PATH_AUTO = 0, PSATTN_PATH_STAGED = 1, PSATTN_PATH_FUSED = 2 };

/* bits of the device status word (psattn_read_status) */
enum {
    PSATTN_STATUS_IDX_CLAMPED = 1u,     /* a sample_idx / row index was out of range and clamped */
    PSATTN_STATUS_LEN_CLAMPED = 2u,     /* a length was outside [0, T_max] and clamped */
    PSATTN_STATUS_WAIT_EXPIRED = 4u     /* a bounded device-side wait gave up; results invalid */
};

typedef struct psattn_desc {
    int32_t B, H, T_max, d_head;        /* d_head must be 64 */
    int32_t dtype;                      /* PSATTN_BF16 | PSATTN_FP32 */
    int32_t fill_mode;                  /* PSATTN_FILL_MEAN_V (default) | PSATTN_FILL_OWN_V */
    int32_t u_override;                 /* > 0: select min(u_override, len) queries instead of n(c, len) */
    int32_t U_override;                 /* > 0: use min(U_override, idx_cols) samples instead of n(c, len) */
    int32_t idx_cols;                   /* row stride (elements) of sample_idx, >= largest U used */
    int32_t idx_per_head;               /* 0: sample_idx is [B][T_max][idx_cols], shared by the heads;
                                           1: [B][H][T_max][idx_cols] */
    int32_t path;                       /* PSATTN_PATH_*: kernel schedule; AUTO picks per shape */
    int32_t idx_shared;                 /* 1: one sample per sequence, used by all its queries (the other
                                           reading of how Sec. 3.2 draws the sampled keys): sample_idx
                                           is [B][idx_cols] (or [B][H][idx_cols] with idx_per_head) */
    double c;                           /* sampling factor of n(c, len) */
    double r_sparse;                    /* 0: u = n(c, len).  In (0, 1]: the count of Sec. 3.2 as the paper states it,
                                           u = clamp(ceil(r_sparse * len), 1, len) from each sequence's own length
                                           (takes precedence over u_override) */
    int64_t q_stride[3], k_stride[3], v_stride[3], o_stride[3];   /* b, h, t strides in elements; all 0 = dense */
} psattn_desc_t;

typedef struct psattn_plan psattn_plan_t;

/* Library version (major * 1000 + minor). */
int psattn_version(void);
/* Static, NUL-terminated description of a status code. */
const char *psattn_status_string(int status);
/* Number of kernels this library has launched in this process so far (all plans, all streams). */
unsigned long long psattn_launch_count(void);
/* cudaError_t of the last failed runtime call seen through this plan (0 if none). */
int psattn_last_cuda_error(const psattn_plan_t *plan);

/* n(c, len) of Sec. 3.2 (host arithmetic in double): the sample size U and the number u of
 * selected queries for a sequence of `len` valid positions.  Returns 0 for len <= 0. */
int psattn_count(double c, int len);

/* Validates the descriptor, builds the per-length tables u[len], U[len] (len = 0..T_max) on
 * the host and uploads them, and records the current device.  *out is NULL on failure. */
int psattn_plan_create(const psattn_desc_t *desc, psattn_plan_t **out);
int psattn_plan_destroy(psattn_plan_t *plan);
/* Test hook for the bounded device-side waits.  Every wait of a kernel on a barrier (a TMA copy, a tensor-core
 * product) gives up after a limit (1 s), sets PSATTN_STATUS_WAIT_EXPIRED and lets the kernel unwind and return.
 * This call shortens the limit (wait_limit_ns, 0 = the default of 1 s, at most 10 s) for the kernels that take it
 * from the plan (the fused forward kernel and the long-row-list / dense attention kernel) and, with
 * extra_expected_bytes > 0, makes the first TMA barrier of those kernels expect that many bytes more than are ever
 * sent, so that the wait really runs out - without any invalid access.  Results of such a call are invalid by
 * design; pass (0, 0) to return to normal operation. */
int psattn_plan_debug_waits(psattn_plan_t *plan, uint64_t wait_limit_ns, uint32_t extra_expected_bytes);

/* Largest u and U over len in [0, T_max]: the widths of sel_idx and the minimum idx_cols. */
int psattn_plan_limits(const psattn_plan_t *plan, int32_t *u_max, int32_t *U_max);
/* Bytes of device workspace every call below needs (the same size for all of them). */
int psattn_workspace_bytes(const psattn_plan_t *plan, size_t *bytes);

/* Steps (a)-(e) (Eq. 11, Sec. 3.2, Eq. 12).  All pointers device.  M_out (fp32
 * [B][H][T_max], zero at padded positions) may be NULL. */
int psattn_forward(psattn_plan_t *plan, const void *Q, const void *K, const void *V,
                   const int32_t *lengths, const int32_t *sample_idx, void *O,
                   int32_t *sel_idx, float *M_out, void *workspace, size_t workspace_bytes,
                   void *stream);

/* Steps (d)-(e) with a given index set (same layout as sel_idx; entries outside
 * [0, lengths[b]) are ignored): the reuse of one layer's selection by the following layers
 * (Sec. 4.4), and the random-selection ablation of Table 1. */
int psattn_forward_with_selection(psattn_plan_t *plan, const void *Q, const void *K,
                                  const void *V, const int32_t *lengths,
                                  const int32_t *sel_idx_in, void *O, void *workspace,
                                  size_t workspace_bytes, void *stream);

/* Steps (a)+(b) only (Eq. 11): M_out fp32 [B][H][T_max], zero at padded positions. */
int psattn_measure(psattn_plan_t *plan, const void *Q, const void *K, const int32_t *lengths,
                   const int32_t *sample_idx, float *M_out, void *workspace,
                   size_t workspace_bytes, void *stream);

/* The exact sparsity measure that Eq. 11 approximates (Eq. 10): M_out[b][h][i] =
 * ln sum_j exp(s_ij) - (1/len) sum_j s_ij over ALL valid keys j < lengths[b]; fp32 [B][H][T_max],
 * zero at padded positions.  A dense pass over the score matrix (cost of dense attention's first
 * half); no sample is involved.  All pointers device. */
int psattn_exact_measure(psattn_plan_t *plan, const void *Q, const void *K, const int32_t *lengths,
                         float *M_out, void *workspace, size_t workspace_bytes, void *stream);

/* The projections that precede the attention (Sec. 3.1: queries, keys and values are the layer input times one matrix each), for all heads
 * at once, written directly in the layout the calls above read.  All pointers device.
 *   X     [B][T_max][d_x], dense, element type of the plan (the layer input; d_x is the model width)
 *   Wt    [3][H * 64][d_x], dense, same type: the matrices stored transposed, role r = 0 (q), 1 (k), 2 (v),
 *         row h * 64 + e of role r = column e of head h's matrix: Wt[r][h*64 + e][x] = W_r^h[x][e]
 *   Q, K, V  outputs of the plan's type with the descriptor's q/k/v strides:
 *         Q[b][h][t][e] = sum_x X[b][t][x] W_q^h[x][e] (fp32 accumulation, rounded to the output type)
 *         for t < lengths[b]; rows at positions >= lengths[b] are NOT written (the attention never reads them)
 *   vbar  optional (may be NULL) fp32 [B][H][64]: mean over t < lengths[b] of V as stored, i.e. the fill
 *         value of step (e), produced while V is written instead of by another pass over it
 * bf16: a tcgen05 GEMM (d_x must be a multiple of 8; otherwise, for fp32, and with PSATTN_PATH_STAGED, a
 * plain fp32-FMA kernel runs).  Base pointers 16-byte aligned.  Uses the workspace (stream-ordered with
 * other calls on it). */
int psattn_project_qkv(psattn_plan_t *plan, const void *X, const void *Wt, int32_t d_x,
                       const int32_t *lengths, void *Q, void *K, void *V, float *vbar,
                       void *workspace, size_t workspace_bytes, void *stream);

/* The output matrix of the attention module, which merges the heads (Sec. 2.2, Eq. 5: the module inside the
 * Conformer block; Sec. 3.1: its heads):  Y[b][t][n] = sum_h sum_e O[b][h][t][e] W_o^h[e][n].  All pointers device.
 *   O        the attention output, plan type, descriptor's o strides (what psattn_forward wrote)
 *   sel_idx  the index sets that psattn_forward wrote for this O ([B][H][u_max], ascending, -1 padded), or NULL
 *   Wot      [d_y][H * 64] dense, plan type: W_o transposed, Wot[n][h * 64 + e] = W_o^h[e][n]
 *   Y        [B][T_max][d_y] dense, plan type; rows at positions >= lengths[b] are NOT written
 * With sel_idx, the mean(V) fill and bf16 (u_max <= 64, H <= 32, d_y a multiple of 8) the call uses the structure
 * Eq. 12 gives O - every valid row of a unit that its index set does not list equals one fill row F_h - and
 * computes Y[b][t][:] = sum_h F_h W_o^h for all positions plus (O[b][h][t][:] - F_h) W_o^h for the listed ones:
 * O(B H u 64 d_y) products instead of O(B T H 64 d_y).  F_h is read from O at the first valid position the set
 * leaves out, so O must really have that structure (rows changed after psattn_forward are not seen).
 * With sel_idx == NULL (any O), the own-value fill, or shapes outside those limits: one dense product (tcgen05 for
 * bf16 with d_y a multiple of 64; one thread per output element for fp32, other d_y, or PSATTN_PATH_STAGED). */
int psattn_project_out(psattn_plan_t *plan, const void *O, const int32_t *sel_idx, const int32_t *lengths,
                       const void *Wot, int32_t d_y, void *Y, void *workspace, size_t workspace_bytes,
                       void *stream);

/* Step (c) only (Sec. 3.2): top-u positions of M (fp32 [B][H][T_max]) among i < lengths[b]. */
int psattn_select(psattn_plan_t *plan, const float *M, const int32_t *lengths,
                  int32_t *sel_idx, void *workspace, size_t workspace_bytes, void *stream);

/* The fill value of step (e): vbar fp32 [B][H][d_head] = mean of V over valid keys (Sec. 3.1). */
int psattn_mean_v(psattn_plan_t *plan, const void *V, const int32_t *lengths, float *vbar,
                  void *workspace, size_t workspace_bytes, void *stream);

/* Step (d) only (Eq. 7-8) for listed rows: row_idx int32 [B][H][n_rows] (entries outside
 * [0, lengths[b]) produce a zero row), out fp32 [B][H][n_rows][d_head]. n_rows <= u_max. */
int psattn_attend_rows(psattn_plan_t *plan, const void *Q, const void *K, const void *V,
                       const int32_t *lengths, const int32_t *row_idx, int32_t n_rows,
                       float *out, void *workspace, size_t workspace_bytes, void *stream);

/* Dense softmax attention (Eq. 6) for every valid query on the same layout: the comparator
 * the sparse path is measured against.  Padded rows of O are zero. */
int psattn_dense_forward(psattn_plan_t *plan, const void *Q, const void *K, const void *V,
                         const int32_t *lengths, void *O, void *workspace,
                         size_t workspace_bytes, void *stream);

/* Copies the device status word of `workspace` to *host_bits and clears it.  Synchronises
 * `stream`. */
int psattn_read_status(psattn_plan_t *plan, void *workspace, void *stream, uint32_t *host_bits);

/* Host-buffer front end.  psattn_plan_enable_host_io allocates, once, device staging for
 * Q, K, V, O, lengths, sample_idx, sel_idx, a workspace, and one internal copy stream with two
 * events, all owned by the plan.
 * psattn_forward_host takes HOST arrays (dense layout, descriptor strides ignored), and returns
 * with O and sel_idx filled in and both streams idle.  Sequences are independent, so the batch
 * goes through in chunks (2 by default; the environment variable PSATTN_HOST_CHUNKS = 1..64
 * overrides it): chunk k is copied in and computed on `stream` while the results of chunk k - 1
 * are copied out on the internal stream.  lengths may be NULL.  Pinned host memory
 * makes the copies asynchronous and lets the two directions overlap; pageable memory works but
 * serialises them. */
int psattn_plan_enable_host_io(psattn_plan_t *plan);
int psattn_forward_host(psattn_plan_t *plan, const void *Q, const void *K, const void *V,
                        const int32_t *lengths, const int32_t *sample_idx, void *O,
                        int32_t *sel_idx, void *stream);

/* Allocation-free variant of psattn_mean_v.  (The paper has no counterpart: this entry point
 * exists for deployment reasons only; it computes the same fill value of step (e).)
 *
 * For callers that cannot allocate device memory where they need the result - code running
 * under a framework that owns all device memory through its own pool, pipelines that forbid
 * allocation after start-up, plug-ins in a process whose memory is already reserved.  It needs
 * no plan and no workspace: its scratch (the column-sum partials) is a fixed array inside the
 * library image, PSATTN_NOALLOC_MAX_PARTIALS * 64 floats (4 MiB) plus 256 bytes, which every
 * GPU that loads the library holds until the process exits.  It calls no cudaMalloc, cudaFree
 * or other allocating routine.
 *
 *   V        device, dense [B][H][T_max][64] of `dtype` (PSATTN_BF16 | PSATTN_FP32), 16-byte aligned
 *   lengths  device int32 [B] or NULL (all T_max); values are clamped to [0, T_max]
 *   vbar     device fp32 [B][H][64]: mean of V over the valid rows (zeros where length is 0)
 *
 * Capacity: B * H * ceil(T_max / 256) <= PSATTN_NOALLOC_MAX_PARTIALS, otherwise
 * PSATTN_ERR_TOO_LARGE is returned and nothing is launched.
 * The first call on each device looks up the array's device address (with that device current);
 * make that first call outside any stream capture.  All calls on a device share the one array:
 * it keeps the previous call's contents (each call rewrites what it reads and clears its status
 * word), and two calls whose kernels may overlap on the GPU (different streams without an
 * ordering between them) race on it - order them. */
#define PSATTN_NOALLOC_MAX_PARTIALS 16384
int psattn_mean_v_noalloc(const void *V, const int32_t *lengths, float *vbar, int32_t B,
                          int32_t H, int32_t T_max, int32_t dtype, void *stream);

/* Microbenchmark of the gather rates that bound steps (a)+(b) (Eq. 11 needs one 128-byte key row per
 * (query, sampled key) pair, at a random position).  Launches ONE kernel on `stream` that gathers
 * n_ctas * warps_per_cta * rounds_per_warp * 16 random rows of 128 bytes and computes nothing; the caller
 * times it (CUDA events) and divides.  No plan, no workspace.
 *   mode 0  rows of a 128 KB chunk resident in shared memory, read with the ldmatrix pattern of the
 *           resident-key measure kernel (`rows`, `n_rows` unused; warps_per_cta <= 32)
 *   mode 1  rows of the device buffer `rows` (n_rows rows of 128 bytes, 16-byte aligned) read from
 *           global memory / L2 into registers, two rounds in flight per warp (warps_per_cta <= 24;
 *           rounds_per_warp is rounded down to a multiple of the rounds in flight)
 *   mode 2  as mode 1 with four rounds in flight per warp
 *   mode 3-5 / 6-8  as mode 0 with the arithmetic of the measure kernel behind the loads (a chain of four
 *           mma.m16n8k16 per round; 1, 2 or 4 rounds interleaved), row numbers from a hash / from a table in shared
 *           memory (one more 4-byte shared-memory load per lane and round, as in the kernel)
 *   mode 9 / 10  rows of the shared memory of the CTAs of a thread-block cluster (distributed shared memory),
 *           read into registers with two / four rounds in flight; n_rows carries the cluster size (1, 2, 4 or 8),
 *           n_ctas is rounded down to a multiple of it
 *   mode 11 as mode 1 through the copy engine: one 128-byte bulk copy per row into a ring in shared memory, two rounds
 *           in flight per warp (rounds_per_warp is rounded down to a multiple of 4)
 *   mode 12 mode 11 and mode 1 in one kernel: every sixth warp uses bulk copies, for half as many rounds; the others
 *           register loads.  It gathers n_ctas * (w - b + b / 2) * rounds * 16 rows, b = the warps among the
 *           warps_per_cta = w whose number is 5 modulo 6.
 *   mode 13 / 14  the inner loop of a chunk-resident form of steps (a)+(b) for long sequences: per work item a 1024-row
 *           chunk of `rows` is copied into shared memory and 2048 queries gather from it the samples that fall into it
 *           (Binomial(46, 1/8) of them per query; a warp's eight queries advance together, two rows per query and
 *           round), their own rows staged through shared memory.  Mode 13: independent counts; mode 14: the counts of
 *           a warp's eight queries are neighbours in the sorted order of a 128-query block.  n_ctas CTAs of 16 warps
 *           (warps_per_cta must be 16), rounds_per_warp = work items per CTA; n_rows >= 4096.  The number of useful
 *           (query, key) pairs is ADDED to the 64-bit counter at sink[2..3] (zero it before the launch; sink 8-byte
 *           aligned).
 * sink: device uint32[4] (sink[0] is written practically never; it keeps the loads alive; sink[1] = 0xdead if a bounded
 * wait of mode 11 / 12 ran out). */
int psattn_probe_gather(int32_t mode, const void *rows, int64_t n_rows, int32_t n_ctas,
                        int32_t warps_per_cta, int32_t rounds_per_warp, uint32_t *sink, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* PSATTN_H_ */
