// C ABI of the library (see include/psattn.h): plan, validation, workspace layout and the
// kernel schedules.  No kernel lives here.
#include "../../include/psattn.h"

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "psattn_launch.h"

using namespace psattn;

struct psattn_plan {
    psattn_desc_t desc;
    int device;
    int u_max, U_max;
    int n_chunks;                 // column-sum partials per unit
    int n_splits;                 // key splits of the SIMT attention kernel
    int *d_tables;                // device: u_tab[T+1] then U_tab[T+1]
    int last_cuda_error;
    // workspace layout (byte offsets)
    size_t off_status, off_M, off_vpart, off_vbar, off_ml, off_acc, off_sel, off_pvsum, off_cand, ws_bytes;
    // host-io staging (psattn_plan_enable_host_io)
    bool host_io;
    void *h_Q, *h_K, *h_V, *h_O, *h_ws;
    int *h_len, *h_idx, *h_sel;
    cudaStream_t h_copy_stream;   // device-to-host copies of finished chunks run here
    cudaEvent_t h_ev[2];          // [0]: a chunk is finished; [1]: its results have been copied out
    int b_override;               // > 0: number of sequences of the current (chunked) call
    // side stream of the staged schedule: the fill of step (e) runs there while steps (a)-(c) run on the caller's
    cudaStream_t side_stream;
    cudaEvent_t side_ev[2];       // [0]: fork (recorded on the caller's stream), [1]: join (recorded on the side stream)
    unsigned long long wait_ns;   // limit of the bounded device-side waits (psattn_plan_debug_waits)
    unsigned debug_extra_tx;
};

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Named ranges around the compute entry points for timeline tools, compiled in only with -DPSATTN_NVTX (a separate
// build of the library; the regular one contains no call into the tools interface).
#ifdef PSATTN_NVTX
#include <nvtx3/nvToolsExt.h>
struct ApiRange {
    explicit ApiRange(const char *name) { nvtxRangePushA(name); }
    ~ApiRange() { nvtxRangePop(); }
};
#else
struct ApiRange {
    explicit ApiRange(const char *) {}
};
#endif
#define PSATTN_RANGE() ApiRange api_range_(__func__)

extern "C" int psattn_version(void) { return 1000; }

extern "C" const char *psattn_status_string(int s) {
    switch (s) {
        case PSATTN_OK: return "ok";
        case PSATTN_ERR_NULL: return "a required pointer is NULL";
        case PSATTN_ERR_BAD_DESC: return "invalid descriptor or argument";
        case PSATTN_ERR_UNSUPPORTED: return "unsupported configuration";
        case PSATTN_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case PSATTN_ERR_MISALIGNED: return "pointer not 16-byte aligned (workspace: 256-byte)";
        case PSATTN_ERR_CUDA: return "CUDA runtime error";
        case PSATTN_ERR_NO_DEVICE: return "no usable CUDA device";
        case PSATTN_ERR_TOO_LARGE: return "problem exceeds a fixed built-in capacity";
        default: return "unknown status";
    }
}

extern "C" unsigned long long psattn_launch_count(void) { return launches_so_far(); }

extern "C" int psattn_last_cuda_error(const psattn_plan_t *p) { return p ? p->last_cuda_error : 0; }

extern "C" int psattn_count(double c, int len) {
    if (len <= 0) return 0;
    double x = std::ceil(c * std::log((double)len));
    if (!(x >= 1.0)) x = 1.0;
    if (x > (double)len) x = (double)len;
    return (int)x;
}

static int cuda_fail(psattn_plan_t *p, cudaError_t e) {
    if (p) p->last_cuda_error = (int)e;
    return PSATTN_ERR_CUDA;
}

static bool strides_zero(const int64_t s[3]) { return s[0] == 0 && s[1] == 0 && s[2] == 0; }

static int check_strides(int64_t s[3], const psattn_desc_t &d) {
    if (strides_zero(s)) {
        s[2] = d.d_head;
        s[1] = (int64_t)d.T_max * d.d_head;
        s[0] = (int64_t)d.H * d.T_max * d.d_head;
        return PSATTN_OK;
    }
    for (int k = 0; k < 3; ++k)
        if (s[k] < 0 || (s[k] % 8) != 0) return PSATTN_ERR_BAD_DESC;
    if (s[2] < d.d_head) return PSATTN_ERR_BAD_DESC;
    return PSATTN_OK;
}

extern "C" int psattn_plan_create(const psattn_desc_t *desc, psattn_plan_t **out) {
    if (out) *out = nullptr;
    if (!desc || !out) return PSATTN_ERR_NULL;
    psattn_desc_t d = *desc;
    if (d.B < 0 || d.H < 1 || d.T_max < 1 || d.B > (1 << 20) || d.H > 4096 || d.T_max > (1 << 20))
        return PSATTN_ERR_BAD_DESC;
    if ((long long)d.B * d.H > (1ll << 24)) return PSATTN_ERR_BAD_DESC;
    if (d.dtype != PSATTN_BF16 && d.dtype != PSATTN_FP32) return PSATTN_ERR_BAD_DESC;
    if (d.fill_mode != PSATTN_FILL_MEAN_V && d.fill_mode != PSATTN_FILL_OWN_V) return PSATTN_ERR_BAD_DESC;
    if (d.path < PSATTN_PATH_AUTO || d.path > PSATTN_PATH_FUSED) return PSATTN_ERR_BAD_DESC;
    if (d.u_override < 0 || d.U_override < 0 || d.idx_cols < 1) return PSATTN_ERR_BAD_DESC;
    if (d.idx_shared != 0 && d.idx_shared != 1) return PSATTN_ERR_BAD_DESC;
    if (!(d.c > 0.0) || !std::isfinite(d.c)) return PSATTN_ERR_BAD_DESC;
    if (!(d.r_sparse >= 0.0) || d.r_sparse > 1.0) return PSATTN_ERR_BAD_DESC;
    if (d.d_head != kD) return PSATTN_ERR_UNSUPPORTED;
    int rc;
    if ((rc = check_strides(d.q_stride, d)) || (rc = check_strides(d.k_stride, d)) ||
        (rc = check_strides(d.v_stride, d)) || (rc = check_strides(d.o_stride, d)))
        return rc;

    // per-length tables of Sec. 3.2's counts, in double on the host
    std::vector<int> tab(2 * (size_t)(d.T_max + 1));
    int u_max = 0, U_max = 0;
    for (int len = 0; len <= d.T_max; ++len) {
        int n = psattn_count(d.c, len);
        int u = d.u_override > 0 ? (d.u_override < len ? d.u_override : len) : n;
        if (d.r_sparse > 0.0 && len > 0) {      // Sec. 3.2: L_sparse = r_sparse L, from the sequence's own length
            double x = std::ceil(d.r_sparse * (double)len);
            if (x < 1.0) x = 1.0;
            if (x > (double)len) x = (double)len;
            u = (int)x;
        }
        int U = d.U_override > 0 ? (len > 0 ? d.U_override : 0) : n;
        if (U > d.idx_cols) {
            if (d.U_override > 0) U = d.idx_cols;
            else return PSATTN_ERR_BAD_DESC;        // idx_cols narrower than the rule's U
        }
        tab[len] = u;
        tab[d.T_max + 1 + len] = U;
        if (u > u_max) u_max = u;
        if (U > U_max) U_max = U;
    }
    if (u_max < 1) u_max = 1;

    int dev = 0, ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) { cudaGetLastError(); return PSATTN_ERR_NO_DEVICE; }
    if (cudaGetDevice(&dev) != cudaSuccess) return PSATTN_ERR_NO_DEVICE;
    int major = 0;
    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (major != 10) return PSATTN_ERR_NO_DEVICE;

    psattn_plan_t *p = new (std::nothrow) psattn_plan_t();
    if (!p) return PSATTN_ERR_CUDA;
    std::memset(p, 0, sizeof(*p));
    p->desc = d;
    p->device = dev;
    p->u_max = u_max;
    p->U_max = U_max;
    p->wait_ns = 1000ull * 1000ull * 1000ull;
    p->debug_extra_tx = 0u;
    p->n_chunks = (d.T_max + kColsumRows - 1) / kColsumRows;
    p->n_splits = (d.T_max + kSplitKeys - 1) / kSplitKeys;       // what the partial buffers are sized for
    {
        const int tiles = (d.T_max + 127) / 128;
        const int tc_splits = tiles < 8 ? tiles : 8;
        if (tc_splits > p->n_splits) p->n_splits = tc_splits;
    }
    cudaError_t e = cudaMalloc((void **)&p->d_tables, tab.size() * sizeof(int));
    if (e != cudaSuccess) { delete p; return PSATTN_ERR_CUDA; }
    e = cudaMemcpy(p->d_tables, tab.data(), tab.size() * sizeof(int), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) { cudaFree(p->d_tables); delete p; return PSATTN_ERR_CUDA; }

    const size_t units = (size_t)d.B * d.H;
    size_t off = 0;
    p->off_status = off; off = align_up(off + 256, 256);
    p->off_M = off;      off = align_up(off + units * d.T_max * sizeof(float), 256);
    p->off_vpart = off;  off = align_up(off + units * p->n_chunks * kD * sizeof(float), 256);
    p->off_vbar = off;   off = align_up(off + units * kD * sizeof(float), 256);
    // split partials: u_max row slots per unit plus one for the all-ones row that yields mean(V)
    p->off_ml = off;     off = align_up(off + units * (u_max + 1) * p->n_splits * 2 * sizeof(float), 256);
    p->off_acc = off;    off = align_up(off + units * (u_max + 1) * p->n_splits * kD * sizeof(float), 256);
    p->off_sel = off;    off = align_up(off + units * u_max * sizeof(int), 256);
    // per-tile column sums of V written by the projection kernel
    p->off_pvsum = off;  off = align_up(off + project_vpart_floats(d.B, d.H, d.T_max) * sizeof(float), 256);
    // candidates of the two-kernel selection
    p->off_cand = off;   off = align_up(off + select_cand_ints((int)units, u_max) * sizeof(int), 256);
    p->ws_bytes = off;
    if (cudaStreamCreateWithFlags(&p->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&p->side_ev[0], cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&p->side_ev[1], cudaEventDisableTiming) != cudaSuccess) {
        if (p->side_ev[0]) cudaEventDestroy(p->side_ev[0]);
        if (p->side_stream) cudaStreamDestroy(p->side_stream);
        cudaFree(p->d_tables);
        delete p;
        return PSATTN_ERR_CUDA;
    }
    *out = p;
    return PSATTN_OK;
}

extern "C" int psattn_plan_destroy(psattn_plan_t *p) {
    if (!p) return PSATTN_ERR_NULL;
    cudaFree(p->d_tables);
    cudaStreamDestroy(p->side_stream); cudaEventDestroy(p->side_ev[0]); cudaEventDestroy(p->side_ev[1]);
    if (p->host_io) {
        cudaFree(p->h_Q); cudaFree(p->h_K); cudaFree(p->h_V); cudaFree(p->h_O); cudaFree(p->h_ws);
        cudaFree(p->h_len); cudaFree(p->h_idx); cudaFree(p->h_sel);
        cudaStreamDestroy(p->h_copy_stream); cudaEventDestroy(p->h_ev[0]); cudaEventDestroy(p->h_ev[1]);
    }
    delete p;
    return PSATTN_OK;
}

extern "C" int psattn_plan_debug_waits(psattn_plan_t *p, uint64_t wait_limit_ns, uint32_t extra_expected_bytes) {
    if (!p) return PSATTN_ERR_NULL;
    if (wait_limit_ns > 10ull * 1000ull * 1000ull * 1000ull) return PSATTN_ERR_BAD_DESC;
    p->wait_ns = wait_limit_ns ? wait_limit_ns : 1000ull * 1000ull * 1000ull;
    p->debug_extra_tx = extra_expected_bytes;
    return PSATTN_OK;
}

extern "C" int psattn_plan_limits(const psattn_plan_t *p, int32_t *u_max, int32_t *U_max) {
    if (!p) return PSATTN_ERR_NULL;
    if (u_max) *u_max = p->u_max;
    if (U_max) *U_max = p->U_max;
    return PSATTN_OK;
}

extern "C" int psattn_workspace_bytes(const psattn_plan_t *p, size_t *bytes) {
    if (!p || !bytes) return PSATTN_ERR_NULL;
    *bytes = p->ws_bytes;
    return PSATTN_OK;
}

// ---- helpers ---------------------------------------------------------------------------
static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// A plan belongs to the device that was current when it was created: its tables, its streams and the
// kernels' shared-memory grants live there.
static int check_device(const psattn_plan_t *p) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return PSATTN_ERR_NO_DEVICE; }
    return dev == p->device ? PSATTN_OK : PSATTN_ERR_BAD_DESC;
}

static int check_ws(const psattn_plan_t *p, const void *ws, size_t bytes) {
    if (int rc = check_device(p)) return rc;
    if (!ws) return PSATTN_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return PSATTN_ERR_MISALIGNED;
    if (bytes < p->ws_bytes) return PSATTN_ERR_WORKSPACE_TOO_SMALL;
    return PSATTN_OK;
}

static int plan_b(const psattn_plan_t *p) { return p->b_override > 0 ? p->b_override : p->desc.B; }

static Geom make_geom(const psattn_plan_t *p, const int32_t *lengths, void *ws) {
    Geom g;
    const psattn_desc_t &d = p->desc;
    g.B = plan_b(p); g.H = d.H; g.T = d.T_max;
    g.idx_cols = d.idx_cols; g.idx_per_head = d.idx_per_head; g.idx_shared = d.idx_shared;
    g.u_max = p->u_max;
    for (int k = 0; k < 3; ++k) {
        g.qs[k] = d.q_stride[k]; g.ks[k] = d.k_stride[k];
        g.vs[k] = d.v_stride[k]; g.os[k] = d.o_stride[k];
    }
    g.lengths = lengths;
    g.u_tab = p->d_tables;
    g.U_tab = p->d_tables + d.T_max + 1;
    g.status = reinterpret_cast<unsigned *>(static_cast<char *>(ws) + p->off_status);
    g.wait_ns = p->wait_ns;
    g.debug_extra_tx = p->debug_extra_tx;
    return g;
}

template <typename T>
static T *ws_at(void *ws, size_t off) { return reinterpret_cast<T *>(static_cast<char *>(ws) + off); }

#define PSATTN_CU(expr)                                         \
    do {                                                        \
        cudaError_t e__ = (expr);                               \
        if (e__ != cudaSuccess) return cuda_fail(plan, e__);    \
    } while (0)

// Steps (a)+(b): resident-key kernel for bf16 inputs when it applies, gather-from-L2 kernel otherwise.
static int run_measure(psattn_plan_t *plan, const Geom &g, const void *Q, const void *K,
                       const int *sample_idx, float *M, cudaStream_t st) {
    const psattn_desc_t &d = plan->desc;
    if (d.idx_shared) {
        // one sample per sequence: the scores of a tile of queries are one dense product on tcgen05
        if (d.dtype == PSATTN_BF16 && d.path != PSATTN_PATH_STAGED) {
            cudaError_t e = launch_measure_shared(g, plan->U_max, Q, K, sample_idx, M, st);
            if (e == cudaSuccess) return PSATTN_OK;
            if (e != cudaErrorNotSupported) return cuda_fail(plan, e);
        }
        PSATTN_CU(launch_measure(d.dtype, g, Q, K, sample_idx, M, st));
        return PSATTN_OK;
    }
    if (d.dtype == PSATTN_BF16 && d.path != PSATTN_PATH_STAGED) {
        cudaError_t e = launch_measure_mma(g, plan->U_max, Q, K, sample_idx, M, st);
        if (e == cudaSuccess) return PSATTN_OK;
        if (e != cudaErrorNotSupported) return cuda_fail(plan, e);
        e = launch_measure_stream(g, plan->U_max, Q, K, sample_idx, M, st);
        if (e == cudaSuccess) return PSATTN_OK;
        if (e != cudaErrorNotSupported) return cuda_fail(plan, e);
    }
    PSATTN_CU(launch_measure(d.dtype, g, Q, K, sample_idx, M, st));
    return PSATTN_OK;
}

// Step (d) for a row list: tensor-core kernel for bf16 inputs (unless the plan asks for the
// staged SIMT schedule or the layout has no tensor map), SIMT kernel otherwise.
static int run_attend(psattn_plan_t *plan, const Geom &g, const void *Q, const void *K, const void *V,
                      const int *rows, int n_rows, int rows_stride, void *out, long long ous,
                      long long ors, int by_pos, int out_fp32, void *ws, cudaStream_t st,
                      float *vbar = nullptr) {
    // vbar != nullptr: the caller has checked attend64_supported(..., with_vbar = 1); mean(V) comes out of
    // the attention kernel (an extra all-ones weight row) instead of a separate pass over V
    const psattn_desc_t &d = plan->desc;
    float *ml = ws_at<float>(ws, plan->off_ml), *acc = ws_at<float>(ws, plan->off_acc);
    if (d.dtype == PSATTN_BF16 && d.path != PSATTN_PATH_STAGED && rows != nullptr && n_rows + (vbar ? 1 : 0) <= 64) {
        // one CTA per SM: split the keys only when there are fewer units than SMs
        const int pairs = (d.T_max + 255) / 256;
        int splits = device_sm_count() / (d.B * d.H > 0 ? d.B * d.H : 1);
        if (splits > plan->n_splits) splits = plan->n_splits;
        if (splits > pairs) splits = pairs;
        if (splits < 1) splits = 1;
        const int split_keys = ((pairs + splits - 1) / splits) * 256;
        splits = (d.T_max + split_keys - 1) / split_keys;
        cudaError_t e = launch_attend64(g, Q, K, V, rows, n_rows, rows_stride, splits, split_keys, ml, acc, out, ous,
                                        ors, by_pos, out_fp32, vbar, st);
        if (e == cudaSuccess) {
            if (splits > 1)
                PSATTN_CU(merge_attend_splits(!out_fp32, g, rows, n_rows, rows_stride, splits, ml, acc, out, ous,
                                              ors, by_pos, vbar, st));
            return PSATTN_OK;
        }
        if (e != cudaErrorNotSupported || vbar != nullptr) return cuda_fail(plan, e);
    }
    if (d.dtype == PSATTN_BF16 && d.path != PSATTN_PATH_STAGED) {
        // key splits: enough CTAs (256 rows each, one per SM) to cover the SMs, never more splits than 128-key tiles
        const int tiles = (d.T_max + 127) / 128;
        const long long ctas = (long long)d.B * d.H * ((n_rows + 255) / 256);
        int splits = (int)((device_sm_count() + ctas - 1) / (ctas > 0 ? ctas : 1));
        if (splits > plan->n_splits) splits = plan->n_splits;
        if (splits > tiles) splits = tiles;
        if (splits < 1 || rows == nullptr) splits = 1;
        const int split_keys = ((tiles + splits - 1) / splits) * 128;
        splits = (d.T_max + split_keys - 1) / split_keys;
        cudaError_t e = launch_attend_tc(g, Q, K, V, rows, n_rows, rows_stride, splits, split_keys, ml, acc, out,
                                         ous, ors, by_pos, out_fp32, st);
        if (e == cudaSuccess) {
            if (splits > 1)
                PSATTN_CU(merge_attend_splits(!out_fp32, g, rows, n_rows, rows_stride, splits, ml, acc, out, ous,
                                              ors, by_pos, nullptr, st));
            return PSATTN_OK;
        }
        if (e != cudaErrorNotSupported) return cuda_fail(plan, e);
    }
    const int splits = rows ? (d.T_max + kSplitKeys - 1) / kSplitKeys : 1;
    PSATTN_CU(launch_attend_simt(d.dtype, out_fp32, g, Q, K, V, rows, n_rows, rows_stride, splits,
                                 rows ? kSplitKeys : d.T_max, ml, acc, out, ous, ors, by_pos, st));
    return PSATTN_OK;
}

// Can mean(V) come out of the attention kernel for this plan and these buffers (bf16, at most 63 rows,
// tensor maps exist, fill value is mean(V))?  Then no separate column-sum pass over V is needed.
static bool vbar_from_attention(const psattn_plan_t *plan, const Geom &g, const void *K, const void *V) {
    const psattn_desc_t &d = plan->desc;
    return d.dtype == PSATTN_BF16 && d.path != PSATTN_PATH_STAGED && d.fill_mode == PSATTN_FILL_MEAN_V &&
           attend64_supported(g, K, V, plan->u_max, 1);
}

// Steps (d)+(e) for a selection that already sits in `sel` (device).  vbar_ready: mean(V) is already
// in the workspace (column-sum pass); otherwise it is produced by the attention kernel, and the fill
// runs after it.
static int run_attend_and_fill(psattn_plan_t *plan, const Geom &g, const void *Q, const void *K,
                               const void *V, const int *sel, void *O, void *ws, cudaStream_t st,
                               bool vbar_ready) {
    const psattn_desc_t &d = plan->desc;
    float *vbar = ws_at<float>(ws, plan->off_vbar);
    if (vbar_ready) {
        PSATTN_CU(launch_fill(d.dtype, g, V, sel, vbar, O, d.fill_mode == PSATTN_FILL_OWN_V, st));
        return run_attend(plan, g, Q, K, V, sel, plan->u_max, plan->u_max, O, 0, 0, 1, 0, ws, st);
    }
    int rc = run_attend(plan, g, Q, K, V, sel, plan->u_max, plan->u_max, O, 0, 0, 1, 0, ws, st, vbar);
    if (rc != PSATTN_OK) return rc;
    PSATTN_CU(launch_fill(d.dtype, g, V, sel, vbar, O, 0, st));
    return PSATTN_OK;
}

extern "C" int psattn_forward(psattn_plan_t *plan, const void *Q, const void *K, const void *V,
                              const int32_t *lengths, const int32_t *sample_idx, void *O,
                              int32_t *sel_idx, float *M_out, void *workspace,
                              size_t workspace_bytes, void *stream) {
    PSATTN_RANGE();
    if (!plan || !Q || !K || !V || !sample_idx || !O || !sel_idx) return PSATTN_ERR_NULL;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return PSATTN_ERR_MISALIGNED;
    int rc = check_ws(plan, workspace, workspace_bytes);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const psattn_desc_t &d = plan->desc;
    Geom g = make_geom(plan, lengths, workspace);
    if (d.dtype == PSATTN_BF16 && d.path != PSATTN_PATH_STAGED && !d.idx_shared) {
        cudaError_t e = launch_forward_fused(g, plan->U_max, d.fill_mode == PSATTN_FILL_OWN_V, Q, K, V, sample_idx, O,
                                             sel_idx, M_out, nullptr, st);
        if (e == cudaSuccess) return PSATTN_OK;
        if (e != cudaErrorNotSupported) return cuda_fail(plan, e);
        if (d.path == PSATTN_PATH_FUSED) return PSATTN_ERR_UNSUPPORTED;
    } else if (d.path == PSATTN_PATH_FUSED) {
        return PSATTN_ERR_UNSUPPORTED;
    }
    float *M = M_out ? M_out : ws_at<float>(workspace, plan->off_M);
    if (vbar_from_attention(plan, g, K, V)) {
        // Steps (a)-(c) do not touch V or O, and they are bound by on-chip gathers, not by HBM: the fill of
        // step (e) - column sums of V, mean(V), every valid row of O - runs beside them on the plan's side
        // stream (forked and joined with events, so the call stays ordered on the caller's stream and can be
        // captured in a graph); step (d) then overwrites the selected rows.
        float *vbar = ws_at<float>(workspace, plan->off_vbar);
        PSATTN_CU(cudaEventRecord(plan->side_ev[0], st));
        PSATTN_CU(cudaStreamWaitEvent(plan->side_stream, plan->side_ev[0], 0));
        cudaError_t se = cudaSuccess;
        if (d.fill_mode == PSATTN_FILL_MEAN_V) {
            se = launch_colsum(d.dtype, g, V, ws_at<float>(workspace, plan->off_vpart), plan->n_chunks, plan->side_stream);
            if (se == cudaSuccess)
                se = launch_select(g, nullptr, nullptr, ws_at<float>(workspace, plan->off_vpart), plan->n_chunks, vbar,
                                   nullptr, plan->side_stream);
        }
        if (se == cudaSuccess)
            se = launch_fill(d.dtype, g, V, nullptr, vbar, O, d.fill_mode == PSATTN_FILL_OWN_V, plan->side_stream);
        // always join, whatever happened on either side
        cudaError_t je = cudaEventRecord(plan->side_ev[1], plan->side_stream);
        rc = run_measure(plan, g, Q, K, sample_idx, M, st);
        cudaError_t le = rc == PSATTN_OK ? launch_select(g, M, sel_idx, nullptr, 0, nullptr, ws_at<int>(workspace, plan->off_cand), st) : cudaSuccess;
        if (je == cudaSuccess) je = cudaStreamWaitEvent(st, plan->side_ev[1], 0);
        if (rc != PSATTN_OK) return rc;
        PSATTN_CU(se); PSATTN_CU(je); PSATTN_CU(le);
        return run_attend(plan, g, Q, K, V, sel_idx, plan->u_max, plan->u_max, O, 0, 0, 1, 0, workspace, st);
    }
    if ((rc = run_measure(plan, g, Q, K, sample_idx, M, st)) != PSATTN_OK) return rc;
    PSATTN_CU(launch_colsum(d.dtype, g, V, ws_at<float>(workspace, plan->off_vpart), plan->n_chunks, st));
    PSATTN_CU(launch_select(g, M, sel_idx, ws_at<float>(workspace, plan->off_vpart), plan->n_chunks,
                            ws_at<float>(workspace, plan->off_vbar), nullptr, st));
    return run_attend_and_fill(plan, g, Q, K, V, sel_idx, O, workspace, st, true);
}

extern "C" int psattn_forward_with_selection(psattn_plan_t *plan, const void *Q, const void *K,
                                             const void *V, const int32_t *lengths,
                                             const int32_t *sel_idx_in, void *O, void *workspace,
                                             size_t workspace_bytes, void *stream) {
    PSATTN_RANGE();
    if (!plan || !Q || !K || !V || !sel_idx_in || !O) return PSATTN_ERR_NULL;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return PSATTN_ERR_MISALIGNED;
    int rc = check_ws(plan, workspace, workspace_bytes);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const psattn_desc_t &d = plan->desc;
    Geom g = make_geom(plan, lengths, workspace);
    if (d.dtype == PSATTN_BF16 && d.path != PSATTN_PATH_STAGED && d.B * d.H >= device_sm_count() / 2) {
        // one kernel for steps (d)+(e), one CTA per unit: where the units cover at least half of the SMs
        cudaError_t e = launch_forward_fused(g, plan->U_max, d.fill_mode == PSATTN_FILL_OWN_V, Q, K, V, nullptr, O,
                                             nullptr, nullptr, sel_idx_in, st);
        if (e == cudaSuccess) return PSATTN_OK;
        if (e != cudaErrorNotSupported) return cuda_fail(plan, e);
    }
    if (vbar_from_attention(plan, g, K, V))
        return run_attend_and_fill(plan, g, Q, K, V, sel_idx_in, O, workspace, st, false);
    // mean(V) by a column-sum pass (the select kernel, run without keys, only finishes the mean)
    PSATTN_CU(launch_colsum(d.dtype, g, V, ws_at<float>(workspace, plan->off_vpart), plan->n_chunks, st));
    PSATTN_CU(launch_select(g, nullptr, nullptr, ws_at<float>(workspace, plan->off_vpart),
                            plan->n_chunks, ws_at<float>(workspace, plan->off_vbar), nullptr, st));
    return run_attend_and_fill(plan, g, Q, K, V, sel_idx_in, O, workspace, st, true);
}

extern "C" int psattn_measure(psattn_plan_t *plan, const void *Q, const void *K,
                              const int32_t *lengths, const int32_t *sample_idx, float *M_out,
                              void *workspace, size_t workspace_bytes, void *stream) {
    PSATTN_RANGE();
    if (!plan || !Q || !K || !sample_idx || !M_out) return PSATTN_ERR_NULL;
    if (!aligned16(Q) || !aligned16(K)) return PSATTN_ERR_MISALIGNED;
    int rc = check_ws(plan, workspace, workspace_bytes);
    if (rc) return rc;
    Geom g = make_geom(plan, lengths, workspace);
    return run_measure(plan, g, Q, K, sample_idx, M_out, static_cast<cudaStream_t>(stream));
}

extern "C" int psattn_exact_measure(psattn_plan_t *plan, const void *Q, const void *K, const int32_t *lengths,
                                    float *M_out, void *workspace, size_t workspace_bytes, void *stream) {
    PSATTN_RANGE();
    if (!plan || !Q || !K || !M_out) return PSATTN_ERR_NULL;
    if (!aligned16(Q) || !aligned16(K)) return PSATTN_ERR_MISALIGNED;
    int rc = check_ws(plan, workspace, workspace_bytes);
    if (rc) return rc;
    Geom g = make_geom(plan, lengths, workspace);
    const psattn_desc_t &d = plan->desc;
    // PSATTN_PATH_STAGED keeps the arithmetic off the tensor cores (one warp per query)
    const int dtype = d.dtype == PSATTN_BF16 && d.path == PSATTN_PATH_STAGED ? 2 : d.dtype;
    PSATTN_CU(launch_exact_measure(dtype, g, Q, K, M_out, static_cast<cudaStream_t>(stream)));
    return PSATTN_OK;
}

extern "C" int psattn_project_qkv(psattn_plan_t *plan, const void *X, const void *Wt, int32_t d_x,
                                  const int32_t *lengths, void *Q, void *K, void *V, float *vbar,
                                  void *workspace, size_t workspace_bytes, void *stream) {
    PSATTN_RANGE();
    if (!plan || !X || !Wt || !Q || !K || !V) return PSATTN_ERR_NULL;
    if (d_x < 1 || d_x > (1 << 20)) return PSATTN_ERR_BAD_DESC;
    if (!aligned16(X) || !aligned16(Wt) || !aligned16(Q) || !aligned16(K) || !aligned16(V)) return PSATTN_ERR_MISALIGNED;
    int rc = check_ws(plan, workspace, workspace_bytes);
    if (rc) return rc;
    const psattn_desc_t &d = plan->desc;
    Geom g = make_geom(plan, lengths, workspace);
    PSATTN_CU(launch_project_qkv(d.dtype, d.path == PSATTN_PATH_STAGED, g, d_x, X, Wt, Q, K, V, vbar,
                                 ws_at<float>(workspace, plan->off_pvsum), static_cast<cudaStream_t>(stream)));
    return PSATTN_OK;
}

extern "C" int psattn_project_out(psattn_plan_t *plan, const void *O, const int32_t *sel_idx, const int32_t *lengths,
                                  const void *Wot, int32_t d_y, void *Y, void *workspace, size_t workspace_bytes,
                                  void *stream) {
    PSATTN_RANGE();
    if (!plan || !O || !Wot || !Y) return PSATTN_ERR_NULL;
    if (d_y < 1 || d_y > (1 << 20)) return PSATTN_ERR_BAD_DESC;
    if (!aligned16(O) || !aligned16(Wot) || !aligned16(Y)) return PSATTN_ERR_MISALIGNED;
    int rc = check_ws(plan, workspace, workspace_bytes);
    if (rc) return rc;
    const psattn_desc_t &d = plan->desc;
    Geom g = make_geom(plan, lengths, workspace);
    // the shortcut needs Eq. 12's structure with the mean(V) fill; any other O goes through the dense product
    const int mode = d.path == PSATTN_PATH_STAGED ? 2 : (sel_idx != nullptr && d.fill_mode == PSATTN_FILL_MEAN_V ? 0 : 1);
    cudaError_t e = launch_project_out(d.dtype, mode, g, d_y, O, sel_idx, Wot, Y, static_cast<cudaStream_t>(stream));
    if (e == cudaErrorNotSupported) return PSATTN_ERR_UNSUPPORTED;
    PSATTN_CU(e);
    return PSATTN_OK;
}

extern "C" int psattn_select(psattn_plan_t *plan, const float *M, const int32_t *lengths,
                             int32_t *sel_idx, void *workspace, size_t workspace_bytes,
                             void *stream) {
    PSATTN_RANGE();
    if (!plan || !M || !sel_idx) return PSATTN_ERR_NULL;
    int rc = check_ws(plan, workspace, workspace_bytes);
    if (rc) return rc;
    Geom g = make_geom(plan, lengths, workspace);
    PSATTN_CU(launch_select(g, M, sel_idx, nullptr, 0, nullptr, ws_at<int>(workspace, plan->off_cand),
                            static_cast<cudaStream_t>(stream)));
    return PSATTN_OK;
}

extern "C" int psattn_mean_v(psattn_plan_t *plan, const void *V, const int32_t *lengths,
                             float *vbar, void *workspace, size_t workspace_bytes, void *stream) {
    PSATTN_RANGE();
    if (!plan || !V || !vbar) return PSATTN_ERR_NULL;
    if (!aligned16(V)) return PSATTN_ERR_MISALIGNED;
    int rc = check_ws(plan, workspace, workspace_bytes);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    Geom g = make_geom(plan, lengths, workspace);
    PSATTN_CU(launch_colsum(plan->desc.dtype, g, V, ws_at<float>(workspace, plan->off_vpart), plan->n_chunks, st));
    PSATTN_CU(launch_select(g, nullptr, nullptr, ws_at<float>(workspace, plan->off_vpart), plan->n_chunks, vbar, nullptr, st));
    return PSATTN_OK;
}

extern "C" int psattn_attend_rows(psattn_plan_t *plan, const void *Q, const void *K, const void *V,
                                  const int32_t *lengths, const int32_t *row_idx, int32_t n_rows,
                                  float *out, void *workspace, size_t workspace_bytes,
                                  void *stream) {
    PSATTN_RANGE();
    if (!plan || !Q || !K || !V || !row_idx || !out) return PSATTN_ERR_NULL;
    if (n_rows < 0 || n_rows > plan->u_max) return PSATTN_ERR_BAD_DESC;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V)) return PSATTN_ERR_MISALIGNED;
    int rc = check_ws(plan, workspace, workspace_bytes);
    if (rc) return rc;
    if (n_rows == 0) return PSATTN_OK;
    Geom g = make_geom(plan, lengths, workspace);
    return run_attend(plan, g, Q, K, V, row_idx, n_rows, n_rows, out, (long long)n_rows * kD, kD, 0, 1,
                      workspace, static_cast<cudaStream_t>(stream));
}

extern "C" int psattn_dense_forward(psattn_plan_t *plan, const void *Q, const void *K,
                                    const void *V, const int32_t *lengths, void *O,
                                    void *workspace, size_t workspace_bytes, void *stream) {
    PSATTN_RANGE();
    if (!plan || !Q || !K || !V || !O) return PSATTN_ERR_NULL;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return PSATTN_ERR_MISALIGNED;
    int rc = check_ws(plan, workspace, workspace_bytes);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const psattn_desc_t &d = plan->desc;
    Geom g = make_geom(plan, lengths, workspace);
    // every position is a listed row (identity list): the attention kernels write the valid rows and the zero
    // rows at padded positions themselves
    return run_attend(plan, g, Q, K, V, nullptr, d.T_max, 0, O, 0, 0, 1, 0, workspace, st);
}

extern "C" int psattn_read_status(psattn_plan_t *plan, void *workspace, void *stream,
                                  uint32_t *host_bits) {
    if (!plan || !workspace || !host_bits) return PSATTN_ERR_NULL;
    if (int rc = check_device(plan)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned *w = ws_at<unsigned>(workspace, plan->off_status);
    PSATTN_CU(cudaMemcpyAsync(host_bits, w, sizeof(unsigned), cudaMemcpyDeviceToHost, st));
    PSATTN_CU(cudaMemsetAsync(w, 0, sizeof(unsigned), st));
    PSATTN_CU(cudaStreamSynchronize(st));
    return PSATTN_OK;
}

// ---- host-buffer front end ------------------------------------------------------------------
extern "C" int psattn_plan_enable_host_io(psattn_plan_t *plan) {
    if (!plan) return PSATTN_ERR_NULL;
    if (int rc = check_device(plan)) return rc;
    if (plan->host_io) return PSATTN_OK;
    const psattn_desc_t &d = plan->desc;
    const size_t es = d.dtype == PSATTN_BF16 ? 2 : 4;
    const size_t n = (size_t)d.B * d.H * d.T_max * kD * es;
    const size_t nidx = (size_t)d.B * (d.idx_per_head ? d.H : 1) * (d.idx_shared ? 1 : d.T_max) * d.idx_cols * sizeof(int);
    void **bufs[] = {&plan->h_Q, &plan->h_K, &plan->h_V, &plan->h_O, &plan->h_ws,
                     (void **)&plan->h_len, (void **)&plan->h_idx, (void **)&plan->h_sel};
    const size_t sizes[] = {n, n, n, n, plan->ws_bytes, (size_t)d.B * sizeof(int) + 16, nidx + 16,
                            (size_t)d.B * d.H * plan->u_max * sizeof(int) + 16};
    for (int k = 0; k < 8; ++k) {
        cudaError_t e = cudaMalloc(bufs[k], sizes[k] ? sizes[k] : 16);
        if (e != cudaSuccess) {
            for (int j = 0; j < k; ++j) { cudaFree(*bufs[j]); *bufs[j] = nullptr; }
            return cuda_fail(plan, e);
        }
    }
    PSATTN_CU(cudaMemset(plan->h_ws, 0, 256));
    PSATTN_CU(cudaStreamCreateWithFlags(&plan->h_copy_stream, cudaStreamNonBlocking));
    PSATTN_CU(cudaEventCreateWithFlags(&plan->h_ev[0], cudaEventDisableTiming));
    PSATTN_CU(cudaEventCreateWithFlags(&plan->h_ev[1], cudaEventDisableTiming));
    plan->host_io = true;
    return PSATTN_OK;
}

extern "C" int psattn_forward_host(psattn_plan_t *plan, const void *Q, const void *K, const void *V,
                                   const int32_t *lengths, const int32_t *sample_idx, void *O,
                                   int32_t *sel_idx, void *stream) {
    PSATTN_RANGE();
    if (!plan || !Q || !K || !V || !sample_idx || !O || !sel_idx) return PSATTN_ERR_NULL;
    if (!plan->host_io) return PSATTN_ERR_BAD_DESC;
    if (int rc = check_device(plan)) return rc;
    psattn_desc_t &d = plan->desc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t es = d.dtype == PSATTN_BF16 ? 2 : 4;
    // Sequences are independent, so the batch goes through in chunks: while chunk k is copied in and
    // computed on `stream`, the results of chunk k - 1 travel back on a second stream (PCIe is full
    // duplex).  All chunks share the one workspace; they are ordered by `stream`.
    const size_t per_b = (size_t)d.H * d.T_max * kD * es;
    const size_t idx_b = (size_t)(d.idx_per_head ? d.H : 1) * (d.idx_shared ? 1 : d.T_max) * d.idx_cols * sizeof(int);
    const size_t sel_b = (size_t)d.H * plan->u_max * sizeof(int);
    if (lengths) PSATTN_CU(cudaMemcpyAsync(plan->h_len, lengths, (size_t)d.B * sizeof(int), cudaMemcpyHostToDevice, st));
    // the staging buffers are dense: run with dense strides whatever the descriptor says
    psattn_desc_t saved = d;
    std::memset(d.q_stride, 0, sizeof(d.q_stride)); std::memset(d.k_stride, 0, sizeof(d.k_stride));
    std::memset(d.v_stride, 0, sizeof(d.v_stride)); std::memset(d.o_stride, 0, sizeof(d.o_stride));
    check_strides(d.q_stride, d); check_strides(d.k_stride, d);
    check_strides(d.v_stride, d); check_strides(d.o_stride, d);
    int n_chunks = 2;       // measured: every extra chunk costs ~50 us of copy set-up, more than it hides
    if (const char *env = std::getenv("PSATTN_HOST_CHUNKS")) { const int v = std::atoi(env); if (v >= 1 && v <= 64) n_chunks = v; }
    if (n_chunks > d.B) n_chunks = d.B > 0 ? d.B : 1;
    int rc = PSATTN_OK;
    cudaError_t ce = cudaSuccess;
    for (int k = 0; k < n_chunks && rc == PSATTN_OK && ce == cudaSuccess; ++k) {
        const int b0 = (int)((long long)d.B * k / n_chunks), b1 = (int)((long long)d.B * (k + 1) / n_chunks);
        const int nb = b1 - b0;
        if (nb == 0) continue;
        char *dq = (char *)plan->h_Q + b0 * per_b, *dk = (char *)plan->h_K + b0 * per_b;
        char *dv = (char *)plan->h_V + b0 * per_b, *dout = (char *)plan->h_O + b0 * per_b;
        char *di = (char *)plan->h_idx + b0 * idx_b, *ds = (char *)plan->h_sel + b0 * sel_b;
        if ((ce = cudaMemcpyAsync(dq, (const char *)Q + b0 * per_b, nb * per_b, cudaMemcpyHostToDevice, st)) != cudaSuccess) break;
        if ((ce = cudaMemcpyAsync(dk, (const char *)K + b0 * per_b, nb * per_b, cudaMemcpyHostToDevice, st)) != cudaSuccess) break;
        if ((ce = cudaMemcpyAsync(dv, (const char *)V + b0 * per_b, nb * per_b, cudaMemcpyHostToDevice, st)) != cudaSuccess) break;
        if ((ce = cudaMemcpyAsync(di, (const char *)sample_idx + b0 * idx_b, nb * idx_b, cudaMemcpyHostToDevice, st)) != cudaSuccess) break;
        plan->b_override = nb;
        rc = psattn_forward(plan, dq, dk, dv, lengths ? plan->h_len + b0 : nullptr, (const int32_t *)di, dout,
                            (int32_t *)ds, nullptr, plan->h_ws, plan->ws_bytes, stream);
        plan->b_override = 0;
        if (rc != PSATTN_OK) break;
        if ((ce = cudaEventRecord(plan->h_ev[0], st)) != cudaSuccess) break;
        if ((ce = cudaStreamWaitEvent(plan->h_copy_stream, plan->h_ev[0], 0)) != cudaSuccess) break;
        if ((ce = cudaMemcpyAsync((char *)O + b0 * per_b, dout, nb * per_b, cudaMemcpyDeviceToHost, plan->h_copy_stream)) != cudaSuccess) break;
        if ((ce = cudaMemcpyAsync((char *)sel_idx + b0 * sel_b, ds, nb * sel_b, cudaMemcpyDeviceToHost, plan->h_copy_stream)) != cudaSuccess) break;
    }
    d = saved;
    plan->b_override = 0;
    // never return with copies in flight, whatever happened above
    cudaStreamSynchronize(plan->h_copy_stream);
    if (rc != PSATTN_OK) { cudaStreamSynchronize(st); return rc; }
    if (ce != cudaSuccess) { cudaStreamSynchronize(st); return cuda_fail(plan, ce); }
    PSATTN_CU(cudaStreamSynchronize(st));
    return PSATTN_OK;
}
