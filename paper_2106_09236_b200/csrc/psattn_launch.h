// Host-callable launchers of the kernels; shared by the translation units of the library.
#pragma once
#include "psattn_common.cuh"

namespace psattn {

constexpr int kColsumRows = 256;      // rows of V per column-sum partial
constexpr int kFillRows = 128;        // rows of O per fill block
constexpr int kSelectThreads = 1024;
constexpr int kSelectSmemKeys = 8192; // keys kept in shared memory by the select kernel (32 KB)
constexpr int kSplitKeys = 1024;      // keys per split of the SIMT attention kernel
constexpr int kMaxDevices = 64;       // device ordinals the per-device records below cover

// Multiprocessors of the current device (read once per device from its attributes).
int device_sm_count();

// cudaFuncAttributeMaxDynamicSharedMemorySize belongs to the current device's context: one record per
// kernel holds, per device, the size already granted there.  grant_dynamic_smem raises it when needed
// (thread safe; `carveout`: also ask for the largest shared-memory carve-out).
struct SmemGrant {
    size_t bytes[kMaxDevices];
};
cudaError_t grant_dynamic_smem_impl(const void *kernel, SmemGrant &rec, size_t smem, bool carveout);
template <typename... KArgs>
inline cudaError_t grant_dynamic_smem(void (*kernel)(KArgs...), SmemGrant &rec, size_t smem, bool carveout = false) {
    return grant_dynamic_smem_impl(reinterpret_cast<const void *>(kernel), rec, smem, carveout);
}

// Launch with programmatic stream serialization: the kernel may be scheduled while its predecessor in the
// stream drains.  Only for kernels that call pdl_enter() before their first global-memory access.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args &&...args) {
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Every kernel launch of the library is counted (process-wide).
void note_launch(int n = 1);
unsigned long long launches_so_far();

cudaError_t launch_measure(int dtype, const Geom &g, const void *Q, const void *K, const int *sidx,
                           float *M, cudaStream_t st);
// Resident-key tensor-datapath form of steps (a)+(b) for bf16 inputs; cudaErrorNotSupported when
// T_max is too long for shared memory, U_max > 64 or the layout has no tensor map (the caller then
// uses launch_measure).
cudaError_t launch_measure_mma(const Geom &g, int U_max, const void *Q, const void *K, const int *sidx, float *M,
                               cudaStream_t st);
// Steps (a)-(e) of every unit in one kernel (bf16, keys resident in shared memory).
// cudaErrorNotSupported: shape outside the kernel's limits; run the staged schedule instead.
// sel_in != nullptr: steps (d)+(e) only, for the given index set [unit][u_max] (sidx, sel, M_out unused).
cudaError_t launch_forward_fused(const Geom &g, int U_max, int own_v, const void *Q, const void *K, const void *V,
                                 const int *sidx, void *O, int *sel, float *M_out, const int *sel_in, cudaStream_t st);
// Streaming tensor-datapath form of steps (a)+(b) for bf16 inputs and any T_max (key rows gathered from L2
// through shared-memory rings); cudaErrorNotSupported when U_max > 64.
cudaError_t launch_measure_stream(const Geom &g, int U_max, const void *Q, const void *K, const int *sidx, float *M,
                                  cudaStream_t st);
// Eq. 10 over all valid keys (dense pass): tcgen05 for bf16 (dtype 0), one warp per query otherwise.
cudaError_t launch_exact_measure(int dtype, const Geom &g, const void *Q, const void *K, float *M, cudaStream_t st);
// One sample per sequence (Geom::idx_shared): the scores of 128 queries are one tcgen05 product.
cudaError_t launch_measure_shared(const Geom &g, int U_max, const void *Q, const void *K, const int *sidx, float *M,
                                  cudaStream_t st);
cudaError_t launch_colsum(int dtype, const Geom &g, const void *V, float *part, int n_chunks,
                          cudaStream_t st);
// cand (optional): scratch of select_cand_ints(units, u_max) ints; with it, few units of long sequences are
// selected in two kernels (ranges of positions first, then their candidates).
size_t select_cand_ints(int units, int u_max);
cudaError_t launch_select(const Geom &g, const float *M, int *sel, const float *vpart, int n_chunks,
                          float *vbar, int *cand, cudaStream_t st);
// rows == nullptr: the row list is the identity (row r is position r).
// out_by_position: write the finished row at its position in O (element type of the inputs,
// strides g.os); otherwise at slot r of `out` with the given unit / row strides.
cudaError_t launch_attend_simt(int dtype, int out_fp32, const Geom &g, const void *Q, const void *K,
                               const void *V, const int *rows, int n_rows, int rows_stride,
                               int n_splits, int split_keys, float *part_ml, float *part_acc,
                               void *out, long long out_unit_stride, long long out_row_stride,
                               int out_by_position, cudaStream_t st);
// Tensor-core (tcgen05) form of the same step for bf16 inputs; same argument meaning, plus
// out_fp32 for row-list output.  split_keys must be a multiple of 128.  Returns
// cudaErrorNotSupported when the layout cannot be described by a TMA tensor map (the caller then
// uses launch_attend_simt); the split partials are merged by merge_attend_splits.
cudaError_t launch_attend_tc(const Geom &g, const void *Q, const void *K, const void *V, const int *rows,
                             int n_rows, int rows_stride, int n_splits, int split_keys, float *part_ml,
                             float *part_acc, void *out, long long out_unit_stride, long long out_row_stride,
                             int out_by_position, int out_fp32, cudaStream_t st);
// Same step for row lists of at most 64 rows (the sparse path): two warpgroups over pairs of key
// tiles.  split_keys must be a multiple of 256.  cudaErrorNotSupported: use launch_attend_tc.
cudaError_t launch_attend64(const Geom &g, const void *Q, const void *K, const void *V, const int *rows,
                            int n_rows, int rows_stride, int n_splits, int split_keys, float *part_ml,
                            float *part_acc, void *out, long long out_unit_stride, long long out_row_stride,
                            int out_by_position, int out_fp32, float *vbar, cudaStream_t st);
// With vbar != nullptr launch_attend64 also produces mean(V) [unit][64] (fp32) from an extra row whose
// weights are all 1, at no extra pass over V; the partials then hold n_rows + 1 row slots per unit.
bool attend64_supported(const Geom &g, const void *K, const void *V, int n_rows, int with_vbar);
// vbar != nullptr: the partials hold one more row slot per unit (the all-ones row), merged into vbar.
cudaError_t merge_attend_splits(int out_is_bf16, const Geom &g, const int *rows, int n_rows, int rows_stride,
                                int n_splits, const float *part_ml, const float *part_acc, void *out,
                                long long out_unit_stride, long long out_row_stride, int out_by_position,
                                float *vbar, cudaStream_t st);
// Sec. 3.1's projections Q = X W_q, K = X W_k, V = X W_v into the attention layout (tcgen05 GEMM for bf16,
// dtype 0; one thread per element for fp32 or with force_simt).  X [B][T][dx], Wt [3][H*64][dx].
// vbar (optional): mean(V) fp32 [B][H][64]; vpart: scratch of project_vpart_floats(B, H, T) floats.
size_t project_vpart_floats(int B, int H, int T);
cudaError_t launch_project_qkv(int dtype, int force_simt, const Geom &g, int dx, const void *X, const void *Wt, void *Q,
                               void *K, void *V, float *vbar, float *vpart, cudaStream_t st);
// The output matrix of the attention module: Y [B][T][dy] = sum_h O[b][h][t][:] W_o^h, Wot [dy][H * 64].
// mode 0: with an index set `sel` ([B][H][g.u_max], as psattn_forward writes it) and the mean(V) fill, the
// broadcast-plus-corrections form; otherwise (and with mode 1) the dense tcgen05 GEMM; mode 2 or fp32: one
// thread per output element.  Rows at padded positions are not written.
cudaError_t launch_project_out(int dtype, int mode, const Geom &g, int dy, const void *O, const int *sel, const void *Wot,
                               void *Y, cudaStream_t st);
cudaError_t launch_fill(int dtype, const Geom &g, const void *V, const int *sel, const float *vbar,
                        void *O, int own_v, cudaStream_t st);

}  // namespace psattn
