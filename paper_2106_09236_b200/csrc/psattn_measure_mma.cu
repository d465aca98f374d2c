// Stand-alone kernel around measure_resident: steps (a)+(b) (Eq. 11) for bf16 inputs.
// One CTA = (unit, slice of its queries).
#include "psattn_launch.h"
#include "psattn_measure_mma.cuh"
#include "psattn_measure_stream.cuh"

namespace psattn {

using namespace sm100;

constexpr int kMeasureThreads = 640;

struct MeasureMmaArgs {
    int q_slices;               // CTAs per unit
    int pos_t, pos_h, pos_b;    // TMA coordinate slots of t, h, b
    uint32_t stage_bytes;       // bytes of one staging buffer (Q tile + sample tile)
    uint32_t k_bytes;           // bytes reserved for the resident keys
};

__global__ void __launch_bounds__(kMeasureThreads, 1) k_measure_mma(Geom g, MeasureMmaArgs a,
                                                                    const __nv_bfloat16 *__restrict__ Q,
                                                                    const int *__restrict__ sidx,
                                                                    float *__restrict__ M,
                                                                    const __grid_constant__ CUtensorMap tmK) {
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ uint64_t bar;
    const int tid = threadIdx.x;
    const int unit = blockIdx.x / a.q_slices, slice = blockIdx.x % a.q_slices;
    const int b = unit / g.H, h = unit % g.H;
    const int L = seq_len(g, b);
    const int U = min(g.U_tab[L], g.idx_cols);
    const int per = (g.T + a.q_slices - 1) / a.q_slices;
    const int q_lo = slice * per, q_hi = min(g.T, q_lo + per);
    const int q_end = min(q_hi, L);
    float *Mu = M + (long long)unit * g.T;

    if (tid == 0) {
        mbar_init(&bar, 1);
        fence_barrier_init();
        if (q_lo < L) measure_issue_keys(smem, &bar, &tmK, L, b, h, a.pos_t, a.pos_h);
    }
    // rows of padded queries are zero
    for (int i = max(q_lo, L) + tid; i < q_hi; i += kMeasureThreads) Mu[i] = 0.f;
    __syncthreads();
    if (L == 0 || q_lo >= L) return;
    measure_resident<kMeasureThreads>(smem, &bar, 0u, a.k_bytes, a.stage_bytes, g, unit, b, h, L, U, q_lo, q_end, Q,
                                      sidx, Mu);
}

// Streaming form (keys gathered from L2 through per-warp rings): any T_max.
constexpr int kStreamThreads = 768;

__global__ void __launch_bounds__(kStreamThreads, 1) k_measure_stream(Geom g, int q_slices, uint32_t stage_bytes,
                                                                      const __nv_bfloat16 *__restrict__ Q,
                                                                      const __nv_bfloat16 *__restrict__ K,
                                                                      const int *__restrict__ sidx,
                                                                      float *__restrict__ M) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x;
    const int unit = blockIdx.x / q_slices, slice = blockIdx.x % q_slices;
    const int b = unit / g.H, h = unit % g.H;
    pdl_enter();
    KernelSpan span(g, kKernelMeasure);
    const int L = seq_len(g, b);
    const int U = min(g.U_tab[L], g.idx_cols);
    // slices in whole staged blocks so that every CTA but the last works on full blocks
    constexpr int kBlock = measure_block_queries(kStreamThreads);
    const int blocks_total = (g.T + kBlock - 1) / kBlock;
    const int per = (blocks_total + q_slices - 1) / q_slices * kBlock;
    const int q_lo = min(g.T, slice * per), q_hi = min(g.T, q_lo + per);
    const int q_end = min(q_hi, L);
    float *Mu = M + (long long)unit * g.T;
    for (int i = max(q_lo, L) + tid; i < q_hi; i += kStreamThreads) Mu[i] = 0.f;   // padded queries
    if (L == 0 || q_lo >= L) return;
    measure_stream<kStreamThreads>(smem, stage_bytes, g, unit, b, h, L, U, q_lo, q_end, Q, K, sidx, Mu);
}

// ---- host side ----------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn2)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);

bool make_rows_map(CUtensorMap *map, const void *base, const Geom &g, const long long s[3], int box_rows,
                   int swizzle128, int pos[3]) {
    static EncodeTiledFn2 enc = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            enc = reinterpret_cast<EncodeTiledFn2>(p);
        else
            cudaGetLastError();
    }
    if (!enc) return false;
    struct Dim { long long size, stride; int which; } dims[3] = {{g.T, s[2], 0}, {g.H, s[1], 1}, {g.B, s[0], 2}};
    for (int x = 0; x < 3; ++x)
        for (int y = x + 1; y < 3; ++y)
            if (dims[y].stride < dims[x].stride) { Dim tmp = dims[x]; dims[x] = dims[y]; dims[y] = tmp; }
    cuuint64_t gdim[4] = {(cuuint64_t)kD, 0, 0, 0};
    cuuint64_t gstr[3];
    cuuint32_t box[4] = {(cuuint32_t)kD, 1, 1, 1}, estr[4] = {1, 1, 1, 1};
    for (int x = 0; x < 3; ++x) {
        if (dims[x].stride <= 0) return false;
        gdim[x + 1] = (cuuint64_t)dims[x].size;
        gstr[x] = (cuuint64_t)dims[x].stride * 2;
        pos[dims[x].which] = x + 1;
        if (dims[x].which == 0) box[x + 1] = (cuuint32_t)box_rows;
    }
    CUresult rc = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), gdim, gstr, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE,
                      swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS;
}

// cudaErrorNotSupported: T_max too long for resident keys, U above four rounds, or no tensor map.
cudaError_t launch_measure_mma(const Geom &g, int U_max, const void *Q, const void *K, const int *sidx, float *M,
                               cudaStream_t st) {
    if (g.B * g.H == 0) return cudaSuccess;
    const size_t k_bytes = measure_k_bytes(g.T);
    const size_t stage_bytes = measure_stage_bytes(kMeasureThreads, g.idx_cols);
    const size_t smem = k_bytes + kMeasureStages * stage_bytes;
    if (smem > 225 * 1024 || U_max > kMeasureMaxU || U_max < 1) return cudaErrorNotSupported;
    CUtensorMap tmK;
    int pos[3];
    if (!make_rows_map(&tmK, K, g, g.ks, kMeasureBoxRows, 0, pos)) return cudaErrorNotSupported;
    MeasureMmaArgs a;
    a.pos_t = pos[0]; a.pos_h = pos[1]; a.pos_b = pos[2];
    a.stage_bytes = (uint32_t)stage_bytes; a.k_bytes = (uint32_t)k_bytes;
    const int units = g.B * g.H;
    // resident CTAs per SM by shared memory; slices so that the grid covers the SMs
    const int per_sm = smem <= 100 * 1024 ? 2 : 1;
    int slices = (device_sm_count() * per_sm) / units;
    if (slices < 1) slices = 1;
    if (slices > 8) slices = 8;
    a.q_slices = slices;
    static SmemGrant grant;
    if (cudaError_t e = grant_dynamic_smem(k_measure_mma, grant, smem)) return e;
    k_measure_mma<<<(unsigned)(units * slices), kMeasureThreads, smem, st>>>(g, a, (const __nv_bfloat16 *)Q, sidx, M, tmK);
    note_launch();
    return cudaGetLastError();
}

}  // namespace psattn

namespace psattn {

// cudaErrorNotSupported: more than 64 samples per query, or key rows of a unit spread over 4 GB or more.
cudaError_t launch_measure_stream(const Geom &g, int U_max, const void *Q, const void *K, const int *sidx, float *M,
                                  cudaStream_t st) {
    if (g.B * g.H == 0) return cudaSuccess;
    if (U_max > kMeasureMaxU || U_max < 1) return cudaErrorNotSupported;
    if (g.ks[2] <= 0 || (long long)g.T * g.ks[2] * 2 >= (1ll << 32)) return cudaErrorNotSupported;
    const size_t stage_bytes = measure_stage_bytes(kStreamThreads, g.idx_cols);
    const size_t smem = (size_t)(kStreamThreads / 32) * kStreamRing * kStreamRoundBytes + 2 * stage_bytes;
    if (smem > 225 * 1024) return cudaErrorNotSupported;
    const int units = g.B * g.H;
    constexpr int kBlock = measure_block_queries(kStreamThreads);
    const int blocks_total = (g.T + kBlock - 1) / kBlock;
    int slices = (2 * device_sm_count() + units - 1) / units;             // about two CTAs' worth of work per SM
    if (slices > blocks_total) slices = blocks_total;
    if (slices < 1) slices = 1;
    static SmemGrant grant;
    if (cudaError_t e = grant_dynamic_smem(k_measure_stream, grant, smem)) return e;
    cudaError_t e = launch_pdl(k_measure_stream, dim3((unsigned)(units * slices)), dim3(kStreamThreads), smem, st, g, slices,
                               (uint32_t)stage_bytes, (const __nv_bfloat16 *)Q, (const __nv_bfloat16 *)K, sidx, M);
    note_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace psattn
