// Steps (a)+(b) (Eq. 11) when one sample of keys serves every query of a sequence (the other reading of
// "a random sampling key matrix" in Sec. 3.2): the sampled scores of a tile of queries are then one dense
// product Q_tile K~^T, which belongs on the tensor cores.
//
// One CTA = (unit, tile of 128 queries), 128 threads:
//   TMA        Q tile (128 rows x 64)           -> shared memory, 128-byte swizzle
//   threads    the U <= 64 sampled key rows     -> shared memory, same layout (rows past U are zero)
//   tcgen05    S = Q_tile K~^T (M = 128, N = 64) -> TMEM, one row per lane
//   threads    row i = TMEM lane i: max and mean over the first U columns, M~_i -> global memory
// A key drawn twice occupies two columns, so it counts twice in the mean.  The step reads Q once and
// writes M~: it is bound by HBM.
#include "psattn_launch.h"
#include "psattn_sm100.cuh"

namespace psattn {

using namespace sm100;

constexpr int kMsRows = 128;                                 // queries per tile
constexpr int kMsMaxU = 64;                                  // columns of the product
constexpr uint32_t kMsOffQ = 0, kMsOffK = kMsRows * 128, kMsOffBar = kMsOffK + kMsMaxU * 128;
constexpr uint32_t kMsSmem = kMsOffBar + 64;
constexpr uint32_t kMsTmemCols = 64;

__global__ void __launch_bounds__(kMsRows) k_measure_shared(Geom g, int pos_t, int pos_h, int pos_b,
                                                            const __nv_bfloat16 *__restrict__ K,
                                                            const int *__restrict__ sidx, float *__restrict__ M,
                                                            const __grid_constant__ CUtensorMap tmQ) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *q_full = reinterpret_cast<uint64_t *>(smem + kMsOffBar), *mma_done = q_full + 1;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(q_full + 2);
    const int tid = threadIdx.x, warp = tid >> 5;
    const int unit = blockIdx.x, tile = blockIdx.y;
    const int b = unit / g.H, h = unit % g.H;
    const int L = seq_len(g, b);
    const int i = tile * kMsRows + tid;
    float *Mu = M + (long long)unit * g.T;
    if (tile * kMsRows >= L) {                                 // a tile of padded queries (uniform over the CTA)
        if (i < g.T) Mu[i] = 0.f;
        return;
    }
    if ((smem_u32(smem) & 1023u) != 0u) {                      // swizzled tiles need a 1024-byte base
        if (tid == 0) atomicOr(g.status, kStatusWaitExpired);
        return;
    }
    const int U = min(min(g.U_tab[L], g.idx_cols), kMsMaxU);
    if (tid == 0) {
        mbar_init(q_full, 1); mbar_init(mma_done, 1);
        fence_barrier_init();
        const int t0 = tile * kMsRows;
        const int c1 = pos_t == 1 ? t0 : (pos_h == 1 ? h : b);
        const int c2 = pos_t == 2 ? t0 : (pos_h == 2 ? h : b);
        const int c3 = pos_t == 3 ? t0 : (pos_h == 3 ? h : b);
        mbar_expect_tx(q_full, kMsRows * 128);
        tma_load_4d(smem + kMsOffQ, &tmQ, q_full, 0, c1, c2, c3);
    }
    __syncwarp();
    if (warp == 0) tmem_alloc(tmem_slot, kMsTmemCols);

    // sampled key rows -> B operand tile: row j, 16-byte chunk c at c ^ (j & 7)
    {
        const int *row = sidx + (g.idx_per_head ? (long long)unit : (long long)b) * g.idx_cols;
        const __nv_bfloat16 *Ku = K + unit_off(g.ks, b, h);
        for (int e = tid; e < kMsMaxU * 8; e += kMsRows) {
            const int j = e >> 3, c = e & 7;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (j < U) {
                int key = __ldg(row + j);
                if (key < 0 || key >= L) { atomicOr(g.status, kStatusIdxClamped); key = key < 0 ? 0 : L - 1; }
                v = __ldg(reinterpret_cast<const uint4 *>(Ku + (long long)key * g.ks[2]) + c);
            }
            *reinterpret_cast<uint4 *>(smem + kMsOffK + j * 128 + ((c ^ (j & 7)) << 4)) = v;
        }
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    bool q_landed = true;
    if (tid == 0) {
        q_landed = mbar_wait(q_full, 0);
        if (q_landed) {
            tc_fence_after();
            constexpr uint32_t kIdesc = umma_idesc_bf16(kMsRows, kMsMaxU, 0);    // B = sampled keys, K-major
            const uint32_t qa = smem_u32(smem + kMsOffQ), ka = smem_u32(smem + kMsOffK);
#pragma unroll
            for (int k = 0; k < kD / 16; ++k)
                umma_bf16(tmem_base, umma_desc_sw128(qa + k * 32, 16, 1024), umma_desc_sw128(ka + k * 32, 16, 1024),
                          kIdesc, k > 0);
            umma_commit(mma_done);
        }                                                      // else: nothing arrives, the wait below expires
    }
    __syncwarp();
    const bool landed = __all_sync(0xffffffffu, mbar_wait(mma_done, 0) ? 1 : 0) != 0;
    tc_fence_after();
    float out = 0.f;
    if (landed) {
        float v[kMsMaxU];
        const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
        tmem_ld32(lane_base, v);
        tmem_ld32(lane_base + 32, v + 32);
        // Eq. 11 relative to the first sampled score: d_j = s_j - s_0, M~ = max_j d_j - (1/U) sum_j d_j
        const float ref = v[0];
        float mx = 0.f, ds = 0.f;
#pragma unroll
        for (int j = 1; j < kMsMaxU; ++j) {
            const float d = v[j] - ref;
            if (j < U) { mx = fmaxf(mx, d); ds += d; }
        }
        out = fmaxf((mx - ds / (float)U) * kScale, 0.f);
    } else if ((tid & 31) == 0) {
        atomicOr(g.status, kStatusWaitExpired);
    }
    if (i < g.T) Mu[i] = (i < L && landed) ? out : 0.f;
    // a copy that did not land in time may still arrive: do not leave while it can write into this CTA's memory
    if (tid == 0 && !q_landed) mbar_wait(q_full, 0);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, kMsTmemCols);
}

bool make_rows_map(CUtensorMap *map, const void *base, const Geom &g, const long long s[3], int box_rows,
                   int swizzle128, int pos[3]);

// cudaErrorNotSupported: more than 64 samples, or no tensor map for the layout of Q.
cudaError_t launch_measure_shared(const Geom &g, int U_max, const void *Q, const void *K, const int *sidx, float *M,
                                  cudaStream_t st) {
    if (g.B * g.H == 0) return cudaSuccess;
    if (U_max > kMsMaxU || U_max < 1) return cudaErrorNotSupported;
    CUtensorMap tmQ;
    int pos[3];
    if (!make_rows_map(&tmQ, Q, g, g.qs, kMsRows, 1, pos)) return cudaErrorNotSupported;
    const dim3 grid((unsigned)(g.B * g.H), (unsigned)((g.T + kMsRows - 1) / kMsRows));
    k_measure_shared<<<grid, kMsRows, kMsSmem, st>>>(g, pos[0], pos[1], pos[2], (const __nv_bfloat16 *)K, sidx, M, tmQ);
    note_launch();
    return cudaGetLastError();
}

}  // namespace psattn
