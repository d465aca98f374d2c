// Steps (a)+(b) (Eq. 11) when one sample of keys serves every query of a sequence (the other reading of
// how Sec. 3.2 draws the sampled keys): the sampled scores of a tile of queries are then one dense
// product Q_tile K~^T, which belongs on the tensor cores.
//
// One CTA = (unit, run of 128-query tiles), 128 threads:
//   threads    the U <= 64 sampled key rows     -> shared memory, 128-byte swizzle (rows past U are zero), once
//   TMA        Q tile (128 rows x 64)           -> shared memory, same layout, two stages
//   tcgen05    S = Q_tile K~^T (M = 128, N = 64) -> TMEM, one row per lane, two accumulators
//   threads    row i = TMEM lane i: max and mean over the first U columns, M~_i -> global memory
// The product of tile t + 1 and the copy of tile t + 2 run while the threads reduce tile t.
// A key drawn twice occupies two columns, so it counts twice in the mean.  The step reads Q once and
// writes M~: it is bound by HBM.
#include "psattn_launch.h"
#include "psattn_sm100.cuh"

namespace psattn {

using namespace sm100;

constexpr int kMsRows = 128;                                 // queries per tile
constexpr int kMsMaxU = 64;                                  // columns of the product
constexpr uint32_t kMsTile = kMsRows * 128;                  // bytes of a Q tile
constexpr uint32_t kMsOffQ = 0, kMsOffK = 2 * kMsTile, kMsOffBar = kMsOffK + kMsMaxU * 128;
constexpr uint32_t kMsSmem = kMsOffBar + 64;
constexpr uint32_t kMsTmemCols = 128;                        // two accumulators of 64 columns

__global__ void __launch_bounds__(kMsRows) k_measure_shared(Geom g, int tiles_per_cta, int pos_t, int pos_h, int pos_b,
                                                            const __nv_bfloat16 *__restrict__ K,
                                                            const int *__restrict__ sidx, float *__restrict__ M,
                                                            const __grid_constant__ CUtensorMap tmQ) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *q_full = reinterpret_cast<uint64_t *>(smem + kMsOffBar), *mma_done = q_full + 2;   // [2] each
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(q_full + 4);
    const int tid = threadIdx.x, warp = tid >> 5;
    const int unit = blockIdx.x;
    const int b = unit / g.H, h = unit % g.H;
    const int L = seq_len(g, b);
    float *Mu = M + (long long)unit * g.T;
    const int tiles_total = (g.T + kMsRows - 1) / kMsRows;
    const int tile0 = blockIdx.y * tiles_per_cta, tile_hi = min(tiles_total, tile0 + tiles_per_cta);
    const int n_live = max(0, min(tile_hi, (L + kMsRows - 1) / kMsRows) - tile0);   // tiles with a valid query
    for (int i = (tile0 + n_live) * kMsRows + tid; i < min(g.T, tile_hi * kMsRows); i += kMsRows) Mu[i] = 0.f;
    if (n_live == 0) return;                                   // only padded queries here (uniform over the CTA)
    if ((smem_u32(smem) & 1023u) != 0u) {                      // swizzled tiles need a 1024-byte base
        if (tid == 0) atomicOr(g.status, kStatusWaitExpired);
        return;
    }
    const int U = min(min(g.U_tab[L], g.idx_cols), kMsMaxU);
    auto load_q = [&](int t) {                                 // thread 0: tile tile0 + t -> stage t & 1
        const int s = t & 1, t0 = (tile0 + t) * kMsRows;
        const int c1 = pos_t == 1 ? t0 : (pos_h == 1 ? h : b);
        const int c2 = pos_t == 2 ? t0 : (pos_h == 2 ? h : b);
        const int c3 = pos_t == 3 ? t0 : (pos_h == 3 ? h : b);
        mbar_expect_tx(&q_full[s], kMsTile);
        tma_load_4d(smem + kMsOffQ + s * kMsTile, &tmQ, &q_full[s], 0, c1, c2, c3);
    };
    if (tid == 0) {
        mbar_init(&q_full[0], 1); mbar_init(&q_full[1], 1);
        mbar_init(&mma_done[0], 1); mbar_init(&mma_done[1], 1);
        fence_barrier_init();
        tma_prefetch_desc(&tmQ);
        load_q(0);
        if (n_live > 1) load_q(1);
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
    const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);

    // thread 0: S of tile t into accumulator t & 1, once its Q tile has landed; false if that wait expired
    auto issue_mma = [&](int t) {
        const int s = t & 1;
        if (!mbar_wait(&q_full[s], (uint32_t)((t >> 1) & 1))) return false;
        tc_fence_after();
        constexpr uint32_t kIdesc = umma_idesc_bf16(kMsRows, kMsMaxU, 0);        // B = sampled keys, K-major
        const uint32_t qa = smem_u32(smem + kMsOffQ + s * kMsTile), ka = smem_u32(smem + kMsOffK);
#pragma unroll
        for (int k = 0; k < kD / 16; ++k)
            umma_bf16(tmem_base + s * kMsMaxU, umma_desc_sw128(qa + k * 32, 16, 1024),
                      umma_desc_sw128(ka + k * 32, 16, 1024), kIdesc, k > 0);
        umma_commit(&mma_done[s]);
        return true;
    };
    bool copies_ok = true;                                     // thread 0: no wait for a Q tile has expired
    int copies_started = min(n_live, 2);
    if (tid == 0) copies_ok = issue_mma(0);
    bool alive = true;
    for (int t = 0; t < n_live && alive; ++t) {
        const int s = t & 1;
        if (tid == 0 && copies_ok && t + 1 < n_live) copies_ok = issue_mma(t + 1);   // its accumulator was read in t - 1
        __syncwarp();
        const bool landed = __all_sync(0xffffffffu, mbar_wait(&mma_done[s], (uint32_t)((t >> 1) & 1)) ? 1 : 0) != 0;
        tc_fence_after();
        float out = 0.f;
        if (landed) {
            float v[kMsMaxU];
            tmem_ld32(lane_base + s * kMsMaxU, v);
            tmem_ld32(lane_base + s * kMsMaxU + 32, v + 32);
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
        const int i = (tile0 + t) * kMsRows + tid;
        if (i < g.T) Mu[i] = (i < L && landed) ? out : 0.f;
        tc_fence_before();
        alive = __syncthreads_and(landed ? 1 : 0) != 0;        // accumulator s and Q stage s are free again
        if (tid == 0 && alive && t + 2 < n_live) { load_q(t + 2); copies_started = t + 3; }
    }
    // copies that were started but never consumed: give them a bounded chance to land before leaving
    if (tid == 0 && !alive)
        for (int t = max(0, copies_started - 2); t < copies_started; ++t) mbar_wait(&q_full[t & 1], (uint32_t)((t >> 1) & 1));
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
    // runs of tiles long enough to amortise the gather of the sampled keys, short enough for a few CTAs per SM
    const int units = g.B * g.H, tiles_total = (g.T + kMsRows - 1) / kMsRows;
    int chunks = (4 * device_sm_count() + units - 1) / units;
    if (chunks > tiles_total) chunks = tiles_total;
    if (chunks < 1) chunks = 1;
    const int tiles_per_cta = (tiles_total + chunks - 1) / chunks;
    chunks = (tiles_total + tiles_per_cta - 1) / tiles_per_cta;
    static SmemGrant grant;
    if (cudaError_t e = grant_dynamic_smem(k_measure_shared, grant, kMsSmem)) return e;
    const dim3 grid((unsigned)units, (unsigned)chunks);
    k_measure_shared<<<grid, kMsRows, kMsSmem, st>>>(g, tiles_per_cta, pos[0], pos[1], pos[2], (const __nv_bfloat16 *)K,
                                                      sidx, M, tmQ);
    note_launch();
    return cudaGetLastError();
}

}  // namespace psattn
