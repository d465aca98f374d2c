// The exact sparsity measure of Eq. 10, M_i = ln sum_j exp(s_ij) - (1/L) sum_j s_ij over ALL valid keys
// (s_ij = q_i . k_j / sqrt(d)): the quantity that the sampled measure of Eq. 11 approximates.  A dense pass
// over the score matrix, so it runs on the tensor cores.
//
// bf16: one CTA = (unit, tile of 128 queries), 128 threads.  K streams in 128-key tiles by TMA (two stages);
// S = Q_tile K_tile^T is a tcgen05.mma (M = 128, N = 128) into one of two TMEM accumulators, so the product
// of tile t + 1 runs while the threads reduce tile t; row i = TMEM lane i keeps the running (max, sum of
// exponentials, sum of scores) of its query in registers.  Nothing but M leaves the SM.
// fp32: one warp per query, lanes stride over the keys, fp32 throughout.
#include "psattn_launch.h"
#include "psattn_sm100.cuh"

namespace psattn {

using namespace sm100;

constexpr int kEmRows = 128, kEmKeys = 128;
constexpr uint32_t kEmTile = 128 * 128;                       // bytes of a Q or K tile
constexpr uint32_t kEmOffQ = 0, kEmOffK = kEmTile, kEmOffBar = 3 * kEmTile;
constexpr uint32_t kEmSmem = kEmOffBar + 64;
constexpr uint32_t kEmTmemCols = 256;                         // two accumulators of 128 columns

__global__ void __launch_bounds__(kEmRows) k_exact_measure(Geom g, int pos_t, int pos_h, int pos_b, float *__restrict__ M,
                                                           const __grid_constant__ CUtensorMap tmQ,
                                                           const __grid_constant__ CUtensorMap tmK) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *k_full = reinterpret_cast<uint64_t *>(smem + kEmOffBar), *mma_done = k_full + 2, *q_full = k_full + 4;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(k_full + 5);
    const int tid = threadIdx.x, warp = tid >> 5;
    const int unit = blockIdx.x, tile = blockIdx.y;
    const int b = unit / g.H, h = unit % g.H;
    const int L = seq_len(g, b);
    const int i = tile * kEmRows + tid;
    float *Mu = M + (long long)unit * g.T;
    if (tile * kEmRows >= L) {                                 // a tile of padded queries (uniform over the CTA)
        if (i < g.T) Mu[i] = 0.f;
        return;
    }
    if ((smem_u32(smem) & 1023u) != 0u) {                      // swizzled tiles need a 1024-byte base
        if (tid == 0) atomicOr(g.status, kStatusWaitExpired);
        return;
    }
    const int n_tiles = (L + kEmKeys - 1) / kEmKeys;
    auto coords = [&](int t0, int &c1, int &c2, int &c3) {
        c1 = pos_t == 1 ? t0 : (pos_h == 1 ? h : b);
        c2 = pos_t == 2 ? t0 : (pos_h == 2 ? h : b);
        c3 = pos_t == 3 ? t0 : (pos_h == 3 ? h : b);
    };
    auto load_k = [&](int t) {                                 // thread 0: key tile t -> stage t & 1
        int c1, c2, c3;
        coords(t * kEmKeys, c1, c2, c3);
        mbar_expect_tx(&k_full[t & 1], kEmTile);
        tma_load_4d(smem + kEmOffK + (t & 1) * kEmTile, &tmK, &k_full[t & 1], 0, c1, c2, c3);
    };
    if (tid == 0) {
        mbar_init(&k_full[0], 1); mbar_init(&k_full[1], 1);
        mbar_init(&mma_done[0], 1); mbar_init(&mma_done[1], 1);
        mbar_init(q_full, 1);
        fence_barrier_init();
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK);
        int c1, c2, c3;
        coords(tile * kEmRows, c1, c2, c3);
        mbar_expect_tx(q_full, kEmTile);
        tma_load_4d(smem + kEmOffQ, &tmQ, q_full, 0, c1, c2, c3);
        load_k(0);
        if (n_tiles > 1) load_k(1);
    }
    __syncwarp();
    if (warp == 0) tmem_alloc(tmem_slot, kEmTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);

    // thread 0: S of key tile t into accumulator t & 1 once the tile has landed; false if that wait expired
    auto issue_mma = [&](int t) {
        const int s = t & 1;
        if (!mbar_wait(&k_full[s], (uint32_t)((t >> 1) & 1))) return false;
        tc_fence_after();
        constexpr uint32_t kIdesc = umma_idesc_bf16(kEmRows, kEmKeys, 0);        // B = K tile, K-major
        const uint32_t qa = smem_u32(smem + kEmOffQ), ka = smem_u32(smem + kEmOffK + s * kEmTile);
#pragma unroll
        for (int k = 0; k < kD / 16; ++k)
            umma_bf16(tmem_base + s * kEmKeys, umma_desc_sw128(qa + k * 32, 16, 1024),
                      umma_desc_sw128(ka + k * 32, 16, 1024), kIdesc, k > 0);
        umma_commit(&mma_done[s]);
        return true;
    };
    bool copies_ok = true;                                     // thread 0 only
    int copies_started = min(n_tiles, 2);
    if (tid == 0) copies_ok = mbar_wait(q_full, 0) && issue_mma(0);

    const float kScaleLog2 = kScale * kLog2e;
    float m_run = -INFINITY, l_run = 0.f, x_sum = 0.f;         // m_run in scaled log2 units; x_sum in raw q.k units
    bool alive = true;
    for (int t = 0; t < n_tiles && alive; ++t) {
        const int s = t & 1;
        if (tid == 0 && copies_ok && t + 1 < n_tiles) copies_ok = issue_mma(t + 1);   // its accumulator was read in t - 1
        __syncwarp();
        const bool landed = __all_sync(0xffffffffu, mbar_wait(&mma_done[s], (uint32_t)((t >> 1) & 1)) ? 1 : 0) != 0;
        tc_fence_after();
        if (landed) {
            const int valid = min(kEmKeys, L - t * kEmKeys);   // keys of this tile that exist
            float v[kEmKeys];
#pragma unroll
            for (int cb = 0; cb < 4; ++cb) tmem_ld32(lane_base + s * kEmKeys + cb * 32, v + cb * 32);
            float mx = -INFINITY, xs = 0.f;
#pragma unroll
            for (int j = 0; j < kEmKeys; ++j)
                if (j < valid) { mx = fmaxf(mx, v[j]); xs += v[j]; }
            const float m_new = fmaxf(m_run, mx * kScaleLog2);
            float lsum = 0.f;
#pragma unroll
            for (int j = 0; j < kEmKeys; ++j)
                if (j < valid) lsum += fast_exp2(fmaf(v[j], kScaleLog2, -m_new));
            l_run = l_run * fast_exp2(m_run - m_new) + lsum;   // the factor is 0 on the first tile
            m_run = m_new;
            x_sum += xs;
        } else if ((tid & 31) == 0) {
            atomicOr(g.status, kStatusWaitExpired);
        }
        tc_fence_before();
        alive = __syncthreads_and(landed ? 1 : 0) != 0;        // accumulator s and key stage s are free again
        if (tid == 0 && alive && t + 2 < n_tiles) { load_k(t + 2); copies_started = t + 3; }
    }
    // Eq. 10: ln sum_j exp(s_j) - mean_j s_j, from the base-2 running state
    if (i < g.T) Mu[i] = (i < L && alive) ? (m_run + log2f(l_run)) * 0.6931471805599453f - kScale * x_sum / (float)L : 0.f;
    if (tid == 0 && !alive) {                                  // copies started but never consumed: bounded drain
        mbar_wait(q_full, 0);
        for (int t = max(0, copies_started - 2); t < copies_started; ++t) mbar_wait(&k_full[t & 1], (uint32_t)((t >> 1) & 1));
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, kEmTmemCols);
}

// fp32 (and any layout the tensor-core form does not take): one warp per query.
template <typename DT>
__global__ void __launch_bounds__(128) k_exact_measure_simt(Geom g, const DT *__restrict__ Q, const DT *__restrict__ K,
                                                            float *__restrict__ M) {
    const int lane = threadIdx.x & 31;
    const long long w = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (w >= (long long)g.B * g.H * g.T) return;
    const int i = (int)(w % g.T), unit = (int)(w / g.T);
    const int b = unit / g.H, h = unit % g.H;
    const int L = seq_len(g, b);
    if (i >= L) { if (lane == 0) M[w] = 0.f; return; }
    float q[kD];
#pragma unroll
    for (int c = 0; c < 8; ++c) load8(Q + unit_off(g.qs, b, h) + (long long)i * g.qs[2], c, q + 8 * c);
    const DT *Ku = K + unit_off(g.ks, b, h);
    float m = -INFINITY, l = 0.f, ssum = 0.f;                  // natural-log units
    for (int j = lane; j < L; j += 32) {
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            float kk[8];
            load8(Ku + (long long)j * g.ks[2], c, kk);
#pragma unroll
            for (int t = 0; t < 8; ++t) s = fmaf(q[8 * c + t], kk[t], s);
        }
        s *= kScale;
        const float m_new = fmaxf(m, s);
        l = l * expf(m - m_new) + expf(s - m_new);
        m = m_new;
        ssum += s;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float m_o = __shfl_xor_sync(0xffffffffu, m, o), l_o = __shfl_xor_sync(0xffffffffu, l, o);
        const float m_new = fmaxf(m, m_o);
        l = (l > 0.f ? l * expf(m - m_new) : 0.f) + (l_o > 0.f ? l_o * expf(m_o - m_new) : 0.f);
        m = m_new;
        ssum += __shfl_xor_sync(0xffffffffu, ssum, o);
    }
    if (lane == 0) M[w] = m + logf(l) - ssum / (float)L;
}

bool make_rows_map(CUtensorMap *map, const void *base, const Geom &g, const long long s[3], int box_rows,
                   int swizzle128, int pos[3]);

// dtype: 0 = bf16, 1 = fp32, 2 = bf16 without the tensor cores
cudaError_t launch_exact_measure(int dtype, const Geom &g, const void *Q, const void *K, float *M, cudaStream_t st) {
    if (g.B * g.H == 0) return cudaSuccess;
    const int units = g.B * g.H;
    if (dtype == 0) {
        CUtensorMap tmQ, tmK;
        int pq[3], pk[3];
        if (make_rows_map(&tmQ, Q, g, g.qs, kEmRows, 1, pq) && make_rows_map(&tmK, K, g, g.ks, kEmKeys, 1, pk) &&
            pq[0] == pk[0] && pq[1] == pk[1] && pq[2] == pk[2]) {
            static SmemGrant grant;
            if (cudaError_t e = grant_dynamic_smem(k_exact_measure, grant, kEmSmem)) return e;
            const dim3 grid((unsigned)units, (unsigned)((g.T + kEmRows - 1) / kEmRows));
            k_exact_measure<<<grid, kEmRows, kEmSmem, st>>>(g, pq[0], pq[1], pq[2], M, tmQ, tmK);
            note_launch();
            return cudaGetLastError();
        }
    }
    const long long warps = (long long)units * g.T;
    const unsigned blocks = (unsigned)((warps + 3) / 4);
    if (dtype == 0 || dtype == 2)
        k_exact_measure_simt<__nv_bfloat16><<<blocks, 128, 0, st>>>(g, (const __nv_bfloat16 *)Q, (const __nv_bfloat16 *)K, M);
    else
        k_exact_measure_simt<float><<<blocks, 128, 0, st>>>(g, (const float *)Q, (const float *)K, M);
    note_launch();
    return cudaGetLastError();
}

}  // namespace psattn
