// The projections that precede the attention (Sec. 3.1): Q = X W_q, K = X W_k, V = X W_v, one
// (d_x x 64) matrix per head and role, written straight into the [B][H][T][64] layout (any b/h/t strides)
// that the attention kernels read, so no transpose pass sits between the two.
//
// bf16: ONE persistent tcgen05 GEMM over all three roles.  A tile is 128 tokens of one sequence x 192 output
// columns (three 64-wide head blocks); CTAs walk the tiles round-robin.  Warp 0 streams 64-deep slabs of X and
// of the transposed weights into a 5-stage shared-memory ring by TMA (128-byte swizzle), warp 1 issues
// tcgen05.mma (M = 128, N = 192, K = 16) into one of two TMEM accumulators, warps 2-5 drain the other
// accumulator: TMEM -> registers -> bf16 -> a swizzled staging tile -> whole 128-byte rows at (b, h, t).  The mainloop of tile i + 1 runs
// under the drain of tile i.  Tiles that lie wholly beyond a sequence's length are skipped; rows beyond it
// are not written.  For the V blocks every drain warp also adds up the columns of its 32 rows (as rounded to
// bf16, read back from the staging tile), in a fixed order, from which mean(V) - the fill value of step (e) - follows without
// another pass over V.
// fp32 (and layouts without a tensor map): one thread per output element, fp32 FMA.
#include "psattn_launch.h"
#include "psattn_sm100.cuh"

namespace psattn {

using namespace sm100;

constexpr int kPjM = 128, kPjN = 192, kPjK = 64, kPjStages = 5;
constexpr int kPjAccCols = 256;                                // TMEM columns reserved per accumulator
constexpr uint32_t kPjBytesA = kPjM * kPjK * 2, kPjBytesB = kPjN * kPjK * 2, kPjStage = kPjBytesA + kPjBytesB;
constexpr uint32_t kPjOffBar = kPjStages * kPjStage;           // mbarriers, TMEM slot, abort flag
constexpr uint32_t kPjOffStage = kPjOffBar + 128;              // [4 warps][32 rows][128 B] output staging (swizzled)
constexpr uint32_t kPjSmem = kPjOffStage + 4 * 4096;
constexpr int kPjThreads = 192;

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *m, uint64_t *bar, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
                 : "memory");
}
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *m, uint64_t *bar, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
                 : "memory");
}

struct ProjArgs {
    int B, H, T, dx;                              // H: 64-column blocks per role (the heads of the outputs)
    int n_blocks;                                 // 64-column blocks of all roles together (3 H for Q, K, V)
    int x_heads;                                  // 0: X is [B][T][dx] (3-D tensor map); 1: X is in the attention layout
    int pos_t, pos_h, pos_b;                      //    [B][H_in][T][64] (4-D map, these coordinate slots), dx = H_in * 64
    int tiles_per_seq, n_tiles_n, n_tiles;        // 128-token tiles per sequence, 192-column tiles, all tiles
    long long qs[3], ks[3], vs[3];                // element strides (b, h, t) of the three outputs
    __nv_bfloat16 *Q, *K, *V;
    const int *lengths;
    float *vpart;                                 // [B][tiles_per_seq][4][H][64] column sums of V per 32 rows, or null
    unsigned *status;
};

__device__ __forceinline__ int proj_len(const ProjArgs &a, int b) {
    if (!a.lengths) return a.T;
    int L = a.lengths[b];
    if (L < 0 || L > a.T) {
        atomicOr(a.status, kStatusLenClamped);
        L = L < 0 ? 0 : a.T;
    }
    return L;
}

__global__ void __launch_bounds__(kPjThreads, 1) k_project_qkv(ProjArgs a, const __grid_constant__ CUtensorMap tmX,
                                                               const __grid_constant__ CUtensorMap tmW) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + kPjOffBar), *empty = full + kPjStages;
    uint64_t *acc_full = empty + kPjStages, *acc_empty = acc_full + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if ((smem_u32(smem) & 1023u) != 0u) {                      // swizzled tiles need a 1024-byte base
        if (tid == 0) atomicOr(a.status, kStatusWaitExpired);
        return;
    }
    if (tid == 0) {
        for (int s = 0; s < kPjStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&acc_full[s], 1); mbar_init(&acc_empty[s], 4); }
        *abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmX); tma_prefetch_desc(&tmW);
    }
    __syncwarp();
    // programmatic dependent launch: the next kernel of the stream may be scheduled now (it waits at its own
    // griddepcontrol.wait); nothing in global memory is touched before the previous grid has completed
    // (the trigger comes after this CTA's TMEM allocation: a dependent CTA that allocates TMEM and then waits
    // for this grid must never get the columns a CTA of this grid still needs)
    if (warp == 1) tmem_alloc(tmem_slot, 512);                 // two accumulators, 192 of 256 columns each
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    const int n_kb = (a.dx + kPjK - 1) / kPjK;

    if (warp == 0) {
        // ---- producer: one lane streams the slabs of every tile of this CTA through the ring ----
        if (lane == 0) {
            uint32_t it = 0;
            for (int tile = blockIdx.x; tile < a.n_tiles && !*abort_flag; tile += gridDim.x) {
                const int n = tile % a.n_tiles_n, m = tile / a.n_tiles_n;
                const int b = m / a.tiles_per_seq, tt = m % a.tiles_per_seq;
                if (tt * kPjM >= proj_len(a, b)) continue;
                for (int kb = 0; kb < n_kb; ++kb, ++it) {
                    const uint32_t s = it % kPjStages, ph = (it / kPjStages) & 1u;
                    if (!mbar_wait(&empty[s], ph ^ 1u)) { atomicOr(a.status, kStatusWaitExpired); *abort_flag = 1; break; }
                    uint8_t *sa = smem + s * kPjStage;
                    mbar_expect_tx(&full[s], kPjStage);
                    if (a.x_heads) {                           // slab kb = head kb of the attention layout
                        const int t0 = tt * kPjM;
                        tma_load_4d(sa, &tmX, &full[s], 0, a.pos_t == 1 ? t0 : (a.pos_h == 1 ? kb : b),
                                    a.pos_t == 2 ? t0 : (a.pos_h == 2 ? kb : b), a.pos_t == 3 ? t0 : (a.pos_h == 3 ? kb : b));
                    } else {
                        tma_load_3d(sa, &tmX, &full[s], kb * kPjK, tt * kPjM, b);
                    }
                    tma_load_2d(sa + kPjBytesA, &tmW, &full[s], kb * kPjK, n * kPjN);
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer: one lane; accumulator (tile count & 1) ----
        if (lane == 0) {
            constexpr uint32_t kIdesc = umma_idesc_bf16(kPjM, kPjN, 0);
            uint32_t it = 0, tc = 0;
            for (int tile = blockIdx.x; tile < a.n_tiles && !*abort_flag; tile += gridDim.x) {
                const int m = tile / a.n_tiles_n;
                const int b = m / a.tiles_per_seq, tt = m % a.tiles_per_seq;
                if (tt * kPjM >= proj_len(a, b)) continue;
                const uint32_t acc = tc & 1u, aph = (tc >> 1) & 1u;
                if (!mbar_wait(&acc_empty[acc], aph ^ 1u)) { atomicOr(a.status, kStatusWaitExpired); *abort_flag = 1; break; }
                tc_fence_after();
                bool ok = true;
                for (int kb = 0; kb < n_kb; ++kb, ++it) {
                    const uint32_t s = it % kPjStages, ph = (it / kPjStages) & 1u;
                    if (!mbar_wait(&full[s], ph)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + s * kPjStage), sb = sa + kPjBytesA;
#pragma unroll
                    for (int k = 0; k < kPjK / 16; ++k)
                        umma_bf16(tmem_base + acc * kPjAccCols, umma_desc_sw128(sa + k * 32, 16, 1024),
                                  umma_desc_sw128(sb + k * 32, 16, 1024), kIdesc, (kb | k) != 0);
                    umma_commit(&empty[s]);                    // the stage is free once these products have run
                }
                if (!ok) { atomicOr(a.status, kStatusWaitExpired); *abort_flag = 1; break; }
                umma_commit(&acc_full[acc]);
                ++tc;
            }
        }
    } else {
        // ---- drain: warp w reads TMEM lanes 32 (w % 4) .. + 31; thread = one token row ----
        const int quarter = warp & 3;
        const int ew = warp - 2;                               // 0..3: slot in the staging buffers
        uint4 *stage = reinterpret_cast<uint4 *>(smem + kPjOffStage + ew * 4096);
        uint32_t tc = 0;
        for (int tile = blockIdx.x; tile < a.n_tiles; tile += gridDim.x) {
            const int n = tile % a.n_tiles_n, m = tile / a.n_tiles_n;
            const int b = m / a.tiles_per_seq, tt = m % a.tiles_per_seq;
            const int L = proj_len(a, b);
            if (tt * kPjM >= L) continue;
            const uint32_t acc = tc & 1u, aph = (tc >> 1) & 1u;
            const bool mine = !*abort_flag && mbar_wait(&acc_full[acc], aph);
            uint32_t landed;                                   // the four drain warps decide together (they meet at
            asm volatile(                                      // barrier 1 below, so none may leave alone)
                "{\n\t.reg .pred p, q;\n\t"
                "setp.ne.u32 q, %1, 0;\n\t"
                "bar.red.and.pred p, 1, 128, q;\n\t"
                "selp.u32 %0, 1, 0, p;\n\t}"
                : "=r"(landed)
                : "r"(mine ? 1u : 0u)
                : "memory");
            if (!landed) {
                if (lane == 0) { atomicOr(a.status, kStatusWaitExpired); *abort_flag = 1; }
                break;
            }
            tc_fence_after();
            const int n_cc = min(kPjN / 64, a.n_blocks - n * (kPjN / 64));   // 64-column blocks of this tile
            const uint32_t tacc = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * kPjAccCols;
            uint32_t ra[64], rb[64];                           // two blocks in flight: the next one loads while
            tmem_ld32_issue(tacc, ra);                         // the current one is converted and stored
            tmem_ld32_issue(tacc + 32, ra + 32);
            auto drain_block = [&](uint32_t (&r)[64], int cc) {
                const int gc = n * (kPjN / 64) + cc;           // role = gc / H, head = gc % H
                const int role = gc / a.H, h = gc - role * a.H;
                uint32_t pk[32];                               // 64 bf16, two per word
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    __nv_bfloat162 p2 = __floats2bfloat162_rn(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
                    pk[j] = *reinterpret_cast<uint32_t *>(&p2);
                }
                // through a swizzled staging tile, so that each store instruction of the warp writes four
                // whole 128-byte rows instead of 16 bytes of 32 different rows
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    stage[lane * 8 + (j ^ (lane & 7))] = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
                __syncwarp();
                const long long *st = role == 0 ? a.qs : (role == 1 ? a.ks : a.vs);
                __nv_bfloat16 *base = (role == 0 ? a.Q : (role == 1 ? a.K : a.V)) + (long long)b * st[0] + (long long)h * st[1];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = 4 * i + (lane >> 3), c = lane & 7;
                    const int tr = tt * kPjM + quarter * 32 + rr;
                    const uint4 val = stage[rr * 8 + (c ^ (rr & 7))];
                    if (tr < L) reinterpret_cast<uint4 *>(base + (long long)tr * st[2])[c] = val;
                }
                if (role == 2 && a.vpart != nullptr) {
                    // column sums of this block over the warp's valid rows, from the values as stored (bf16):
                    // lane l adds up word l (columns 2 l and 2 l + 1) of every row of the staging tile
                    const int n_valid = min(32, max(0, L - (tt * kPjM + quarter * 32)));
                    const uint32_t *words = reinterpret_cast<const uint32_t *>(stage);
                    uint32_t wv[32];                           // all loads first: nothing else hides their latency here
#pragma unroll
                    for (int rr = 0; rr < 32; ++rr)
                        wv[rr] = rr < n_valid ? words[rr * 32 + ((((lane >> 2) ^ (rr & 7)) << 2) | (lane & 3))] : 0u;
                    float e0[4] = {0.f, 0.f, 0.f, 0.f}, e1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int rr = 0; rr < 32; ++rr) {          // four independent chains, combined in a fixed order
                        e0[rr & 3] += __uint_as_float(wv[rr] << 16);
                        e1[rr & 3] += __uint_as_float(wv[rr] & 0xffff0000u);
                    }
                    const float s0 = (e0[0] + e0[1]) + (e0[2] + e0[3]), s1 = (e1[0] + e1[1]) + (e1[2] + e1[3]);
                    float2 *dst = reinterpret_cast<float2 *>(
                        a.vpart + ((((long long)b * a.tiles_per_seq + tt) * 4 + quarter) * a.H + h) * 64);
                    dst[lane] = make_float2(s0, s1);
                }
                __syncwarp();
            };
#pragma unroll
            for (int cc = 0; cc < kPjN / 64; cc += 2) {
                if (cc < n_cc) {
                    tmem_ld_wait();
                    tmem_ld_fence32(ra); tmem_ld_fence32(ra + 32);
                    if (cc + 1 < n_cc) { tmem_ld32_issue(tacc + (cc + 1) * 64, rb); tmem_ld32_issue(tacc + (cc + 1) * 64 + 32, rb + 32); }
                    drain_block(ra, cc);
                }
                if (cc + 1 < n_cc) {
                    tmem_ld_wait();
                    tmem_ld_fence32(rb); tmem_ld_fence32(rb + 32);
                    if (cc + 2 < n_cc) { tmem_ld32_issue(tacc + (cc + 2) * 64, ra); tmem_ld32_issue(tacc + (cc + 2) * 64 + 32, ra + 32); }
                    drain_block(rb, cc + 1);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[acc]);
            ++tc;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, 512);
}

// mean(V) of every unit from the partial column sums: eight groups of 64 threads take every eighth partial
// (in order), the eight group sums are then added in order.
__global__ void __launch_bounds__(512) k_project_vbar(ProjArgs a, float *__restrict__ vbar) {
    __shared__ float red[8][64];
    const int unit = blockIdx.x, b = unit / a.H, h = unit % a.H, e = threadIdx.x & 63, grp = threadIdx.x >> 6;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");        // the partial sums of the kernel before
    const int L = proj_len(a, b);
    const int n_part = ((L + kPjM - 1) / kPjM) * 4;            // one partial per 32 rows of every tile in use
    const float *base = a.vpart + ((long long)b * a.tiles_per_seq * 4 * a.H + h) * 64 + e;
    float s = 0.f;
#pragma unroll 4
    for (int p = grp; p < n_part; p += 8) s += base[(long long)p * a.H * 64];
    red[grp][e] = s;
    __syncthreads();
    if (grp == 0) {
        float t = 0.f;
#pragma unroll
        for (int q = 0; q < 8; ++q) t += red[q][e];
        vbar[(long long)unit * 64 + e] = L > 0 ? t / (float)L : 0.f;
    }
}

// Any element type and layout: one thread per output element (64 threads = one head block of one token).
template <typename DT>
__global__ void __launch_bounds__(64) k_project_simt(ProjArgs a, const DT *__restrict__ X, const DT *__restrict__ Wt,
                                                     DT *Q, DT *K, DT *V) {
    const int e = threadIdx.x, gc = blockIdx.y;
    const int b = blockIdx.x / a.T, t = blockIdx.x % a.T;
    if (t >= proj_len(a, b)) return;
    const int role = gc / a.H, h = gc - role * a.H;
    const DT *x = X + ((long long)b * a.T + t) * a.dx;
    const DT *w = Wt + ((long long)gc * 64 + e) * a.dx;
    float acc = 0.f;
    for (int k = 0; k < a.dx; ++k) acc = fmaf((float)x[k], (float)w[k], acc);
    const long long *st = role == 0 ? a.qs : (role == 1 ? a.ks : a.vs);
    DT *base = role == 0 ? Q : (role == 1 ? K : V);
    base[(long long)b * st[0] + (long long)h * st[1] + (long long)t * st[2] + e] = (DT)acc;
}

// mean(V) from the stored V (SIMT path): one block per unit, fixed order over t.
template <typename DT>
__global__ void __launch_bounds__(64) k_project_vbar_simt(ProjArgs a, const DT *__restrict__ V, float *__restrict__ vbar) {
    const int unit = blockIdx.x, b = unit / a.H, h = unit % a.H, e = threadIdx.x;
    const int L = proj_len(a, b);
    const DT *v = V + (long long)b * a.vs[0] + (long long)h * a.vs[1] + e;
    float s = 0.f;
    for (int t = 0; t < L; ++t) s += (float)v[(long long)t * a.vs[2]];
    vbar[(long long)unit * 64 + e] = L > 0 ? s / (float)L : 0.f;
}

typedef CUresult (*EncodeTiledFnP)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);

static EncodeTiledFnP proj_encode_fn() {
    static EncodeTiledFnP fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFnP>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

size_t project_vpart_floats(int B, int H, int T) { return (size_t)B * ((T + kPjM - 1) / kPjM) * 4 * H * 64; }

// dtype 0 = bf16, 1 = fp32.  X [B][T][dx], Wt [3][H*64][dx], outputs with g.qs / g.ks / g.vs strides.
// vbar (optional) fp32 [B][H][64]; vpart = scratch of project_vpart_floats() floats (needed with vbar on the
// tensor-core path).  force_simt keeps bf16 inputs off the tensor cores.
cudaError_t launch_project_qkv(int dtype, int force_simt, const Geom &g, int dx, const void *X, const void *Wt, void *Q,
                               void *K, void *V, float *vbar, float *vpart, cudaStream_t st) {
    if (g.B * g.H == 0) return cudaSuccess;
    ProjArgs a;
    a.B = g.B; a.H = g.H; a.T = g.T; a.dx = dx;
    a.n_blocks = 3 * g.H; a.x_heads = 0; a.pos_t = a.pos_h = a.pos_b = 0;
    a.tiles_per_seq = (g.T + kPjM - 1) / kPjM;
    a.n_tiles_n = (3 * g.H * 64 + kPjN - 1) / kPjN;
    a.n_tiles = g.B * a.tiles_per_seq * a.n_tiles_n;
    for (int k = 0; k < 3; ++k) { a.qs[k] = g.qs[k]; a.ks[k] = g.ks[k]; a.vs[k] = g.vs[k]; }
    a.Q = (__nv_bfloat16 *)Q; a.K = (__nv_bfloat16 *)K; a.V = (__nv_bfloat16 *)V;
    a.lengths = g.lengths; a.status = g.status;
    a.vpart = vbar ? vpart : nullptr;
    EncodeTiledFnP enc = proj_encode_fn();
    if (dtype == 0 && !force_simt && enc && dx % 8 == 0 && (vbar == nullptr || vpart != nullptr)) {
        CUtensorMap tmX, tmW;
        const cuuint64_t xdim[3] = {(cuuint64_t)dx, (cuuint64_t)g.T, (cuuint64_t)g.B};
        const cuuint64_t xstr[2] = {(cuuint64_t)dx * 2, (cuuint64_t)g.T * dx * 2};
        const cuuint32_t xbox[3] = {kPjK, kPjM, 1}, one3[3] = {1, 1, 1};
        const cuuint64_t wdim[2] = {(cuuint64_t)dx, (cuuint64_t)3 * g.H * 64};
        const cuuint64_t wstr[1] = {(cuuint64_t)dx * 2};
        const cuuint32_t wbox[2] = {kPjK, kPjN}, one2[2] = {1, 1};
        const bool ok =
            enc(&tmX, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(X), xdim, xstr, xbox, one3,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS &&
            enc(&tmW, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(Wt), wdim, wstr, wbox, one2,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
        if (ok) {
            static SmemGrant grant;
            if (cudaError_t e = grant_dynamic_smem(k_project_qkv, grant, kPjSmem)) return e;
            // both kernels carry a programmatic dependency on their predecessor in the stream
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)(a.n_tiles < device_sm_count() ? a.n_tiles : device_sm_count()));
            cfg.blockDim = dim3(kPjThreads);
            cfg.dynamicSmemBytes = kPjSmem;
            cfg.stream = st;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            cudaError_t e = cudaLaunchKernelEx(&cfg, k_project_qkv, a, tmX, tmW);
            note_launch();
            if (e == cudaSuccess) e = cudaGetLastError();
            if (e != cudaSuccess || vbar == nullptr) return e;
            cfg.gridDim = dim3((unsigned)(g.B * g.H));
            cfg.blockDim = dim3(512);
            cfg.dynamicSmemBytes = 0;
            e = cudaLaunchKernelEx(&cfg, k_project_vbar, a, vbar);
            note_launch();
            return e != cudaSuccess ? e : cudaGetLastError();
        }
    }
    const dim3 grid((unsigned)(g.B * g.T), (unsigned)(3 * g.H));
    if (dtype == 0) {
        k_project_simt<__nv_bfloat16><<<grid, 64, 0, st>>>(a, (const __nv_bfloat16 *)X, (const __nv_bfloat16 *)Wt,
                                                            (__nv_bfloat16 *)Q, (__nv_bfloat16 *)K, (__nv_bfloat16 *)V);
        note_launch();
        if (vbar) { k_project_vbar_simt<__nv_bfloat16><<<g.B * g.H, 64, 0, st>>>(a, (const __nv_bfloat16 *)V, vbar); note_launch(); }
    } else {
        k_project_simt<float><<<grid, 64, 0, st>>>(a, (const float *)X, (const float *)Wt, (float *)Q, (float *)K, (float *)V);
        note_launch();
        if (vbar) { k_project_vbar_simt<float><<<g.B * g.H, 64, 0, st>>>(a, (const float *)V, vbar); note_launch(); }
    }
    return cudaGetLastError();
}


bool make_rows_map(CUtensorMap *map, const void *base, const Geom &g, const long long s[3], int box_rows,
                   int swizzle128, int pos[3]);

// Dense form of the output matrix of the attention module (see psattn_project_out.cu): Y[b][t][:] =
// sum_h O[b][h][t][:] W_o^h as ONE GEMM on the kernel above, the K dimension running over the heads of the
// attention layout (slab kb = head kb, fetched through a 4-D tensor map of O), the 64-column blocks of Y
// standing where the heads of one role stand for the projections.  bf16, dy a multiple of 64.
// cudaErrorNotSupported: no tensor map for the layout.
cudaError_t launch_project_out_dense(const Geom &g, int dy, const void *O, const void *Wot, void *Y, cudaStream_t st) {
    if (g.B * g.H == 0) return cudaSuccess;
    EncodeTiledFnP enc = proj_encode_fn();
    if (!enc || dy % 64 != 0 || dy < 64) return cudaErrorNotSupported;
    ProjArgs a;
    a.B = g.B; a.H = dy / 64; a.T = g.T; a.dx = g.H * 64;
    a.n_blocks = dy / 64; a.x_heads = 1;
    a.tiles_per_seq = (g.T + kPjM - 1) / kPjM;
    a.n_tiles_n = (dy + kPjN - 1) / kPjN;
    a.n_tiles = g.B * a.tiles_per_seq * a.n_tiles_n;
    // Y [B][T][dy] seen as [B][dy / 64][T][64]: block stride 64, token stride dy
    const long long ys[3] = {(long long)g.T * dy, 64, dy};
    for (int k = 0; k < 3; ++k) { a.qs[k] = ys[k]; a.ks[k] = ys[k]; a.vs[k] = ys[k]; }
    a.Q = (__nv_bfloat16 *)Y; a.K = nullptr; a.V = nullptr;
    a.lengths = g.lengths; a.status = g.status; a.vpart = nullptr;
    CUtensorMap tmX, tmW;
    int pos[3];
    if (!make_rows_map(&tmX, O, g, g.os, kPjM, 1, pos)) return cudaErrorNotSupported;
    a.pos_t = pos[0]; a.pos_h = pos[1]; a.pos_b = pos[2];
    const cuuint64_t wdim[2] = {(cuuint64_t)a.dx, (cuuint64_t)dy};
    const cuuint64_t wstr[1] = {(cuuint64_t)a.dx * 2};
    const cuuint32_t wbox[2] = {kPjK, kPjN}, one2[2] = {1, 1};
    if (enc(&tmW, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(Wot), wdim, wstr, wbox, one2,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorNotSupported;
    static SmemGrant grant;
    if (cudaError_t e = grant_dynamic_smem(k_project_qkv, grant, kPjSmem)) return e;
    const int sms = device_sm_count();
    cudaError_t e = launch_pdl(k_project_qkv, dim3((unsigned)(a.n_tiles < sms ? a.n_tiles : sms)), dim3(kPjThreads), kPjSmem,
                               st, a, tmX, tmW);
    note_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace psattn
