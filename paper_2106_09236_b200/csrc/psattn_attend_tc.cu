// Step (d) on the tensor cores (bf16 inputs): softmax attention (Eq. 7-8) of a list of query
// rows over all valid keys of their unit, flash style.
//
// One CTA = (unit, tile of up to 128 listed rows, key split).  Per 128-key tile:
//   TMA        K tile, V tile  -> shared memory (128-byte swizzle), two stages
//   tcgen05    S = Qsel K^T    -> TMEM (128 lanes = rows, 128 fp32 columns = keys)
//   threads    row r = TMEM lane r: masked online softmax in registers, P (bf16) -> shared memory
//   tcgen05    O_t = P V       -> TMEM (64 columns); V is the MN-major B operand as TMA wrote it
//   threads    acc = acc * alpha + O_t   (fp32 registers, one row per thread)
// With one split the rows are finished here; otherwise (m, l, acc) go to the workspace and the
// split-merge kernel of the staged schedule finishes them.
#include "psattn_launch.h"
#include "psattn_sm100.cuh"

namespace psattn {

using namespace sm100;

constexpr int kTileKeys = 128;
constexpr int kTileRows = 128;
constexpr uint32_t kTileBytes = kTileKeys * kD * 2;          // 16 KB: one K, V or Q tile
constexpr uint32_t kTmemCols = 256;                          // S: [0,128), O_t: [128,192)
constexpr uint32_t kOffQ = 0, kOffK = kTileBytes, kOffV = 3 * kTileBytes, kOffP = 5 * kTileBytes,
                   kOffBar = 7 * kTileBytes;
constexpr uint32_t kAttendSmem = kOffBar + 128;

struct AttendTcArgs {
    const int *rows;            // [unit][rows_stride] listed positions, or null = identity
    int n_rows, rows_stride;
    int n_splits, split_keys;   // split_keys is a multiple of kTileKeys
    float *part_ml, *part_acc;  // split partials (n_splits > 1)
    void *out;                  // finished rows (n_splits == 1)
    long long out_unit_stride, out_row_stride;
    int out_by_position, out_fp32;
    int pos_t, pos_h, pos_b;    // which TMA coordinate (1..3) carries t, h, b
};

__global__ void __launch_bounds__(128, 2) k_attend_tc(Geom g, AttendTcArgs a,
                                                      const __nv_bfloat16 *__restrict__ Q,
                                                      const __grid_constant__ CUtensorMap tmK,
                                                      const __grid_constant__ CUtensorMap tmV) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *full_k = reinterpret_cast<uint64_t *>(smem + kOffBar);        // [2]
    uint64_t *full_v = full_k + 2;                                          // [2]
    uint64_t *mma_s = full_k + 4, *mma_o = full_k + 5;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(full_k + 6);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int tid = threadIdx.x, warp = tid >> 5;
    const int split = blockIdx.x, row_tile = blockIdx.y, unit = blockIdx.z;
    const int b = unit / g.H, h = unit % g.H;
    const int L = seq_len(g, b);
    const int r = row_tile * kTileRows + tid;                  // slot in the row list
    const int lo = min(L, split * a.split_keys), hi = min(L, lo + a.split_keys);
    const int n_tiles = (hi - lo + kTileKeys - 1) / kTileKeys;

    if ((smem_u32(smem) & 1023u) != 0u) {                      // swizzled tiles need a 1024-byte base
        if (tid == 0) atomicOr(g.status, kStatusWaitExpired);
        return;
    }
    if (tid == 0) {
        mbar_init(&full_k[0], 1); mbar_init(&full_k[1], 1);
        mbar_init(&full_v[0], 1); mbar_init(&full_v[1], 1);
        mbar_init(mma_s, 1); mbar_init(mma_o, 1);
        *abort_flag = 0u;
        fence_barrier_init();
        tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
    }
    __syncwarp();
    if (warp == 0) tmem_alloc(tmem_slot, kTmemCols);

    // the listed row of this thread
    int i = -1;
    if (r < a.n_rows) i = a.rows ? a.rows[(long long)unit * a.rows_stride + r] : r;
    const bool row_ok = i >= 0 && i < L;
    {   // Q row -> shared memory, K-major, 128-byte swizzle (16-byte chunk c of row t at c ^ (t & 7))
        uint4 *dst = reinterpret_cast<uint4 *>(smem + kOffQ + tid * 128);
        const uint4 *src = reinterpret_cast<const uint4 *>(Q + unit_off(g.qs, b, h) + (long long)(row_ok ? i : 0) * g.qs[2]);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (row_ok) v = __ldg(src + c);
            dst[c ^ (tid & 7)] = v;
        }
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);

    auto issue_loads = [&](int t) {            // thread 0 only
        const int s = t & 1;
        const int key0 = lo + t * kTileKeys;
        const int c1 = a.pos_t == 1 ? key0 : (a.pos_h == 1 ? h : b);
        const int c2 = a.pos_t == 2 ? key0 : (a.pos_h == 2 ? h : b);
        const int c3 = a.pos_t == 3 ? key0 : (a.pos_h == 3 ? h : b);
        mbar_expect_tx(&full_k[s], kTileBytes);
        tma_load_4d(smem + kOffK + s * kTileBytes, &tmK, &full_k[s], 0, c1, c2, c3);
        mbar_expect_tx(&full_v[s], kTileBytes);
        tma_load_4d(smem + kOffV + s * kTileBytes, &tmV, &full_v[s], 0, c1, c2, c3);
    };
    int loads_issued = 0;
    if (tid == 0) {
        for (; loads_issued < min(2, n_tiles); ++loads_issued) issue_loads(loads_issued);
    }

    constexpr uint32_t kIdescS = umma_idesc_bf16(kTileRows, kTileKeys, 0);   // B = K tile, K-major
    constexpr uint32_t kIdescO = umma_idesc_bf16(kTileRows, kD, 1);          // B = V tile, MN-major
    const float kScaleLog2 = kScale * kLog2e;
    float m_run = -INFINITY, l_run = 0.f;                      // m_run in scaled log2 units
    float acc[kD];
#pragma unroll
    for (int c = 0; c < kD; ++c) acc[c] = 0.f;
    const bool warp_has_rows = (row_tile * kTileRows + warp * 32) < a.n_rows;

    // thread 0: S = Q K^T of key tile t once the tile has landed (the S accumulator must be free)
    auto issue_s = [&](int t) {
        const int s = t & 1;
        if (!mbar_wait(&full_k[s], (uint32_t)((t >> 1) & 1))) { *abort_flag = 1u; atomicOr(g.status, kStatusWaitExpired); return; }
        tc_fence_after();
        const uint32_t qa = smem_u32(smem + kOffQ), ka = smem_u32(smem + kOffK + s * kTileBytes);
#pragma unroll
        for (int k = 0; k < kD / 16; ++k)
            umma_bf16(tmem_base, umma_desc_sw128(qa + k * 32, 16, 1024), umma_desc_sw128(ka + k * 32, 16, 1024),
                      kIdescS, k > 0);
        umma_commit(mma_s);
    };
    if (tid == 0 && n_tiles > 0) issue_s(0);

    for (int t = 0; t < n_tiles; ++t) {
        const int s = t & 1;
        const uint32_t ph_load = (uint32_t)((t >> 1) & 1), ph_mma = (uint32_t)(t & 1);
        __syncwarp();
        if (!*abort_flag && !mbar_wait(mma_s, ph_mma)) { *abort_flag = 1u; atomicOr(g.status, kStatusWaitExpired); }
        tc_fence_after();
        // ---- masked online softmax of this thread's row; P -> shared memory -------------------
        // two passes over the 128 scores in TMEM, 64 at a time with both loads of a half in flight
        const int valid = min(kTileKeys, hi - (lo + t * kTileKeys));     // keys of this tile that exist
        float alpha = 1.f;
        __syncwarp();
        if (warp_has_rows && !*abort_flag) {
            uint32_t sv[2][32];
            float mx = -INFINITY;
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                tmem_ld32_issue(lane_base + hf * 64, sv[0]);
                tmem_ld32_issue(lane_base + hf * 64 + 32, sv[1]);
                tmem_ld_wait();
                tmem_ld_fence32(sv[0]); tmem_ld_fence32(sv[1]);
#pragma unroll
                for (int x = 0; x < 64; ++x)
                    if (hf * 64 + x < valid) mx = fmaxf(mx, __uint_as_float(sv[x >> 5][x & 31]));
            }
            const float m_new = fmaxf(m_run, mx * kScaleLog2);
            alpha = fast_exp2(m_run - m_new);                   // 0 on the first tile
            float lsum = 0.f;
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                tmem_ld32_issue(lane_base + hf * 64, sv[0]);
                tmem_ld32_issue(lane_base + hf * 64 + 32, sv[1]);
                tmem_ld_wait();
                tmem_ld_fence32(sv[0]); tmem_ld_fence32(sv[1]);
                uint8_t *prow = smem + kOffP + hf * kTileBytes + tid * 128;    // panel hf: keys 64 * hf ..
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {                // 8 keys = one 16-byte chunk
                    uint32_t packed[4];
#pragma unroll
                    for (int x = 0; x < 8; x += 2) {
                        const int col = ch * 8 + x;
                        const float s0 = __uint_as_float(sv[col >> 5][col & 31]);
                        const float s1 = __uint_as_float(sv[(col + 1) >> 5][(col + 1) & 31]);
                        const float p0 = (hf * 64 + col < valid) ? fast_exp2(fmaf(s0, kScaleLog2, -m_new)) : 0.f;
                        const float p1 = (hf * 64 + col + 1 < valid) ? fast_exp2(fmaf(s1, kScaleLog2, -m_new)) : 0.f;
                        __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
                        // the weights that multiply V are the rounded ones: sum those for the denominator
                        lsum += __low2float(pk) + __high2float(pk);
                        packed[x >> 1] = *reinterpret_cast<uint32_t *>(&pk);
                    }
                    *reinterpret_cast<uint4 *>(prow + ((ch ^ (tid & 7)) << 4)) =
                        make_uint4(packed[0], packed[1], packed[2], packed[3]);
                }
            }
            l_run = l_run * alpha + lsum;
            m_run = m_new;
        }
        // rows of V past the valid length may hold anything (even NaN): zero them so that 0 * x stays 0
        if (valid < kTileKeys) {                                // uniform over the CTA
            if (!*abort_flag && !mbar_wait(&full_v[s], ph_load)) { *abort_flag = 1u; atomicOr(g.status, kStatusWaitExpired); }
            __syncthreads();
            if (!*abort_flag) {
                uint4 *vrows = reinterpret_cast<uint4 *>(smem + kOffV + s * kTileBytes);
                for (int e = valid * 8 + tid; e < kTileKeys * 8; e += 128) vrows[e] = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();                                        // P is written, everybody has read S
        // ---- O_t = P V, then S of the next tile while the threads add O_t ---------------------
        if (tid == 0 && !*abort_flag) {
            if (!mbar_wait(&full_v[s], ph_load)) { *abort_flag = 1u; atomicOr(g.status, kStatusWaitExpired); }
            else {
                tc_fence_after();
                const uint32_t pa = smem_u32(smem + kOffP), va = smem_u32(smem + kOffV + s * kTileBytes);
#pragma unroll
                for (int k = 0; k < kTileKeys / 16; ++k)
                    umma_bf16(tmem_base + 128,
                              umma_desc_sw128(pa + (k >> 2) * kTileBytes + (k & 3) * 32, 16, 1024),
                              umma_desc_sw128(va + k * 2048, 16, 1024), kIdescO, k > 0);
                umma_commit(mma_o);
                if (t + 1 < n_tiles) issue_s(t + 1);
            }
        }
        __syncwarp();
        if (!*abort_flag && !mbar_wait(mma_o, ph_mma)) { *abort_flag = 1u; atomicOr(g.status, kStatusWaitExpired); }
        tc_fence_after();
        __syncwarp();
        if (warp_has_rows && !*abort_flag) {
            uint32_t ov[2][32];
            tmem_ld32_issue(lane_base + 128, ov[0]);
            tmem_ld32_issue(lane_base + 160, ov[1]);
            tmem_ld_wait();
            tmem_ld_fence32(ov[0]); tmem_ld_fence32(ov[1]);
#pragma unroll
            for (int x = 0; x < 64; ++x) acc[x] = fmaf(acc[x], alpha, __uint_as_float(ov[x >> 5][x & 31]));
        }
        tc_fence_before();
        __syncthreads();                                        // stage s, P and O_t are free again
        if (tid == 0 && !*abort_flag && loads_issued < n_tiles) { issue_loads(loads_issued); ++loads_issued; }
    }

    // ---- results -------------------------------------------------------------------------
    if (r < a.n_rows && !*abort_flag) {
        if (a.n_splits == 1) {
            const float inv = (row_ok && l_run > 0.f) ? 1.f / l_run : 0.f;
            float o[kD];
#pragma unroll
            for (int c = 0; c < kD; ++c) o[c] = row_ok ? acc[c] * inv : 0.f;
            if (a.out_by_position) {
                if (row_ok) {
                    __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(a.out) + unit_off(g.os, b, h) + (long long)i * g.os[2];
#pragma unroll
                    for (int c8 = 0; c8 < 8; ++c8) store8(dst, c8, o + 8 * c8);
                }
            } else if (a.out_fp32) {
                float *dst = reinterpret_cast<float *>(a.out) + (long long)unit * a.out_unit_stride + (long long)r * a.out_row_stride;
#pragma unroll
                for (int c8 = 0; c8 < 8; ++c8) store8(dst, c8, o + 8 * c8);
            } else {
                __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(a.out) + (long long)unit * a.out_unit_stride + (long long)r * a.out_row_stride;
#pragma unroll
                for (int c8 = 0; c8 < 8; ++c8) store8(dst, c8, o + 8 * c8);
            }
        } else {
            const long long slot = ((long long)unit * a.n_rows + r) * a.n_splits + split;
            a.part_ml[2 * slot] = row_ok ? m_run : -INFINITY;
            a.part_ml[2 * slot + 1] = row_ok ? l_run : 0.f;
            float *dst = a.part_acc + slot * kD;
#pragma unroll
            for (int c8 = 0; c8 < 8; ++c8) store8(dst, c8, acc + 8 * c8);
        }
    }
    // ---- teardown: nothing of this CTA may still be in flight when its TMEM is released ---------
    if (tid == 0 && *abort_flag) {
        // loads that were issued but never consumed: give them a bounded chance to land
        for (int t = 0; t < loads_issued; ++t) {
            mbar_wait(&full_k[t & 1], (uint32_t)((t >> 1) & 1));
            mbar_wait(&full_v[t & 1], (uint32_t)((t >> 1) & 1));
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, kTmemCols);
}

// ---- host side -------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

// Tensor map over a [B][H][T][64] bf16 array with arbitrary b/h/t strides: dimensions ordered by
// stride, box = 64 x 128 rows of t, 128-byte swizzle.  pos[] receives the coordinate slot of t, h, b.
static bool make_kv_map(CUtensorMap *map, const void *base, const Geom &g, const long long s[3], int pos[3]) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    struct Dim { long long size, stride; int which; } dims[3] = {
        {g.T, s[2], 0}, {g.H, s[1], 1}, {g.B, s[0], 2}};
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
        if (dims[x].which == 0) box[x + 1] = (cuuint32_t)kTileKeys;
    }
    CUresult rc = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), gdim, gstr, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS;
}

// Returns cudaErrorNotSupported when this kernel cannot take the call (the caller then uses the
// SIMT kernel): non-bf16 handled by the caller; here: tensor map not encodable.
cudaError_t launch_attend_tc(const Geom &g, const void *Q, const void *K, const void *V, const int *rows,
                             int n_rows, int rows_stride, int n_splits, int split_keys, float *part_ml,
                             float *part_acc, void *out, long long out_unit_stride, long long out_row_stride,
                             int out_by_position, int out_fp32, cudaStream_t st) {
    if (g.B * g.H == 0 || n_rows == 0) return cudaSuccess;
    if ((long long)g.B * g.H > 65535 || (n_rows + kTileRows - 1) / kTileRows > 65535) return cudaErrorNotSupported;   // gridDim.z, .y
    AttendTcArgs a;
    a.rows = rows; a.n_rows = n_rows; a.rows_stride = rows_stride;
    a.n_splits = n_splits; a.split_keys = split_keys;
    a.part_ml = part_ml; a.part_acc = part_acc; a.out = out;
    a.out_unit_stride = out_unit_stride; a.out_row_stride = out_row_stride;
    a.out_by_position = out_by_position; a.out_fp32 = out_fp32;
    CUtensorMap tmK, tmV;
    int posK[3], posV[3];
    if (!make_kv_map(&tmK, K, g, g.ks, posK) || !make_kv_map(&tmV, V, g, g.vs, posV)) return cudaErrorNotSupported;
    if (posK[0] != posV[0] || posK[1] != posV[1] || posK[2] != posV[2]) return cudaErrorNotSupported;
    a.pos_t = posK[0]; a.pos_h = posK[1]; a.pos_b = posK[2];
    // two CTAs fit an SM (2 x 113 KB of shared memory, 2 x 256 TMEM columns) and hide each other's waits
    static SmemGrant grant;
    if (cudaError_t e = grant_dynamic_smem(k_attend_tc, grant, kAttendSmem, true)) return e;
    dim3 grid((unsigned)n_splits, (unsigned)((n_rows + kTileRows - 1) / kTileRows), (unsigned)(g.B * g.H));
    k_attend_tc<<<grid, 128, kAttendSmem, st>>>(g, a, (const __nv_bfloat16 *)Q, tmK, tmV);
    note_launch();
    return cudaGetLastError();
}

}  // namespace psattn
