// Stand-alone kernel around attend64_run: step (d) for row lists of at most 64 rows per unit
// (the selected queries of the sparse path).  One CTA = (unit, key split).
#include "psattn_attend64.cuh"
#include "psattn_launch.h"

namespace psattn {

using namespace sm100;

struct Attend64Args {
    const int *rows;            // [unit][rows_stride]
    int n_rows, rows_stride;
    int n_splits, split_keys;   // split_keys is a multiple of 256
    float *part_ml, *part_acc;
    void *out;
    long long out_unit_stride, out_row_stride;
    int out_by_position, out_fp32;
    int pos_t, pos_h, pos_b;
    float *vbar;                // if non-null: mean(V) [unit][64], from an extra all-weights-1 row (slot n_rows)
};

constexpr int kA64Threads = 384;        // warp 0: control, warps 4-7 and 8-11: the two warpgroups

__global__ void __launch_bounds__(kA64Threads, 1) k_attend64(Geom g, Attend64Args a,
                                                             const __nv_bfloat16 *__restrict__ Q,
                                                             const __grid_constant__ CUtensorMap tmK,
                                                             const __grid_constant__ CUtensorMap tmV) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint32_t *tmem_slot_p = reinterpret_cast<uint32_t *>(smem + kA64OffBar + 120);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int split = blockIdx.x, unit = blockIdx.y;
    if ((smem_u32(smem) & 1023u) != 0u) {                      // swizzled tiles need a 1024-byte base
        if (tid == 0) atomicOr(g.status, kStatusWaitExpired);
        return;
    }
    if (warp == 0) tmem_alloc(tmem_slot_p, kA64TmemCols);
    if (tid == 32) { tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_p;
    // Programmatic dependent launch (see pdl_enter), only now that this CTA holds its TMEM: a dependent CTA
    // that starts early allocates TMEM too and then sits in its griddepcontrol.wait; if it could take the
    // columns before a CTA of this grid had allocated, that CTA would block in tcgen05.alloc for good.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");                // nothing above touches global data
    KernelSpan span(g, kKernelAttend64);

    Attend64Job j;
    j.b = unit / g.H; j.h = unit % g.H; j.L = seq_len(g, j.b);
    j.lo = min(j.L, split * a.split_keys); j.hi = min(j.L, j.lo + a.split_keys);
    j.rows = a.rows + (long long)unit * a.rows_stride; j.n_rows = a.n_rows;
    j.pos_t = a.pos_t; j.pos_h = a.pos_h; j.pos_b = a.pos_b;
    j.ctrl_warp = 0; j.wg_warp0 = 4; j.sum_row = a.vbar ? a.n_rows : -1; j.started = 0;
    float m_run, l_run, acc[kD];
    const bool ok = attend64_run(smem, tmem_base, g, j, Q, &tmK, &tmV, m_run, l_run, acc);

    if (ok && warp >= 4 && warp < 8 && lane < 16) {
        const int r = 16 * (warp - 4) + lane;
        const int n_slots = a.n_rows + (a.vbar ? 1 : 0);           // row slots per unit in the split partials
        if (r < a.n_rows) {
            const int i = j.rows[r];
            const bool row_ok = i >= 0 && i < j.L;
            if (a.n_splits == 1) {
                const float inv = (row_ok && l_run > 0.f) ? 1.f / l_run : 0.f;
#pragma unroll
                for (int c = 0; c < kD; ++c) acc[c] = row_ok ? acc[c] * inv : 0.f;
                if (a.out_by_position) {
                    if (row_ok) {
                        __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(a.out) + unit_off(g.os, j.b, j.h) + (long long)i * g.os[2];
#pragma unroll
                        for (int c8 = 0; c8 < 8; ++c8) store8(dst, c8, acc + 8 * c8);
                    }
                } else if (a.out_fp32) {
                    float *dst = reinterpret_cast<float *>(a.out) + (long long)unit * a.out_unit_stride + (long long)r * a.out_row_stride;
#pragma unroll
                    for (int c8 = 0; c8 < 8; ++c8) store8(dst, c8, acc + 8 * c8);
                } else {
                    __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(a.out) + (long long)unit * a.out_unit_stride + (long long)r * a.out_row_stride;
#pragma unroll
                    for (int c8 = 0; c8 < 8; ++c8) store8(dst, c8, acc + 8 * c8);
                }
            } else {
                const long long slot = ((long long)unit * n_slots + r) * a.n_splits + split;
                a.part_ml[2 * slot] = row_ok ? m_run : -INFINITY;
                a.part_ml[2 * slot + 1] = row_ok ? l_run : 0.f;
                float *dst = a.part_acc + slot * kD;
#pragma unroll
                for (int c8 = 0; c8 < 8; ++c8) store8(dst, c8, acc + 8 * c8);
            }
        } else if (r == j.sum_row) {                             // column sums of V over [lo, hi), l = key count
            if (a.n_splits == 1) {
                const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
#pragma unroll
                for (int c = 0; c < kD; ++c) acc[c] *= inv;
                float *dst = a.vbar + (long long)unit * kD;
#pragma unroll
                for (int c8 = 0; c8 < 8; ++c8) store8(dst, c8, acc + 8 * c8);
            } else {
                const long long slot = ((long long)unit * n_slots + r) * a.n_splits + split;
                a.part_ml[2 * slot] = l_run > 0.f ? m_run : -INFINITY;
                a.part_ml[2 * slot + 1] = l_run;
                float *dst = a.part_acc + slot * kD;
#pragma unroll
                for (int c8 = 0; c8 < 8; ++c8) store8(dst, c8, acc + 8 * c8);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, kA64TmemCols);
}

bool make_rows_map(CUtensorMap *map, const void *base, const Geom &g, const long long s[3], int box_rows,
                   int swizzle128, int pos[3]);

// Host-side check with no side effect: would launch_attend64 take this call?
bool attend64_supported(const Geom &g, const void *K, const void *V, int n_rows, int with_vbar) {
    if (n_rows + (with_vbar ? 1 : 0) > kA64MaxRows) return false;
    CUtensorMap tmK, tmV;
    int posK[3], posV[3];
    if (!make_rows_map(&tmK, K, g, g.ks, 128, 1, posK) || !make_rows_map(&tmV, V, g, g.vs, 128, 1, posV)) return false;
    return posK[0] == posV[0] && posK[1] == posV[1] && posK[2] == posV[2];
}

// cudaErrorNotSupported: more than 64 rows (63 with vbar), no row list, or no tensor map for the layout.
cudaError_t launch_attend64(const Geom &g, const void *Q, const void *K, const void *V, const int *rows,
                            int n_rows, int rows_stride, int n_splits, int split_keys, float *part_ml,
                            float *part_acc, void *out, long long out_unit_stride, long long out_row_stride,
                            int out_by_position, int out_fp32, float *vbar, cudaStream_t st) {
    if (g.B * g.H == 0 || n_rows == 0) return cudaSuccess;
    if (n_rows + (vbar ? 1 : 0) > kA64MaxRows || rows == nullptr || (split_keys % 256) != 0) return cudaErrorNotSupported;
    if ((long long)g.B * g.H > 65535) return cudaErrorNotSupported;         // the unit index is gridDim.y
    Attend64Args a;
    a.rows = rows; a.n_rows = n_rows; a.rows_stride = rows_stride;
    a.n_splits = n_splits; a.split_keys = split_keys;
    a.part_ml = part_ml; a.part_acc = part_acc; a.out = out;
    a.out_unit_stride = out_unit_stride; a.out_row_stride = out_row_stride;
    a.out_by_position = out_by_position; a.out_fp32 = out_fp32; a.vbar = vbar;
    CUtensorMap tmK, tmV;
    int posK[3], posV[3];
    if (!make_rows_map(&tmK, K, g, g.ks, 128, 1, posK) || !make_rows_map(&tmV, V, g, g.vs, 128, 1, posV))
        return cudaErrorNotSupported;
    if (posK[0] != posV[0] || posK[1] != posV[1] || posK[2] != posV[2]) return cudaErrorNotSupported;
    a.pos_t = posK[0]; a.pos_h = posK[1]; a.pos_b = posK[2];
    static SmemGrant grant;
    if (cudaError_t e = grant_dynamic_smem(k_attend64, grant, kA64Bytes)) return e;
    dim3 grid((unsigned)n_splits, (unsigned)(g.B * g.H));
    cudaError_t le = launch_pdl(k_attend64, grid, dim3(kA64Threads), kA64Bytes, st, g, a, (const __nv_bfloat16 *)Q, tmK, tmV);
    if (le != cudaSuccess) { note_launch(); return le; }
    note_launch();
    return cudaGetLastError();
}

}  // namespace psattn
