// The whole path (steps a-e) of one (batch, head) unit in one CTA, bf16 inputs, for sequences
// whose keys fit in shared memory.
//
//   1. TMA brings the unit's K rows in once; the measure routine (ldmatrix gather + mma.sync)
//      leaves M~ of every query in shared memory                              (Eq. 11)
//   2. block-wide radix select picks the u queries, in place                  (Sec. 3.2)
//   3. the shared memory of step 1 is reused for the tcgen05 attention of the selected rows
//      over all valid keys; an extra all-ones weight row accumulates the column sums of V on the
//      tensor cores while V streams through, so V is read from HBM once        (Eq. 7-8; Sec. 3.1)
//   4. mean(V) (or the query's own value row) is written to every other valid row of O, zeros
//      to padded rows                                                         (Eq. 12)
// With a given index set (the reuse of one layer's selection by the following layers, Sec. 4.4) steps
// 1 and 2 are skipped and the kernel is steps (d)+(e) in one launch.
// HBM traffic is the algorithmic minimum: Q, K, V read once (K a second time out of L2), O
// written once.  M~ never leaves the SM unless the caller asks for it.
#include "psattn_attend64.cuh"
#include "psattn_launch.h"
#include "psattn_measure_mma.cuh"
#include "psattn_select.cuh"

namespace psattn {

using namespace sm100;

constexpr int kFusedThreads = 512;       // warp 0: control; warps 4-7, 8-11: attention warpgroups; all 16 warps measure

struct FusedArgs {
    uint32_t k_bytes, stage_bytes;       // measure phase: resident keys, one staging buffer
    uint32_t off_persist;                // M~, selection, flags: live through all phases
    int pos_t, pos_h, pos_b;             // TMA coordinate slots (same for the three maps)
    int own_v;                           // fill with the query's own value row instead of mean(V)
    int by_length;                       // CTAs take the sequences in descending order of length
    const int *sel_in;                   // non-null: a given index set [unit][u_max] replaces steps (a)-(c)
};

struct FusedPersist {                    // at smem + off_persist + 4 * T (after the M~ array)
    SelectScratch select;
    int sel[kA64MaxRows];
    float vbar[kD];
    uint64_t bar;
    uint32_t tmem_slot;
};

__global__ void __launch_bounds__(kFusedThreads, 1) k_forward_fused(
    Geom g, FusedArgs a, const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ V,
    const int *__restrict__ sidx, __nv_bfloat16 *__restrict__ O, int *__restrict__ sel_out, float *__restrict__ M_out,
    const __grid_constant__ CUtensorMap tmKrows, const __grid_constant__ CUtensorMap tmK,
    const __grid_constant__ CUtensorMap tmV) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    float *M_s = reinterpret_cast<float *>(smem + a.off_persist);
    unsigned char *chosen = reinterpret_cast<unsigned char *>(M_s + g.T);
    FusedPersist &P = *reinterpret_cast<FusedPersist *>(smem + a.off_persist + ((5 * (size_t)g.T + 127) / 128) * 128);

    if ((smem_u32(smem) & 1023u) != 0u) {                      // swizzled tiles need a 1024-byte base
        if (tid == 0) atomicOr(g.status, kStatusWaitExpired);
        return;
    }
    // Programmatic dependent launch: let the next kernel of the stream be scheduled already (its CTAs
    // wait at their own griddepcontrol.wait until this grid has completed and its writes are visible),
    // and do not touch global memory before the previous grid has completed.  Both are no-ops when the
    // launch carries no programmatic dependency.
    // The trigger comes after this CTA's TMEM allocation (below, behind the barrier that publishes the slot):
    // a dependent CTA allocates TMEM and then waits for this grid, so it must never get columns that a CTA
    // of this grid still needs.
    if (warp == 0) tmem_alloc(&P.tmem_slot, kA64TmemCols);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // Which unit this CTA works on.  With ragged lengths the CTAs take the sequences longest first
    // (CTA x gets the sequence of rank x / H in descending length, ties by position): when there are
    // more units than SMs the long ones start in the first wave and the short ones fill the tail.
    int b = blockIdx.x / g.H;
    const int h = blockIdx.x % g.H;
    if (a.by_length) {
        __shared__ int b_ranked;
        const int rank = b;
        for (int c = tid; c < g.B; c += kFusedThreads) {
            const int lc = min(max(g.lengths[c], 0), g.T);
            int before = 0;
            for (int o = 0; o < g.B; ++o) {
                const int lo = min(max(g.lengths[o], 0), g.T);
                before += (lo > lc) || (lo == lc && o < c);
            }
            if (before == rank) b_ranked = c;
        }
        __syncthreads();
        b = b_ranked;
    }
    const int unit = b * g.H + h;
    const int L = seq_len(g, b);
    const int U = min(g.U_tab[L], g.idx_cols);
    const int u = min(min(g.u_tab[L], g.u_max), L);
    const bool given = a.sel_in != nullptr;                    // steps (d)+(e) only, for a given index set
    if (tid == 32) {
        mbar_init(&P.bar, 1);
        fence_barrier_init();
        if (L > 0 && !given) measure_issue_keys(smem, &P.bar, &tmKrows, L, b, h, a.pos_t, a.pos_h, g.debug_extra_tx);
        tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
    }
    for (int i = tid; i < g.T; i += kFusedThreads) { chosen[i] = 0; if (i >= L) M_s[i] = 0.f; }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = P.tmem_slot;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    phase_stamp(g, 0);

    // ---- steps (a)+(b) ------------------------------------------------------------------------
    bool ok = true;
    if (L > 0 && !given)
        ok = measure_resident<kFusedThreads>(smem, &P.bar, 0u, a.k_bytes, a.stage_bytes, g, unit, b, h, L, U, 0, L, Q,
                                             sidx, M_s);
    __syncthreads();
    phase_stamp(g, 2);                                         // steps (a)+(b) done (stamp 1: the keys had landed)
    if (M_out != nullptr && !given)
        for (int i = tid; i < g.T; i += kFusedThreads) M_out[(long long)unit * g.T + i] = M_s[i];

    // The attention phase reuses the shared memory of the measure phase, which is free now; its first
    // K/V tiles depend only on the unit, so their copies start before the selection and land behind it.
    Attend64Job j;
    j.b = b; j.h = h; j.L = L; j.lo = 0; j.hi = L;
    const int n_rows = given ? g.u_max : u;                    // a given list is taken at its full width
    j.rows = P.sel; j.n_rows = n_rows;
    j.pos_t = a.pos_t; j.pos_h = a.pos_h; j.pos_b = a.pos_b;
    j.ctrl_warp = 0; j.wg_warp0 = 4;
    j.sum_row = a.own_v ? -1 : n_rows;
    j.started = 1;
    if (ok && L > 0 && tid == 0) attend64_start(smem, j, &tmK, &tmV);

    // ---- step (c) -----------------------------------------------------------------------------
    if (!given) {
        block_select([&](int i) { return float_key(M_s[i]); }, L, u, kA64MaxRows, P.sel, P.select);
        for (int r = tid; r < g.u_max; r += kFusedThreads) {
            const int i = r < kA64MaxRows ? P.sel[r] : -1;
            sel_out[(long long)unit * g.u_max + r] = i;
            if (i >= 0) chosen[i] = 1;
        }
    } else {
        for (int r = tid; r < kA64MaxRows; r += kFusedThreads) {
            const int i = r < g.u_max ? a.sel_in[(long long)unit * g.u_max + r] : -1;
            P.sel[r] = (i >= 0 && i < L) ? i : -1;              // entries outside the sequence are ignored
            if (i >= 0 && i < L) chosen[i] = 1;
        }
    }
    __syncthreads();
    phase_stamp(g, 3);                                         // step (c) done

    // ---- step (d), with the column sums of V riding along ------------------------------------------
    if (ok && L > 0) {
        float m_run, l_run, acc[kD];
        ok = attend64_run(smem, tmem_base, g, j, Q, &tmK, &tmV, m_run, l_run, acc);
        if (ok && warp >= 4 && warp < 8 && lane < 16) {
            const int r = 16 * (warp - 4) + lane;
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            if (r < n_rows) {
                const int i = P.sel[r];
                if (i >= 0) {
#pragma unroll
                    for (int c = 0; c < kD; ++c) acc[c] *= inv;
                    __nv_bfloat16 *dst = O + unit_off(g.os, b, h) + (long long)i * g.os[2];
#pragma unroll
                    for (int c8 = 0; c8 < 8; ++c8) store8(dst, c8, acc + 8 * c8);
                }
            } else if (r == j.sum_row) {
#pragma unroll
                for (int c = 0; c < kD; ++c) P.vbar[c] = acc[c] * inv;     // l = number of valid keys
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    phase_stamp(g, 4);                                         // step (d) done

    // ---- step (e) -----------------------------------------------------------------------------
    {
        const int sub = tid & 7, r0 = tid >> 3;
        float fillv[8], zero8[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) { fillv[t] = (L > 0 && !a.own_v && ok) ? P.vbar[sub * 8 + t] : 0.f; zero8[t] = 0.f; }
        __nv_bfloat16 *Ou = O + unit_off(g.os, b, h);
        const __nv_bfloat16 *Vu = V + unit_off(g.vs, b, h);
        for (int i = r0; i < g.T; i += kFusedThreads / 8) {
            __nv_bfloat16 *dst = Ou + (long long)i * g.os[2];
            if (i >= L) store8(dst, sub, zero8);
            else if (chosen[i] && ok) continue;
            else if (a.own_v) { float v[8]; load8(Vu + (long long)i * g.vs[2], sub, v); store8(dst, sub, v); }
            else store8(dst, sub, fillv);
        }
    }
    __syncthreads();
    phase_stamp(g, 5);                                         // step (e) done
    if (warp == 0) tmem_dealloc(tmem_base, kA64TmemCols);
}

bool make_rows_map(CUtensorMap *map, const void *base, const Geom &g, const long long s[3], int box_rows,
                   int swizzle128, int pos[3]);

// cudaErrorNotSupported when the shape does not fit this kernel (the caller runs the staged schedule):
// keys + staging beyond shared memory, more than 63 selected rows or 64 samples, no tensor map.
cudaError_t launch_forward_fused(const Geom &g, int U_max, int own_v, const void *Q, const void *K, const void *V,
                                 const int *sidx, void *O, int *sel, float *M_out, const int *sel_in, cudaStream_t st) {
    if (g.B * g.H == 0) return cudaSuccess;
    if (g.u_max > kA64MaxRows - 1) return cudaErrorNotSupported;
    if (sel_in == nullptr && (U_max > kMeasureMaxU || U_max < 1)) return cudaErrorNotSupported;
    FusedArgs a;
    a.k_bytes = (uint32_t)measure_k_bytes(g.T);
    a.stage_bytes = (uint32_t)measure_stage_bytes(kFusedThreads, g.idx_cols);
    size_t phase = (size_t)a.k_bytes + kMeasureStages * (size_t)a.stage_bytes;
    if (phase < kA64Bytes) phase = kA64Bytes;
    a.off_persist = (uint32_t)((phase + 1023) / 1024 * 1024);
    const size_t smem = a.off_persist + ((5 * (size_t)g.T + 127) / 128) * 128 + sizeof(FusedPersist) + 128;
    if (smem > 227 * 1024) return cudaErrorNotSupported;
    CUtensorMap tmKrows, tmK, tmV;
    int p0[3], p1[3], p2[3];
    if (!make_rows_map(&tmKrows, K, g, g.ks, kMeasureBoxRows, 0, p0) || !make_rows_map(&tmK, K, g, g.ks, 128, 1, p1) ||
        !make_rows_map(&tmV, V, g, g.vs, 128, 1, p2))
        return cudaErrorNotSupported;
    for (int x = 0; x < 3; ++x)
        if (p0[x] != p1[x] || p1[x] != p2[x]) return cudaErrorNotSupported;
    a.pos_t = p0[0]; a.pos_h = p0[1]; a.pos_b = p0[2];
    a.own_v = own_v;
    a.sel_in = sel_in;
    // the ranking costs B comparisons per sequence in every CTA: only where a second wave exists and B is small
    a.by_length = g.lengths != nullptr && g.B * g.H > device_sm_count() && g.B <= 256;
    static SmemGrant grant;
    if (cudaError_t e = grant_dynamic_smem(k_forward_fused, grant, smem)) return e;
    // launched with programmatic stream serialization: the kernel may be scheduled while the previous
    // kernel of the stream drains; it orders itself with griddepcontrol.wait before its first read
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(g.B * g.H));
    cfg.blockDim = dim3(kFusedThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, k_forward_fused, g, a, (const __nv_bfloat16 *)Q, (const __nv_bfloat16 *)V,
                                       sidx, (__nv_bfloat16 *)O, sel, M_out, tmKrows, tmK, tmV);
    note_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace psattn
