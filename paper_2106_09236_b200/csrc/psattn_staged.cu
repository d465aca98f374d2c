// Staged (one kernel per step) schedule of prob-sparse attention: plain SIMT kernels that
// run for any T_max, both element types, and serve the per-step entry points.
//   measure  : steps (a)+(b), Eq. 11           select : step (c), Sec. 3.2
//   colsum   : partial column sums of V        fill   : step (e), Eq. 12 else-branch
//   attend   : step (d), Eq. 7-8, flash-decoding form with one key per lane
#include "psattn_launch.h"
#include "psattn_select.cuh"

#include <atomic>
#include <mutex>

namespace psattn {

// ---------------------------------------------------------------------------------------
// Steps (a)+(b): one warp per query.  The warp is four groups of eight lanes; a group
// reads one sampled key row per step (lane `sub` holds columns 8*sub..8*sub+7 of q and of
// the key), reduces the dot product over its eight lanes and keeps a MeasureState.
// ---------------------------------------------------------------------------------------
template <typename DT>
__global__ void __launch_bounds__(256) k_measure(Geom g, const DT *__restrict__ Q,
                                                 const DT *__restrict__ K,
                                                 const int *__restrict__ sidx,
                                                 float *__restrict__ M) {
    const int lane = threadIdx.x & 31, sub = lane & 7, grp = lane >> 3;
    const long long w = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long long total = (long long)g.B * g.H * g.T;
    if (w >= total) return;
    const int i = (int)(w % g.T);
    const int unit = (int)(w / g.T);
    const int b = unit / g.H, h = unit % g.H;
    const int L = seq_len(g, b);
    if (i >= L) { if (lane == 0) M[w] = 0.f; return; }
    const int U = min(g.U_tab[L], g.idx_cols);

    float q[8];
    load8(Q + unit_off(g.qs, b, h) + (long long)i * g.qs[2], sub, q);
    const DT *Ku = K + unit_off(g.ks, b, h);
    const int *row = sidx + (g.idx_shared ? (g.idx_per_head ? (long long)unit : (long long)b)
                                          : (g.idx_per_head ? (long long)unit : (long long)b) * g.T + i) * g.idx_cols;

    MeasureState st = measure_init();
    for (int base = 0; base < U; base += 32) {
        int my = 0;
        if (base + lane < U) {
            my = __ldg(row + base + lane);
            if (my < 0 || my >= L) { atomicOr(g.status, kStatusIdxClamped); my = my < 0 ? 0 : L - 1; }
        }
        const int steps = (min(32, U - base) + 3) >> 2;
        // four steps (16 sampled keys) at a time, all their row reads in flight together; a lane
        // without a sample reads row 0 (always valid) and its result is dropped
        for (int s0 = 0; s0 < steps; s0 += 4) {
            float kk[4][8], part[4];
            bool active[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int src = (s0 + x) * 4 + grp;
                const int key = __shfl_sync(0xffffffffu, my, src & 31);
                active[x] = s0 + x < steps && base + src < U;
                load8(Ku + (long long)(active[x] ? key : 0) * g.ks[2], sub, kk[x]);
            }
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                part[x] = 0.f;
#pragma unroll
                for (int t = 0; t < 8; ++t) part[x] = fmaf(q[t], kk[x][t], part[x]);
            }
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                part[x] += __shfl_xor_sync(0xffffffffu, part[x], 1);
                part[x] += __shfl_xor_sync(0xffffffffu, part[x], 2);
                part[x] += __shfl_xor_sync(0xffffffffu, part[x], 4);
            }
#pragma unroll
            for (int x = 0; x < 4; ++x)
                if (active[x]) measure_push(st, part[x] * kScale);
        }
    }
#pragma unroll
    for (int o = 8; o <= 16; o <<= 1) {
        MeasureState other;
        other.m = __shfl_xor_sync(0xffffffffu, st.m, o);
        other.D = __shfl_xor_sync(0xffffffffu, st.D, o);
        other.n = __shfl_xor_sync(0xffffffffu, st.n, o);
        // merge in a fixed (lower group first) order so that all lanes agree bit for bit
        st = (lane & o) ? measure_merge(other, st) : measure_merge(st, other);
    }
    if (lane == 0) M[w] = U > 0 ? st.D / (float)U : 0.f;
}

// ---------------------------------------------------------------------------------------
// Column sums of V over blocks of kColsumRows valid rows: part[unit][chunk][64].
// ---------------------------------------------------------------------------------------
template <typename DT>
__global__ void __launch_bounds__(256) k_colsum(Geom g, const DT *__restrict__ V,
                                                float *__restrict__ part, int n_chunks) {
    __shared__ float red[32][kD + 1];
    const int unit = blockIdx.x, chunk = blockIdx.y;
    const int b = unit / g.H, h = unit % g.H;
    pdl_enter();
    KernelSpan span(g, kKernelColsum);
    const int L = seq_len(g, b);
    const int sub = threadIdx.x & 7, r0 = threadIdx.x >> 3;
    const int lo = chunk * kColsumRows, hi = min(L, lo + kColsumRows);
    const DT *Vu = V + unit_off(g.vs, b, h);
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int r = lo + r0; r < hi; r += 32) {
        float v[8];
        load8(Vu + (long long)r * g.vs[2], sub, v);
#pragma unroll
        for (int t = 0; t < 8; ++t) acc[t] += v[t];
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) red[r0][sub * 8 + t] = acc[t];
    __syncthreads();
    if (threadIdx.x < kD) {
        float s = 0.f;
#pragma unroll
        for (int r = 0; r < 32; ++r) s += red[r][threadIdx.x];
        part[((long long)unit * n_chunks + chunk) * kD + threadIdx.x] = s;
    }
}

// ---------------------------------------------------------------------------------------
// Step (c): one block per unit.  Four 8-bit radix passes over order-preserving keys find
// the u-th largest value tau; the result is every position with key > tau plus the first
// (in position order) positions with key == tau, written in ascending position order.
// The same block finishes mean(V) from the column-sum partials.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSelectThreads) k_select(Geom g, const float *__restrict__ M,
                                                           int *__restrict__ sel,
                                                           const float *__restrict__ vpart,
                                                           int n_chunks, float *__restrict__ vbar) {
    __shared__ SelectScratch scratch;
    const int unit = blockIdx.x;
    const int b = unit / g.H;
    pdl_enter();
    KernelSpan span(g, kKernelSelect);
    const int L = seq_len(g, b);
    const int u = min(min(g.u_tab[L], g.u_max), L);
    const float *Mu = M + (long long)unit * g.T;
    int *out = sel + (long long)unit * g.u_max;

    if (vbar != nullptr && threadIdx.x < kD) {
        float s = 0.f;
        for (int c = 0; c < n_chunks; ++c) s += vpart[((long long)unit * n_chunks + c) * kD + threadIdx.x];
        vbar[(long long)unit * kD + threadIdx.x] = L > 0 ? s / (float)L : 0.f;
    }
    if (M == nullptr) return;                  // mean(V) only
    // the routine reads every key several times: keep them in shared memory when they fit
    __shared__ unsigned keys[kSelectSmemKeys];
    if (L <= kSelectSmemKeys) {
        for (int i = threadIdx.x; i < L; i += blockDim.x) keys[i] = float_key(Mu[i]);
        __syncthreads();
        block_select([&](int i) { return keys[i]; }, L, u, g.u_max, out, scratch);
    } else {
        block_select([&](int i) { return float_key(Mu[i]); }, L, u, g.u_max, out, scratch);
    }
}

// ---------------------------------------------------------------------------------------
// Step (c) for few units with long sequences, in two kernels: every unit is cut into `slices` ranges of
// `width` positions; one block per (unit, range) finds the top-u of its range (an element of the unit's
// top-u is also in the top-u of its own range); one small block per unit then picks the top-u among the
// slices * u candidates, which sit in position order, so that the tie rule (equal values: lower position
// first) carries over.  Four times as many SMs work on the long scan, and each block's scan is short.
// ---------------------------------------------------------------------------------------
constexpr int kSelectMaxSlices = 8;

__global__ void __launch_bounds__(kSelectThreads) k_select_slice(Geom g, const float *__restrict__ M, int slices,
                                                                 int width, int *__restrict__ cand) {
    __shared__ SelectScratch scratch;
    __shared__ unsigned keys[kSelectSmemKeys];
    const int unit = blockIdx.x / slices, sl = blockIdx.x % slices;
    const int b = unit / g.H;
    pdl_enter();
    KernelSpan span(g, kKernelSelectSlice);
    const int L = seq_len(g, b);
    const int u = min(min(g.u_tab[L], g.u_max), L);
    const int lo = sl * width, n = max(0, min(L - lo, width));
    const float *Mu = M + (long long)unit * g.T + lo;
    int *out = cand + ((long long)unit * slices + sl) * g.u_max;
    for (int i = threadIdx.x; i < n; i += blockDim.x) keys[i] = float_key(Mu[i]);
    __syncthreads();
    block_select([&](int i) { return keys[i]; }, n, min(u, n), g.u_max, out, scratch);
    for (int r = threadIdx.x; r < g.u_max; r += blockDim.x) {       // positions within the range -> positions of the unit
        const int p = out[r];
        if (p >= 0) out[r] = p + lo;
    }
}

__global__ void __launch_bounds__(256) k_select_merge(Geom g, const float *__restrict__ M, int slices,
                                                      const int *__restrict__ cand, int *__restrict__ sel) {
    __shared__ SelectScratch scratch;
    __shared__ unsigned ckey[kSelectMaxSlices * 64];
    __shared__ int cidx[kSelectMaxSlices * 64];
    const int unit = blockIdx.x;
    const int b = unit / g.H;
    pdl_enter();
    KernelSpan span(g, kKernelSelectMerge);
    const int L = seq_len(g, b);
    const int u = min(min(g.u_tab[L], g.u_max), L);
    const int n = slices * g.u_max;                            // candidate slots, -1 padded per range
    const float *Mu = M + (long long)unit * g.T;
    for (int p = threadIdx.x; p < n; p += blockDim.x) {
        const int i = cand[(long long)unit * n + p];
        cidx[p] = i;
        ckey[p] = i >= 0 ? float_key(Mu[i]) : 0u;              // 0 lies below the key of every float
    }
    __syncthreads();
    int *out = sel + (long long)unit * g.u_max;
    block_select([&](int p) { return ckey[p]; }, n, u, g.u_max, out, scratch);
    for (int r = threadIdx.x; r < g.u_max; r += blockDim.x) {
        const int p = out[r];
        if (p >= 0) out[r] = cidx[p];
    }
}

// ---------------------------------------------------------------------------------------
// Step (d), SIMT form: one warp per (unit, listed row, key split).  Lane l owns keys
// lo + l, lo + l + 32, ... and keeps its own online-softmax state (m, l, acc[64]) in base-2
// exponent form; the 32 states are merged at the end.  With one split the row is finished
// here; otherwise (m, l, acc) goes to the workspace for k_attend_combine.
// ---------------------------------------------------------------------------------------
template <typename DT>
__device__ __forceinline__ void load_row64(const DT *row, float out[kD]) {
#pragma unroll
    for (int s = 0; s < 8; ++s) load8(row, s, out + 8 * s);
}

template <typename DT, typename OT>
__global__ void __launch_bounds__(128) k_attend(Geom g, const DT *__restrict__ Q,
                                                const DT *__restrict__ K,
                                                const DT *__restrict__ V,
                                                const int *__restrict__ rows, int n_rows,
                                                int rows_stride, int n_splits, int split_keys,
                                                float *__restrict__ part_ml,
                                                float *__restrict__ part_acc,
                                                OT *__restrict__ out, long long out_unit_stride,
                                                long long out_row_stride, int out_by_position) {
    const int lane = threadIdx.x & 31;
    const long long w = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long long total = (long long)g.B * g.H * n_rows * n_splits;
    if (w >= total) return;
    const int split = (int)(w % n_splits);
    const int r = (int)((w / n_splits) % n_rows);
    const int unit = (int)(w / ((long long)n_splits * n_rows));
    const int b = unit / g.H, h = unit % g.H;
    const int L = seq_len(g, b);
    const int i = rows ? rows[(long long)unit * rows_stride + r] : r;
    const bool row_ok = i >= 0 && i < L;
    // where the finished row goes: at its position i of O, or at its slot r of a row-list output
    OT *dst = nullptr;
    // (with the identity list every position is a row: the padded ones get their zero rows here)
    if (out_by_position) { if (row_ok || (rows == nullptr && i < g.T)) dst = out + unit_off(g.os, b, h) + (long long)i * g.os[2]; }
    else dst = out + (long long)unit * out_unit_stride + (long long)r * out_row_stride;

    float m = -INFINITY, l = 0.f;
    float acc[kD];
#pragma unroll
    for (int c = 0; c < kD; ++c) acc[c] = 0.f;
    if (row_ok) {
        float q[kD];
        load_row64(Q + unit_off(g.qs, b, h) + (long long)i * g.qs[2], q);
        const DT *Ku = K + unit_off(g.ks, b, h);
        const DT *Vu = V + unit_off(g.vs, b, h);
        const int lo = split * split_keys, hi = min(L, lo + split_keys);
        for (int j = lo + lane; j < hi; j += 32) {
            float x[kD];
            load_row64(Ku + (long long)j * g.ks[2], x);
            float s = 0.f;
#pragma unroll
            for (int c = 0; c < kD; ++c) s = fmaf(q[c], x[c], s);
            s *= kScale * kLog2e;
            if (s > m) {
                const float f = exp2f(m - s);          // 0 on the first key (m = -inf)
                l *= f;
#pragma unroll
                for (int c = 0; c < kD; ++c) acc[c] *= f;
                m = s;
            }
            const float p = exp2f(s - m);
            l += p;
            load_row64(Vu + (long long)j * g.vs[2], x);
#pragma unroll
            for (int c = 0; c < kD; ++c) acc[c] = fmaf(p, x[c], acc[c]);
        }
    }
    // merge the 32 lane states
    float mw = m;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mw = fmaxf(mw, __shfl_xor_sync(0xffffffffu, mw, o));
    const float f = (l > 0.f) ? exp2f(m - mw) : 0.f;
    float lw = l * f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) lw += __shfl_xor_sync(0xffffffffu, lw, o);
    float mine[2] = {0.f, 0.f};
#pragma unroll
    for (int c = 0; c < kD; ++c) {
        float v = acc[c] * f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == (c & 31)) mine[c >> 5] = v;
    }
    if (n_splits == 1) {
        if (dst) {
            const float inv = lw > 0.f ? 1.f / lw : 0.f;
            dst[lane] = (OT)(mine[0] * inv);
            dst[lane + 32] = (OT)(mine[1] * inv);
        }
    } else {
        const long long slot = ((long long)unit * n_rows + r) * n_splits + split;
        if (lane == 0) { part_ml[2 * slot] = mw; part_ml[2 * slot + 1] = lw; }
        part_acc[slot * kD + lane] = mine[0];
        part_acc[slot * kD + lane + 32] = mine[1];
    }
}

// Merge of the key splits of one row: 64 threads per row.
template <typename OT>
__global__ void __launch_bounds__(256) k_attend_combine(Geom g, const int *__restrict__ rows,
                                                        int n_rows, int rows_stride, int n_splits,
                                                        const float *__restrict__ part_ml,
                                                        const float *__restrict__ part_acc,
                                                        OT *__restrict__ out,
                                                        long long out_unit_stride,
                                                        long long out_row_stride,
                                                        int out_by_position, float *__restrict__ vbar) {
    const int n_slots = n_rows + (vbar ? 1 : 0);           // slot n_rows (if any) is the all-ones row
    pdl_enter();
    KernelSpan span(g, kKernelCombine);
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long rowid = t / kD;
    const int c = (int)(t % kD);
    if (rowid >= (long long)g.B * g.H * n_slots) return;
    const int r = (int)(rowid % n_slots);
    const int unit = (int)(rowid / n_slots);
    const int b = unit / g.H, h = unit % g.H;
    const int L = seq_len(g, b);
    if (r == n_rows) {                                     // mean(V) = merged column sums / merged key count
        float lw = 0.f, a = 0.f;
        for (int s = 0; s < n_splits; ++s) {
            lw += part_ml[2 * (rowid * n_splits + s) + 1];
            a += part_acc[(rowid * n_splits + s) * kD + c];
        }
        vbar[(long long)unit * kD + c] = lw > 0.f ? a / lw : 0.f;
        return;
    }
    const int i = rows ? rows[(long long)unit * rows_stride + r] : r;
    const bool row_ok = i >= 0 && i < L;
    OT *dst;
    if (out_by_position) {
        if (!row_ok && !(rows == nullptr && i < g.T)) return;   // identity list: padded positions get zero rows
        dst = out + unit_off(g.os, b, h) + (long long)i * g.os[2];
    } else {
        dst = out + (long long)unit * out_unit_stride + (long long)r * out_row_stride;
    }
    const long long slot0 = rowid * n_splits;
    float mw = -INFINITY;
    for (int s = 0; s < n_splits; ++s) mw = fmaxf(mw, part_ml[2 * (slot0 + s)]);
    float lw = 0.f, a = 0.f;
    for (int s = 0; s < n_splits; ++s) {
        const float ls = part_ml[2 * (slot0 + s) + 1];
        const float f = ls > 0.f ? exp2f(part_ml[2 * (slot0 + s)] - mw) : 0.f;
        lw += ls * f;
        a += part_acc[(slot0 + s) * kD + c] * f;
    }
    dst[c] = (OT)(lw > 0.f ? a / lw : 0.f);
}

// ---------------------------------------------------------------------------------------
// Step (e): every valid, non-selected row of O receives mean(V) (or its own value row);
// padded rows receive zeros; selected rows are left to step (d).  One block covers
// kFillRows rows of one unit.
// ---------------------------------------------------------------------------------------
template <typename DT>
__global__ void __launch_bounds__(256) k_fill(Geom g, const DT *__restrict__ V,
                                              const int *__restrict__ sel,
                                              const float *__restrict__ vbar, DT *__restrict__ O,
                                              int own_v) {
    __shared__ unsigned char chosen[kFillRows];
    const int unit = blockIdx.x;
    const int b = unit / g.H, h = unit % g.H;
    pdl_enter();
    KernelSpan span(g, kKernelFill);
    const int L = seq_len(g, b);
    const int lo = blockIdx.y * kFillRows;
    for (int t = threadIdx.x; t < kFillRows; t += blockDim.x) chosen[t] = 0;
    __syncthreads();
    if (sel != nullptr)                                    // no list: every valid row is filled
        for (int r = threadIdx.x; r < g.u_max; r += blockDim.x) {
            const int i = sel[(long long)unit * g.u_max + r];
            if (i >= lo && i < lo + kFillRows && i < L) chosen[i - lo] = 1;
        }
    __syncthreads();
    const int sub = threadIdx.x & 7, r0 = threadIdx.x >> 3;
    float mean8[8], zero8[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) { mean8[t] = vbar[(long long)unit * kD + sub * 8 + t]; zero8[t] = 0.f; }
    DT *Ou = O + unit_off(g.os, b, h);
    const DT *Vu = V + unit_off(g.vs, b, h);
    const int hi = min(g.T, lo + kFillRows);
    for (int i = lo + r0; i < hi; i += 32) {
        DT *dst = Ou + (long long)i * g.os[2];
        if (i >= L) store8(dst, sub, zero8);
        else if (chosen[i - lo]) continue;
        else if (own_v) { float v[8]; load8(Vu + (long long)i * g.vs[2], sub, v); store8(dst, sub, v); }
        else store8(dst, sub, mean8);
    }
}

// ---------------------------------------------------------------------------------------
// Host-side launchers
// ---------------------------------------------------------------------------------------
static std::atomic<unsigned long long> g_launches{0};
int device_sm_count() {
    static std::atomic<int> cached[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 1; }
    const bool slot = dev >= 0 && dev < kMaxDevices;
    int n = slot ? cached[dev].load(std::memory_order_relaxed) : 0;
    if (n <= 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) { cudaGetLastError(); n = 1; }
        if (slot) cached[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

cudaError_t grant_dynamic_smem_impl(const void *kernel, SmemGrant &rec, size_t smem, bool carveout) {
    static std::mutex mu;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const bool slot = dev >= 0 && dev < kMaxDevices;
    std::lock_guard<std::mutex> lock(mu);
    if (slot && rec.bytes[dev] >= smem) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess && carveout)
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    if (slot) rec.bytes[dev] = smem;
    return cudaSuccess;
}

void note_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }
unsigned long long launches_so_far() { return g_launches.load(std::memory_order_relaxed); }

template <typename DT>
static cudaError_t launch_measure_t(const Geom &g, const void *Q, const void *K, const int *sidx,
                                    float *M, cudaStream_t st) {
    const long long total = (long long)g.B * g.H * g.T;
    if (total == 0) return cudaSuccess;
    const unsigned blocks = (unsigned)((total + 7) / 8);
    k_measure<DT><<<blocks, 256, 0, st>>>(g, (const DT *)Q, (const DT *)K, sidx, M); note_launch();
    return cudaGetLastError();
}
cudaError_t launch_measure(int dtype, const Geom &g, const void *Q, const void *K, const int *sidx,
                           float *M, cudaStream_t st) {
    return dtype == 0 ? launch_measure_t<__nv_bfloat16>(g, Q, K, sidx, M, st)
                      : launch_measure_t<float>(g, Q, K, sidx, M, st);
}

cudaError_t launch_colsum(int dtype, const Geom &g, const void *V, float *part, int n_chunks,
                          cudaStream_t st) {
    if (g.B * g.H == 0 || n_chunks == 0) return cudaSuccess;
    dim3 grid((unsigned)(g.B * g.H), (unsigned)n_chunks);
    cudaError_t e;
    if (dtype == 0) e = launch_pdl(k_colsum<__nv_bfloat16>, grid, dim3(256), 0, st, g, (const __nv_bfloat16 *)V, part, n_chunks);
    else e = launch_pdl(k_colsum<float>, grid, dim3(256), 0, st, g, (const float *)V, part, n_chunks);
    if (e != cudaSuccess) return e;
    note_launch();
    return cudaGetLastError();
}

size_t select_cand_ints(int units, int u_max) { return (size_t)units * kSelectMaxSlices * u_max; }

cudaError_t launch_select(const Geom &g, const float *M, int *sel, const float *vpart, int n_chunks,
                          float *vbar, int *cand, cudaStream_t st) {
    if (g.B * g.H == 0) return cudaSuccess;
    const int units = g.B * g.H;
    int slices = device_sm_count() / units;
    if (slices > kSelectMaxSlices) slices = kSelectMaxSlices;
    if (M != nullptr && vbar == nullptr && cand != nullptr && slices >= 2 && g.u_max <= 64 && g.T / slices >= 1024) {
        const int width = (g.T + slices - 1) / slices;
        if (width <= kSelectSmemKeys) {
            cudaError_t e = launch_pdl(k_select_slice, dim3((unsigned)(units * slices)), dim3(kSelectThreads), 0, st, g, M,
                                       slices, width, cand);
            note_launch();
            if (e != cudaSuccess) return e;
            e = launch_pdl(k_select_merge, dim3((unsigned)units), dim3(256), 0, st, g, M, slices, (const int *)cand, sel);
            note_launch();
            return e != cudaSuccess ? e : cudaGetLastError();
        }
    }
    cudaError_t e = launch_pdl(k_select, dim3((unsigned)(g.B * g.H)), dim3(kSelectThreads), 0, st, g, M, sel, vpart, n_chunks, vbar);
    note_launch();
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

template <typename DT, typename OT>
static cudaError_t launch_attend_t(const Geom &g, const void *Q, const void *K, const void *V,
                                   const int *rows, int n_rows, int rows_stride, int n_splits,
                                   int split_keys, float *part_ml, float *part_acc, void *out,
                                   long long ous, long long ors, int by_pos, cudaStream_t st) {
    const long long warps = (long long)g.B * g.H * n_rows * n_splits;
    if (warps == 0) return cudaSuccess;
    k_attend<DT, OT><<<(unsigned)((warps + 3) / 4), 128, 0, st>>>(
        g, (const DT *)Q, (const DT *)K, (const DT *)V, rows, n_rows, rows_stride, n_splits,
        split_keys, part_ml, part_acc, (OT *)out, ous, ors, by_pos); note_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || n_splits == 1) return e;
    const long long threads = (long long)g.B * g.H * n_rows * kD;
    k_attend_combine<OT><<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(
        g, rows, n_rows, rows_stride, n_splits, part_ml, part_acc, (OT *)out, ous, ors, by_pos, nullptr); note_launch();
    return cudaGetLastError();
}

cudaError_t launch_attend_simt(int dtype, int out_fp32, const Geom &g, const void *Q, const void *K,
                               const void *V, const int *rows, int n_rows, int rows_stride,
                               int n_splits, int split_keys, float *part_ml, float *part_acc,
                               void *out, long long out_unit_stride, long long out_row_stride,
                               int out_by_position, cudaStream_t st) {
#define PSATTN_ATT(DT, OT)                                                                      \
    launch_attend_t<DT, OT>(g, Q, K, V, rows, n_rows, rows_stride, n_splits, split_keys, part_ml, \
                            part_acc, out, out_unit_stride, out_row_stride, out_by_position, st)
    if (dtype == 0) return out_fp32 ? PSATTN_ATT(__nv_bfloat16, float) : PSATTN_ATT(__nv_bfloat16, __nv_bfloat16);
    return PSATTN_ATT(float, float);
#undef PSATTN_ATT
}

cudaError_t merge_attend_splits(int out_is_bf16, const Geom &g, const int *rows, int n_rows, int rows_stride,
                                int n_splits, const float *part_ml, const float *part_acc, void *out,
                                long long out_unit_stride, long long out_row_stride, int out_by_position,
                                float *vbar, cudaStream_t st) {
    const long long threads = (long long)g.B * g.H * (n_rows + (vbar ? 1 : 0)) * kD;
    if (threads == 0) return cudaSuccess;
    const unsigned blocks = (unsigned)((threads + 255) / 256);
    cudaError_t e;
    if (out_is_bf16)
        e = launch_pdl(k_attend_combine<__nv_bfloat16>, dim3(blocks), dim3(256), 0, st, g, rows, n_rows, rows_stride,
                       n_splits, part_ml, part_acc, (__nv_bfloat16 *)out, out_unit_stride, out_row_stride,
                       out_by_position, vbar);
    else
        e = launch_pdl(k_attend_combine<float>, dim3(blocks), dim3(256), 0, st, g, rows, n_rows, rows_stride, n_splits,
                       part_ml, part_acc, (float *)out, out_unit_stride, out_row_stride, out_by_position, vbar);
    note_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_fill(int dtype, const Geom &g, const void *V, const int *sel, const float *vbar,
                        void *O, int own_v, cudaStream_t st) {
    if (g.B * g.H == 0 || g.T == 0) return cudaSuccess;
    dim3 grid((unsigned)(g.B * g.H), (unsigned)((g.T + kFillRows - 1) / kFillRows));
    cudaError_t e;
    if (dtype == 0)
        e = launch_pdl(k_fill<__nv_bfloat16>, grid, dim3(256), 0, st, g, (const __nv_bfloat16 *)V, sel, vbar,
                       (__nv_bfloat16 *)O, own_v);
    else
        e = launch_pdl(k_fill<float>, grid, dim3(256), 0, st, g, (const float *)V, sel, vbar, (float *)O, own_v);
    note_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace psattn
