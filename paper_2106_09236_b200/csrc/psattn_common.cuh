// Shared device-side definitions of the prob-sparse attention kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace psattn {

constexpr int kD = 64;                    // d_head, fixed (Sec. 4.2: d_model / heads = 64)
constexpr float kScale = 0.125f;          // 1 / sqrt(64), exact
constexpr float kLog2e = 1.4426950408889634f;

constexpr unsigned kStatusIdxClamped = 1u;
constexpr unsigned kStatusLenClamped = 2u;
constexpr unsigned kStatusWaitExpired = 4u;

// Geometry of one call, passed by value to every kernel.
struct Geom {
    int B, H, T;                          // T = T_max
    int idx_cols, idx_per_head;
    int idx_shared;                       // one sample row per sequence (or unit) instead of one per query
    int u_max;
    long long qs[3], ks[3], vs[3], os[3]; // element strides of the b, h, t axes
    const int *lengths;                   // device, may be null
    const int *u_tab;                     // device [T + 1]: number of selected queries by length
    const int *U_tab;                     // device [T + 1]: number of sampled keys by length
    unsigned *status;                     // device status word
    unsigned long long wait_ns;           // limit of the bounded device-side waits that take it from here (1 s unless a
                                          // test shortens it, see psattn_plan_debug_waits)
    unsigned debug_extra_tx;              // test hook: bytes added to the first expected-bytes count of a kernel's
                                          // first TMA barrier, so that the barrier never completes and the wait runs out
};

// Programmatic dependent launch, for kernels that are launched with launch_pdl (psattn_launch.h): lets the
// next kernel of the stream be scheduled already, then waits until the previous kernel of the stream has
// completed and its writes are visible.  Must run before the first access to global memory; both
// instructions do nothing in a launch without the programmatic attribute.
__device__ __forceinline__ void pdl_enter() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Phase timing of the fused forward kernel, compiled in only with -DPSATTN_PHASE_STAMPS (a separate build of
// the library that the benchmark's --phases mode makes and loads; the regular build contains none of it).
// Called by all threads right after a block-wide barrier; thread 0 adds the time since the CTA's previous stamp
// to accumulator k (nanoseconds, 64-bit) in the status area of the workspace: bytes [64 + 8 k, 72 + 8 k),
// k = 1 .. 7; accumulator 0 counts the CTAs.
#ifdef PSATTN_PHASE_STAMPS
__device__ __forceinline__ void phase_stamp(const Geom &g, int k) {
    __shared__ unsigned long long phase_last;
    if (threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        unsigned long long *acc = reinterpret_cast<unsigned long long *>(g.status) + 8;
        if (k == 0) atomicAdd(acc, 1ull);
        else atomicAdd(acc + k, t - phase_last);
        phase_last = t;
    }
}
#else
__device__ __forceinline__ void phase_stamp(const Geom &, int) {}
#endif

// Begin and end of a kernel of the staged schedule, same build only: the earliest moment a block got past its
// wait for the grid before it and the latest moment a block ended (%globaltimer, nanoseconds), in the status area at
// bytes [128 + 16 k, 144 + 16 k), k = which kernel (KernelId).  The host sets begin to a large value and end to 0.
enum KernelId { kKernelMeasure = 0, kKernelSelectSlice, kKernelSelectMerge, kKernelAttend64, kKernelCombine, kKernelColsum,
                kKernelSelect, kKernelFill };
#ifdef PSATTN_PHASE_STAMPS
struct KernelSpan {
    unsigned long long *slot;
    __device__ __forceinline__ KernelSpan(const Geom &g, int k) {
        slot = reinterpret_cast<unsigned long long *>(g.status) + 16 + 2 * k;
        if (threadIdx.x == 0) { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); atomicMin(slot, t); }
    }
    __device__ __forceinline__ ~KernelSpan() {
        if (threadIdx.x == 0) { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); atomicMax(slot + 1, t); }
    }
};
#else
struct KernelSpan {
    __device__ __forceinline__ KernelSpan(const Geom &, int) {}
};
#endif

__device__ __forceinline__ int seq_len(const Geom &g, int b) {
    if (!g.lengths) return g.T;
    int L = g.lengths[b];
    if (L < 0 || L > g.T) {
        atomicOr(g.status, kStatusLenClamped);
        L = L < 0 ? 0 : g.T;
    }
    return L;
}

__device__ __forceinline__ long long unit_off(const long long s[3], int b, int h) {
    return (long long)b * s[0] + (long long)h * s[1];
}

// Eight consecutive elements (columns 8*sub .. 8*sub+7) of a row, widened to fp32.
__device__ __forceinline__ void load8(const __nv_bfloat16 *row, int sub, float out[8]) {
    uint4 r = __ldg(reinterpret_cast<const uint4 *>(row) + sub);
    out[0] = __uint_as_float(r.x << 16); out[1] = __uint_as_float(r.x & 0xffff0000u);
    out[2] = __uint_as_float(r.y << 16); out[3] = __uint_as_float(r.y & 0xffff0000u);
    out[4] = __uint_as_float(r.z << 16); out[5] = __uint_as_float(r.z & 0xffff0000u);
    out[6] = __uint_as_float(r.w << 16); out[7] = __uint_as_float(r.w & 0xffff0000u);
}
__device__ __forceinline__ void load8(const float *row, int sub, float out[8]) {
    float4 a = __ldg(reinterpret_cast<const float4 *>(row) + 2 * sub);
    float4 b = __ldg(reinterpret_cast<const float4 *>(row) + 2 * sub + 1);
    out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
    out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
}

__device__ __forceinline__ void store8(__nv_bfloat16 *row, int sub, const float v[8]) {
    __nv_bfloat162 p0 = __floats2bfloat162_rn(v[0], v[1]);
    __nv_bfloat162 p1 = __floats2bfloat162_rn(v[2], v[3]);
    __nv_bfloat162 p2 = __floats2bfloat162_rn(v[4], v[5]);
    __nv_bfloat162 p3 = __floats2bfloat162_rn(v[6], v[7]);
    uint4 r;
    r.x = *reinterpret_cast<unsigned *>(&p0); r.y = *reinterpret_cast<unsigned *>(&p1);
    r.z = *reinterpret_cast<unsigned *>(&p2); r.w = *reinterpret_cast<unsigned *>(&p3);
    reinterpret_cast<uint4 *>(row)[sub] = r;
}
__device__ __forceinline__ void store8(float *row, int sub, const float v[8]) {
    reinterpret_cast<float4 *>(row)[2 * sub] = make_float4(v[0], v[1], v[2], v[3]);
    reinterpret_cast<float4 *>(row)[2 * sub + 1] = make_float4(v[4], v[5], v[6], v[7]);
}

// Running state of Eq. 11 in the form  M~ = (1/U) sum_j (max - s_j):
//   m = largest score so far, n = scores seen, D = sum over them of (m - s_j).
// Every update adds non-negative terms only, so D >= 0 always and D == 0 exactly when all
// scores are equal.  Two states merge the same way, which lets lanes work on disjoint keys.
struct MeasureState {
    float m, D;
    int n;
};
__device__ __forceinline__ MeasureState measure_init() { return {-INFINITY, 0.f, 0}; }
__device__ __forceinline__ void measure_push(MeasureState &st, float s) {
    if (st.n == 0) { st.m = s; st.D = 0.f; st.n = 1; return; }
    if (s > st.m) { st.D += (float)st.n * (s - st.m); st.m = s; }
    else          { st.D += st.m - s; }
    st.n += 1;
}
__device__ __forceinline__ MeasureState measure_merge(const MeasureState &a, const MeasureState &b) {
    if (a.n == 0) return b;
    if (b.n == 0) return a;
    MeasureState r;
    r.m = fmaxf(a.m, b.m);
    r.D = (a.D + (float)a.n * (r.m - a.m)) + (b.D + (float)b.n * (r.m - b.m));
    r.n = a.n + b.n;
    return r;
}

// Order-preserving map float -> uint32 (larger float <=> larger key).
__device__ __forceinline__ unsigned float_key(float f) {
    unsigned b = __float_as_uint(f);
    if (b == 0x80000000u) b = 0u;                          // -0 and +0 are one value: they tie, the lower position first
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

}  // namespace psattn
