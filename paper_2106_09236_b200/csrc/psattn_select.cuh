// Step (c) (Sec. 3.2): the u positions with the largest M~ among i < L, equal values ordered by
// position, written in ascending position order.  A block-wide routine shared by the stand-alone
// select kernel and the fused forward kernel.
#pragma once
#include "psattn_common.cuh"

namespace psattn {

struct SelectScratch {
    int hist[256];
    int wtot_gt[32], wtot_eq[32];
    int wpre_gt[33], wpre_eq[33];
    unsigned prefix;
    int remaining;
    int done;
};

// All threads of the block call this with the same arguments (blockDim.x a multiple of 32, <= 1024).
// key_of(i) returns the order-preserving key of position i (larger key = larger M~); it is called
// several times per position and must be cheap (a global or shared-memory read).
// Four 8-bit radix passes find tau, the u-th largest key; the result is every position with
// key > tau plus the first `remaining` positions with key == tau.  out[0..u_max) receives the
// positions in ascending order, -1 padded.  Ends with a __syncthreads().
template <class KeyFn>
__device__ __forceinline__ void block_select(KeyFn key_of, int L, int u, int u_max, int *out, SelectScratch &s) {
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, wid = tid >> 5, nw = nthr >> 5;
    if (u <= 0) {
        for (int r = tid; r < u_max; r += nthr) out[r] = -1;
        __syncthreads();
        return;
    }
    if (tid == 0) { s.prefix = 0u; s.remaining = u; s.done = 0; }
    unsigned known = 0u;                                   // key bits fixed so far
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (tid < 256) s.hist[tid] = 0;
        __syncthreads();
        const unsigned prefix = s.prefix;
        for (int i = tid; i < L; i += nthr) {
            const unsigned k = key_of(i);
            if (((k ^ prefix) & known) == 0u) atomicAdd(&s.hist[(k >> shift) & 255u], 1);
        }
        __syncthreads();
        if (wid == 0) {                                    // find the bin that holds the remaining-th largest
            int h[8], mine = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { h[j] = s.hist[lane * 8 + j]; mine += h[j]; }
            int incl = mine;                               // becomes the count of bins >= this lane's first bin
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_down_sync(0xffffffffu, incl, o);
                if (lane + o < 32) incl += y;
            }
            const int above = incl - mine, rem = s.remaining;
            __syncwarp();
            if (above < rem && incl >= rem) {              // exactly one lane
                int r = rem - above, bin = 7;
                for (; bin > 0; --bin) {
                    if (h[bin] >= r) break;
                    r -= h[bin];
                }
                const unsigned value = prefix | ((unsigned)(lane * 8 + bin) << shift);
                if (h[bin] == r && value != 0u) {
                    // every key of this bin is taken: the result is "all keys >= value"; no need to
                    // resolve the lower bits
                    s.prefix = value - 1u;
                    s.remaining = 0;
                    s.done = 1;
                } else {
                    s.prefix = value;
                    s.remaining = r;
                }
            }
        }
        known |= 0xffu << shift;
        __syncthreads();
        if (s.done) break;
    }
    const unsigned tau = s.prefix;
    const int need_eq = s.remaining;                       // positions with key == tau to take, lowest first
    int gt_seen = 0, eq_seen = 0;
    for (int base = 0; base < L; base += nthr) {
        const int i = base + tid;
        const bool valid = i < L;
        const unsigned k = valid ? key_of(i) : 0u;
        const int is_gt = valid && k > tau, is_eq = valid && k == tau;
        int xg = is_gt, xe = is_eq;                        // inclusive warp scans of both flags
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int yg = __shfl_up_sync(0xffffffffu, xg, o), ye = __shfl_up_sync(0xffffffffu, xe, o);
            if (lane >= o) { xg += yg; xe += ye; }
        }
        if (lane == 31) { s.wtot_gt[wid] = xg; s.wtot_eq[wid] = xe; }
        __syncthreads();
        if (wid == 0) {                                        // exclusive scan of the warp totals; grand totals in [nw]
            int tg = lane < nw ? s.wtot_gt[lane] : 0, te = lane < nw ? s.wtot_eq[lane] : 0;
            const int og = tg, oe = te;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int yg = __shfl_up_sync(0xffffffffu, tg, o), ye = __shfl_up_sync(0xffffffffu, te, o);
                if (lane >= o) { tg += yg; te += ye; }
            }
            s.wpre_gt[lane] = tg - og; s.wpre_eq[lane] = te - oe;
            if (lane == 31) { s.wpre_gt[32] = tg; s.wpre_eq[32] = te; }
        }
        __syncthreads();
        const int bg = s.wpre_gt[wid], be = s.wpre_eq[wid], tg = s.wpre_gt[32], te = s.wpre_eq[32];
        const int gt_before = gt_seen + bg + xg - is_gt, eq_before = eq_seen + be + xe - is_eq;
        // taken positions before this one: all greater ones, and the equal ones up to need_eq
        if (is_gt || (is_eq && eq_before < need_eq)) {
            const int pos = gt_before + min(eq_before, need_eq);
            if (pos < u_max) out[pos] = i;
        }
        gt_seen += tg; eq_seen += te;
        __syncthreads();
    }
    for (int r = u + tid; r < u_max; r += nthr) out[r] = -1;
    __syncthreads();
}

}  // namespace psattn
