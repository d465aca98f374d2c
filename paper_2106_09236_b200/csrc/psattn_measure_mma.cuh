// Steps (a)+(b) (Eq. 11) for bf16 inputs with the keys of a unit resident in shared memory, as
// CTA-wide device routines (used by the stand-alone measure kernel and by the fused forward kernel).
//
// The unit's K rows [len][64] are brought in once by TMA, unswizzled (row pitch 128 B).  A warp then
// works on eight queries at a time and lets the tensor-core datapath do the 64-term dot products of
// a *gather*:
//   - A operand of mma.m16n8k16 = 16 sampled key rows, fetched with ldmatrix from arbitrary row
//     addresses: rows i and i + 8 are two sampled keys of query i (i = 0..7).  In k-step s row i
//     supplies its 16-byte chunk (s + i) mod 8 instead of chunk s, so the eight rows of every 8x8
//     ldmatrix tile hit eight different bank groups whatever the sampled keys are (a plain "same
//     chunk for all rows" access would serialise 8-fold).
//   - B operand: column n = query n, rotated by n chunks; then D[i][i mod 8] is the full dot product
//     of key row i with its own query.  Only that diagonal is read, and the lane that holds
//     D[i][i] also holds D[i + 8][i]: every score of a query lands in one lane, so the running
//     max and sum of Eq. 11 need no cross-lane step at all.
// Every (query, key) pair costs one 128-byte shared-memory row read, the floor of this step.
// Q rows and sample rows are staged through shared memory with cp.async, double buffered.
#pragma once
#include "psattn_common.cuh"
#include "psattn_sm100.cuh"

namespace psattn {

constexpr int kMeasureBoxRows = 256;      // K rows per TMA box
constexpr int kMeasureMaxU = 64;          // four rounds of 16 sampled keys
constexpr int kMeasureStages = 2;         // staging buffers for Q rows and sample rows (2 blocks in flight)

// The shared-memory reads of the gather are not volatile asm, so that the compiler may interleave
// independent rounds.  What they read is constant between the two barriers around a staged block;
// the extra `epoch` operand (a value produced by a volatile asm right after the first barrier)
// keeps them from being hoisted above that barrier or merged with an identical read of an earlier
// block that used the same buffer.
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t epoch, uint32_t &r0, uint32_t &r1, uint32_t &r2,
                                            uint32_t &r3) {
    asm("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4]; // %5"
        : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
        : "r"(addr), "r"(epoch));
}
__device__ __forceinline__ int lds_b32(uint32_t addr, uint32_t epoch) {
    int v;
    asm("ld.shared.b32 %0, [%1]; // %2" : "=r"(v) : "r"(addr), "r"(epoch));
    return v;
}
__device__ __forceinline__ void mma_bf16_16816(float c[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// Same with a zero accumulator coming in: the first k-step of a chain (saves clearing four registers).
__device__ __forceinline__ void mma_bf16_16816_first(float c[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                     uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%10, %10, %10, %10};"
        : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_4(uint32_t dst, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Shared-memory budget of the routine for a THREADS-thread CTA: resident keys + kMeasureStages
// staging buffers.
__host__ __device__ constexpr int measure_block_queries(int threads) { return threads / 32 * 8; }
__host__ __device__ inline size_t measure_k_bytes(int T) {
    return (size_t)((T + kMeasureBoxRows - 1) / kMeasureBoxRows * kMeasureBoxRows) * 128;
}
__host__ __device__ inline size_t measure_stage_bytes(int threads, int idx_cols) {
    const size_t q = measure_block_queries(threads);
    return (q * 128 + q * idx_cols * 4 + 127) / 128 * 128;
}

struct MeasureCtx {
    uint32_t k_base, q_tile, idx_tile;      // shared-memory addresses
    int rows, U, L, idx_cols;
    uint32_t epoch;                         // see ldmatrix_x4
    float *out;                             // M~ of the first query of the block (global or shared)
    unsigned *status;
};

// One round of the gather: 16 key rows (two per query) against the eight queries of the warp.
__device__ __forceinline__ void measure_round(float c[4], uint32_t row_addr, const uint32_t off[4], const uint32_t bq[8],
                                              uint32_t epoch) {
    uint32_t a0, a1, a2, a3;
    ldmatrix_x4(row_addr + off[0], epoch, a0, a1, a2, a3);
    mma_bf16_16816_first(c, a0, a1, a2, a3, bq[0], bq[1]);
#pragma unroll
    for (int t = 1; t < 4; ++t) {
        ldmatrix_x4(row_addr + off[t], epoch, a0, a1, a2, a3);
        mma_bf16_16816(c, a0, a1, a2, a3, bq[2 * t], bq[2 * t + 1]);
    }
}

// The queries of one staged block: every warp takes eight consecutive queries.
template <int THREADS>
__device__ __forceinline__ void measure_block(const MeasureCtx &cx) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int l7 = lane & 7;
    const int q0 = warp * 8;
    if (q0 >= cx.rows) return;
    const int qn = min(q0 + l7, cx.rows - 1);                  // tail: recompute the last row
    // B fragments through ldmatrix: matrix m = l >> 3 holds k8-step s0 + m; its row n = l & 7 is the
    // 16-byte chunk (s0 + m + n) mod 8 of query n's row
    uint32_t bq[8];
    {
        const uint32_t qa = cx.q_tile + (uint32_t)qn * 128u;
        ldmatrix_x4(qa + ((uint32_t)(((lane >> 3) + l7) & 7) << 4), cx.epoch, bq[0], bq[1], bq[2], bq[3]);
        ldmatrix_x4(qa + ((uint32_t)(((lane >> 3) + l7 + 4) & 7) << 4), cx.epoch, bq[4], bq[5], bq[6], bq[7]);
    }
    // A rows: lane l addresses row (l & 7) + 8 * ((l >> 3) & 1), i.e. query l & 7, sample 2r + ((l >> 3) & 1)
    // of round r, k half l >> 4 -> chunk (2t + (l >> 4) + (l & 7)) mod 8 in k-step t
    uint32_t off[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) off[t] = (uint32_t)((2 * t + (lane >> 4) + l7) & 7) << 4;
    const uint32_t krow = cx.idx_tile + (uint32_t)(qn * cx.idx_cols + ((lane >> 3) & 1)) * 4u;
    // D: lane 4g + g / 2 holds D[g][g] (register g & 1) and D[g + 8][g] (register 2 + (g & 1)):
    // the two scores of query g in this round
    const int g = lane >> 2;
    const bool de = g & 1;
    const int full_rounds = cx.U >> 1;

    auto key_of = [&](int sample0) {                           // sample0 = 2r; this lane's sample is 2r or 2r + 1
        int key = lds_b32(krow + (uint32_t)sample0 * 4u, cx.epoch);
        if ((unsigned)key >= (unsigned)cx.L) {                 // rare: clamp and report
            atomicOr(cx.status, kStatusIdxClamped);
            key = key < 0 ? 0 : cx.L - 1;
        }
        return cx.k_base + (uint32_t)key * 128u;
    };
    // Eq. 11 relative to the first sampled score `ref`: with d_j = s_j - ref,
    // M~ = max_j d_j - (1/U) sum_j d_j.  Constant scores give exactly 0; rounding is clamped at 0.
    float ref = 0.f, mx = 0.f, ds = 0.f;
    int r = 0;
    if (full_rounds > 0) {
        float c[4];
        measure_round(c, key_of(0), off, bq, cx.epoch);
        ref = de ? c[1] : c[0];
        const float d_hi = (de ? c[3] : c[2]) - ref;
        mx = fmaxf(0.f, d_hi); ds = d_hi;
        r = 1;
    }
    for (; r + 1 < full_rounds; r += 2) {                      // two independent chains per trip
        float c0[4], c1[4];
        const uint32_t ra0 = key_of(2 * r), ra1 = key_of(2 * r + 2);
        measure_round(c0, ra0, off, bq, cx.epoch);
        measure_round(c1, ra1, off, bq, cx.epoch);
        const float a_lo = (de ? c0[1] : c0[0]) - ref, a_hi = (de ? c0[3] : c0[2]) - ref;
        const float b_lo = (de ? c1[1] : c1[0]) - ref, b_hi = (de ? c1[3] : c1[2]) - ref;
        mx = fmaxf(mx, fmaxf(fmaxf(a_lo, a_hi), fmaxf(b_lo, b_hi)));
        ds += (a_lo + a_hi) + (b_lo + b_hi);
    }
    if (r < full_rounds) {
        float c[4];
        measure_round(c, key_of(2 * r), off, bq, cx.epoch);
        const float a_lo = (de ? c[1] : c[0]) - ref, a_hi = (de ? c[3] : c[2]) - ref;
        mx = fmaxf(mx, fmaxf(a_lo, a_hi));
        ds += a_lo + a_hi;
    }
    if (cx.U & 1) {                                            // last sample: only the rows 0-7 count
        float c[4];
        // rows 8-15 would be sample U: point them at sample U - 1 as well (in range, result unused)
        const uint32_t back = ((lane >> 3) & 1) ? 4u : 0u;
        int key = lds_b32(krow + (uint32_t)(cx.U - 1) * 4u - back, cx.epoch);
        if ((unsigned)key >= (unsigned)cx.L) { atomicOr(cx.status, kStatusIdxClamped); key = key < 0 ? 0 : cx.L - 1; }
        measure_round(c, cx.k_base + (uint32_t)key * 128u, off, bq, cx.epoch);
        const float s_lo = de ? c[1] : c[0];
        if (full_rounds == 0) ref = s_lo;
        const float a_lo = s_lo - ref;
        mx = fmaxf(mx, a_lo);
        ds += a_lo;
    }
    if ((lane & 3) == (g >> 1) && q0 + g < cx.rows)
        cx.out[q0 + g] = fmaxf((mx - ds / (float)cx.U) * kScale, 0.f);
}

// One thread: start the TMA copies of the unit's key rows [0, L) into shared memory at `smem`
// (row pitch 128 B), all arriving on `bar` (initialised, count 1).  Returns the number of boxes.
__device__ __forceinline__ int measure_issue_keys(uint8_t *smem, uint64_t *bar, const CUtensorMap *tmK, int L, int b,
                                                  int h, int pos_t, int pos_h, uint32_t extra_tx = 0u) {
    using namespace sm100;
    const int n_boxes = (L + kMeasureBoxRows - 1) / kMeasureBoxRows;
    if (n_boxes == 0) return 0;
    mbar_expect_tx(bar, (uint32_t)n_boxes * kMeasureBoxRows * 128u + extra_tx);   // extra_tx: test hook, see Geom
    for (int x = 0; x < n_boxes; ++x) {
        const int key0 = x * kMeasureBoxRows;
        const int c1 = pos_t == 1 ? key0 : (pos_h == 1 ? h : b);
        const int c2 = pos_t == 2 ? key0 : (pos_h == 2 ? h : b);
        const int c3 = pos_t == 3 ? key0 : (pos_h == 3 ? h : b);
        tma_load_4d(smem + (size_t)key0 * 128, tmK, bar, 0, c1, c2, c3);
    }
    return n_boxes;
}

// All THREADS threads of the CTA: M~ of the queries [q_lo, q_end) (q_end <= L, L >= 1) of unit
// (b, h) into out[i] (global or shared).  The key copies must have been started on `bar`
// (phase `bar_phase`).  Shared memory: keys at smem[0, k_bytes), staging buffers after them.
// Contains __syncthreads.  Returns false if the bounded wait for the keys expired.
template <int THREADS>
__device__ __forceinline__ bool measure_resident(uint8_t *smem, uint64_t *bar, uint32_t bar_phase, uint32_t k_bytes,
                                                 uint32_t stage_bytes, const Geom &g, int unit, int b, int h, int L,
                                                 int U, int q_lo, int q_end, const __nv_bfloat16 *__restrict__ Q,
                                                 const int *__restrict__ sidx, float *out) {
    using namespace sm100;
    constexpr int kBlock = measure_block_queries(THREADS);
    const int tid = threadIdx.x;
    const int *idx_base = sidx + ((g.idx_per_head ? (long long)unit : (long long)b) * g.T) * g.idx_cols;
    const __nv_bfloat16 *Qu = Q + unit_off(g.qs, b, h);
    const uint32_t stage0 = smem_u32(smem) + k_bytes;
    const int n_blocks = (q_end - q_lo + kBlock - 1) / kBlock;
    // Every warp stages the rows of its own eight queries of a block (Q rows, then sample rows, at the warp's
    // place in the block's buffer) and nobody else reads them, so the warps run through the blocks without
    // meeting at a barrier.  Always commits a group, even an empty one.
    const int warp = tid >> 5, lane = tid & 31;
    auto stage_block = [&](int blk) {
        if (blk < n_blocks) {
            const int i0 = q_lo + blk * kBlock + warp * 8;
            const int rows = min(8, q_end - i0);
            if (rows > 0) {
                const uint32_t base = stage0 + (uint32_t)(blk % kMeasureStages) * stage_bytes;
                const uint32_t qdst = base + (uint32_t)warp * 1024u;
                for (int e = lane; e < rows * 8; e += 32)
                    cp_async_16(qdst + (uint32_t)e * 16u, Qu + (long long)(i0 + (e >> 3)) * g.qs[2] + (e & 7) * 8);
                const int words = rows * g.idx_cols;
                const int *src = idx_base + (long long)i0 * g.idx_cols;
                const uint32_t idst = base + kBlock * 128u + (uint32_t)(warp * 8 * g.idx_cols) * 4u;
                if (((reinterpret_cast<uintptr_t>(src) | (uintptr_t)(words * 4)) & 15u) == 0u) {
                    for (int w = lane; w < words / 4; w += 32) cp_async_16(idst + (uint32_t)w * 16u, src + 4 * w);
                } else {
                    for (int w = lane; w < words; w += 32) cp_async_4(idst + (uint32_t)w * 4u, src + w);
                }
            }
        }
        cp_async_commit();
    };
    for (int blk = 0; blk < kMeasureStages - 1; ++blk) stage_block(blk);

    // every thread must take the same branch (both contain barriers): agree on the outcome
    if (!__syncthreads_and(mbar_wait(bar, bar_phase, g.wait_ns) ? 1 : 0)) {   // bounded wait expired: report, produce zeros
        if ((tid & 31) == 0) atomicOr(g.status, kStatusWaitExpired);
        for (int i = q_lo + tid; i < q_end; i += THREADS) out[i] = 0.f;
        cp_async_wait<0>();
        // the bulk copies may still land: do not go on while they can write into this CTA's memory
        mbar_wait(bar, bar_phase, g.wait_ns);
        __syncthreads();
        return false;
    }
    phase_stamp(g, 1);                                    // the unit's keys are in shared memory
    U = min(U, kMeasureMaxU);
    MeasureCtx cx;
    cx.k_base = smem_u32(smem); cx.U = U; cx.L = L; cx.idx_cols = g.idx_cols; cx.status = g.status;

    for (int blk = 0; blk < n_blocks; ++blk) {
        stage_block(blk + kMeasureStages - 1);            // into the buffer this warp left at the end of the trip before
        cp_async_wait<kMeasureStages - 1>();              // this lane's part of block blk has landed
        __syncwarp();                                     // ... and the other lanes' parts
        asm volatile("mov.u32 %0, %1;" : "=r"(cx.epoch) : "r"(blk) : "memory");
        cx.q_tile = stage0 + (uint32_t)(blk % kMeasureStages) * stage_bytes;
        cx.idx_tile = cx.q_tile + kBlock * 128u;
        const int i0 = q_lo + blk * kBlock;
        cx.rows = min(kBlock, q_end - i0);
        cx.out = out + i0;
        measure_block<THREADS>(cx);
        __syncwarp();                                 // the warp's part of the buffer may be restaged from now on
    }
    return true;
}

}  // namespace psattn
