// Steps (a)+(b) (Eq. 11) for bf16 inputs of any sequence length: the streaming form of the
// gather-dot routine of psattn_measure_mma.cuh (same eight-queries-per-warp layout of the mma
// operands; the key rows come from global memory instead of a resident copy).
#pragma once
#include "psattn_measure_mma.cuh"

namespace psattn {

// ---------------------------------------------------------------------------------------------
// Streaming form for sequences whose keys do not fit in shared memory: the same eight-queries-per-
// warp gather-dot, but the 16 sampled key rows of a round are first copied from global memory (L2)
// into a small per-warp ring in shared memory with cp.async (16 bytes per lane, four copies per
// round), one round ahead.  Random 128-byte row reads out of L2 run far faster than a warp can
// unpack and multiply them with ordinary instructions, so the arithmetic stays on the tensor-core
// datapath here too.  Every pair costs one L2 row read, one shared-memory write and one read.
// ---------------------------------------------------------------------------------------------
constexpr int kStreamRing = 2;                                  // rounds in flight per warp (the code below is written for 2)
constexpr uint32_t kStreamRoundBytes = 16 * 128;

struct StreamCtx {
    uint32_t ring;                        // shared-memory address of this warp's ring
    uint32_t q_tile, idx_tile;            // staged Q rows and sample rows of the block
    int rows, U, L, idx_cols;
    uint32_t epoch0;                      // see ldmatrix_x4: produced after the barrier that published the block
    const __nv_bfloat16 *Ku;              // key rows of the unit
    uint32_t k_row_bytes;                 // row pitch of K in bytes (T_max * pitch < 2^32, checked by the launcher)
    float *out;
    unsigned *status;
};

// The ring accesses are volatile asm in program order, with the stage and copy offsets as immediates.
template <int OFF>
__device__ __forceinline__ void stream_ldmatrix(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4+%5];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr), "n"(OFF)
                 : "memory");
}
template <int OFF>
__device__ __forceinline__ void stream_copy16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0+%2], [%1], 16;" ::"r"(dst), "l"(src), "n"(OFF) : "memory");
}

struct StreamLane {                       // per-lane constants of one staged block
    uint32_t la[4];                       // ldmatrix row addresses in ring stage 0, one per k-step
    uint32_t dst;                         // this lane's 16-byte slot in ring stage 0 (copy k adds 512 k)
    uint32_t kp, kp_last;                 // address of this lane's sample of round 0; of the query's last sample
    const char *kb;                       // key rows of the unit, at this lane's 16-byte chunk
    uint32_t k_row_bytes;
    int src0;                             // copy k moves row src0 + 4k of the round; its key sits in lane src0 + 4k
    int L;
    unsigned *status;
};

// Start the copies of round r (16 key rows) into ring stage STAGE and commit them as one group.
template <int STAGE>
__device__ __forceinline__ void stream_issue(const StreamLane &ln, int r) {
    // odd U: in the last round the second sample does not exist; both halves then use the last sample
    const uint32_t ka = min(ln.kp + 8u * (uint32_t)r, ln.kp_last);
    int key;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(key) : "r"(ka) : "memory");
    if ((unsigned)key >= (unsigned)ln.L) {                     // rare: clamp and report
        atomicOr(ln.status, kStatusIdxClamped);
        key = key < 0 ? 0 : ln.L - 1;
    }
    __syncwarp();
    const uint32_t k0 = (uint32_t)__shfl_sync(0xffffffffu, key, ln.src0);
    const uint32_t k1 = (uint32_t)__shfl_sync(0xffffffffu, key, ln.src0 + 4);
    const uint32_t k2 = (uint32_t)__shfl_sync(0xffffffffu, key, ln.src0 + 8);
    const uint32_t k3 = (uint32_t)__shfl_sync(0xffffffffu, key, ln.src0 + 12);
    stream_copy16<STAGE * (int)kStreamRoundBytes>(ln.dst, ln.kb + (unsigned long long)k0 * ln.k_row_bytes);
    stream_copy16<STAGE * (int)kStreamRoundBytes + 512>(ln.dst, ln.kb + (unsigned long long)k1 * ln.k_row_bytes);
    stream_copy16<STAGE * (int)kStreamRoundBytes + 1024>(ln.dst, ln.kb + (unsigned long long)k2 * ln.k_row_bytes);
    stream_copy16<STAGE * (int)kStreamRoundBytes + 1536>(ln.dst, ln.kb + (unsigned long long)k3 * ln.k_row_bytes);
    cp_async_commit();
}

// The 16 dot products of the round that sits in ring stage STAGE (after PENDING younger groups at most
// are still in flight).  The accumulators are pinned behind a volatile asm so that every read of the
// stage precedes the next copy into it in program order.
template <int STAGE, int PENDING>
__device__ __forceinline__ void stream_round(const StreamLane &ln, const uint32_t bq[8], float c[4]) {
    cp_async_wait<PENDING>();                                  // this lane's copies of the round have landed
    __syncwarp();                                              // ... and everybody else's
    uint32_t a0, a1, a2, a3;
    stream_ldmatrix<STAGE * (int)kStreamRoundBytes>(ln.la[0], a0, a1, a2, a3);
    mma_bf16_16816_first(c, a0, a1, a2, a3, bq[0], bq[1]);
    stream_ldmatrix<STAGE * (int)kStreamRoundBytes>(ln.la[1], a0, a1, a2, a3);
    mma_bf16_16816(c, a0, a1, a2, a3, bq[2], bq[3]);
    stream_ldmatrix<STAGE * (int)kStreamRoundBytes>(ln.la[2], a0, a1, a2, a3);
    mma_bf16_16816(c, a0, a1, a2, a3, bq[4], bq[5]);
    stream_ldmatrix<STAGE * (int)kStreamRoundBytes>(ln.la[3], a0, a1, a2, a3);
    mma_bf16_16816(c, a0, a1, a2, a3, bq[6], bq[7]);
    asm volatile("" ::"f"(c[0]), "f"(c[1]), "f"(c[2]), "f"(c[3]) : "memory");
}

template <int THREADS>
__device__ __forceinline__ void measure_stream_block(const StreamCtx &cx) {
    static_assert(kStreamRing == 2, "two ring stages");
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int l7 = lane & 7;
    const int q0 = warp * 8;
    if (q0 >= cx.rows) return;
    const int qn = min(q0 + l7, cx.rows - 1);
    uint32_t bq[8];
    {
        const uint32_t qa = cx.q_tile + (uint32_t)qn * 128u;
        ldmatrix_x4(qa + ((uint32_t)(((lane >> 3) + l7) & 7) << 4), cx.epoch0, bq[0], bq[1], bq[2], bq[3]);
        ldmatrix_x4(qa + ((uint32_t)(((lane >> 3) + l7 + 4) & 7) << 4), cx.epoch0, bq[4], bq[5], bq[6], bq[7]);
    }
    const int slot = (lane >> 3) & 1;                          // this lane's A row is (query l7, sample 2r + slot)
    StreamLane ln;
#pragma unroll
    for (int t = 0; t < 4; ++t)
        ln.la[t] = cx.ring + (uint32_t)(l7 + 8 * slot) * 128u + ((uint32_t)((2 * t + (lane >> 4) + l7) & 7) << 4);
    ln.dst = cx.ring + (uint32_t)lane * 16u;
    ln.kp = cx.idx_tile + (uint32_t)(qn * cx.idx_cols + slot) * 4u;
    ln.kp_last = cx.idx_tile + (uint32_t)(qn * cx.idx_cols + cx.U - 1) * 4u;
    ln.kb = reinterpret_cast<const char *>(cx.Ku) + l7 * 16;
    ln.k_row_bytes = cx.k_row_bytes;
    ln.src0 = lane >> 3;
    ln.L = cx.L;
    ln.status = cx.status;
    const int g = lane >> 2;
    const bool de = g & 1;
    const int rounds = (cx.U + 1) >> 1;
    const bool odd = cx.U & 1;

    // Eq. 11 relative to the first sampled score `ref` (see measure_block)
    float ref = 0.f, mx = 0.f, ds = 0.f, c[4] = {0.f, 0.f, 0.f, 0.f};
    auto take = [&](bool hi_ok) {
        const float d_lo = (de ? c[1] : c[0]) - ref, d_hi = (de ? c[3] : c[2]) - ref;
        mx = fmaxf(mx, fmaxf(d_lo, hi_ok ? d_hi : d_lo));
        ds += d_lo + (hi_ok ? d_hi : 0.f);
    };
    stream_issue<0>(ln, 0);
    if (rounds == 1) {
        stream_round<0, 0>(ln, bq, c);
        ref = de ? c[1] : c[0];
        take(!odd);
    } else {
        stream_issue<1>(ln, 1);
        stream_round<0, 1>(ln, bq, c);
        ref = de ? c[1] : c[0];
        take(true);
        int r = 1;                                             // round r sits (or lands) in stage 1, stage 0 is free
        for (; r + 2 < rounds; r += 2) {                       // rounds r and r + 1, neither is the last
            stream_issue<0>(ln, r + 1);
            stream_round<1, 1>(ln, bq, c);
            take(true);
            stream_issue<1>(ln, r + 2);
            stream_round<0, 1>(ln, bq, c);
            take(true);
        }
        if (rounds - r == 2) {
            stream_issue<0>(ln, r + 1);
            stream_round<1, 1>(ln, bq, c);
            take(true);
            stream_round<0, 0>(ln, bq, c);
            take(!odd);
        } else {
            stream_round<1, 0>(ln, bq, c);
            take(!odd);
        }
    }
    if ((lane & 3) == (g >> 1) && q0 + g < cx.rows)
        cx.out[q0 + g] = fmaxf((mx - ds / (float)cx.U) * kScale, 0.f);
}

// All THREADS threads of the CTA: M~ of the queries [q_lo, q_end) (q_end <= L, L >= 1) of unit (b, h)
// into out[i].  Shared memory: THREADS / 32 rings, then two staging buffers of stage_bytes.
// No block-wide barrier inside: the caller orders the result with one of its own where it needs to.
template <int THREADS>
__device__ __forceinline__ void measure_stream(uint8_t *smem, uint32_t stage_bytes, const Geom &g, int unit, int b, int h,
                                               int L, int U, int q_lo, int q_end, const __nv_bfloat16 *__restrict__ Q,
                                               const __nv_bfloat16 *__restrict__ K, const int *__restrict__ sidx,
                                               float *out) {
    using namespace sm100;
    constexpr int kBlock = measure_block_queries(THREADS);
    constexpr uint32_t kRingBytes = (THREADS / 32) * kStreamRing * kStreamRoundBytes;
    const int tid = threadIdx.x;
    const int *idx_base = sidx + ((g.idx_per_head ? (long long)unit : (long long)b) * g.T) * g.idx_cols;
    const __nv_bfloat16 *Qu = Q + unit_off(g.qs, b, h);
    const uint32_t stage0 = smem_u32(smem) + kRingBytes;
    const int n_blocks = (q_end - q_lo + kBlock - 1) / kBlock;
    // every warp stages the rows of its own eight queries (see measure_resident): no barrier between blocks,
    // so the warps drift apart and the pipeline bubble at the start of a group of queries does not hit all
    // of them at once
    const int warp = tid >> 5, lane = tid & 31;
    auto stage_block = [&](int blk) {
        if (blk < n_blocks) {
            const int i0 = q_lo + blk * kBlock + warp * 8;
            const int rows = min(8, q_end - i0);
            if (rows > 0) {
                const uint32_t base = stage0 + (uint32_t)(blk & 1) * stage_bytes;
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
    StreamCtx cx;
    cx.ring = smem_u32(smem) + (uint32_t)(tid >> 5) * kStreamRing * kStreamRoundBytes;
    cx.U = min(U, kMeasureMaxU); cx.L = L; cx.idx_cols = g.idx_cols; cx.status = g.status;
    cx.Ku = K + unit_off(g.ks, b, h); cx.k_row_bytes = (uint32_t)(g.ks[2] * 2);
    stage_block(0);
    for (int blk = 0; blk < n_blocks; ++blk) {
        cp_async_wait<0>();                                    // this lane's part of block blk (nothing else is pending)
        __syncwarp();
        asm volatile("mov.u32 %0, %1;" : "=r"(cx.epoch0) : "r"(blk << 8) : "memory");
        stage_block(blk + 1);                                  // lands while this block is worked on
        cx.q_tile = stage0 + (uint32_t)(blk & 1) * stage_bytes;
        cx.idx_tile = cx.q_tile + kBlock * 128u;
        const int i0 = q_lo + blk * kBlock;
        cx.rows = min(kBlock, q_end - i0);
        cx.out = out + i0;
        measure_stream_block<THREADS>(cx);
        __syncwarp();                                          // the warp's part of buffer blk & 1 may be restaged next time
    }
    cp_async_wait<0>();
}

}  // namespace psattn
