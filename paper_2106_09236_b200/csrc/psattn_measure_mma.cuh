// Steps (a)+(b) (Eq. 11) for bf16 inputs with the keys of a unit resident in shared memory, as
// CTA-wide device routines (used by the stand-alone measure kernel and by the fused forward kernel).
//
// The unit's K rows [len][64] are brought in once by TMA, unswizzled (row pitch 128 B).  A warp then
// works on four queries at a time and lets the tensor-core datapath do the 64-term dot products of a
// *gather*:
//   - A operand of mma.m16n8k16 = 16 sampled key rows, fetched with ldmatrix from arbitrary row
//     addresses.  In k-step s row i supplies its 16-byte chunk (s + i) mod 8 instead of chunk s,
//     so the eight rows of every 8x8 ldmatrix tile hit eight different bank groups whatever the
//     sampled keys are (a plain "same chunk for all rows" access would serialise 8-fold).
//   - B operand = the query, column n holding q rotated by n chunks; then D[i][i mod 8] is the
//     full dot product of key row i with q.  Only that diagonal is read.
// Every (query, key) pair costs one 128-byte shared-memory row read, the floor of this step.
// Q rows and sample rows are staged through shared memory with cp.async, double buffered.
#pragma once
#include "psattn_common.cuh"
#include "psattn_sm100.cuh"

namespace psattn {

constexpr int kMeasureBoxRows = 256;      // K rows per TMA box
constexpr int kMeasureMaxU = 64;          // four rounds of 16 sampled keys

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    // not volatile: what it reads is constant between the barriers around it, and leaving the
    // compiler free to reorder these lets independent rounds overlap
    asm("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
        : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
        : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t addr, uint32_t &r0, uint32_t &r1) {
    asm("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float c[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
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

// Shared-memory budget of the routine for a THREADS-thread CTA: resident keys + two staging buffers.
__host__ __device__ constexpr int measure_block_queries(int threads) { return threads / 32 * 4; }
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
    float *out;                             // M~ of the first query of the block (global or shared)
    unsigned *status;
};

// The queries of one staged block.  ROUNDS rounds of 16 sampled keys; with HALF the last round
// has at most 8 keys and loads only the A rows 0-7 (ldmatrix.x2).
template <int THREADS, int ROUNDS, bool HALF>
__device__ __forceinline__ void measure_block(const MeasureCtx &cx) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int l7 = lane & 7;
    // Full round (ldmatrix.x4): lane -> A row (l & 7) + 8 * ((l >> 3) & 1), k half l >> 4.
    // Half round (ldmatrix.x2, lanes 0-15 address): A row l & 7, k half (l >> 3) & 1.
    const int row_full = l7 + ((lane >> 3) & 1) * 8;
    const int hl_full = (lane >> 4) + l7, hl_half = ((lane >> 3) & 1) + l7;
    uint32_t off_full[4], off_half[4], j_off[ROUNDS];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        off_full[t] = (uint32_t)((2 * t + hl_full) & 7) << 4;
        off_half[t] = (uint32_t)((2 * t + hl_half) & 7) << 4;
    }
#pragma unroll
    for (int r = 0; r < ROUNDS; ++r) {
        const int j = r * 16 + ((HALF && r == ROUNDS - 1) ? l7 : row_full);
        j_off[r] = (uint32_t)(j < cx.U ? j : 0) * 4u;
    }
    // B fragments through ldmatrix: matrix m = l >> 3 holds k8-step s0 + m, its row n = l & 7 is the
    // 16-byte chunk (s0 + m + n) mod 8 of the q row
    const uint32_t q_off0 = (uint32_t)(((lane >> 3) + l7) & 7) << 4, q_off4 = (uint32_t)(((lane >> 3) + l7 + 4) & 7) << 4;
    // D: this lane holds rows dg and dg + 8, columns 2 * (l & 3) + {0, 1}; the wanted entry of row i
    // is column i mod 8, which sits in lane 4 * dg + dg / 2, register dg & 1 (+ 2 for row dg + 8)
    const int dg = lane >> 2;
    const bool de = dg & 1;
    const bool last_lo = (ROUNDS - 1) * 16 + dg < cx.U, last_hi = (ROUNDS - 1) * 16 + dg + 8 < cx.U;
    const float inv_U = 1.f / (float)cx.U;

    // A warp takes four consecutive queries of the block.  Their cross-lane reductions are done
    // together: only one lane per quad (the "diagonal" lane) holds wanted scores, so lane q of each
    // quad adopts query q's partials from its quad's diagonal lane, and three xor steps across the
    // quads finish all four queries at once.
    constexpr int kPerWarp = 4;
    const int quad_src = (lane & ~3) | (dg >> 1);
    float my_mx = -INFINITY, my_ds = 0.f;
#pragma unroll
    for (int k = 0; k < kPerWarp; ++k) {
        const int ql = min(warp * kPerWarp + k, cx.rows - 1);      // tail: recompute the last row
        uint32_t bq[8];
        ldmatrix_x4(cx.q_tile + (uint32_t)ql * 128u + q_off0, bq[0], bq[1], bq[2], bq[3]);
        ldmatrix_x4(cx.q_tile + (uint32_t)ql * 128u + q_off4, bq[4], bq[5], bq[6], bq[7]);
        const uint32_t krow = cx.idx_tile + (uint32_t)(ql * cx.idx_cols) * 4u;
        int key[ROUNDS];
        bool bad = false;
#pragma unroll
        for (int r = 0; r < ROUNDS; ++r) {
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(key[r]) : "r"(krow + j_off[r]));
            bad |= (unsigned)key[r] >= (unsigned)cx.L;
        }
        if (bad) {                                                 // rare: clamp and report
            atomicOr(cx.status, kStatusIdxClamped);
#pragma unroll
            for (int r = 0; r < ROUNDS; ++r) key[r] = key[r] < 0 ? 0 : min(key[r], cx.L - 1);
        }
        float c[ROUNDS][4];
#pragma unroll
        for (int r = 0; r < ROUNDS; ++r) c[r][0] = c[r][1] = c[r][2] = c[r][3] = 0.f;
        // the rounds are independent accumulation chains: step t of every round, then step t + 1
#pragma unroll
        for (int t = 0; t < 4; ++t) {
#pragma unroll
            for (int r = 0; r < ROUNDS; ++r) {
                const uint32_t row_addr = cx.k_base + (uint32_t)key[r] * 128u;
                uint32_t a0, a1 = 0u, a2, a3 = 0u;
                if (HALF && r == ROUNDS - 1) ldmatrix_x2(row_addr + off_half[t], a0, a2);
                else ldmatrix_x4(row_addr + off_full[t], a0, a1, a2, a3);
                mma_bf16_16816(c[r], a0, a1, a2, a3, bq[2 * t], bq[2 * t + 1]);
            }
        }
        // Eq. 11 relative to the first sampled score `ref` (always present): with d_j = s_j - ref,
        // M~ = max_j d_j - (1/U) sum_j d_j.  Constant scores give exactly 0; rounding is clamped at 0.
        const float ref = __shfl_sync(0xffffffffu, c[0][0], 0);
        float mx = -INFINITY, ds = 0.f;
#pragma unroll
        for (int r = 0; r < ROUNDS; ++r) {
            const float d_lo = (de ? c[r][1] : c[r][0]) - ref, d_hi = (de ? c[r][3] : c[r][2]) - ref;
            if (r < ROUNDS - 1) {
                mx = fmaxf(mx, fmaxf(d_lo, d_hi));
                ds += d_lo + d_hi;
            } else {
                mx = fmaxf(mx, fmaxf(last_lo ? d_lo : -INFINITY, last_hi ? d_hi : -INFINITY));
                ds += (last_lo ? d_lo : 0.f) + (last_hi ? d_hi : 0.f);
            }
        }
        const float q_mx = __shfl_sync(0xffffffffu, mx, quad_src);
        const float q_ds = __shfl_sync(0xffffffffu, ds, quad_src);
        if ((lane & 3) == k) { my_mx = q_mx; my_ds = q_ds; }
    }
#pragma unroll
    for (int o = 4; o <= 16; o <<= 1) {
        my_mx = fmaxf(my_mx, __shfl_xor_sync(0xffffffffu, my_mx, o));
        my_ds += __shfl_xor_sync(0xffffffffu, my_ds, o);
    }
    const int ql_out = warp * kPerWarp + lane;
    if (lane < kPerWarp && ql_out < cx.rows) cx.out[ql_out] = fmaxf((my_mx - my_ds * inv_U) * kScale, 0.f);
}

// One thread: start the TMA copies of the unit's key rows [0, L) into shared memory at `smem`
// (row pitch 128 B), all arriving on `bar` (initialised, count 1).  Returns the number of boxes.
__device__ __forceinline__ int measure_issue_keys(uint8_t *smem, uint64_t *bar, const CUtensorMap *tmK, int L, int b,
                                                  int h, int pos_t, int pos_h) {
    using namespace sm100;
    const int n_boxes = (L + kMeasureBoxRows - 1) / kMeasureBoxRows;
    if (n_boxes == 0) return 0;
    mbar_expect_tx(bar, (uint32_t)n_boxes * kMeasureBoxRows * 128u);
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
    auto stage_block = [&](int blk) {
        const int i0 = q_lo + blk * kBlock;
        const int rows = min(kBlock, q_end - i0);
        const uint32_t base = stage0 + (uint32_t)(blk & 1) * stage_bytes;
        if (tid < rows * 8)
            cp_async_16(base + (uint32_t)tid * 16u, Qu + (long long)(i0 + (tid >> 3)) * g.qs[2] + (tid & 7) * 8);
        const int words = rows * g.idx_cols;
        const int *src = idx_base + (long long)i0 * g.idx_cols;
        for (int w = tid; w < words; w += THREADS) cp_async_4(base + kBlock * 128u + (uint32_t)w * 4u, src + w);
        cp_async_commit();
    };
    const int n_blocks = (q_end - q_lo + kBlock - 1) / kBlock;
    if (n_blocks > 0) stage_block(0);

    // every thread must take the same branch (both contain barriers): agree on the outcome
    if (!__syncthreads_and(mbar_wait(bar, bar_phase) ? 1 : 0)) {   // bounded wait expired: report, produce zeros
        if ((tid & 31) == 0) atomicOr(g.status, kStatusWaitExpired);
        for (int i = q_lo + tid; i < q_end; i += THREADS) out[i] = 0.f;
        cp_async_wait<0>();
        // the bulk copies may still land: do not go on while they can write into this CTA's memory
        mbar_wait(bar, bar_phase);
        __syncthreads();
        return false;
    }
    U = min(U, kMeasureMaxU);
    const int rounds = (U + 15) >> 4;
    const bool last_half = (U - (rounds - 1) * 16) <= 8;        // last round has at most 8 rows: x2 loads
    MeasureCtx cx;
    cx.k_base = smem_u32(smem); cx.U = U; cx.L = L; cx.idx_cols = g.idx_cols; cx.status = g.status;

    for (int blk = 0; blk < n_blocks; ++blk) {
        if (blk + 1 < n_blocks) { stage_block(blk + 1); cp_async_wait<1>(); }
        else cp_async_wait<0>();
        __syncthreads();
        cx.q_tile = stage0 + (uint32_t)(blk & 1) * stage_bytes;
        cx.idx_tile = cx.q_tile + kBlock * 128u;
        const int i0 = q_lo + blk * kBlock;
        cx.rows = min(kBlock, q_end - i0);
        cx.out = out + i0;
        switch (rounds * 2 + (last_half ? 1 : 0)) {
            case 2: measure_block<THREADS, 1, false>(cx); break;
            case 3: measure_block<THREADS, 1, true>(cx); break;
            case 4: measure_block<THREADS, 2, false>(cx); break;
            case 5: measure_block<THREADS, 2, true>(cx); break;
            case 6: measure_block<THREADS, 3, false>(cx); break;
            case 7: measure_block<THREADS, 3, true>(cx); break;
            case 8: measure_block<THREADS, 4, false>(cx); break;
            default: measure_block<THREADS, 4, true>(cx); break;
        }
        __syncthreads();                              // the buffer is restaged two steps from now
    }
    return true;
}

}  // namespace psattn
