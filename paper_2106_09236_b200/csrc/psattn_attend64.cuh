// Step (d) (Eq. 7-8) for up to 64 listed rows of one unit, as a CTA-wide routine on tcgen05.
//
// Work is cut into pairs of 128-key tiles.  Two warpgroups alternate over the pairs; inside a
// warpgroup lanes 0-15 of every warp work on the first tile of the pair and lanes 16-31 on the
// second one: tcgen05.mma with M = 64 puts row m of its accumulator in TMEM lane
// (m mod 16) + 32 * (m / 16), so two such accumulators interleave in one column range (the second
// at lane offset 16) and one tcgen05.ld serves both.  Per pair and warpgroup:
//   control thread   TMA K pair, V pair -> shared memory (128-byte swizzle)
//   control thread   S_a = Q K_a^T, S_b = Q K_b^T -> TMEM
//   warpgroup        masked online softmax of (row, tile) per thread; P_a, P_b (bf16) -> shared memory
//   control thread   O_a = P_a V_a, O_b = P_b V_b -> TMEM
//   warpgroup        acc = acc * alpha + O
// Each warpgroup has its own control thread (lane 0 of warps ctrl_warp and ctrl_warp + 1), so neither
// waits for the other.  A warpgroup owns two score accumulators (TMEM columns [256 wg, 256 wg + 128) and the 128
// after them) used by alternate pairs; O of a pair is written over the first 64 columns of the scores it came
// from.  So the scores of the next pair are computed as soon as its keys have landed and the other accumulator
// has been read out, under the softmax of the current pair.
// At the end the (m, l, acc) states of the two tiles of a pair and of the two warpgroups are merged.
// Every wait is bounded; on expiry the routine sets the status bit and unwinds.
#pragma once
#include "psattn_common.cuh"
#include "psattn_sm100.cuh"

namespace psattn {

constexpr uint32_t kA64Tile = 16384;                         // one 128-key K or V tile
constexpr uint32_t kA64OffQ = 0;                             // 64 rows x 128 B
constexpr uint32_t kA64OffWg = 8192;                         // per warpgroup: K pair, V pair, P pair
constexpr uint32_t kA64WgBytes = 6 * kA64Tile;
constexpr uint32_t kA64OffBar = kA64OffWg + 2 * kA64WgBytes;
constexpr uint32_t kA64Bytes = kA64OffBar + 128;
constexpr uint32_t kA64TmemCols = 512;                       // per warpgroup: two score accumulators of 128 columns
constexpr int kA64MaxRows = 64;

struct Attend64Job {
    int b, h, L;                 // unit and its valid length
    int lo, hi;                  // key range of this CTA (lo a multiple of 128 relative to 0)
    const int *rows;             // listed positions (global or shared), or null = identity
    int n_rows;                  // <= 64
    int pos_t, pos_h, pos_b;     // TMA coordinate slots
    int ctrl_warp, wg_warp0;     // warps ctrl_warp, ctrl_warp + 1: control threads; first warp of warpgroup 0 (multiple of 4)
    int started;                 // attend64_start was already run for this job
    int sum_row;                 // slot (>= n_rows, < 64) kept active although it lists no query: its zero
                                 // query row gets weight 1 on every key, so it returns the column sums of V
                                 // over [lo, hi) with l = number of keys; -1 = none
};

// Control thread only: initialise the barriers of the routine and start the TMA copies of the first
// key-tile pair of each warpgroup.  They depend only on the unit and its length, not on the listed
// rows, so a caller may run this early (set Attend64Job::started) to hide the copy latency behind
// other work; the shared memory of the routine must be free by then.
__device__ __forceinline__ void attend64_start(uint8_t *smem, const Attend64Job &j, const CUtensorMap *tmK,
                                               const CUtensorMap *tmV) {
    using namespace sm100;
    uint64_t *kfull = reinterpret_cast<uint64_t *>(smem + kA64OffBar);
    uint64_t *vfull = kfull + 2, *sfull = kfull + 4, *pready = kfull + 8, *ofull = kfull + 10, *sfree = kfull + 12;
    volatile uint32_t *abort_flag = reinterpret_cast<uint32_t *>(kfull + 14);
    const int n_tiles = (j.hi - j.lo + 127) / 128, n_pairs = (n_tiles + 1) / 2;
    for (int x = 0; x < 2; ++x) {
        mbar_init(&kfull[x], 1); mbar_init(&vfull[x], 1); mbar_init(&sfull[2 * x], 1); mbar_init(&sfull[2 * x + 1], 1);
        mbar_init(&pready[x], 128); mbar_init(&ofull[x], 1); mbar_init(&sfree[x], 128);
    }
    *abort_flag = 0u;
    fence_barrier_init();
    for (int wg = 0; wg < 2 && wg < n_pairs; ++wg) {
        for (int is_v = 0; is_v < 2; ++is_v) {
            uint8_t *dst = smem + kA64OffWg + wg * kA64WgBytes + (is_v ? 2 * kA64Tile : 0);
            uint64_t *bar = is_v ? &vfull[wg] : &kfull[wg];
            const int two = (2 * wg + 1 < n_tiles) ? 1 : 0;
            mbar_expect_tx(bar, kA64Tile * (1 + two));
            for (int s = 0; s <= two; ++s) {
                const int key0 = j.lo + (2 * wg + s) * 128;
                const int c1 = j.pos_t == 1 ? key0 : (j.pos_h == 1 ? j.h : j.b);
                const int c2 = j.pos_t == 2 ? key0 : (j.pos_h == 2 ? j.h : j.b);
                const int c3 = j.pos_t == 3 ? key0 : (j.pos_h == 3 ? j.h : j.b);
                tma_load_4d(dst + s * kA64Tile, is_v ? tmV : tmK, bar, 0, c1, c2, c3);
            }
        }
    }
}

// Masked online softmax of one thread's (row, key tile): two passes over its 128 scores in TMEM,
// 64 at a time with both loads of a half in flight together; P (bf16) goes to the thread's row of
// the A-operand tile.  FULL: all 128 keys exist (no masks).  A row whose query is zero gets equal
// weights exp2(0) = 1 with m = 0, so its accumulator row is the column sum of V and its l the
// number of keys: that is how the all-ones row works, without any special case here.
template <bool FULL>
__device__ __forceinline__ void a64_softmax(uint32_t t_lane, uint8_t *prow, int row, int valid, float &m_run,
                                            float &l_run, float &alpha) {
    using namespace sm100;
    const float kScaleLog2 = kScale * kLog2e;
    uint32_t sv[2][32];
    float mx = -INFINITY;
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
        tmem_ld32_issue(t_lane + hf * 64, sv[0]);
        tmem_ld32_issue(t_lane + hf * 64 + 32, sv[1]);
        tmem_ld_wait();
        tmem_ld_fence32(sv[0]); tmem_ld_fence32(sv[1]);
#pragma unroll
        for (int x = 0; x < 64; ++x)
            if (FULL || hf * 64 + x < valid) mx = fmaxf(mx, __uint_as_float(sv[x >> 5][x & 31]));
    }
    const bool any = FULL || valid > 0;                        // an absent tile contributes nothing
    const float m_new = fmaxf(m_run, mx * kScaleLog2);
    const float m_use = any ? m_new : 0.f;
    alpha = any ? fast_exp2(m_run - m_new) : 1.f;              // 0 on a thread's first tile
    float lsum = 0.f;
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
        tmem_ld32_issue(t_lane + hf * 64, sv[0]);
        tmem_ld32_issue(t_lane + hf * 64 + 32, sv[1]);
        tmem_ld_wait();
        tmem_ld_fence32(sv[0]); tmem_ld_fence32(sv[1]);
        uint8_t *pp = prow + hf * 8192;                        // panel hf: keys 64 * hf ..
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {                       // 8 keys = one 16-byte chunk
            uint32_t packed[4];
#pragma unroll
            for (int x = 0; x < 8; x += 2) {
                const int col = ch * 8 + x;
                const float s0 = __uint_as_float(sv[col >> 5][col & 31]);
                const float s1 = __uint_as_float(sv[(col + 1) >> 5][(col + 1) & 31]);
                const float p0 = (FULL || hf * 64 + col < valid) ? fast_exp2(fmaf(s0, kScaleLog2, -m_use)) : 0.f;
                const float p1 = (FULL || hf * 64 + col + 1 < valid) ? fast_exp2(fmaf(s1, kScaleLog2, -m_use)) : 0.f;
                lsum += p0 + p1;
                __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
                packed[x >> 1] = *reinterpret_cast<uint32_t *>(&pk);
            }
            *reinterpret_cast<uint4 *>(pp + ((ch ^ (row & 7)) << 4)) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
        }
    }
    if (any) { l_run = l_run * alpha + lsum; m_run = m_new; }
}

// All threads of the CTA call this (it contains __syncthreads).  On return the threads of
// warpgroup 0 with lane < 16 hold, for row 16 * (warp - wg_warp0) + lane, the softmax state over
// [lo, hi): m (scaled log2 units), l, acc[64] (unnormalised).  Returns false if a wait expired.
__device__ __forceinline__ bool attend64_run(uint8_t *smem, uint32_t tmem_base, const Geom &g,
                                             const Attend64Job &j, const __nv_bfloat16 *__restrict__ Q,
                                             const CUtensorMap *tmK, const CUtensorMap *tmV, float &m_out,
                                             float &l_out, float acc[kD]) {
    using namespace sm100;
    uint64_t *kfull = reinterpret_cast<uint64_t *>(smem + kA64OffBar);   // [2] per warpgroup
    // sfull[2 wg + x]: scores in accumulator x of warpgroup wg; sfree[wg]: the warpgroup has read O of a pair
    uint64_t *vfull = kfull + 2, *sfull = kfull + 4, *pready = kfull + 8, *ofull = kfull + 10, *sfree = kfull + 12;
    volatile uint32_t *abort_flag = reinterpret_cast<uint32_t *>(kfull + 14);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_tiles = (j.hi - j.lo + 127) / 128, n_pairs = (n_tiles + 1) / 2;

    auto coords = [&](int tile, int &c1, int &c2, int &c3) {
        const int key0 = j.lo + tile * 128;
        c1 = j.pos_t == 1 ? key0 : (j.pos_h == 1 ? j.h : j.b);
        c2 = j.pos_t == 2 ? key0 : (j.pos_h == 2 ? j.h : j.b);
        c3 = j.pos_t == 3 ? key0 : (j.pos_h == 3 ? j.h : j.b);
    };
    auto load_pair = [&](int wg, int q, bool is_v) {            // control thread only
        uint8_t *dst = smem + kA64OffWg + wg * kA64WgBytes + (is_v ? 2 * kA64Tile : 0);
        uint64_t *bar = is_v ? &vfull[wg] : &kfull[wg];
        const int two = (2 * q + 1 < n_tiles) ? 1 : 0;
        mbar_expect_tx(bar, kA64Tile * (1 + two));
        for (int s = 0; s <= two; ++s) {
            int c1, c2, c3;
            coords(2 * q + s, c1, c2, c3);
            tma_load_4d(dst + s * kA64Tile, is_v ? tmV : tmK, bar, 0, c1, c2, c3);
        }
    };
    if (!j.started && warp == j.ctrl_warp && lane == 0) attend64_start(smem, j, tmK, tmV);
    // Q rows -> shared memory, K-major, 128-byte swizzle; unused rows are zero
    for (int e = tid; e < kA64MaxRows * 8; e += blockDim.x) {
        const int r = e >> 3, c = e & 7;
        int i = -1;
        if (r < j.n_rows) i = j.rows ? j.rows[r] : r;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (i >= 0 && i < j.L)
            v = __ldg(reinterpret_cast<const uint4 *>(Q + unit_off(g.qs, j.b, j.h) + (long long)i * g.qs[2]) + c);
        *reinterpret_cast<uint4 *>(smem + kA64OffQ + r * 128 + ((c ^ (r & 7)) << 4)) = v;
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    float m_run = -INFINITY, l_run = 0.f;
#pragma unroll
    for (int c = 0; c < kD; ++c) acc[c] = 0.f;

    if (warp >= j.ctrl_warp && warp < j.ctrl_warp + 2) {
        const int wg = warp - j.ctrl_warp;
        if (lane == 0 && wg < n_pairs) {
            // ---------------- control thread of warpgroup wg: a straight-line program per pair -------------
            constexpr uint32_t kIdescS = umma_idesc_bf16(64, 128, 0);       // B = K tile, K-major
            constexpr uint32_t kIdescO = umma_idesc_bf16(64, kD, 1);        // B = V tile, MN-major
            const uint32_t wg_smem = smem_u32(smem + kA64OffWg + wg * kA64WgBytes);
            const uint32_t qa = smem_u32(smem + kA64OffQ);
            const uint32_t t_wg = tmem_base + wg * 256;
            auto issue_s = [&](int q, int x) {                 // S_a = Q K_a^T, S_b = Q K_b^T into accumulator x
                const int two = (2 * q + 1 < n_tiles) ? 1 : 0;
                for (int s = 0; s <= two; ++s)
#pragma unroll
                    for (int k = 0; k < kD / 16; ++k)
                        umma_bf16(t_wg + x * 128 + ((uint32_t)(16 * s) << 16), umma_desc_sw128(qa + k * 32, 16, 1024),
                                  umma_desc_sw128(wg_smem + s * kA64Tile + k * 32, 16, 1024), kIdescS, k > 0);
                umma_commit(&sfull[2 * wg + x]);
            };
            auto give_up = [&]() { *abort_flag = 1u; atomicOr(g.status, kStatusWaitExpired); };
            bool alive = !*abort_flag;
            if (alive && !mbar_wait(&kfull[wg], 0)) { give_up(); alive = false; }
            if (alive) { tc_fence_after(); issue_s(wg, 0); }
            int cnt = 0;
            for (int q = wg; alive && q < n_pairs; q += 2, ++cnt) {
                const uint32_t ph = (uint32_t)(cnt & 1);
                const int x = cnt & 1;
                const bool more = q + 2 < n_pairs;
                const int two = (2 * q + 1 < n_tiles) ? 1 : 0;
                // the K buffers are free once S is done: bring in the next pair's keys
                if (!mbar_wait(&sfull[2 * wg + x], (uint32_t)((cnt >> 1) & 1))) { give_up(); break; }
                if (more) load_pair(wg, q + 2, false);
                // Two things are due now, in whichever order they become possible:
                //   the next pair's scores, once its keys have landed and the other accumulator has been read out
                //   (O of the pair before this one sat there);
                //   O_a = P_a V_a, O_b = P_b V_b of this pair, once the warpgroup has written P and V has landed.
                bool s_due = more, o_due = true, other_free = cnt == 0;
                const unsigned long long t0 = global_ns();
                for (int spin = 0; s_due || o_due; ++spin) {
                    if (!other_free) other_free = mbar_test(&sfree[wg], ph ^ 1u);
                    if (s_due && other_free && mbar_test(&kfull[wg], ph ^ 1u)) {
                        tc_fence_after();
                        issue_s(q + 2, x ^ 1);
                        s_due = false;
                    }
                    if (o_due && mbar_test(&pready[wg], ph) && mbar_test(&vfull[wg], ph)) {
                        tc_fence_after();
                        for (int s = 0; s <= two; ++s)
#pragma unroll
                            for (int k = 0; k < 8; ++k)
                                umma_bf16(t_wg + x * 128 + ((uint32_t)(16 * s) << 16),
                                          umma_desc_sw128(wg_smem + (4 + s) * kA64Tile + (k >> 2) * 8192 + (k & 3) * 32, 16, 1024),
                                          umma_desc_sw128(wg_smem + (2 + s) * kA64Tile + k * 2048, 16, 1024), kIdescO, k > 0);
                        umma_commit(&ofull[wg]);
                        o_due = false;
                    }
                    if ((spin & 63) == 63 && (*abort_flag || global_ns() - t0 > kWaitNs)) { give_up(); alive = false; break; }
                }
                if (!alive) break;
                // the V buffers are free once O is done
                if (!mbar_wait(&ofull[wg], ph)) { give_up(); break; }
                if (more) load_pair(wg, q + 2, true);
                if (*abort_flag) break;
            }
        }
    } else if (warp >= j.wg_warp0 && warp < j.wg_warp0 + 8) {
        // ---------------------------------- warpgroups ------------------------------------------------
        const int wg = (warp - j.wg_warp0) >> 2, w4 = (warp - j.wg_warp0) & 3;
        const int sub = lane >> 4, row = 16 * w4 + (lane & 15);
        const bool warp_active = 16 * w4 < max(j.n_rows, j.sum_row + 1);
        const int wtid = (warp - j.wg_warp0 - 4 * wg) * 32 + lane;          // 0..127 inside the warpgroup
        uint8_t *wg_smem = smem + kA64OffWg + wg * kA64WgBytes;
        const uint32_t t_lane0 = tmem_base + wg * 256 + ((uint32_t)(32 * w4) << 16);
        uint8_t *prow = wg_smem + (4 + sub) * kA64Tile + row * 128;
        int cnt = 0;
        for (int q = wg; q < n_pairs; q += 2, ++cnt) {
            const uint32_t ph = (uint32_t)(cnt & 1);
            if (*abort_flag) break;
            const uint32_t t_lane = t_lane0 + (uint32_t)(cnt & 1) * 128u;   // this pair's accumulator
            if (!mbar_wait(&sfull[2 * wg + (cnt & 1)], (uint32_t)((cnt >> 1) & 1))) { *abort_flag = 1u; atomicOr(g.status, kStatusWaitExpired); break; }
            tc_fence_after();
            const int valid_a = min(128, j.hi - (j.lo + 2 * q * 128));
            const int valid_b = max(0, min(128, j.hi - (j.lo + (2 * q + 1) * 128)));
            const int valid = sub ? valid_b : valid_a;
            float alpha = 1.f;
            __syncwarp();
            if (warp_active) {
                if (valid_a == 128 && valid_b == 128) a64_softmax<true>(t_lane, prow, row, 128, m_run, l_run, alpha);
                else a64_softmax<false>(t_lane, prow, row, valid, m_run, l_run, alpha);
            }
            // rows of V past the valid length may hold anything (even NaN): zero them so that 0 * x stays 0
            if (valid_a < 128 || (valid_b > 0 && valid_b < 128)) {          // uniform over the warpgroup
                if (!mbar_wait(&vfull[wg], ph)) { *abort_flag = 1u; atomicOr(g.status, kStatusWaitExpired); break; }
                uint4 *va = reinterpret_cast<uint4 *>(wg_smem + 2 * kA64Tile), *vb = reinterpret_cast<uint4 *>(wg_smem + 3 * kA64Tile);
                for (int e = valid_a * 8 + wtid; e < 128 * 8; e += 128) va[e] = make_uint4(0u, 0u, 0u, 0u);
                if (valid_b > 0)
                    for (int e = valid_b * 8 + wtid; e < 128 * 8; e += 128) vb[e] = make_uint4(0u, 0u, 0u, 0u);
            }
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(&pready[wg]);
            if (!mbar_wait(&ofull[wg], ph)) { *abort_flag = 1u; atomicOr(g.status, kStatusWaitExpired); break; }
            tc_fence_after();
            __syncwarp();
            if (warp_active) {
                uint32_t ov[2][32];
                tmem_ld32_issue(t_lane, ov[0]);                 // O sits over the first 64 score columns
                tmem_ld32_issue(t_lane + 32, ov[1]);
                tmem_ld_wait();
                tmem_ld_fence32(ov[0]); tmem_ld_fence32(ov[1]);
                if (valid > 0) {
#pragma unroll
                    for (int x = 0; x < 64; ++x) acc[x] = fmaf(acc[x], alpha, __uint_as_float(ov[x >> 5][x & 31]));
                }
            }
            tc_fence_before();
            mbar_arrive(&sfree[wg]);                           // this accumulator may take the scores of pair q + 4
        }
        // merge the two tiles of the pair stream: lanes l and l ^ 16 hold the same row
        __syncwarp();
        {
            const float m_o = __shfl_xor_sync(0xffffffffu, m_run, 16);
            const float m_new = fmaxf(m_run, m_o);
            const float f = l_run > 0.f ? fast_exp2(m_run - m_new) : 0.f;
            l_run *= f;
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 16);
#pragma unroll
            for (int c = 0; c < kD; ++c) {
                const float x = acc[c] * f;
                acc[c] = x + __shfl_xor_sync(0xffffffffu, x, 16);
            }
            m_run = m_new;
        }
    }
    tc_fence_before();
    __syncthreads();
    // merge warpgroup 1 into warpgroup 0 through shared memory (the P area of warpgroup 1 is free now)
    float *xchg = reinterpret_cast<float *>(smem + kA64OffWg + kA64WgBytes + 4 * kA64Tile);
    if (warp >= j.wg_warp0 + 4 && warp < j.wg_warp0 + 8 && lane < 16) {
        const int row = 16 * (warp - j.wg_warp0 - 4) + lane;
        xchg[row * 66] = m_run; xchg[row * 66 + 1] = l_run;
#pragma unroll
        for (int c = 0; c < kD; ++c) xchg[row * 66 + 2 + c] = acc[c];
    }
    __syncthreads();
    if (warp >= j.wg_warp0 && warp < j.wg_warp0 + 4 && lane < 16) {
        const int row = 16 * (warp - j.wg_warp0) + lane;
        const float m1 = xchg[row * 66], l1 = xchg[row * 66 + 1];
        const float m_new = fmaxf(m_run, m1);
        const float f0 = l_run > 0.f ? fast_exp2(m_run - m_new) : 0.f, f1 = l1 > 0.f ? fast_exp2(m1 - m_new) : 0.f;
        l_run = l_run * f0 + l1 * f1;
#pragma unroll
        for (int c = 0; c < kD; ++c) acc[c] = acc[c] * f0 + xchg[row * 66 + 2 + c] * f1;
        m_run = m_new;
    }
    m_out = m_run; l_out = l_run;
    const bool ok = *abort_flag == 0u;
    if (!ok && tid == 0) {
        // copies that were issued but never consumed: give them a bounded chance to land
        for (int x = 0; x < 2; ++x) { mbar_wait(&kfull[x], 0); mbar_wait(&vfull[x], 0); }
    }
    __syncthreads();
    return ok;
}

}  // namespace psattn
