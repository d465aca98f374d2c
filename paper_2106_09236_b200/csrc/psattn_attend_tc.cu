// Step (d) on the tensor cores (bf16 inputs): softmax attention (Eq. 7-8) of a list of query
// rows over all valid keys of their unit, flash style, for row lists longer than 64 (Sec. 3.2's own
// count L_sparse = r_sparse L) and for the dense comparator (Eq. 6: every valid query).
//
// One CTA = (unit, two tiles of up to 128 listed rows, key split), 320 threads:
//   warps 0-3 / 4-7  softmax warpgroups A / B: thread = one row of the warpgroup's query tile = one TMEM lane
//   warp 8           one thread issues every tcgen05.mma
//   warp 9           one thread streams 128-key K and V tiles through two 3-stage rings by TMA (128-byte swizzle);
//                    both query tiles use the same key tile, so K and V cross L2 -> shared memory once per 256 rows
// Per key tile t and warpgroup w:
//   tcgen05   S_w = Q_w K_t^T            -> TMEM (128 lanes x 128 fp32 columns)
//   threads   one pass over the row's 128 scores (32 at a time in registers, the next 32 in flight): exponentials
//             relative to the row's reference, P (bf16) -> shared memory (A-operand layout), the maximum on the side
//   tcgen05   O_w += P_w V_t             -> TMEM (64 columns), accumulated across key tiles; V is the MN-major B
//                                           operand exactly as TMA wrote it
// The issuing thread runs "P V of tile t, then S of tile t + 1" for A and for B in turn, so the tensor pipe
// works on one warpgroup's tiles while the other warpgroup does its softmax.  O never leaves TMEM between
// tiles: the exponentials are taken relative to a per-row reference that only moves when the row maximum
// exceeds it by more than 2^8 (the weights then stay below 2^8, fine for bf16 and fp32), and only then is the
// row of O read, scaled and written back (tcgen05.ld / tcgen05.st).  Because tcgen05.commit tracks every
// product issued before it, "S of tile t has arrived" also says that P V of tile t - 1 has finished: at that
// point the warpgroup may rescale O and overwrite P.
// With one split the rows are finished here; otherwise (reference, l, acc) go to the workspace and the
// split-merge kernel of the staged schedule finishes them.
#include "psattn_launch.h"
#include "psattn_sm100.cuh"

namespace psattn {

using namespace sm100;

constexpr int kTileKeys = 128;
constexpr int kTileRows = 128;
constexpr int kCtaRows = 2 * kTileRows;                      // two query tiles per CTA
constexpr int kTcThreads = 320;
constexpr int kTcStages = 3;
constexpr uint32_t kTileBytes = kTileKeys * kD * 2;          // 16 KB: one K, V, Q or half-P tile
constexpr uint32_t kTmemCols = 512;                          // S_A [0,128) S_B [128,256) O_A [256,320) O_B [320,384)
constexpr uint32_t kOffQ = 0, kOffK = 2 * kTileBytes, kOffV = kOffK + kTcStages * kTileBytes,
                   kOffP = kOffV + kTcStages * kTileBytes,   // per warpgroup: two panels of 64 keys, 16 KB each
                   kOffBar = kOffP + 4 * kTileBytes;
constexpr uint32_t kAttendSmem = kOffBar + 256;
static_assert(kAttendSmem <= 227 * 1024, "the CTA's tiles must fit the shared memory of one SM");
static_assert(kAttendSmem <= 227 * 1024, "the CTA's tiles must fit the shared memory of one SM");
constexpr bool kTakeTurns = true;                            // the softmax warpgroups alternate on the exponential unit
constexpr float kRefSlack = 8.f;                             // the reference follows the row maximum in steps of 2^8

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

// 32 consecutive fp32 columns of this thread's TMEM lane, written from registers.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t r[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// One pass over a row's 128 scores in TMEM, 32 columns at a time, the next block of 32 in flight while the
// current one is worked on.  EXP: the exponentials relative to `ref` (scaled log2 units) go to the row's place in
// P as bf16 (two panels of 64 keys in the A-operand layout, 128-byte swizzle) and their sum to `lsum`; the largest
// raw score of the valid columns goes to `mx` in any case.  FULL: all 128 keys exist.
template <bool EXP, bool FULL>
__device__ __forceinline__ void tc_row_pass(uint32_t t_s, float ref, int valid, uint8_t *prow, int row, float &mx, float &lsum) {
    const float kScaleLog2 = kScale * kLog2e;
    uint32_t buf[2][32];
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    tmem_ld32_issue(t_s, buf[0]);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint32_t (&cur)[32] = buf[q & 1];
        tmem_ld_wait();
        tmem_ld_fence32(cur);
        if (q < 3) tmem_ld32_issue(t_s + (q + 1) * 32, buf[(q + 1) & 1]);
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {                        // 8 keys = one 16-byte chunk of P
            uint32_t packed[4];
#pragma unroll
            for (int x = 0; x < 8; x += 2) {
                const int c = ch * 8 + x, col = q * 32 + c;
                const float s0 = __uint_as_float(cur[c]), s1 = __uint_as_float(cur[c + 1]);
                if (FULL || col < valid) m0 = fmaxf(m0, s0);
                if (FULL || col + 1 < valid) m1 = fmaxf(m1, s1);
                if (EXP) {
                    const float p0 = (FULL || col < valid) ? fast_exp2(fmaf(s0, kScaleLog2, -ref)) : 0.f;
                    const float p1 = (FULL || col + 1 < valid) ? fast_exp2(fmaf(s1, kScaleLog2, -ref)) : 0.f;
                    l0 += p0; l1 += p1;
                    __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
                    packed[x >> 1] = *reinterpret_cast<uint32_t *>(&pk);
                }
            }
            if (EXP)
                *reinterpret_cast<uint4 *>(prow + (q >> 1) * kTileBytes + ((((q & 1) * 4 + ch) ^ (row & 7)) << 4)) =
                    make_uint4(packed[0], packed[1], packed[2], packed[3]);
        }
    }
    mx = fmaxf(m0, m1);
    lsum = l0 + l1;
}

__global__ void __launch_bounds__(kTcThreads, 1) k_attend_tc(Geom g, AttendTcArgs a,
                                                             const __nv_bfloat16 *__restrict__ Q,
                                                             const __grid_constant__ CUtensorMap tmK,
                                                             const __grid_constant__ CUtensorMap tmV) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *k_full = reinterpret_cast<uint64_t *>(smem + kOffBar);        // [3]
    uint64_t *k_empty = k_full + kTcStages, *v_full = k_empty + kTcStages, *v_empty = v_full + kTcStages;
    uint64_t *s_full = v_empty + kTcStages;                                 // [2] scores of warpgroup w have arrived
    uint64_t *p_ready = s_full + 2;                                         // [2] warpgroup w has written P (128 arrivals)
    uint64_t *o_final = p_ready + 2;                                        // [2] the last P V of warpgroup w has finished
    uint64_t *turn = o_final + 2;                                           // [2] warpgroup w may take the exponential unit (128 arrivals)
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(turn + 2);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int split = blockIdx.x, pair = blockIdx.y, unit = blockIdx.z;
    const int b = unit / g.H, h = unit % g.H;
    const int L = seq_len(g, b);
    const int lo = min(L, split * a.split_keys), hi = min(L, lo + a.split_keys);
    const int n_tiles = (hi - lo + kTileKeys - 1) / kTileKeys;
    const bool has_b = pair * kCtaRows + kTileRows < a.n_rows;  // the second query tile lists rows

    if ((smem_u32(smem) & 1023u) != 0u) {                      // swizzled tiles need a 1024-byte base
        if (tid == 0) atomicOr(g.status, kStatusWaitExpired);
        return;
    }
    if (tid == 9 * 32) {
        for (int s = 0; s < kTcStages; ++s) { mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1); mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1); }
        for (int w = 0; w < 2; ++w) { mbar_init(&s_full[w], 1); mbar_init(&p_ready[w], 128); mbar_init(&o_final[w], 1); mbar_init(&turn[w], 128); }
        *abort_flag = 0u;
        fence_barrier_init();
        tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
    }
    if (warp == 8) tmem_alloc(tmem_slot, kTmemCols);

    // the listed row of this thread (softmax warpgroups) and its Q row -> shared memory, K-major, 128-byte swizzle
    const int wg = warp >> 2, wrow = tid & 127;
    const int r = pair * kCtaRows + wg * kTileRows + wrow;     // slot in the row list
    int i = -1;
    if (warp < 8 && r < a.n_rows) i = a.rows ? a.rows[(long long)unit * a.rows_stride + r] : r;
    const bool row_ok = i >= 0 && i < L;
    if (warp < 8) {
        uint4 *dst = reinterpret_cast<uint4 *>(smem + kOffQ + wg * kTileBytes + wrow * 128);
        const uint4 *src = reinterpret_cast<const uint4 *>(Q + unit_off(g.qs, b, h) + (long long)(row_ok ? i : 0) * g.qs[2]);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (row_ok) v = __ldg(src + c);
            dst[c ^ (wrow & 7)] = v;
        }
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    auto give_up = [&]() { *abort_flag = 1u; atomicOr(g.status, kStatusWaitExpired); };

    float m_ref = -INFINITY, l_run = 0.f;                      // softmax state of this thread's row
    if (warp == 9) {
        // ---------------- producer: K and V tiles through their rings ----------------------------------------
        if (lane == 0) {
            for (int t = 0; t < n_tiles && !*abort_flag; ++t) {
                const int s = t % kTcStages;
                const uint32_t ph = (uint32_t)((t / kTcStages) & 1);
                const int key0 = lo + t * kTileKeys;
                const int c1 = a.pos_t == 1 ? key0 : (a.pos_h == 1 ? h : b);
                const int c2 = a.pos_t == 2 ? key0 : (a.pos_h == 2 ? h : b);
                const int c3 = a.pos_t == 3 ? key0 : (a.pos_h == 3 ? h : b);
                if (!mbar_wait(&k_empty[s], ph ^ 1u, g.wait_ns)) { give_up(); break; }
                mbar_expect_tx(&k_full[s], kTileBytes + (t == 0 ? g.debug_extra_tx : 0u));
                tma_load_4d(smem + kOffK + s * kTileBytes, &tmK, &k_full[s], 0, c1, c2, c3);
                if (!mbar_wait(&v_empty[s], ph ^ 1u, g.wait_ns)) { give_up(); break; }
                mbar_expect_tx(&v_full[s], kTileBytes);
                tma_load_4d(smem + kOffV + s * kTileBytes, &tmV, &v_full[s], 0, c1, c2, c3);
            }
        }
    } else if (warp == 8) {
        // ---------------- the thread that issues every product -----------------------------------------------
        if (lane == 0 && n_tiles > 0) {
            constexpr uint32_t kIdescS = umma_idesc_bf16(kTileRows, kTileKeys, 0);   // B = K tile, K-major
            constexpr uint32_t kIdescO = umma_idesc_bf16(kTileRows, kD, 1);          // B = V tile, MN-major
            const int n_wg = has_b ? 2 : 1;
            // The descriptors are built once; a k-step or a ring stage only adds to the start-address field (in
            // 16-byte units; shared-memory addresses stay below 2^18, so the 14-bit field never carries over).  The
            // issuing thread shares its scheduler with two softmax warps: every instruction it saves shortens the
            // time from "P is written" to "the products are queued".
            const uint64_t dq = umma_desc_sw128(smem_u32(smem + kOffQ), 16, 1024), dk = umma_desc_sw128(smem_u32(smem + kOffK), 16, 1024);
            const uint64_t dp = umma_desc_sw128(smem_u32(smem + kOffP), 16, 1024), dv = umma_desc_sw128(smem_u32(smem + kOffV), 16, 1024);
            constexpr uint64_t kTile16 = kTileBytes >> 4;
            auto issue_s = [&](int w, int t) {
                const uint64_t a0 = dq + (uint64_t)w * kTile16, b0 = dk + (uint64_t)(t % kTcStages) * kTile16;
#pragma unroll
                for (int k = 0; k < kD / 16; ++k) umma_bf16(tmem_base + w * 128, a0 + 2 * k, b0 + 2 * k, kIdescS, k > 0);
                umma_commit(&s_full[w]);
            };
            bool alive = !*abort_flag;
            if (alive && !mbar_wait(&k_full[0], 0u, g.wait_ns)) { give_up(); alive = false; }
            if (alive) {
                tc_fence_after();
                for (int w = 0; w < n_wg; ++w) issue_s(w, 0);
                umma_commit(&k_empty[0]);
            }
            for (int t = 0; alive && t < n_tiles; ++t) {
                const int s = t % kTcStages, sn = (t + 1) % kTcStages;
                const uint32_t ph = (uint32_t)((t / kTcStages) & 1), phn = (uint32_t)(((t + 1) / kTcStages) & 1);
                for (int w = 0; w < n_wg; ++w) {
                    if (!mbar_wait(&p_ready[w], (uint32_t)(t & 1), g.wait_ns)) { give_up(); alive = false; break; }
                    if (w == 0 && !mbar_wait(&v_full[s], ph, g.wait_ns)) { give_up(); alive = false; break; }
                    tc_fence_after();
                    const uint64_t pa = dp + (uint64_t)(2 * w) * kTile16, va = dv + (uint64_t)s * kTile16;
#pragma unroll
                    for (int k = 0; k < kTileKeys / 16; ++k)
                        umma_bf16(tmem_base + 256 + w * 64, pa + (uint64_t)((k >> 2) * kTile16 + (k & 3) * 2), va + (uint64_t)(k * 128),
                                  kIdescO, (t > 0 || k > 0) ? 1u : 0u);
                    if (w == n_wg - 1) umma_commit(&v_empty[s]);
                    if (t + 1 < n_tiles) {
                        if (w == 0 && !mbar_wait(&k_full[sn], phn, g.wait_ns)) { give_up(); alive = false; break; }
                        tc_fence_after();
                        issue_s(w, t + 1);
                        if (w == n_wg - 1) umma_commit(&k_empty[sn]);
                    } else {
                        umma_commit(&o_final[w]);
                    }
                }
                if (*abort_flag) break;
            }
        }
    } else if (wg == 0 || has_b) {
        // ---------------- softmax warpgroups: thread = row = TMEM lane ------------------------------------------
        const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t t_s = lane_base + wg * 128, t_o = lane_base + 256 + wg * 64;
        uint8_t *prow = smem + kOffP + wg * 2 * kTileBytes + wrow * 128;
        const float kScaleLog2 = kScale * kLog2e;
        for (int t = 0; t < n_tiles; ++t) {
            if (*abort_flag) break;
            if (!mbar_wait(&s_full[wg], (uint32_t)(t & 1), g.wait_ns)) { give_up(); break; }
            tc_fence_after();
            const int valid = min(kTileKeys, hi - (lo + t * kTileKeys));     // keys of this tile that exist (>= 1)
            const bool full = valid == kTileKeys;
            float mx, lsum;
            // The exponentials are bound by the special-function unit (16 per clock and SM).  Left alone, the two
            // warpgroups fall into step: both take it at half speed, then both wait for their products while it idles.
            // So they take turns: B starts the exponentials of tile t when A has issued its own, A those of tile t + 1
            // when B has; each one's wait for the tensor pipe then lies under the other one's exponentials.
            if (kTakeTurns && has_b && (wg == 1 || t > 0)) {
                if (!mbar_wait(&turn[wg], (uint32_t)((wg == 1 ? t : t - 1) & 1), g.wait_ns)) { give_up(); break; }
            }
            if (t == 0) {
                // the first tile fixes the reference: a pass for the maximum, then the exponentials
                if (full) tc_row_pass<false, true>(t_s, 0.f, valid, prow, wrow, mx, lsum);
                else tc_row_pass<false, false>(t_s, 0.f, valid, prow, wrow, mx, lsum);
                m_ref = mx * kScaleLog2;
                if (full) tc_row_pass<true, true>(t_s, m_ref, valid, prow, wrow, mx, lsum);
                else tc_row_pass<true, false>(t_s, m_ref, valid, prow, wrow, mx, lsum);
                l_run = lsum;
            } else {
                // Later tiles take ONE pass: the exponentials relative to the standing reference, the maximum on the
                // side.  P V of tile t - 1 has finished (see the head of the file), so P may be overwritten.
                if (full) tc_row_pass<true, true>(t_s, m_ref, valid, prow, wrow, mx, lsum);
                else tc_row_pass<true, false>(t_s, m_ref, valid, prow, wrow, mx, lsum);
                const float mxs = mx * kScaleLog2;
                const bool moved = mxs > m_ref + kRefSlack;
                if (__any_sync(0xffffffffu, moved)) {
                    // rare: the maximum has run away from the reference (the weights just written may even have
                    // overflowed).  The reference follows, the row of O (stable: no product is in flight) and the
                    // row sum are scaled, and the row's weights are written again.
                    const float alpha = moved ? fast_exp2(m_ref - mxs) : 1.f;
                    uint32_t ov[2][32];
                    tmem_ld32_issue(t_o, ov[0]);
                    tmem_ld32_issue(t_o + 32, ov[1]);
                    tmem_ld_wait();
                    tmem_ld_fence32(ov[0]); tmem_ld_fence32(ov[1]);
#pragma unroll
                    for (int x = 0; x < 64; ++x) ov[x >> 5][x & 31] = __float_as_uint(__uint_as_float(ov[x >> 5][x & 31]) * alpha);
                    tmem_st32(t_o, ov[0]);
                    tmem_st32(t_o + 32, ov[1]);
                    tmem_st_wait();
                    if (moved) m_ref = mxs;
                    if (full) tc_row_pass<true, true>(t_s, m_ref, valid, prow, wrow, mx, lsum);
                    else tc_row_pass<true, false>(t_s, m_ref, valid, prow, wrow, mx, lsum);
                    l_run = l_run * alpha + lsum;
                } else {
                    l_run += lsum;
                }
            }
            if (kTakeTurns && has_b && (wg == 0 || t + 1 < n_tiles)) mbar_arrive(&turn[wg ^ 1]);
            // rows of V past the valid length may hold anything (even NaN): zero them so that 0 * x stays 0
            if (valid < kTileKeys) {                                // uniform over the CTA (both warpgroups write zeros)
                const int s = t % kTcStages;
                if (!mbar_wait(&v_full[s], (uint32_t)((t / kTcStages) & 1), g.wait_ns)) { give_up(); break; }
                uint4 *vrows = reinterpret_cast<uint4 *>(smem + kOffV + s * kTileBytes);
                for (int e = valid * 8 + wrow; e < kTileKeys * 8; e += 128) vrows[e] = make_uint4(0u, 0u, 0u, 0u);
            }
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(&p_ready[wg]);
        }
        // ---- results: the row of O, divided by the row sum ---------------------------------------------------
        float acc[kD];
#pragma unroll
        for (int c = 0; c < kD; ++c) acc[c] = 0.f;
        if (n_tiles > 0 && !*abort_flag) {
            if (!mbar_wait(&o_final[wg], 0u, g.wait_ns)) give_up();
            else {
                tc_fence_after();
                uint32_t ov[2][32];
                tmem_ld32_issue(t_o, ov[0]);
                tmem_ld32_issue(t_o + 32, ov[1]);
                tmem_ld_wait();
                tmem_ld_fence32(ov[0]); tmem_ld_fence32(ov[1]);
#pragma unroll
                for (int x = 0; x < 64; ++x) acc[x] = __uint_as_float(ov[x >> 5][x & 31]);
            }
        }
        if (r < a.n_rows && !*abort_flag) {
            if (a.n_splits == 1) {
                const float inv = (row_ok && l_run > 0.f) ? 1.f / l_run : 0.f;
                float o[kD];
#pragma unroll
                for (int c = 0; c < kD; ++c) o[c] = row_ok ? acc[c] * inv : 0.f;
                if (a.out_by_position) {
                    // with the identity list (every position is a row) the padded positions get their zero rows here
                    if (row_ok || (a.rows == nullptr && i >= 0 && i < g.T)) {
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
                a.part_ml[2 * slot] = (row_ok && n_tiles > 0) ? m_ref : -INFINITY;
                a.part_ml[2 * slot + 1] = (row_ok && n_tiles > 0) ? l_run : 0.f;
                float *dst = a.part_acc + slot * kD;
#pragma unroll
                for (int c8 = 0; c8 < 8; ++c8) store8(dst, c8, acc + 8 * c8);
            }
        }
    }
    // ---- teardown: nothing of this CTA may still be in flight when its TMEM is released ---------
    tc_fence_before();
    __syncthreads();
    if (tid == 9 * 32 && *abort_flag) {
        // tiles that were requested but perhaps never consumed: give every ring slot a bounded chance to land
        for (int s = 0; s < kTcStages && s < n_tiles; ++s) {
            const int t_last = ((n_tiles - 1 - s) / kTcStages) * kTcStages + s;     // the last tile that uses slot s
            mbar_wait(&k_full[s], (uint32_t)((t_last / kTcStages) & 1), g.wait_ns);
            mbar_wait(&v_full[s], (uint32_t)((t_last / kTcStages) & 1), g.wait_ns);
        }
    }
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem_base, kTmemCols);
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
    if ((long long)g.B * g.H > 65535 || (n_rows + kCtaRows - 1) / kCtaRows > 65535) return cudaErrorNotSupported;   // gridDim.z, .y
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
    // one CTA per SM: 192 KB of shared memory, all 512 TMEM columns
    static SmemGrant grant;
    if (cudaError_t e = grant_dynamic_smem(k_attend_tc, grant, kAttendSmem, true)) return e;
    dim3 grid((unsigned)n_splits, (unsigned)((n_rows + kCtaRows - 1) / kCtaRows), (unsigned)(g.B * g.H));
    k_attend_tc<<<grid, kTcThreads, kAttendSmem, st>>>(g, a, (const __nv_bfloat16 *)Q, tmK, tmV);
    note_launch();
    return cudaGetLastError();
}

}  // namespace psattn
