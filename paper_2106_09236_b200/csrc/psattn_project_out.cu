// The output matrix of the attention module (Sec. 2.2, Eq. 5: the module inside the Conformer block; Sec. 3.1:
// its heads): Y[b][t][:] = sum_h O[b][h][t][:] W_o^h, W_o stored transposed (Wot[n][h * 64 + e]).
//
// After Eq. 12 with the mean(V) fill almost all rows of a unit are one and the same vector F_h (the fill row), so
//   Y[b][t][:] = base_b + sum over the heads h that selected t of (O[b][h][t][:] - F_h) W_o^h,
//   base_b = sum_h F_h W_o^h,
// i.e. one row per sequence broadcast to every position, plus a correction for the H * u selected (head,
// position) pairs: O(B H u d d_y) products instead of the O(B T (H d) d_y) of the dense GEMM.
//
// k_project_out_rows: one CTA = (64 output columns, a range of positions of one sequence).  It keeps its
// 64 x (H * 64) slice of the weights in shared memory, computes c_h = F_h W_o^h and base for its columns,
// lists the (head, position) pairs of its range (every head's rows padded to whole 16-row tiles) and runs
// them through mma.sync (A = the rows of O, read in place, B = the head's block of the weight slice), keeps the products
// in shared memory, and writes its 64-column slice of every valid row of its range: base for the positions
// nobody picked, base + sum over the picking heads (in head order, so the result does not depend on timing)
// of (product - c_h) for the others.  Padded rows are not written.
// The dense form (any O, no index set) runs as one tcgen05 GEMM (psattn_project.cu); fp32 and odd shapes
// run one thread per output element.
#include "psattn_launch.h"
#include "psattn_sm100.cuh"

namespace psattn {

constexpr int kPoThreads = 256;
constexpr int kPoCols = 64;                  // output columns per CTA
constexpr int kPoMaxRows = 64;               // selected rows of one head (u_max <= 64)
constexpr int kPoMaxChunk = 1024;            // positions per CTA at most

struct OutArgs {
    int B, H, T, dy, u_max, t_chunk, max_slots, max_pairs;
    long long os[3];
    const __nv_bfloat16 *O, *Wot;
    const int *sel, *lengths;
    __nv_bfloat16 *Y;
    unsigned *status;
};

__host__ __device__ inline uint32_t po_w_pitch(int H) { return (uint32_t)(H * 64 + 8) * 2u; }   // bytes per weight row
__host__ __device__ inline size_t po_align16(size_t x) { return (x + 15) / 16 * 16; }

__device__ __forceinline__ void po_mma(float c[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__global__ void __launch_bounds__(kPoThreads, 1) k_project_out_rows(OutArgs a) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ int head_base[33], head_cnt[32], fill_t[32], n_pairs_s, n_slots_s, warp_tot[kPoThreads / 32];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n0 = blockIdx.x * kPoCols, chunk = blockIdx.y, b = blockIdx.z;
    const uint32_t wpitch = po_w_pitch(a.H);
    // shared memory: weight slice | fill rows | c | base | pair positions | slot positions |
    // pair of (head, slot) | slots | products of the pairs
    uint8_t *Ws = smem;
    __nv_bfloat16 *Fs = reinterpret_cast<__nv_bfloat16 *>(Ws + (size_t)kPoCols * wpitch);   // [H][64]
    float *cs = reinterpret_cast<float *>(Fs + (size_t)a.H * 64);                           // [H][64]
    float *base = cs + (size_t)a.H * 64;                                                    // [64]
    int *pair_t = reinterpret_cast<int *>(base + 64);                                       // [max_pairs] position, -1 = padding
    int *slot_t = pair_t + a.max_pairs;                                                     // [max_slots] position of a slot
    short *pair_of = reinterpret_cast<short *>(slot_t + a.max_slots);                       // [H][max_slots] pair of (head, slot) or -1
    // (H * max_slots may be odd: the arrays behind it start on the next 16-byte boundary of the block's memory)
    short *slot_of = reinterpret_cast<short *>(smem + po_align16((size_t)(reinterpret_cast<uint8_t *>(pair_of) - smem) +
                                                                 (size_t)a.H * a.max_slots * 2));   // [t_chunk] slot of a position or -1
    float *P = reinterpret_cast<float *>(smem + po_align16((size_t)(reinterpret_cast<uint8_t *>(slot_of) - smem) +
                                                           (size_t)a.t_chunk * 2));              // [max_pairs][64]

    pdl_enter();
    int L = a.lengths ? a.lengths[b] : a.T;
    if (L < 0 || L > a.T) { if (tid == 0) atomicOr(a.status, kStatusLenClamped); L = L < 0 ? 0 : a.T; }
    const int t0 = chunk * a.t_chunk, t1 = min(t0 + a.t_chunk, L);
    if (t0 >= L) return;

    // the weight slice: rows n0 .. n0 + 63 of Wot (zeros past dy), H * 64 bf16 each
    {
        const int chunks_per_row = a.H * 8;
        for (int e = tid; e < kPoCols * chunks_per_row; e += kPoThreads) {
            const int n = e / chunks_per_row, c = e - n * chunks_per_row;
            const uint32_t dst = sm100::smem_u32(Ws + (size_t)n * wpitch + c * 16);
            if (n0 + n < a.dy)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(a.Wot + ((size_t)(n0 + n) * a.H * 64 + c * 8)) : "memory");
            else
                *reinterpret_cast<uint4 *>(Ws + (size_t)n * wpitch + c * 16) = make_uint4(0u, 0u, 0u, 0u);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    for (int i = tid; i < a.t_chunk; i += kPoThreads) slot_of[i] = 0;
    for (int i = tid; i < a.H * a.max_slots; i += kPoThreads) pair_of[i] = -1;
    for (int i = tid; i < a.max_pairs; i += kPoThreads) pair_t[i] = -1;
    __syncthreads();
    // positions of this range picked by any head; per head (one warp each): how many of its rows lie in the range
    for (int h = warp; h < a.H; h += kPoThreads / 32) {
        const int *s = a.sel + ((size_t)b * a.H + h) * a.u_max;
        // the fill row of the head is the first valid position its index set (ascending, -1 padded) leaves
        // out: the number of leading entries r with sel[r] == r
        int cnt = 0, lead = 0;
        bool leading = true;
        for (int r0 = 0; r0 < a.u_max; r0 += 32) {
            const int t = r0 + lane < a.u_max ? s[r0 + lane] : -1;
            const bool in = t >= t0 && t < t1;
            if (in) slot_of[t - t0] = 1;
            cnt += __popc(__ballot_sync(0xffffffffu, in));
            const unsigned same = __ballot_sync(0xffffffffu, t == r0 + lane);
            if (leading) {
                const int run = same == 0xffffffffu ? 32 : __ffs(~same) - 1;
                lead += run;
                leading = run == 32;
            }
        }
        if (lane == 0) {
            head_cnt[h] = cnt;
            fill_t[h] = lead < L ? lead : -1;                    // -1: every valid row is selected, no fill row
        }
    }
    __syncthreads();
    if (tid == 0) {                                              // the heads' pairs start at multiples of 16 rows
        int off = 0;
        for (int h = 0; h < a.H; ++h) { head_base[h] = off; off += (head_cnt[h] + 15) & ~15; }
        head_base[a.H] = off;
        n_pairs_s = off;
    }
    for (int e = tid; e < a.H * 8; e += kPoThreads) {
        const int h = e >> 3, c = e & 7, t = fill_t[h];
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (t >= 0) v = __ldg(reinterpret_cast<const uint4 *>(a.O + (long long)b * a.os[0] + (long long)h * a.os[1] + (long long)t * a.os[2]) + c);
        reinterpret_cast<uint4 *>(Fs)[e] = v;
    }
    // ordered compaction of the marked positions into slots (thread i owns positions i * per .. + per - 1)
    {
        const int per = (a.t_chunk + kPoThreads - 1) / kPoThreads;
        const int lo = tid * per, hi = min(lo + per, t1 - t0);
        int cnt = 0;
        for (int i = lo; i < hi; ++i) cnt += slot_of[i];
        int incl = cnt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += v;
        }
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        int off = incl - cnt;
        for (int w = 0; w < warp; ++w) off += warp_tot[w];
        for (int i = lo; i < hi; ++i) {
            if (slot_of[i]) {
                if (off < a.max_slots) { slot_of[i] = (short)off; slot_t[off] = t0 + i; }
                else slot_of[i] = -1;
                ++off;
            } else {
                slot_of[i] = -1;
            }
        }
        if (tid == kPoThreads - 1) n_slots_s = min(off, a.max_slots);
    }
    __syncthreads();
    // pairs (head, row inside the range), in the order of the head's index set: pair -> position, (head, slot) -> pair
    for (int h = warp; h < a.H; h += kPoThreads / 32) {
        const int *s = a.sel + ((size_t)b * a.H + h) * a.u_max;
        int seen = 0;
        for (int r0 = 0; r0 < a.u_max; r0 += 32) {
            const int t = r0 + lane < a.u_max ? s[r0 + lane] : -1;
            const bool in = t >= t0 && t < t1 && slot_of[t - t0] >= 0;
            const unsigned bal = __ballot_sync(0xffffffffu, in);
            if (in) {
                const int p = head_base[h] + seen + __popc(bal & ((1u << lane) - 1u));
                if (p < a.max_pairs) { pair_t[p] = t; pair_of[(size_t)h * a.max_slots + slot_of[t - t0]] = (short)p; }
            }
            seen += __popc(bal);
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    const int n_pairs = min(n_pairs_s, a.max_pairs), n_slots = n_slots_s;
    // c_h[n] = F_h . W_o^h[:, n] for the CTA's columns; base = their sum over the heads, in head order
    {
        const int n = tid & 63;
        for (int h = tid >> 6; h < a.H; h += kPoThreads / 64) {
            const uint4 *w = reinterpret_cast<const uint4 *>(Ws + (size_t)n * wpitch + h * 128);
            const uint4 *f = reinterpret_cast<const uint4 *>(Fs + h * 64);
            float acc = 0.f;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint4 wv = w[c], fv = f[c];
                const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w}, ff[4] = {fv.x, fv.y, fv.z, fv.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    acc = fmaf(__uint_as_float(ff[k] << 16), __uint_as_float(ww[k] << 16), acc);
                    acc = fmaf(__uint_as_float(ff[k] & 0xffff0000u), __uint_as_float(ww[k] & 0xffff0000u), acc);
                }
            }
            cs[h * 64 + n] = acc;
        }
    }

    // ---- products of the pairs: P[pair][:] = O[b][h][t][:] W_o^h (the CTA's columns) ----------------------------
    // One task = 16 pairs (of one head) x 32 columns on mma.m16n8k16, operands straight from where they are: the
    // sum over k does not care in which order the 64 elements of a row meet their weights, so lane (g, q) takes
    // the 32 contiguous bytes [32 q, 32 q + 32) of rows g and g + 8 (two 16-byte loads each, no staging) and
    // gives four of those elements to every k-step; the B fragments read the same elements of the weight rows.
    {
        const int n_tasks = (n_pairs >> 4) * 2;
        const int g = lane >> 2, q = lane & 3;
        auto load_rows = [&](int task, uint4 (&v)[4], int &h) {
            const int mt = task >> 1;
            h = 0;
            while (head_base[h + 1] <= mt * 16) ++h;            // a tile of 16 pairs lies within one head
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int t = pair_t[mt * 16 + g + 8 * half];
                if (t >= 0) {
                    const uint4 *src = reinterpret_cast<const uint4 *>(a.O + (long long)b * a.os[0] + (long long)h * a.os[1] + (long long)t * a.os[2]) + 2 * q;
                    v[2 * half] = __ldg(src); v[2 * half + 1] = __ldg(src + 1);
                } else {
                    v[2 * half] = v[2 * half + 1] = make_uint4(0u, 0u, 0u, 0u);
                }
            }
        };
        uint4 cur[4], nxt[4];
        int h_cur = 0, h_nxt = 0;
        if (warp < n_tasks) load_rows(warp, cur, h_cur);
        for (int task = warp; task < n_tasks; task += kPoThreads / 32) {
            const bool more = task + kPoThreads / 32 < n_tasks;
            if (more) load_rows(task + kPoThreads / 32, nxt, h_nxt);
            const int mt = task >> 1, nh = task & 1;
            const uint32_t A0[8] = {cur[0].x, cur[0].y, cur[0].z, cur[0].w, cur[1].x, cur[1].y, cur[1].z, cur[1].w};
            const uint32_t A1[8] = {cur[2].x, cur[2].y, cur[2].z, cur[2].w, cur[3].x, cur[3].y, cur[3].z, cur[3].w};
            float acc[4][4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int x = 0; x < 4; ++x) acc[j][x] = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint8_t *wrow = Ws + (size_t)(nh * 32 + j * 8 + g) * wpitch + h_cur * 128 + q * 32;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const uint2 bw = *reinterpret_cast<const uint2 *>(wrow + ks * 8);
                    po_mma(acc[j], A0[2 * ks], A1[2 * ks], A0[2 * ks + 1], A1[2 * ks + 1], bw.x, bw.y);
                }
            }
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                float *y = P + (size_t)(mt * 16 + g + 8 * half) * 64 + nh * 32 + 2 * q;
#pragma unroll
                for (int j = 0; j < 4; ++j) *reinterpret_cast<float2 *>(y + j * 8) = make_float2(acc[j][2 * half], acc[j][2 * half + 1]);
            }
            if (more) {
#pragma unroll
                for (int x = 0; x < 4; ++x) cur[x] = nxt[x];
                h_cur = h_nxt;
            }
        }
    }
    __syncthreads();
    if (tid < 64) {
        float s = 0.f;
        for (int h = 0; h < a.H; ++h) s += cs[h * 64 + tid];
        base[tid] = s;
    }
    __syncthreads();

    // ---- write the CTA's 64-column slice of every valid row of its range: base, plus for a selected position the
    //      corrections (product - c_h) of the heads that picked it, in head order ------------------------------------
    const int c8 = tid & 7;                                     // 8 columns = 16 bytes per thread
    if (n0 + c8 * 8 < a.dy) {
        float bv[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) bv[x] = base[c8 * 8 + x];
        for (int i = (tid >> 3); i < t1 - t0; i += kPoThreads / 8)
            if (slot_of[i] < 0) store8(a.Y + ((size_t)b * a.T + t0 + i) * a.dy + n0, c8, bv);
        // the picked positions, slot by slot (the heads' pair numbers of a slot are read together: a chain of
        // dependent look-ups per row would leave the few warps of the CTA waiting)
        for (int s = (tid >> 3); s < n_slots; s += kPoThreads / 8) {
            float v[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) v[x] = bv[x];
            for (int h0 = 0; h0 < a.H; h0 += 8) {
                int pr[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) pr[k] = h0 + k < a.H ? pair_of[(size_t)(h0 + k) * a.max_slots + s] : -1;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    if (pr[k] >= 0) {
                        const float4 *pp = reinterpret_cast<const float4 *>(P + (size_t)pr[k] * 64 + c8 * 8);
                        const float4 *ch = reinterpret_cast<const float4 *>(cs + (h0 + k) * 64 + c8 * 8);
                        const float4 p0 = pp[0], p1 = pp[1], c0 = ch[0], c1 = ch[1];
                        v[0] += p0.x - c0.x; v[1] += p0.y - c0.y; v[2] += p0.z - c0.z; v[3] += p0.w - c0.w;
                        v[4] += p1.x - c1.x; v[5] += p1.y - c1.y; v[6] += p1.z - c1.z; v[7] += p1.w - c1.w;
                    }
                }
            }
            store8(a.Y + ((size_t)b * a.T + slot_t[s]) * a.dy + n0, c8, v);
        }
    }
}

// Any element type, any O: one thread per output element.
template <typename DT>
__global__ void __launch_bounds__(128) k_project_out_simt(OutArgs a, const DT *__restrict__ O, const DT *__restrict__ Wot,
                                                          DT *__restrict__ Y) {
    const int n = blockIdx.x * 128 + threadIdx.x, t = blockIdx.y, b = blockIdx.z;
    pdl_enter();
    int L = a.lengths ? a.lengths[b] : a.T;
    if (L < 0 || L > a.T) { if (threadIdx.x == 0) atomicOr(a.status, kStatusLenClamped); L = L < 0 ? 0 : a.T; }
    if (t >= L || n >= a.dy) return;
    float acc = 0.f;
    for (int h = 0; h < a.H; ++h) {
        const DT *o = O + (long long)b * a.os[0] + (long long)h * a.os[1] + (long long)t * a.os[2];
        const DT *w = Wot + ((size_t)n * a.H + h) * 64;
        for (int e = 0; e < 64; ++e) acc = fmaf((float)o[e], (float)w[e], acc);
    }
    Y[((size_t)b * a.T + t) * a.dy + n] = (DT)acc;
}

cudaError_t launch_project_out_dense(const Geom &g, int dy, const void *O, const void *Wot, void *Y, cudaStream_t st);

// mode 0: pick (shortcut when an index set is given and the shape fits, else the dense GEMM, else one thread
// per element); 1: never the shortcut; 2: one thread per element.
cudaError_t launch_project_out(int dtype, int mode, const Geom &g, int dy, const void *O, const int *sel, const void *Wot,
                               void *Y, cudaStream_t st) {
    if (g.B * g.H == 0 || dy == 0) return cudaSuccess;
    OutArgs a;
    a.B = g.B; a.H = g.H; a.T = g.T; a.dy = dy; a.u_max = g.u_max;
    for (int k = 0; k < 3; ++k) a.os[k] = g.os[k];
    a.O = (const __nv_bfloat16 *)O; a.Wot = (const __nv_bfloat16 *)Wot; a.Y = (__nv_bfloat16 *)Y;
    a.sel = sel; a.lengths = g.lengths; a.status = g.status;
    a.t_chunk = 0; a.max_slots = 0; a.max_pairs = 0;
    if (dtype == 0 && mode == 0 && sel != nullptr && g.u_max <= kPoMaxRows && g.H <= 32 && dy % 8 == 0) {
        const int sms = device_sm_count();
        const int slices = (dy + kPoCols - 1) / kPoCols;
        // ranges of positions: about one CTA per SM (every CTA loads its weight slice once), 256 .. 1024 positions each
        int chunks = sms / (slices * g.B);
        if (chunks < 1) chunks = 1;
        int t_chunk = (g.T + chunks - 1) / chunks;
        t_chunk = ((t_chunk + 63) / 64) * 64;
        if (t_chunk < 256) t_chunk = 256;
        if (t_chunk > kPoMaxChunk) t_chunk = kPoMaxChunk;
        chunks = (g.T + t_chunk - 1) / t_chunk;
        a.t_chunk = t_chunk;
        a.max_slots = g.H * g.u_max < t_chunk ? g.H * g.u_max : t_chunk;
        a.max_pairs = g.H * ((g.u_max + 15) / 16 * 16);         // every head's rows padded to whole 16-row tiles
        // the kernel's layout: weights, fill rows, c, base, pair positions, slot positions, pair_of | slot_of | P
        size_t smem = (size_t)kPoCols * po_w_pitch(g.H) + (size_t)g.H * 64 * 2 + (size_t)g.H * 64 * 4 + 64 * 4 +
                      (size_t)a.max_pairs * 4 + (size_t)a.max_slots * 4;
        smem = po_align16(smem + (size_t)g.H * a.max_slots * 2);
        smem = po_align16(smem + (size_t)t_chunk * 2);
        smem += (size_t)a.max_pairs * 64 * 4 + 128;
        if (smem <= 200 * 1024 && chunks <= 65535 && g.B <= 65535) {
            static SmemGrant grant;
            if (cudaError_t e = grant_dynamic_smem(k_project_out_rows, grant, smem)) return e;
            cudaError_t e = launch_pdl(k_project_out_rows, dim3((unsigned)slices, (unsigned)chunks, (unsigned)g.B),
                                       dim3(kPoThreads), smem, st, a);
            note_launch();
            return e != cudaSuccess ? e : cudaGetLastError();
        }
    }
    if (dtype == 0 && mode != 2) {
        cudaError_t e = launch_project_out_dense(g, dy, O, Wot, Y, st);
        if (e != cudaErrorNotSupported) return e;
    }
    if (g.T > 65535 || g.B > 65535) return cudaErrorNotSupported;
    const dim3 grid((unsigned)((dy + 127) / 128), (unsigned)g.T, (unsigned)g.B);
    cudaError_t e;
    if (dtype == 0)
        e = launch_pdl(k_project_out_simt<__nv_bfloat16>, grid, dim3(128), 0, st, a, (const __nv_bfloat16 *)O,
                       (const __nv_bfloat16 *)Wot, (__nv_bfloat16 *)Y);
    else
        e = launch_pdl(k_project_out_simt<float>, grid, dim3(128), 0, st, a, (const float *)O, (const float *)Wot, (float *)Y);
    note_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace psattn
