// Microbenchmarks of the two gather rates that bound steps (a)+(b) (Eq. 11): every (query, sampled key)
// pair needs one 128-byte key row, read at a random position
//   mode 0  out of shared memory (keys of a unit resident: T_max <= ~1100), with the ldmatrix access
//           pattern of psattn_measure_mma.cuh (16 rows per round, rotated 16-byte chunks);
//   mode 1  out of L2 into registers (longer sequences), with the access pattern of
//           psattn_measure_stream.cuh (16 rows per round, four 16-byte loads per lane).
// Nothing is computed: the loaded words are xor-ed into a sink so that the loads stay.  The benchmark
// times these kernels with CUDA events and reports the measure kernels against the rates found.
#include "../../include/psattn.h"

#include "psattn_launch.h"
#include <cmath>
#include "psattn_sm100.cuh"

namespace psattn {

constexpr int kProbeSmemRows = 1024;                       // 128 KB of 128-byte rows

__device__ __forceinline__ uint32_t probe_hash(uint32_t x) {
    x ^= x >> 16; x *= 0x7feb352du; x ^= x >> 15; x *= 0x846ca68bu; x ^= x >> 16;
    return x;
}

__global__ void __launch_bounds__(1024, 1) k_probe_smem(int rounds, uint32_t *__restrict__ sink) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int e = tid; e < kProbeSmemRows * 32; e += blockDim.x) reinterpret_cast<uint32_t *>(smem)[e] = (uint32_t)e;
    __syncthreads();
    const uint32_t base = sm100::smem_u32(smem);
    const int l7 = lane & 7;
    uint32_t off[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) off[t] = (uint32_t)((2 * t + (lane >> 4) + l7) & 7) << 4;
    uint32_t acc = 0;
    uint32_t seed = (blockIdx.x * 64u + warp) * 65536u;
#pragma unroll 2
    for (int r = 0; r < rounds; ++r) {
        // lane l addresses row (l & 7) + 8 * ((l >> 3) & 1) of the round: a random key of the resident chunk
        const uint32_t row = probe_hash(seed + (uint32_t)r * 16u + (uint32_t)(l7 + 8 * ((lane >> 3) & 1))) % kProbeSmemRows;
        const uint32_t ra = base + row * 128u;
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            uint32_t a0, a1, a2, a3;
            asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                         : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3)
                         : "r"(ra + off[t]));
            acc ^= a0 ^ a1 ^ a2 ^ a3;
        }
    }
    if (acc == 0x12345678u) sink[0] = acc;                 // practically never: keeps the loads alive
}

// Same gather with the arithmetic of the measure kernel behind it: the four ldmatrix tiles of a round feed a
// chain of four mma.m16n8k16; kChains rounds are interleaved.  kIdx: the row numbers come from a table in
// shared memory (one 4-byte load per lane and round) instead of a hash.
template <int kChains, bool kIdx>
__global__ void __launch_bounds__(1024, 1) k_probe_smem_mma(int rounds, uint32_t *__restrict__ sink) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int e = tid; e < kProbeSmemRows * 32; e += blockDim.x) reinterpret_cast<uint32_t *>(smem)[e] = (uint32_t)e;
    uint32_t *table = reinterpret_cast<uint32_t *>(smem + kProbeSmemRows * 128);        // 4096 row numbers
    for (int e = tid; e < 4096; e += blockDim.x) table[e] = probe_hash((uint32_t)e * 7919u + blockIdx.x) % kProbeSmemRows;
    __syncthreads();
    const uint32_t base = sm100::smem_u32(smem), tbase = sm100::smem_u32(table);
    const int l7 = lane & 7;
    uint32_t off[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) off[t] = (uint32_t)((2 * t + (lane >> 4) + l7) & 7) << 4;
    uint32_t bq[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) bq[t] = 0x3f803f80u + (uint32_t)(lane + t);
    float mx = 0.f, ds = 0.f;
    const uint32_t seed = (blockIdx.x * 64u + warp) * 65536u;
    const uint32_t slot = (uint32_t)(l7 + 8 * ((lane >> 3) & 1));
    for (int r = 0; r + kChains <= rounds; r += kChains) {
        float c[kChains][4];
        uint32_t ra[kChains];
#pragma unroll
        for (int k = 0; k < kChains; ++k) {
            uint32_t row;
            if (kIdx) {
                const uint32_t ta = tbase + ((((uint32_t)(r + k) * 16u + slot + (uint32_t)warp * 64u) & 4095u) << 2);
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(row) : "r"(ta));
            } else {
                row = probe_hash(seed + (uint32_t)(r + k) * 16u + slot) % kProbeSmemRows;
            }
            ra[k] = base + row * 128u;
        }
#pragma unroll
        for (int k = 0; k < kChains; ++k) {
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                uint32_t a0, a1, a2, a3;
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                             : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3)
                             : "r"(ra[k] + off[t]));
                if (t == 0)
                    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%10, %10, %10, %10};"
                                 : "=f"(c[k][0]), "=f"(c[k][1]), "=f"(c[k][2]), "=f"(c[k][3])
                                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(bq[0]), "r"(bq[1]), "f"(0.f));
                else
                    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                                 : "+f"(c[k][0]), "+f"(c[k][1]), "+f"(c[k][2]), "+f"(c[k][3])
                                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(bq[2 * t]), "r"(bq[2 * t + 1]));
            }
        }
#pragma unroll
        for (int k = 0; k < kChains; ++k) {
            mx = fmaxf(mx, fmaxf(c[k][0], c[k][2]));
            ds += c[k][1] + c[k][3];
        }
    }
    if (mx + ds == 0.12345f) sink[0] = 1u;
}

// The same register gather out of the shared memory of the CTAs of a thread-block cluster (distributed shared
// memory): every CTA holds 1024 rows, a warp reads random rows of random CTAs of its cluster.
template <int kInFlight>
__global__ void __launch_bounds__(768, 1) k_probe_dsmem(int rounds, int cluster_size, uint32_t *__restrict__ sink) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int e = tid; e < kProbeSmemRows * 32; e += blockDim.x) reinterpret_cast<uint32_t *>(smem)[e] = (uint32_t)e;
    // every CTA of the cluster has filled its rows before anybody reads them
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    const uint32_t base = sm100::smem_u32(smem);
    const int g = lane >> 2, t = lane & 3;
    uint32_t acc = 0;
    const uint32_t seed = (blockIdx.x * 64u + warp) * 65536u;
    for (int r0 = 0; r0 + kInFlight <= rounds; r0 += kInFlight) {
        uint32_t v[kInFlight][4][4];
#pragma unroll
        for (int k = 0; k < kInFlight; ++k) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const uint32_t hsh = probe_hash(seed + (uint32_t)(r0 + k) * 16u + (uint32_t)(g + 8 * half));
                const uint32_t row = hsh % kProbeSmemRows, rank = (hsh >> 16) % (uint32_t)cluster_size;
                uint32_t remote;
                asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(base + row * 128u + (uint32_t)t * 16u), "r"(rank));
                asm volatile("ld.shared::cluster.v4.u32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(v[k][2 * half][0]), "=r"(v[k][2 * half][1]), "=r"(v[k][2 * half][2]), "=r"(v[k][2 * half][3]) : "r"(remote));
                asm volatile("ld.shared::cluster.v4.u32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(v[k][2 * half + 1][0]), "=r"(v[k][2 * half + 1][1]), "=r"(v[k][2 * half + 1][2]), "=r"(v[k][2 * half + 1][3]) : "r"(remote + 64u));
            }
        }
#pragma unroll
        for (int k = 0; k < kInFlight; ++k)
#pragma unroll
            for (int x = 0; x < 4; ++x) acc ^= v[k][x][0] ^ v[k][x][1] ^ v[k][x][2] ^ v[k][x][3];
    }
    if (acc == 0x12345678u) sink[0] = acc;
    // nobody leaves while its rows may still be read
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <int kInFlight>
__global__ void __launch_bounds__(768, 1) k_probe_l2(const uint4 *__restrict__ rows, uint32_t n_rows, int rounds,
                                                     uint32_t *__restrict__ sink) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    uint32_t acc = 0;
    const uint32_t seed = (blockIdx.x * 64u + warp) * 65536u;
    for (int r0 = 0; r0 < rounds; r0 += kInFlight) {
        uint4 v[kInFlight][4];
#pragma unroll
        for (int k = 0; k < kInFlight; ++k) {
            // rows g and g + 8 of the round; lanes t = 0..3 read the four 16-byte pieces of each half row
            const uint32_t ra = probe_hash(seed + (uint32_t)(r0 + k) * 16u + (uint32_t)g) % n_rows;
            const uint32_t rb = probe_hash(seed + (uint32_t)(r0 + k) * 16u + (uint32_t)(g + 8)) % n_rows;
            const uint4 *pa = rows + (size_t)ra * 8 + t, *pb = rows + (size_t)rb * 8 + t;
            asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(v[k][0].x), "=r"(v[k][0].y), "=r"(v[k][0].z), "=r"(v[k][0].w) : "l"(pa));
            asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(v[k][1].x), "=r"(v[k][1].y), "=r"(v[k][1].z), "=r"(v[k][1].w) : "l"(pa + 4));
            asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(v[k][2].x), "=r"(v[k][2].y), "=r"(v[k][2].z), "=r"(v[k][2].w) : "l"(pb));
            asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(v[k][3].x), "=r"(v[k][3].y), "=r"(v[k][3].z), "=r"(v[k][3].w) : "l"(pb + 4));
        }
#pragma unroll
        for (int k = 0; k < kInFlight; ++k)
#pragma unroll
            for (int x = 0; x < 4; ++x) acc ^= v[k][x].x ^ v[k][x].y ^ v[k][x].z ^ v[k][x].w;
    }
    if (acc == 0x12345678u) sink[0] = acc;
}


// The L2 gather through the copy engine instead of the load/store unit: lanes 0-15 of a warp each ask for one row
// with a 128-byte bulk copy into the warp's ring in shared memory (one mbarrier per ring slot counts the bytes), two
// rounds in flight.  MIXED: only every sixth warp does so, with half as many rounds; the others read their rows with
// 16-byte register loads as k_probe_l2 - does the copy engine add to what the load/store unit gets out of L2?
template <bool MIXED>
__global__ void __launch_bounds__(768, 1) k_probe_bulk(const uint4 *__restrict__ rows, uint32_t n_rows, int rounds,
                                                       uint32_t *__restrict__ sink) {
    constexpr int kInFlight = 2;
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nw = blockDim.x >> 5;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + (size_t)nw * kInFlight * 2048);
    if (lane == 0)
        for (int s = 0; s < kInFlight; ++s) sm100::mbar_init(&bars[warp * kInFlight + s], 1);
    sm100::fence_barrier_init();
    __syncthreads();
    const uint32_t seed = (blockIdx.x * 64u + warp) * 65536u;
    uint32_t acc = 0;
    if (MIXED && (warp % 6) != 5) {
        const int g = lane >> 2, t = lane & 3;
        for (int r0 = 0; r0 < rounds; r0 += kInFlight) {
            uint4 v[kInFlight][4];
#pragma unroll
            for (int k = 0; k < kInFlight; ++k) {
                const uint32_t ra = probe_hash(seed + (uint32_t)(r0 + k) * 16u + (uint32_t)g) % n_rows;
                const uint32_t rb = probe_hash(seed + (uint32_t)(r0 + k) * 16u + (uint32_t)(g + 8)) % n_rows;
                const uint4 *pa = rows + (size_t)ra * 8 + t, *pb = rows + (size_t)rb * 8 + t;
                asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(v[k][0].x), "=r"(v[k][0].y), "=r"(v[k][0].z), "=r"(v[k][0].w) : "l"(pa));
                asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(v[k][1].x), "=r"(v[k][1].y), "=r"(v[k][1].z), "=r"(v[k][1].w) : "l"(pa + 4));
                asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(v[k][2].x), "=r"(v[k][2].y), "=r"(v[k][2].z), "=r"(v[k][2].w) : "l"(pb));
                asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(v[k][3].x), "=r"(v[k][3].y), "=r"(v[k][3].z), "=r"(v[k][3].w) : "l"(pb + 4));
            }
#pragma unroll
            for (int k = 0; k < kInFlight; ++k)
#pragma unroll
                for (int x = 0; x < 4; ++x) acc ^= v[k][x].x ^ v[k][x].y ^ v[k][x].z ^ v[k][x].w;
        }
    } else {
        if (MIXED) rounds /= 2;
        uint8_t *ring = smem + (size_t)warp * kInFlight * 2048;
        uint64_t *bar = &bars[warp * kInFlight];
        auto issue = [&](int r) {
            const int s = r % kInFlight;
            if (lane == 0) sm100::mbar_expect_tx(&bar[s], 2048);
            __syncwarp();
            if (lane < 16) {
                const uint32_t row = probe_hash(seed + (uint32_t)r * 16u + (uint32_t)lane) % n_rows;
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], 128, [%2];"
                             ::"r"(sm100::smem_u32(ring + s * 2048 + lane * 128)), "l"(rows + (size_t)row * 8),
                               "r"(sm100::smem_u32(&bar[s])) : "memory");
            }
        };
        for (int r = 0; r < kInFlight && r < rounds; ++r) issue(r);
        bool ok = true;
        for (int r = 0; r < rounds && ok; ++r) {
            const int s = r % kInFlight;
            ok = sm100::mbar_wait(&bar[s], (uint32_t)((r / kInFlight) & 1));     // bounded
            acc ^= *reinterpret_cast<const uint32_t *>(ring + s * 2048 + lane * 64);
            __syncwarp();
            if (ok && r + kInFlight < rounds) issue(r + kInFlight);
        }
        if (!ok) {                                             // give the copies in flight a bounded chance to land
            for (int s = 0; s < kInFlight; ++s) sm100::mbar_wait(&bar[s], 0);
            sink[1] = 0xdeadu;
        }
    }
    if (acc == 0x12345678u) sink[0] = acc;
}


// What a chunk-resident form of steps (a)+(b) could reach for long sequences: a 1024-key chunk (128 KB) sits in shared
// memory, and the (query, sampled key) pairs whose key lies in the chunk are gathered from there.  A query has
// Binomial(U, 1/8) samples in one of eight chunks; the mma layout gives each of a warp's eight queries two rows per
// round, so a group of eight costs max over its queries of ceil(n / 2) rounds.  Per work item (one chunk, 2048
// queries): the chunk is copied in, then every warp takes groups of eight queries - their rows of Q staged through
// shared memory (cp.async, three groups ahead) and read as mma fragments, their row numbers read from a table, the rounds
// as in k_probe_smem_mma.  kSorted: the counts of a group are neighbours in the sorted order of their 128-query block
// (what a pre-pass that orders the queries of a block by count would deliver); otherwise they are independent draws.
// counts: 128 quantiles of the count distribution.  The kernel adds the useful pairs to sink[2..3] (64 bit).
struct ProbeCounts { unsigned char q[128]; };

template <bool kSorted>
__global__ void __launch_bounds__(512, 1) k_probe_bucketed(const uint4 *__restrict__ rows, uint32_t n_rows, int items,
                                                           ProbeCounts counts, uint32_t *__restrict__ sink) {
    extern __shared__ __align__(1024) uint8_t smem[];
    constexpr int kQueries = 2048;
    constexpr int kAhead = 3;                                            // groups of Q rows requested ahead of the one in work
    uint8_t *qstage = smem + kProbeSmemRows * 128;                       // [16 warps][kAhead + 1][1 KB]
    uint32_t *table = reinterpret_cast<uint32_t *>(qstage + 16 * (kAhead + 1) * 1024);   // 4096 row numbers
    unsigned char *cnt = reinterpret_cast<unsigned char *>(table + 4096);     // counts of the item's queries
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int e = tid; e < 4096; e += blockDim.x) table[e] = probe_hash((uint32_t)e * 7919u + blockIdx.x) % kProbeSmemRows;
    const uint32_t base = sm100::smem_u32(smem), tbase = sm100::smem_u32(table);
    const int l7 = lane & 7;
    uint32_t off[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) off[t] = (uint32_t)((2 * t + (lane >> 4) + l7) & 7) << 4;
    const uint32_t slot = (uint32_t)(l7 + 8 * ((lane >> 3) & 1));
    float mx = 0.f, ds = 0.f;
    unsigned long long pairs = 0;
    for (int item = 0; item < items; ++item) {
        const uint32_t work = (uint32_t)(blockIdx.x * items + item);
        __syncthreads();                                                 // everybody has left the chunk of the item before
        // the chunk: 1024 consecutive rows
        const uint32_t c0 = (work * 1024u) % (n_rows - 1024u);
        for (int e = tid; e < kProbeSmemRows * 8; e += blockDim.x) reinterpret_cast<uint4 *>(smem)[e] = __ldg(rows + (size_t)c0 * 8 + e);
        for (int q = tid; q < kQueries; q += blockDim.x)
            cnt[q] = kSorted ? counts.q[q & 127] : counts.q[probe_hash(work * 4096u + (uint32_t)q) & 127];
        __syncthreads();
        const uint32_t q0 = (work * 2048u + 12345u) % (n_rows - 2048u);  // the item's rows of Q, consecutive
        uint8_t *st = qstage + warp * (kAhead + 1) * 1024;
        auto stage_q = [&](int grp, int buf) {                           // 8 rows x 128 B: two 16-byte pieces per lane
            const uint4 *src = rows + (size_t)(q0 + grp * 8) * 8;
#pragma unroll
            for (int x = 0; x < 2; ++x) {                                // piece c of row r goes to place (c + r) mod 8 of the row
                const int pc = lane + 32 * x, r = pc >> 3, c = pc & 7;
                const uint32_t dst = sm100::smem_u32(st + buf * 1024) + (uint32_t)(r * 128 + (((c + r) & 7) << 4));
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src + pc) : "memory");
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        int it = 0;
        for (int a = 0; a < kAhead; ++a) stage_q(warp + 16 * a, a);      // (2048 queries: every warp has 16 groups)
        for (int grp = warp; grp < kQueries / 8; grp += 16, ++it) {
            // one commit per trip, empty at the end, so that "all but the newest kAhead groups" is always this trip's rows
            if (grp + 16 * kAhead < kQueries / 8) stage_q(grp + 16 * kAhead, (it + kAhead) % (kAhead + 1));
            else asm volatile("cp.async.commit_group;" ::: "memory");
            asm volatile("cp.async.wait_group %0;" ::"n"(kAhead) : "memory");
            __syncwarp();
            uint32_t bq[8];
            const uint32_t qa = sm100::smem_u32(st + (it % (kAhead + 1)) * 1024) + (uint32_t)l7 * 128u;
            asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                         : "=r"(bq[0]), "=r"(bq[1]), "=r"(bq[2]), "=r"(bq[3]) : "r"(qa + (uint32_t)((((lane >> 3) + l7) & 7) << 4)));
            asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                         : "=r"(bq[4]), "=r"(bq[5]), "=r"(bq[6]), "=r"(bq[7]) : "r"(qa + (uint32_t)((((lane >> 3) + 4 + l7) & 7) << 4)));
            int n = cnt[grp * 8 + l7];                                   // lanes with the same l7 agree
            int rounds = (n + 1) >> 1;
#pragma unroll
            for (int o = 1; o < 8; o <<= 1) rounds = max(rounds, __shfl_xor_sync(0xffffffffu, rounds, o));
            if (lane < 8) pairs += (unsigned long long)n;
            for (int r = 0; r < rounds; ++r) {
                uint32_t row;
                const uint32_t ta = tbase + ((((uint32_t)(it * 16 + r) * 16u + slot + (uint32_t)warp * 64u) & 4095u) << 2);
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(row) : "r"(ta));
                const uint32_t ra = base + row * 128u;
                float c[4];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    uint32_t a0, a1, a2, a3;
                    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3) : "r"(ra + off[t]));
                    if (t == 0)
                        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%10, %10, %10, %10};"
                                     : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
                                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(bq[0]), "r"(bq[1]), "f"(0.f));
                    else
                        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(bq[2 * t]), "r"(bq[2 * t + 1]));
                }
                mx = fmaxf(mx, fmaxf(c[0], c[2]));
                ds += c[1] + c[3];
            }
            __syncwarp();
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) pairs += __shfl_xor_sync(0xffffffffu, pairs, o);
    if (lane == 0) atomicAdd(reinterpret_cast<unsigned long long *>(sink + 2), pairs);
    if (mx + ds == 0.12345f) sink[0] = 1u;
}

}  // namespace psattn

using namespace psattn;

extern "C" int psattn_probe_gather(int32_t mode, const void *rows, int64_t n_rows, int32_t n_ctas,
                                   int32_t warps_per_cta, int32_t rounds_per_warp, uint32_t *sink,
                                   void *stream) {
    if (!sink) return PSATTN_ERR_NULL;
    if (n_ctas < 1 || n_ctas > 65535 || rounds_per_warp < 1 || warps_per_cta < 1) return PSATTN_ERR_BAD_DESC;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (mode == 0) {
        if (warps_per_cta > 32) return PSATTN_ERR_BAD_DESC;
        static SmemGrant grant;
        const size_t smem = (size_t)kProbeSmemRows * 128;
        if (grant_dynamic_smem(k_probe_smem, grant, smem) != cudaSuccess) return PSATTN_ERR_CUDA;
        k_probe_smem<<<(unsigned)n_ctas, (unsigned)warps_per_cta * 32, smem, st>>>(rounds_per_warp, sink);
    } else if (mode >= 3 && mode <= 8) {
        if (warps_per_cta > 32) return PSATTN_ERR_BAD_DESC;
        const size_t smem = (size_t)kProbeSmemRows * 128 + 4096 * 4;
        static SmemGrant g3, g4, g5, g6, g7, g8;
        const dim3 grid((unsigned)n_ctas), block((unsigned)warps_per_cta * 32);
#define PSATTN_PROBE_CASE(M, G, CH, IDX)                                                                   \
        case M:                                                                                            \
            if (grant_dynamic_smem(k_probe_smem_mma<CH, IDX>, G, smem) != cudaSuccess) return PSATTN_ERR_CUDA; \
            k_probe_smem_mma<CH, IDX><<<grid, block, smem, st>>>(rounds_per_warp, sink);                   \
            break;
        switch (mode) {
            PSATTN_PROBE_CASE(3, g3, 1, false)
            PSATTN_PROBE_CASE(4, g4, 2, false)
            PSATTN_PROBE_CASE(5, g5, 4, false)
            PSATTN_PROBE_CASE(6, g6, 1, true)
            PSATTN_PROBE_CASE(7, g7, 2, true)
            PSATTN_PROBE_CASE(8, g8, 4, true)
        }
#undef PSATTN_PROBE_CASE
    } else if (mode == 9 || mode == 10) {
        // n_rows carries the cluster size here (1, 2, 4 or 8); n_ctas is rounded down to a multiple of it
        const int cs = (int)n_rows;
        if ((cs != 1 && cs != 2 && cs != 4 && cs != 8) || warps_per_cta > 24) return PSATTN_ERR_BAD_DESC;
        const int ctas = n_ctas / cs * cs;
        if (ctas < cs) return PSATTN_ERR_BAD_DESC;
        const size_t smem = (size_t)kProbeSmemRows * 128;
        static SmemGrant g9, g10;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)ctas);
        cfg.blockDim = dim3((unsigned)warps_per_cta * 32);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t e;
        if (mode == 9) {
            if (grant_dynamic_smem(k_probe_dsmem<2>, g9, smem) != cudaSuccess) return PSATTN_ERR_CUDA;
            e = cudaLaunchKernelEx(&cfg, k_probe_dsmem<2>, rounds_per_warp, cs, sink);
        } else {
            if (grant_dynamic_smem(k_probe_dsmem<4>, g10, smem) != cudaSuccess) return PSATTN_ERR_CUDA;
            e = cudaLaunchKernelEx(&cfg, k_probe_dsmem<4>, rounds_per_warp, cs, sink);
        }
        note_launch();
        return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? PSATTN_OK : PSATTN_ERR_CUDA;
    } else if (mode == 11 || mode == 12) {
        if (!rows) return PSATTN_ERR_NULL;
        if (n_rows < 1 || n_rows > (1ll << 31) || warps_per_cta > 24) return PSATTN_ERR_BAD_DESC;
        if ((reinterpret_cast<uintptr_t>(rows) & 15u) != 0) return PSATTN_ERR_MISALIGNED;
        const size_t smem = (size_t)warps_per_cta * 2 * 2048 + (size_t)warps_per_cta * 2 * 8 + 64;
        static SmemGrant g11, g12;
        const dim3 grid((unsigned)n_ctas), block((unsigned)warps_per_cta * 32);
        if (mode == 11) {
            if (grant_dynamic_smem(k_probe_bulk<false>, g11, smem) != cudaSuccess) return PSATTN_ERR_CUDA;
            k_probe_bulk<false><<<grid, block, smem, st>>>((const uint4 *)rows, (uint32_t)n_rows, rounds_per_warp / 4 * 4, sink);
        } else {
            if (grant_dynamic_smem(k_probe_bulk<true>, g12, smem) != cudaSuccess) return PSATTN_ERR_CUDA;
            k_probe_bulk<true><<<grid, block, smem, st>>>((const uint4 *)rows, (uint32_t)n_rows, rounds_per_warp / 4 * 4, sink);
        }
    } else if (mode == 13 || mode == 14) {
        if (!rows) return PSATTN_ERR_NULL;
        if (n_rows < 4096 || n_rows > (1ll << 31) || warps_per_cta != 16) return PSATTN_ERR_BAD_DESC;
        if ((reinterpret_cast<uintptr_t>(rows) & 15u) != 0 || (reinterpret_cast<uintptr_t>(sink) & 7u) != 0) return PSATTN_ERR_MISALIGNED;
        // 128 quantiles of Binomial(46, 1/8): the number of a query's 46 samples that fall into one of eight chunks
        ProbeCounts pc;
        {
            double pmf[47], cdf = 0.0;
            for (int k = 0; k <= 46; ++k) {
                double c = 1.0;
                for (int j = 0; j < k; ++j) c = c * (46 - j) / (j + 1);
                pmf[k] = c * std::pow(0.125, k) * std::pow(0.875, 46 - k);
            }
            int k = 0;
            cdf = pmf[0];
            for (int i = 0; i < 128; ++i) {
                const double u = (i + 0.5) / 128.0;
                while (cdf < u && k < 46) cdf += pmf[++k];
                pc.q[i] = (unsigned char)k;
            }
        }
        const size_t smem = (size_t)kProbeSmemRows * 128 + 16 * 4 * 1024 + 4096 * 4 + 2048;
        static SmemGrant g13, g14;
        const dim3 grid((unsigned)n_ctas), block(512);
        if (mode == 13) {
            if (grant_dynamic_smem(k_probe_bucketed<false>, g13, smem) != cudaSuccess) return PSATTN_ERR_CUDA;
            k_probe_bucketed<false><<<grid, block, smem, st>>>((const uint4 *)rows, (uint32_t)n_rows, rounds_per_warp, pc, sink);
        } else {
            if (grant_dynamic_smem(k_probe_bucketed<true>, g14, smem) != cudaSuccess) return PSATTN_ERR_CUDA;
            k_probe_bucketed<true><<<grid, block, smem, st>>>((const uint4 *)rows, (uint32_t)n_rows, rounds_per_warp, pc, sink);
        }
    } else if (mode == 1 || mode == 2) {
        if (!rows) return PSATTN_ERR_NULL;
        if (n_rows < 1 || n_rows > (1ll << 31) || warps_per_cta > 24) return PSATTN_ERR_BAD_DESC;
        if ((reinterpret_cast<uintptr_t>(rows) & 15u) != 0) return PSATTN_ERR_MISALIGNED;
        if (mode == 1)
            k_probe_l2<2><<<(unsigned)n_ctas, (unsigned)warps_per_cta * 32, 0, st>>>((const uint4 *)rows, (uint32_t)n_rows,
                                                                                  rounds_per_warp / 2 * 2, sink);
        else
            k_probe_l2<4><<<(unsigned)n_ctas, (unsigned)warps_per_cta * 32, 0, st>>>((const uint4 *)rows, (uint32_t)n_rows,
                                                                                  rounds_per_warp / 4 * 4, sink);
    } else {
        return PSATTN_ERR_BAD_DESC;
    }
    note_launch();
    return cudaGetLastError() == cudaSuccess ? PSATTN_OK : PSATTN_ERR_CUDA;
}
