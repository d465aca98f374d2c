// psattn_mean_v_noalloc: the fill value of step (e) for callers that may not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need mean(V):
// code that runs inside a memory-pool-managed region of a framework (every byte of device
// memory is handed out by the framework's own allocator and a raw cudaMalloc either fails under
// a hard memory cap or fragments the pool), real-time audio pipelines that forbid allocation
// after start-up, and plug-ins that are loaded into a process whose device memory is already
// fully reserved.  The regular entry point needs a plan (device tables, allocated at plan
// creation) and a caller-provided workspace; this one needs neither.  Its scratch - the
// column-sum partials - lives in a fixed array that is part of the library image, so every GPU
// that loads the library holds kNoAllocScratchBytes of device memory until the process exits.
#include "../../include/psattn.h"

#include <mutex>

#include "psattn_launch.h"

namespace psattn {

constexpr size_t kNoAllocScratchFloats = (size_t)PSATTN_NOALLOC_MAX_PARTIALS * kD;   // 4 MiB
constexpr size_t kNoAllocStatusFloats = 64;                                          // 256 B

// [0, 64) floats: the device status word (bit 1 = a length was clamped); then the partials.
static __device__ __align__(256) float g_noalloc_scratch[kNoAllocStatusFloats + kNoAllocScratchFloats];

// Finishes mean(V): sums the partials of one unit in chunk order (the same order the planned
// path uses, so both give the same bits) and divides by the valid length.
__global__ void __launch_bounds__(kD) k_mean_finish(Geom g, const float *__restrict__ part,
                                                    int n_chunks, float *__restrict__ vbar) {
    const int unit = blockIdx.x;
    const int L = seq_len(g, unit / g.H);
    float s = 0.f;
    for (int c = 0; c < n_chunks; ++c) s += part[((long long)unit * n_chunks + c) * kD + threadIdx.x];
    vbar[(long long)unit * kD + threadIdx.x] = L > 0 ? s / (float)L : 0.f;
}

static std::mutex g_setup_mutex;
static float *g_scratch_addr[kMaxDevices];          // device address of the array, per device

// The array's name is only a handle on the host; its device address differs per GPU and has
// to be asked for with that GPU current.  Done once per device, on the first call.
static int scratch_for_current_device(float **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PSATTN_ERR_NO_DEVICE;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        float *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress((void **)&ptr, g_noalloc_scratch);
        if (e != cudaSuccess || ptr == nullptr) { cudaGetLastError(); return PSATTN_ERR_CUDA; }
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return PSATTN_OK;
}

}  // namespace psattn

using namespace psattn;

extern "C" int psattn_mean_v_noalloc(const void *V, const int32_t *lengths, float *vbar,
                                     int32_t B, int32_t H, int32_t T_max, int32_t dtype,
                                     void *stream) {
    if (!V || !vbar) return PSATTN_ERR_NULL;
    if (B < 0 || H < 1 || T_max < 1 || B > (1 << 20) || H > 4096 || T_max > (1 << 20)) return PSATTN_ERR_BAD_DESC;
    if (dtype != PSATTN_BF16 && dtype != PSATTN_FP32) return PSATTN_ERR_BAD_DESC;
    if ((reinterpret_cast<uintptr_t>(V) & 15u) != 0) return PSATTN_ERR_MISALIGNED;
    const long long units = (long long)B * H;
    const int n_chunks = (T_max + kColsumRows - 1) / kColsumRows;
    if (units * n_chunks > (long long)PSATTN_NOALLOC_MAX_PARTIALS) return PSATTN_ERR_TOO_LARGE;
    if (units == 0) return PSATTN_OK;
    float *scratch = nullptr;
    int rc = scratch_for_current_device(&scratch);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    Geom g;
    g.B = B; g.H = H; g.T = T_max;
    g.idx_cols = 0; g.idx_per_head = 0; g.idx_shared = 0; g.u_max = 0;
    const long long dense[3] = {(long long)H * T_max * kD, (long long)T_max * kD, kD};
    for (int k = 0; k < 3; ++k) { g.qs[k] = g.ks[k] = g.vs[k] = g.os[k] = dense[k]; }
    g.lengths = lengths;
    g.u_tab = nullptr; g.U_tab = nullptr;
    g.status = reinterpret_cast<unsigned *>(scratch);
    g.wait_ns = 1000ull * 1000ull * 1000ull; g.debug_extra_tx = 0u;
    float *part = scratch + kNoAllocStatusFloats;
    // The array keeps whatever the previous call left.  The partials of this call's units are all
    // rewritten by the column-sum kernel before they are read; only the status word has to start
    // from zero.
    if (cudaMemsetAsync(scratch, 0, sizeof(unsigned), st) != cudaSuccess) { cudaGetLastError(); return PSATTN_ERR_CUDA; }
    if (launch_colsum(dtype, g, V, part, n_chunks, st) != cudaSuccess) return PSATTN_ERR_CUDA;
    k_mean_finish<<<(unsigned)units, kD, 0, st>>>(g, part, n_chunks, vbar);
    note_launch();
    if (cudaGetLastError() != cudaSuccess) return PSATTN_ERR_CUDA;
    return PSATTN_OK;
}
