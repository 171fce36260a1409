// luvc_spu_prune_static: the Spectrum Pruning Unit for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the moment they need a prune: an
// inference server whose own allocator has already claimed the device's memory, a latency-bound
// loop in which an allocation's implicit device synchronisation is not acceptable, or code running
// under a memory budget it has promised not to exceed.  The other SPU entry points either grow a
// library-owned buffer with cudaMalloc or ask the caller for a workspace.  This one does neither:
// its workspace is the fixed array below, which is part of the library's device image, so every
// device that loads that image holds these bytes until the process exits (with lazy module
// loading the image arrives with the first call on a device: see the warm-up note in luvc.h).
//
// The array's name is only a handle on the host side; the device address is looked up once per
// device with cudaGetSymbolAddress (with that device current) and handed to the kernels.

#include <mutex>

#include "luvc_internal.h"

namespace {

constexpr size_t kStatusBytes = 256;                                    // status word, kept apart from the workspace
constexpr size_t kStaticBytes = kStatusBytes + LUVC_SPU_STATIC_MAX_BYTES;

static __device__ __align__(256) unsigned char g_spu_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
unsigned char* g_base[kMaxDevices];      // device address of the array, per device ordinal
std::mutex g_setup_mutex;

// Device address of the scratch array on the current device; looked up on the first call per device.
int scratch_base(unsigned char** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LUVC_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_base[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_spu_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return LUVC_ERR_CUDA;
        }
        g_base[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_base[dev];
    return LUVC_OK;
}

}  // namespace

extern "C" int luvc_spu_prune_static(const void* hidden, int B, int N, int D, float cutoff, int keep, int dtype,
                                     void* cuda_stream, int32_t* out_idx, void* out_hidden) {
    using namespace luvc;
    if (!hidden || !out_idx || !out_hidden) return LUVC_ERR_NULL;
    if (dtype != LUVC_BF16 && dtype != LUVC_F32) return LUVC_ERR_DTYPE;
    if (B < 1 || N < 1 || D < 1 || B > 65535 || (long long)B * N > (1ll << 31) - 1) return LUVC_ERR_SHAPE;
    if (keep < 1 || keep > N) return LUVC_ERR_KEEP;
    const int sigma = luvc_spu_sigma(N, cutoff);
    if (sigma < 0) return LUVC_ERR_CUTOFF;
    const size_t es = dtype == LUVC_F32 ? 4 : 2;
    if (((size_t)D * es) % 16 != 0) return LUVC_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(hidden) & 15u) || (reinterpret_cast<uintptr_t>(out_hidden) & 15u) ||
        (reinterpret_cast<uintptr_t>(out_idx) & 3u))
        return LUVC_ERR_ALIGN;
    if (spu_workspace_bytes(B, N, D, sigma, dtype) > (size_t)LUVC_SPU_STATIC_MAX_BYTES) return LUVC_ERR_WORKSPACE;

    unsigned char* base = nullptr;
    const int rc = scratch_base(&base);
    if (rc != LUVC_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // the array keeps whatever the previous call left: the status word must start at zero (every
    // other part of the workspace is fully rewritten by the kernels before it is read)
    if (cudaMemsetAsync(base, 0, kStatusBytes, stream) != cudaSuccess) return LUVC_ERR_CUDA;

    SpuProblem p;
    p.hidden = hidden; p.B = B; p.N = N; p.D = D; p.sigma = sigma; p.keep = keep; p.dtype = dtype;
    p.no_window = 0;
    p.out_idx = out_idx; p.out_hidden = out_hidden; p.out_scores = nullptr;
    p.workspace = base + kStatusBytes;
    p.status = reinterpret_cast<int*>(base);
    p.stream = stream;
    return spu_run(p);
}

extern "C" int luvc_spu_static_status(void* cuda_stream) {
    unsigned char* base = nullptr;
    const int rc = scratch_base(&base);
    if (rc != LUVC_OK) return rc;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return LUVC_ERR_CUDA;
    int host = 0;
    if (cudaMemcpy(&host, base, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return LUVC_ERR_CUDA;
    return host;
}
