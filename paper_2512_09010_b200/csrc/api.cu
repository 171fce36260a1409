// C ABI of the library: argument checks, stream and scratch handling, and the
// host-buffer variants.  All arithmetic lives in oim.cu and spu.cu.

#include <atomic>
#include <cmath>
#include <mutex>

#include "luvc_internal.h"

namespace luvc {

static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

static std::atomic<int> g_profile{0};
static cudaEvent_t g_ev[LUVC_PHASE_COUNT][2];
static bool g_ev_made = false, g_ev_used[LUVC_PHASE_COUNT];
static std::mutex g_ev_mutex;

void phase_begin(int phase, cudaStream_t stream) {
    if (!g_profile.load(std::memory_order_relaxed)) return;
    std::lock_guard<std::mutex> lock(g_ev_mutex);
    if (!g_ev_made) {
        for (auto& pair : g_ev) { cudaEventCreate(&pair[0]); cudaEventCreate(&pair[1]); }
        g_ev_made = true;
    }
    cudaEventRecord(g_ev[phase][0], stream);
}

void phase_end(int phase, cudaStream_t stream) {
    if (!g_profile.load(std::memory_order_relaxed)) return;
    std::lock_guard<std::mutex> lock(g_ev_mutex);
    if (!g_ev_made) return;
    cudaEventRecord(g_ev[phase][1], stream);
    g_ev_used[phase] = true;
}

namespace {

thread_local cudaStream_t t_stream = nullptr;

// Library-owned scratch: one growing buffer per purpose and per device (keyed by the ordinal of the
// device that is current at the call), shared by all threads and streams of the process.  Calls
// whose GPU work overlaps race on it (documented in luvc.h); the lock only covers (re)allocation.
enum Slot { kOimWs = 0, kSpuWs, kIoIn, kIoOut, kStatus, kCascade, kIoInSpu, kIoOutSpu, kSlots };
constexpr int kMaxDevices = 64;
struct Scratch { void* ptr = nullptr; size_t bytes = 0; };
Scratch g_scratch[kMaxDevices][kSlots];
std::mutex g_mutex;

int current_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
    return dev;
}

void* scratch(Slot s, size_t bytes) {
    const int dev = current_device();
    if (dev < 0) return nullptr;
    std::lock_guard<std::mutex> lock(g_mutex);
    Scratch& sc = g_scratch[dev][s];
    if (sc.bytes >= bytes && sc.ptr) return sc.ptr;
    if (sc.ptr) { cudaDeviceSynchronize(); cudaFree(sc.ptr); sc.ptr = nullptr; sc.bytes = 0; }
    void* p = nullptr;
    if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    sc.ptr = p; sc.bytes = bytes;
    return p;
}

// The current device's status block: 256 bytes allocated once and zeroed, kept until luvc_shutdown.
int* status_word() {
    const int dev = current_device();
    if (dev < 0) return nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (g_scratch[dev][kStatus].ptr) return static_cast<int*>(g_scratch[dev][kStatus].ptr);
    }
    void* p = scratch(kStatus, 256);
    if (p && cudaMemset(p, 0, 256) != cudaSuccess) return nullptr;
    return static_cast<int*>(p);
}

// Reads (after synchronising the stream) and clears the first word of a status block.
int read_status_block(int* block, cudaStream_t stream) {
    if (cudaStreamSynchronize(stream) != cudaSuccess) return LUVC_ERR_CUDA;
    int host = 0;
    if (cudaMemcpy(&host, block, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return LUVC_ERR_CUDA;
    if (host != 0 && cudaMemset(block, 0, sizeof(int)) != cudaSuccess) return LUVC_ERR_CUDA;
    return host;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
size_t elem_size(int dtype) { return dtype == LUVC_F32 ? 4 : 2; }

// Merge numbers per axis: the axis' own field, else the common one, else the appendix's 2.
int oim_r_w(const luvc_oim_opts& o) { return o.merge_per_step_w ? o.merge_per_step_w : (o.merge_per_step ? o.merge_per_step : 2); }
int oim_r_h(const luvc_oim_opts& o) { return o.merge_per_step_h ? o.merge_per_step_h : (o.merge_per_step ? o.merge_per_step : 2); }

int check_oim(const void* tokens, int B, int H, int W, int D, int target, const void* out_tokens,
              const void* out_sizes, const void* out_map, const luvc_oim_opts& o, int* Hf, int* Wf) {
    if (!tokens || !out_tokens || !out_sizes || !out_map) return LUVC_ERR_NULL;
    if (o.dtype != LUVC_BF16 && o.dtype != LUVC_F32) return LUVC_ERR_DTYPE;
    if (B < 1 || H < 1 || W < 1 || D < 1 || B > 65535) return LUVC_ERR_SHAPE;
    if ((long long)H * W > (1ll << 30) || (long long)B * H * W > (1ll << 31) - 1) return LUVC_ERR_SHAPE;
    if (((size_t)D * elem_size(o.dtype)) % 16 != 0) return LUVC_ERR_ALIGN;
    if (!aligned16(tokens) || !aligned16(out_tokens) || (reinterpret_cast<uintptr_t>(out_sizes) & 3u) ||
        (reinterpret_cast<uintptr_t>(out_map) & 3u))
        return LUVC_ERR_ALIGN;
    if (o.merge_per_step < 0 || o.merge_per_step_h < 0 || o.merge_per_step_w < 0) return LUVC_ERR_TARGET;
    if (o.device_status && (reinterpret_cast<uintptr_t>(o.device_status) & 15u)) return LUVC_ERR_ALIGN;
    if (o.matching != LUVC_OIM_MATCH_ADJACENT && o.matching != LUVC_OIM_MATCH_BIPARTITE) return LUVC_ERR_SHAPE;
    if (o.matching == LUVC_OIM_MATCH_BIPARTITE && (H > 256 || W > 256)) return LUVC_ERR_SHAPE;
    if (o.matching == LUVC_OIM_MATCH_BIPARTITE && D % 8 != 0) return LUVC_ERR_ALIGN;
    if (o.out_h || o.out_w) {
        if (o.out_h < 1 || o.out_w < 1 || o.out_h > H || o.out_w > W) return LUVC_ERR_TARGET;
        if ((long long)o.out_h * o.out_w != (long long)target) return LUVC_ERR_TARGET;
        *Hf = o.out_h; *Wf = o.out_w;
    } else if (!oim_final_dims(H, W, target, Hf, Wf)) {
        return LUVC_ERR_TARGET;
    }
    int n = 0;
    if (!oim_schedule(H, W, *Hf, *Wf, oim_r_w(o), oim_r_h(o), o.height_first, nullptr, 0, &n)) return LUVC_ERR_TARGET;
    if (o.trace) {
        if (reinterpret_cast<uintptr_t>(o.trace) & 3u) return LUVC_ERR_ALIGN;
        const size_t need = (size_t)B * ((size_t)H * W - (size_t)*Hf * *Wf) * sizeof(int32_t);
        if (o.trace_bytes < need) return LUVC_ERR_WORKSPACE;
    }
    return LUVC_OK;
}

int check_spu(const void* hidden, int B, int N, int D, float cutoff, int keep, const void* out_idx,
              const void* out_hidden, int dtype, int* sigma) {
    if (!hidden || !out_idx || !out_hidden) return LUVC_ERR_NULL;
    if (dtype != LUVC_BF16 && dtype != LUVC_F32) return LUVC_ERR_DTYPE;
    if (B < 1 || N < 1 || D < 1 || B > 65535 || (long long)B * N > (1ll << 31) - 1) return LUVC_ERR_SHAPE;
    if (keep < 1 || keep > N) return LUVC_ERR_KEEP;
    *sigma = luvc_spu_sigma(N, cutoff);
    if (*sigma < 0) return LUVC_ERR_CUTOFF;
    if (((size_t)D * elem_size(dtype)) % 16 != 0) return LUVC_ERR_ALIGN;
    if (!aligned16(hidden) || !aligned16(out_hidden) || (reinterpret_cast<uintptr_t>(out_idx) & 3u))
        return LUVC_ERR_ALIGN;
    return LUVC_OK;
}

}  // namespace
}  // namespace luvc

using namespace luvc;

extern "C" {

int luvc_version(void) { return 1000; }

const char* luvc_status_string(int status) {
    switch (status) {
        case LUVC_OK: return "ok";
        case LUVC_ERR_NULL: return "a required pointer is NULL";
        case LUVC_ERR_SHAPE: return "a dimension is out of range";
        case LUVC_ERR_TARGET: return "the target grid cannot be reached from the input grid";
        case LUVC_ERR_KEEP: return "keep is outside [1, N]";
        case LUVC_ERR_CUTOFF: return "cutoff is NaN or larger than 1";
        case LUVC_ERR_ALIGN: return "a pointer or the row size is not 16-byte aligned";
        case LUVC_ERR_DTYPE: return "unknown element type";
        case LUVC_ERR_WORKSPACE: return "workspace too small or misaligned";
        case LUVC_ERR_CUDA: return "a CUDA call failed";
        case LUVC_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        case LUVC_ERR_INTERNAL: return "internal error";
        default: return "unknown status";
    }
}

int luvc_set_stream(void* cuda_stream) {
    t_stream = static_cast<cudaStream_t>(cuda_stream);
    return LUVC_OK;
}

int luvc_shutdown(void) {
    const int dev = current_device();
    if (dev < 0) return LUVC_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    cudaDeviceSynchronize();
    for (auto& sc : g_scratch[dev]) {
        if (sc.ptr) cudaFree(sc.ptr);
        sc.ptr = nullptr; sc.bytes = 0;
    }
    return LUVC_OK;
}

int luvc_check_status(void* cuda_stream) {
    int* word = status_word();
    if (!word) return LUVC_ERR_CUDA;
    return read_status_block(word, static_cast<cudaStream_t>(cuda_stream));
}

int luvc_read_status(int32_t* device_status, void* cuda_stream) {
    if (!device_status) return LUVC_ERR_NULL;
    return read_status_block(device_status, static_cast<cudaStream_t>(cuda_stream));
}

int luvc_debug_wait_probes(int probes, int hold_back, int32_t* device_status, void* cuda_stream) {
    if (probes < 0 || hold_back < 0) return LUVC_ERR_SHAPE;
    int* block = device_status ? device_status : status_word();
    if (!block) return LUVC_ERR_CUDA;
    const int knobs[2] = {probes, hold_back};
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(block + kStatusProbeLimit, knobs, sizeof(knobs), cudaMemcpyHostToDevice, st) != cudaSuccess)
        return LUVC_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? LUVC_OK : LUVC_ERR_CUDA;   // `knobs` lives on this stack
}

long long luvc_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

int luvc_profile_enable(int on) {
    g_profile.store(on ? 1 : 0, std::memory_order_relaxed);
    return LUVC_OK;
}

int luvc_profile_read(float* ms, int count) {
    if (!ms) return LUVC_ERR_NULL;
    std::lock_guard<std::mutex> lock(g_ev_mutex);
    for (int i = 0; i < count; ++i) {
        ms[i] = 0.f;
        if (i >= LUVC_PHASE_COUNT || !g_ev_made || !g_ev_used[i]) continue;
        if (cudaEventSynchronize(g_ev[i][1]) != cudaSuccess) return LUVC_ERR_CUDA;
        if (cudaEventElapsedTime(&ms[i], g_ev[i][0], g_ev[i][1]) != cudaSuccess) return LUVC_ERR_CUDA;
        g_ev_used[i] = false;
    }
    return LUVC_OK;
}

// ---- OIM ---------------------------------------------------------------------

int luvc_oim_plan(int H, int W, int target_count, int merge_per_step, int* out_h, int* out_w, int* n_steps) {
    if (!out_h || !out_w || !n_steps) return LUVC_ERR_NULL;
    if (H < 1 || W < 1) return LUVC_ERR_SHAPE;
    int hf, wf, n;
    if (merge_per_step < 0 || !oim_final_dims(H, W, target_count, &hf, &wf)) return LUVC_ERR_TARGET;
    const int r = merge_per_step ? merge_per_step : 2;
    if (!oim_schedule(H, W, hf, wf, r, r, 0, nullptr, 0, &n)) return LUVC_ERR_TARGET;
    *out_h = hf; *out_w = wf; *n_steps = n;
    return LUVC_OK;
}

int luvc_oim_plan_anyres(int H, int W, int n_ops, int merge_per_step, int* merge_h, int* merge_w, int* out_h,
                         int* out_w, int* n_steps) {
    if (!merge_h || !merge_w || !out_h || !out_w || !n_steps) return LUVC_ERR_NULL;
    if (H < 1 || W < 1) return LUVC_ERR_SHAPE;
    if (n_ops < 0 || merge_per_step < 0) return LUVC_ERR_TARGET;
    const long long r = merge_per_step ? merge_per_step : 2;
    // the longer side's number is r * long / short rounded to the nearest integer (halves up), in integers
    const long long lo = H < W ? H : W, hi = H < W ? W : H;
    const long long r_long = (2 * r * hi + lo) / (2 * lo);
    const long long rh = H > W ? r_long : r, rw = W > H ? r_long : r;
    const long long hf = H - n_ops * rh, wf = W - n_ops * rw;
    if (hf < 1 || wf < 1 || rh > 0x7fffffffll || rw > 0x7fffffffll) return LUVC_ERR_TARGET;
    int n = 0;
    if (!oim_schedule(H, W, (int)hf, (int)wf, (int)rw, (int)rh, 0, nullptr, 0, &n)) return LUVC_ERR_TARGET;
    *merge_h = (int)rh; *merge_w = (int)rw; *out_h = (int)hf; *out_w = (int)wf; *n_steps = n;
    return LUVC_OK;
}

size_t luvc_oim_workspace_bytes(int B, int H, int W, int D, int dtype) {
    if (B < 1 || H < 1 || W < 1 || D < 1) return 0;
    return oim_workspace_bytes(B, H, W, D, dtype);
}

size_t luvc_oim_workspace_bytes_ex(int B, int H, int W, int D, int dtype, int matching) {
    if (B < 1 || H < 1 || W < 1 || D < 1) return 0;
    if (matching != LUVC_OIM_MATCH_ADJACENT && matching != LUVC_OIM_MATCH_BIPARTITE) return 0;
    return oim_workspace_bytes(B, H, W, D, dtype, matching);
}

int luvc_oim_merge_ex(const void* tokens, int B, int H, int W, int D, int target_count, void* out_tokens,
                      int32_t* out_sizes, int32_t* out_map, const luvc_oim_opts* opts) {
    if (!opts) return LUVC_ERR_NULL;
    int Hf = 0, Wf = 0;
    const int rc = check_oim(tokens, B, H, W, D, target_count, out_tokens, out_sizes, out_map, *opts, &Hf, &Wf);
    if (rc) return rc;
    const size_t need = oim_workspace_bytes(B, H, W, D, opts->dtype, opts->matching);
    void* ws = opts->workspace;
    if (ws) {
        if (opts->workspace_bytes < need || (reinterpret_cast<uintptr_t>(ws) & 255u)) return LUVC_ERR_WORKSPACE;
    } else {
        ws = scratch(kOimWs, need);
        if (!ws) return LUVC_ERR_CUDA;
    }
    OimProblem p;
    p.tokens = tokens; p.B = B; p.H = H; p.W = W; p.D = D; p.Hf = Hf; p.Wf = Wf;
    p.r_w = oim_r_w(*opts); p.r_h = oim_r_h(*opts);
    p.height_first = opts->height_first ? 1 : 0;
    p.dtype = opts->dtype;
    p.out_tokens = out_tokens; p.out_sizes = out_sizes; p.out_map = out_map; p.trace = opts->trace;
    p.out_log_sizes = opts->out_log_sizes;
    p.matching = opts->matching;
    p.workspace = ws; p.stream = static_cast<cudaStream_t>(opts->stream);
    p.status = opts->device_status ? opts->device_status : status_word();
    if (!p.status) return LUVC_ERR_CUDA;
    return oim_run(p);
}

int luvc_oim_merge(const void* tokens, int B, int H, int W, int D, int target_count, void* out_tokens,
                   int32_t* out_sizes, int32_t* out_map) {
    luvc_oim_opts o = {};
    o.dtype = LUVC_BF16; o.stream = t_stream;
    return luvc_oim_merge_ex(tokens, B, H, W, D, target_count, out_tokens, out_sizes, out_map, &o);
}

int luvc_oim_merge_f32(const float* tokens, int B, int H, int W, int D, int target_count, float* out_tokens,
                       int32_t* out_sizes, int32_t* out_map) {
    luvc_oim_opts o = {};
    o.dtype = LUVC_F32; o.stream = t_stream;
    return luvc_oim_merge_ex(tokens, B, H, W, D, target_count, out_tokens, out_sizes, out_map, &o);
}

int luvc_oim_merge_host(const void* tokens, int B, int H, int W, int D, int target_count, int dtype,
                        void* out_tokens, int32_t* out_sizes, int32_t* out_map) {
    if (!tokens || !out_tokens || !out_sizes || !out_map) return LUVC_ERR_NULL;
    if (dtype != LUVC_BF16 && dtype != LUVC_F32) return LUVC_ERR_DTYPE;
    {   // every argument rule of the device form, before anything is allocated or copied (host
        // pointers need no alignment, so an aligned stand-in goes through the pointer checks)
        luvc_oim_opts probe = {};
        probe.dtype = dtype;
        int hf = 0, wf = 0;
        void* const aligned = reinterpret_cast<void*>(uintptr_t{256});
        const int rc = check_oim(aligned, B, H, W, D, target_count, aligned, aligned, aligned, probe, &hf, &wf);
        if (rc) return rc;
    }
    const size_t es = elem_size(dtype), hw = (size_t)H * W;
    const size_t in_bytes = (size_t)B * hw * D * es;
    const size_t tok_bytes = align_up((size_t)B * target_count * D * es);
    const size_t sz_bytes = align_up((size_t)B * target_count * 4), map_bytes = align_up((size_t)B * hw * 4);
    unsigned char* din = static_cast<unsigned char*>(scratch(kIoIn, in_bytes));
    unsigned char* dout = static_cast<unsigned char*>(scratch(kIoOut, tok_bytes + sz_bytes + map_bytes));
    if (!din || !dout) return LUVC_ERR_CUDA;
    cudaStream_t st = t_stream;
    if (cudaMemcpyAsync(din, tokens, in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return LUVC_ERR_CUDA;
    luvc_oim_opts o = {};
    o.dtype = dtype; o.stream = st;
    int32_t* dsz = reinterpret_cast<int32_t*>(dout + tok_bytes);
    int32_t* dmap = reinterpret_cast<int32_t*>(dout + tok_bytes + sz_bytes);
    const int rc = luvc_oim_merge_ex(din, B, H, W, D, target_count, dout, dsz, dmap, &o);
    if (rc) return rc;
    cudaMemcpyAsync(out_tokens, dout, (size_t)B * target_count * D * es, cudaMemcpyDeviceToHost, st);
    cudaMemcpyAsync(out_sizes, dsz, (size_t)B * target_count * 4, cudaMemcpyDeviceToHost, st);
    cudaMemcpyAsync(out_map, dmap, (size_t)B * hw * 4, cudaMemcpyDeviceToHost, st);
    return cudaStreamSynchronize(st) == cudaSuccess ? LUVC_OK : LUVC_ERR_CUDA;
}

int luvc_oim_value_enhance(const void* values, const int32_t* sizes, int B, int T, int D, int dtype, void* out,
                           void* cuda_stream) {
    if (!values || !sizes || !out) return LUVC_ERR_NULL;
    if (dtype != LUVC_BF16 && dtype != LUVC_F32) return LUVC_ERR_DTYPE;
    if (B < 1 || T < 1 || D < 1 || (long long)B * T > (1ll << 31) - 1) return LUVC_ERR_SHAPE;
    if (((size_t)D * elem_size(dtype)) % 16 != 0 || !aligned16(values) || !aligned16(out) ||
        (reinterpret_cast<uintptr_t>(sizes) & 3u))
        return LUVC_ERR_ALIGN;
    return oim_value_enhance(values, sizes, (long long)B * T, D, dtype, out, static_cast<cudaStream_t>(cuda_stream));
}

// ---- SPU ---------------------------------------------------------------------

int luvc_spu_sigma(int N, float cutoff) {
    if (N < 1 || cutoff != cutoff || cutoff > 1.0f) return -1;
    const double c = cutoff <= 0.0f ? (double)LUVC_SPU_DEFAULT_CUTOFF : (double)cutoff;
    return (int)std::floor(c * (double)(N / 2));
}

size_t luvc_spu_workspace_bytes(int B, int N, int D, float cutoff, int dtype) {
    const int sigma = luvc_spu_sigma(N, cutoff);
    if (B < 1 || N < 1 || D < 1 || sigma < 0) return 0;
    return spu_workspace_bytes(B, N, D, sigma, dtype);
}

int luvc_spu_prune_ex(const void* hidden, int B, int N, int D, float cutoff, int keep, int32_t* out_idx,
                      void* out_hidden, const luvc_spu_opts* opts) {
    if (!opts) return LUVC_ERR_NULL;
    int sigma = 0;
    const int rc = check_spu(hidden, B, N, D, cutoff, keep, out_idx, out_hidden, opts->dtype, &sigma);
    if (rc) return rc;
    if (opts->device_status && (reinterpret_cast<uintptr_t>(opts->device_status) & 15u)) return LUVC_ERR_ALIGN;
    const size_t need = spu_workspace_bytes(B, N, D, sigma, opts->dtype);
    void* ws = opts->workspace;
    if (ws) {
        if (opts->workspace_bytes < need || (reinterpret_cast<uintptr_t>(ws) & 255u)) return LUVC_ERR_WORKSPACE;
    } else {
        ws = scratch(kSpuWs, need);
        if (!ws) return LUVC_ERR_CUDA;
    }
    SpuProblem p;
    p.hidden = hidden; p.B = B; p.N = N; p.D = D; p.sigma = sigma; p.keep = keep; p.dtype = opts->dtype;
    p.no_window = opts->no_window ? 1 : 0;
    p.out_idx = out_idx; p.out_hidden = out_hidden; p.out_scores = opts->out_scores;
    p.workspace = ws; p.stream = static_cast<cudaStream_t>(opts->stream);
    p.status = opts->device_status ? opts->device_status : status_word();
    if (!p.status) return LUVC_ERR_CUDA;
    return spu_run(p);
}

int luvc_spu_prune(const void* hidden, int B, int N, int D, float cutoff, int keep, int32_t* out_idx,
                   void* out_hidden) {
    luvc_spu_opts o = {};
    o.dtype = LUVC_BF16; o.stream = t_stream;
    return luvc_spu_prune_ex(hidden, B, N, D, cutoff, keep, out_idx, out_hidden, &o);
}

int luvc_spu_prune_f32(const float* hidden, int B, int N, int D, float cutoff, int keep, int32_t* out_idx,
                       float* out_hidden) {
    luvc_spu_opts o = {};
    o.dtype = LUVC_F32; o.stream = t_stream;
    return luvc_spu_prune_ex(hidden, B, N, D, cutoff, keep, out_idx, out_hidden, &o);
}

int luvc_spu_cascade(const void* hidden, int B, int N, int D, int n_stages, const int* keeps, const float* cutoffs,
                     int dtype, void* cuda_stream, int32_t* out_idx, void* out_hidden) {
    if (!hidden || !keeps || !out_idx || !out_hidden) return LUVC_ERR_NULL;
    if (dtype != LUVC_BF16 && dtype != LUVC_F32) return LUVC_ERR_DTYPE;
    if (B < 1 || N < 1 || D < 1 || n_stages < 1) return LUVC_ERR_SHAPE;
    int prev = N;
    for (int t = 0; t < n_stages; ++t) {
        if (keeps[t] < 1 || keeps[t] > prev) return LUVC_ERR_KEEP;
        if (cutoffs && (cutoffs[t] != cutoffs[t] || cutoffs[t] > 1.0f)) return LUVC_ERR_CUTOFF;
        prev = keeps[t];
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    luvc_spu_opts o = {};
    o.dtype = dtype; o.stream = cuda_stream;
    if (n_stages == 1) return luvc_spu_prune_ex(hidden, B, N, D, cutoffs ? cutoffs[0] : 0.f, keeps[0], out_idx, out_hidden, &o);
    {   // pointer and row-size rules of a single prune (the stages run through the internal entry point)
        int sg = 0;
        const int rc = check_spu(hidden, B, N, D, cutoffs ? cutoffs[0] : 0.f, keeps[0], out_idx, out_hidden, dtype, &sg);
        if (rc) return rc;
    }
    // Stage t > 0 reads the survivors' rows straight out of `hidden` through the index list composed so far
    // (gather on load) whenever a sequence of that length runs the dense contractions anyway; only a stage
    // long enough for the two-stage kernels, which walk dense memory, gets its rows copied out first.  The
    // survivors' rows are written once, by the last stage.
    const size_t es = elem_size(dtype);
    int sigmas[64];
    if (n_stages > 64) return LUVC_ERR_SHAPE;
    size_t ws_need = 0, rows_need = 0;
    int n_in = N;
    for (int t = 0; t < n_stages; ++t) {
        sigmas[t] = luvc_spu_sigma(n_in, cutoffs ? cutoffs[t] : 0.f);
        if (sigmas[t] < 0) return LUVC_ERR_CUTOFF;
        const bool fuse = t > 0 && spu_dense_is_natural(B, n_in, D, sigmas[t], dtype);
        const size_t need = spu_workspace_bytes(B, n_in, D, sigmas[t], dtype, fuse);
        ws_need = need > ws_need ? need : ws_need;
        if (t > 0 && !fuse) rows_need = align_up((size_t)B * n_in * D * es) > rows_need ? align_up((size_t)B * n_in * D * es) : rows_need;
        n_in = keeps[t];
    }
    const size_t idxb = align_up((size_t)B * keeps[0] * 4);
    unsigned char* sc = static_cast<unsigned char*>(scratch(kCascade, rows_need + 3 * idxb));
    void* ws = scratch(kSpuWs, ws_need);
    int* status = status_word();
    if (!sc || !ws || !status) return LUVC_ERR_CUDA;
    void* rows_buf = sc;
    int32_t* idx_stage = reinterpret_cast<int32_t*>(sc + rows_need);
    int32_t* idx_tot[2] = {reinterpret_cast<int32_t*>(sc + rows_need + idxb), reinterpret_cast<int32_t*>(sc + rows_need + 2 * idxb)};
    const int32_t* cur = nullptr;      // survivors so far as rows of `hidden` (null: all N, in order)
    n_in = N;
    for (int t = 0; t < n_stages; ++t) {
        const bool last = t == n_stages - 1;
        const bool fuse = t > 0 && spu_dense_is_natural(B, n_in, D, sigmas[t], dtype);
        SpuProblem p;
        p.B = B; p.N = n_in; p.D = D; p.sigma = sigmas[t]; p.keep = keeps[t]; p.dtype = dtype; p.no_window = 0;
        p.out_idx = idx_stage; p.out_hidden = nullptr; p.out_scores = nullptr;
        p.workspace = ws; p.status = status; p.stream = st;
        if (t == 0) {
            p.hidden = hidden;
        } else if (fuse) {
            p.hidden = hidden; p.row_index = cur; p.src_rows = N;
        } else {
            int rc = spu_gather_rows(hidden, cur, rows_buf, B, N, n_in, D, dtype, st);
            if (rc) return rc;
            p.hidden = rows_buf;
        }
        int rc = spu_run(p);
        if (rc) return rc;
        int32_t* tot = last ? out_idx : idx_tot[t & 1];
        rc = spu_compose_indices(cur, idx_stage, tot, B, t == 0 ? 0 : keeps[t - 1], keeps[t], st);
        if (rc) return rc;
        cur = tot;
        n_in = keeps[t];
    }
    return spu_gather_rows(hidden, out_idx, out_hidden, B, N, keeps[n_stages - 1], D, dtype, st);
}

int luvc_spu_prune_host(const void* hidden, int B, int N, int D, float cutoff, int keep, int dtype,
                        int32_t* out_idx, void* out_hidden) {
    if (!hidden || !out_idx || !out_hidden) return LUVC_ERR_NULL;
    if (dtype != LUVC_BF16 && dtype != LUVC_F32) return LUVC_ERR_DTYPE;
    {   // the device form's argument rules first: nothing is allocated or copied for a bad request
        int sigma = 0;
        void* const aligned = reinterpret_cast<void*>(uintptr_t{256});
        const int rc = check_spu(aligned, B, N, D, cutoff, keep, aligned, aligned, dtype, &sigma);
        if (rc) return rc;
    }
    const size_t es = elem_size(dtype);
    const size_t in_bytes = (size_t)B * N * D * es, hid_bytes = align_up((size_t)B * keep * D * es);
    unsigned char* din = static_cast<unsigned char*>(scratch(kIoInSpu, in_bytes));
    unsigned char* dout = static_cast<unsigned char*>(scratch(kIoOutSpu, hid_bytes + align_up((size_t)B * keep * 4)));
    if (!din || !dout) return LUVC_ERR_CUDA;
    cudaStream_t st = t_stream;
    if (cudaMemcpyAsync(din, hidden, in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return LUVC_ERR_CUDA;
    luvc_spu_opts o = {};
    o.dtype = dtype; o.stream = st;
    int32_t* didx = reinterpret_cast<int32_t*>(dout + hid_bytes);
    const int rc = luvc_spu_prune_ex(din, B, N, D, cutoff, keep, didx, dout, &o);
    if (rc) return rc;
    cudaMemcpyAsync(out_hidden, dout, (size_t)B * keep * D * es, cudaMemcpyDeviceToHost, st);
    cudaMemcpyAsync(out_idx, didx, (size_t)B * keep * 4, cudaMemcpyDeviceToHost, st);
    return cudaStreamSynchronize(st) == cudaSuccess ? LUVC_OK : LUVC_ERR_CUDA;
}

}  // extern "C"
