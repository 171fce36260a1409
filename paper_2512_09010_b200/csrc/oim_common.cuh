// Definitions shared by the two OIM chain kernels (adjacent-pair matching and full-line
// bipartite matching): the cell-grid encoding, the step table, the kernel arguments, the
// vector loads and the bounded wait on an image's line counter.  Device-only, header-only.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "luvc_internal.h"

namespace luvc {
namespace {

constexpr unsigned kMergedBit = 0x80000000u;
constexpr int kSpinLimit = 1 << 20;        // about a microsecond per probe: gives up after roughly a second

template <typename T> struct Elem;
template <> struct Elem<__nv_bfloat16> { static constexpr int kVec = 8; };   // elements per 16 bytes
template <> struct Elem<float> { static constexpr int kVec = 4; };

__device__ __forceinline__ float bf16lo(unsigned u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(unsigned u) { return __uint_as_float(u & 0xffff0000u); }

// Loads kVec consecutive elements starting at element e of a cell's vector as fp32:
// from the fp32 sum row when the cell is merged (written during this kernel: L2 only),
// else from the caller's read-only input row.
template <typename T>
__device__ __forceinline__ void load_vec(const T* __restrict__ tok_row, const float* acc_row, bool merged, int e,
                                         float (&v)[Elem<T>::kVec]) {
    constexpr int V = Elem<T>::kVec;
    if (merged) {
#pragma unroll
        for (int q = 0; q < V; q += 4) {
            const float4 f = __ldcg(reinterpret_cast<const float4*>(acc_row + e + q));
            v[q] = f.x; v[q + 1] = f.y; v[q + 2] = f.z; v[q + 3] = f.w;
        }
    } else if constexpr (sizeof(T) == 4) {
        const float4 f = __ldg(reinterpret_cast<const float4*>(tok_row + e));
        v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
    } else {
        const uint4 u = __ldg(reinterpret_cast<const uint4*>(tok_row + e));
        v[0] = bf16lo(u.x); v[1] = bf16hi(u.x); v[2] = bf16lo(u.y); v[3] = bf16hi(u.y);
        v[4] = bf16lo(u.z); v[5] = bf16hi(u.z); v[6] = bf16lo(u.w); v[7] = bf16hi(u.w);
    }
}

}  // namespace

// One entry per merge step, built on the device by the set-up kernel.
struct StepDesc {
    int axis;        // 0: lines are rows, the width shrinks; 1: lines are columns, the height shrinks
    int m;           // cells removed per line
    int h, w;        // grid before the step
    int item_begin;  // first work item of the step (items are step-major, then image, then line)
    int trace_off;   // offset of the step's decisions inside one image's trace
};

struct ChainArgs {
    const void* tokens;   // [B][HW][D] caller input
    float* acc;           // [B][HW][D] fp32 sums of merged cells
    int32_t* cell[2];     // [B][HW] grid of (root | merged bit), ping-pong by step parity
    int32_t* size;        // [B][HW] by root
    int32_t* parent;      // [B][HW] by root: the root this one was merged into, or -1
    int32_t* trace;       // [B][HW - target] or null
    const StepDesc* steps;
    int* done;            // [n_steps][B] finished lines
    int* next_item;       // work counter
    int* status;          // device status word (0 = ok)
    int B, HW, D, n_steps, total_items, trace_stride;
};

namespace {

__device__ __forceinline__ int load_acquire(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Thread 0 of a CTA waits until *ctr reaches `target`.  Gives up after kSpinLimit probes (or as soon
// as another CTA has reported a failure) and records LUVC_ERR_TIMEOUT in the status word.  The
// second word of the status block, when positive, replaces the probe limit (test knob).
__device__ __forceinline__ bool wait_for_count(const int* ctr, int target, int* status) {
    if (load_acquire(ctr) >= target) return true;                   // the usual case: nothing else is read
    const int knob = load_acquire(status + kStatusProbeLimit);      // 0 unless a test shortened the wait
    const int limit = knob > 0 ? knob : kSpinLimit;
    for (int it = 0; it < limit; ++it) {
        if (load_acquire(ctr) >= target) return true;
        if (load_acquire(status) != 0) return false;
        __nanosleep(it < 64 ? 32 : 256);
    }
    atomicCAS(status, 0, (int)LUVC_ERR_TIMEOUT);
    return false;
}

}  // namespace

// The chain of merge steps with the full-line bipartite matching (oim_bipartite.cu).
// dtype: LUVC_BF16 or LUVC_F32; max_len: longest line of the schedule; r: merge number.
// It keeps, beside the chain's own scratch, split[B][HW][2][D] (bf16 hi and lo parts of every fp32
// row) and nrm2[B][HW] (squared norm by root); oim_bipartite_prepare fills nrm2 (and, for fp32
// input, split) from the input tokens.  They travel apart from ChainArgs, whose layout the
// adjacent-pair kernel's register allocation is tuned to.
cudaError_t oim_bipartite_prepare(const ChainArgs& a, __nv_bfloat16* split, float* nrm2, int dtype, cudaStream_t stream);
cudaError_t oim_bipartite_launch(const ChainArgs& a, __nv_bfloat16* split, float* nrm2, int dtype, int max_len, int r,
                                 cudaStream_t stream);

}  // namespace luvc
