// Orthogonal Iterative Merger (Section 3.2 of the paper) for sm_100a.
//
// Data layout.  The token vectors never move.  A cell of the current grid is
// named by its root: the index (0 .. H*W-1) of one of its source tokens.  A
// cell that has absorbed nothing reads its vector straight from the caller's
// input row; a cell that has absorbed others keeps the fp32 SUM of its sources
// in row `root` of a scratch matrix acc[B][H*W][D] (cosines are scale-free, so
// sums serve for the similarity; the mean is formed once, at the end).  The
// grid itself is a small int32 matrix of roots that is compacted every step.
// A step therefore reads every live vector once (that is the algorithm: all
// neighbour similarities along the axis change when the orthogonal axis was
// compacted) and writes only the merged rows.
//
// One CTA owns one line (row or column) of one image for one step: its warps
// stream the line's vectors with 128-bit loads and fp32 accumulation, warp 0
// ranks the even-position cells, then the warps apply the merges and close the
// line up.  Lines are independent inside a step, so a step is one launch.

#include <cuda_bf16.h>
#include <float.h>

#include "luvc_internal.h"

namespace luvc {
namespace {

constexpr int kStepThreads = 256;
constexpr unsigned kMergedBit = 0x80000000u;

template <typename T> struct Elem;
template <> struct Elem<__nv_bfloat16> { static constexpr int kVec = 8; };   // elements per 16 bytes
template <> struct Elem<float> { static constexpr int kVec = 4; };

__device__ __forceinline__ float bf16lo(unsigned u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(unsigned u) { return __uint_as_float(u & 0xffff0000u); }

// Loads kVec consecutive elements starting at element e of a cell's vector as fp32:
// from the fp32 sum row when the cell is merged, else from the caller's input row.
template <typename T>
__device__ __forceinline__ void load_vec(const T* __restrict__ tok_row, const float* __restrict__ acc_row,
                                         bool merged, int e, float (&v)[Elem<T>::kVec]) {
    constexpr int V = Elem<T>::kVec;
    if (merged) {
#pragma unroll
        for (int q = 0; q < V; q += 4) {
            const float4 f = *reinterpret_cast<const float4*>(acc_row + e + q);
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

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

__global__ void oim_init_kernel(int32_t* cell, int32_t* size, int32_t* parent, int HW, long long total) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    cell[i] = (int32_t)(i % HW);
    size[i] = 1;
    parent[i] = -1;
}

struct StepArgs {
    const void* tokens;   // [B][HW][D] caller input
    float* acc;           // [B][HW][D] fp32 sums of merged cells
    const int32_t* cell_in;
    int32_t* cell_out;
    int32_t* size;        // [B][HW] by root
    int32_t* parent;      // [B][HW] by root: the root this one was merged into, or -1
    int32_t* trace;       // this step's slice of image 0, or null
    long long trace_stride;  // ints per image in the trace
    int h, w, axis, m, D, HW;
};

// |x|^2 and <x, y> over one lane's share of two vectors.  NCHUNK > 0: D == NCHUNK * 32 * kVec and
// the loop is fully unrolled so that all of a lane's loads are in flight together.
template <typename T, int NCHUNK>
__device__ __forceinline__ void pair_stats(const T* __restrict__ t0, const float* __restrict__ a0, bool m0,
                                           const T* __restrict__ t1, const float* __restrict__ a1, bool m1,
                                           bool has_next, int lane, int D, float& nn, float& dd) {
    constexpr int V = Elem<T>::kVec;
    if (has_next) {
        if constexpr (NCHUNK > 0) {
#pragma unroll
            for (int c = 0; c < NCHUNK; ++c) {
                float x[V], y[V];
                load_vec<T>(t0, a0, m0, (c * 32 + lane) * V, x);
                load_vec<T>(t1, a1, m1, (c * 32 + lane) * V, y);
#pragma unroll
                for (int q = 0; q < V; ++q) { nn = fmaf(x[q], x[q], nn); dd = fmaf(x[q], y[q], dd); }
            }
        } else {
#pragma unroll 2
            for (int e = lane * V; e < D; e += 32 * V) {
                float x[V], y[V];
                load_vec<T>(t0, a0, m0, e, x);
                load_vec<T>(t1, a1, m1, e, y);
#pragma unroll
                for (int q = 0; q < V; ++q) { nn = fmaf(x[q], x[q], nn); dd = fmaf(x[q], y[q], dd); }
            }
        }
    } else {
        if constexpr (NCHUNK > 0) {
#pragma unroll
            for (int c = 0; c < NCHUNK; ++c) {
                float x[V];
                load_vec<T>(t0, a0, m0, (c * 32 + lane) * V, x);
#pragma unroll
                for (int q = 0; q < V; ++q) nn = fmaf(x[q], x[q], nn);
            }
        } else {
#pragma unroll 2
            for (int e = lane * V; e < D; e += 32 * V) {
                float x[V];
                load_vec<T>(t0, a0, m0, e, x);
#pragma unroll
                for (int q = 0; q < V; ++q) nn = fmaf(x[q], x[q], nn);
            }
        }
    }
}

template <typename T, int NCHUNK>
__global__ void __launch_bounds__(kStepThreads, 3) oim_step_kernel(const StepArgs a) {
    constexpr int V = Elem<T>::kVec;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int len = a.axis == 0 ? a.w : a.h;
    const int ncand = (len + 1) >> 1;
    float* s_dot = reinterpret_cast<float*>(smem_raw);          // <v_j, v_{j+1}>
    float* s_nrm = s_dot + len;                                  // |v_j|^2
    float* s_score = s_nrm + len;                                // best cosine of even cell 2c
    unsigned* s_root = reinterpret_cast<unsigned*>(s_score + ncand);   // root | merged bit
    int* s_dir = reinterpret_cast<int*>(s_root + len);           // best direction of even cell 2c
    int* s_sel = s_dir + ncand;                                  // chosen (pos * 2 + dir), m entries

    const int b = blockIdx.y, line = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = kStepThreads >> 5;
    const int base = a.axis == 0 ? line * a.w : line;
    const int stride = a.axis == 0 ? 1 : a.w;
    const size_t img = (size_t)b * a.HW;
    const int32_t* cell_in = a.cell_in + img;
    int32_t* size = a.size + img;
    const T* tokens = reinterpret_cast<const T*>(a.tokens) + img * a.D;
    float* acc = a.acc + img * a.D;
    const int D = a.D;

    for (int j = tid; j < len; j += kStepThreads) {
        const unsigned r = (unsigned)cell_in[base + j * stride];
        s_root[j] = r | (size[r] > 1 ? kMergedBit : 0u);
    }
    __syncthreads();

    // ---- similarity pass: one warp per cell, norm of v_j and dot with its successor
    for (int j = warp; j < len; j += nwarps) {
        const unsigned r0 = s_root[j];
        const bool m0 = r0 & kMergedBit;
        const size_t o0 = (size_t)(r0 & ~kMergedBit) * D;
        const bool has_next = j + 1 < len;
        const unsigned r1 = has_next ? s_root[j + 1] : r0;
        const bool m1 = r1 & kMergedBit;
        const size_t o1 = (size_t)(r1 & ~kMergedBit) * D;
        float nn = 0.f, dd = 0.f;
        pair_stats<T, NCHUNK>(tokens + o0, acc + o0, m0, tokens + o1, acc + o1, m1, has_next, lane, D, nn, dd);
        nn = warp_sum(nn);
        dd = warp_sum(dd);
        if (lane == 0) { s_nrm[j] = nn; s_dot[j] = dd; }
    }
    __syncthreads();

    // ---- ranking: warp 0 scores the even cells and takes the m best
    if (warp == 0) {
        for (int c = lane; c < ncand; c += 32) {
            const int j = 2 * c;
            const float nj = sqrtf(s_nrm[j]);
            float cl = -FLT_MAX, cr = -FLT_MAX;
            if (j >= 1) {
                const float nb = sqrtf(s_nrm[j - 1]);
                cl = (nj == 0.f || nb == 0.f) ? 0.f : s_dot[j - 1] / (nj * nb);
                if (!(cl == cl)) cl = -FLT_MAX;
            }
            if (j + 1 < len) {
                const float nb = sqrtf(s_nrm[j + 1]);
                cr = (nj == 0.f || nb == 0.f) ? 0.f : s_dot[j] / (nj * nb);
                if (!(cr == cr)) cr = -FLT_MAX;
            }
            const bool right = (j < 1) || (j + 1 < len && cr > cl);   // ties stay with the previous cell
            s_dir[c] = right ? 1 : 0;
            s_score[c] = right ? cr : cl;
        }
        __syncwarp();
        for (int k = 0; k < a.m; ++k) {
            float best = -INFINITY;
            int best_c = 0x7fffffff;
            for (int c = lane; c < ncand; c += 32) {
                const float s = s_score[c];
                if (s > best) { best = s; best_c = c; }   // ascending c: the first maximum stays
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ob = __shfl_xor_sync(0xffffffffu, best, o);
                const int oc = __shfl_xor_sync(0xffffffffu, best_c, o);
                if (ob > best || (ob == best && oc < best_c)) { best = ob; best_c = oc; }
            }
            if (lane == 0) {
                s_sel[k] = (2 * best_c) * 2 + s_dir[best_c];
                s_score[best_c] = -INFINITY;             // taken
            }
            __syncwarp();
        }
        if (a.trace != nullptr)
            for (int k = lane; k < a.m; k += 32)
                a.trace[(size_t)b * a.trace_stride + (size_t)line * a.m + k] = s_sel[k];
    }
    __syncthreads();

    // ---- close the line up: surviving cells keep their order
    {
        int32_t* cell_out = a.cell_out + img;
        const int out_w = a.axis == 0 ? a.w - a.m : a.w;
        for (int j = tid; j < len; j += kStepThreads) {
            int before = 0;
            bool removed = false;
            for (int k = 0; k < a.m; ++k) {
                const int p = s_sel[k] >> 1;   // position of the merged cell
                removed |= p == j;
                before += p < j;
            }
            if (!removed) {
                const int nj = j - before;
                const int dst = a.axis == 0 ? line * out_w + nj : nj * out_w + line;
                cell_out[dst] = (int32_t)(s_root[j] & ~kMergedBit);
            }
        }
    }

    // ---- merges: one warp per destination cell; its new sum is written as fp32
    for (int k = warp; k < a.m; k += nwarps) {
        const int pos = s_sel[k] >> 1, dst = pos + ((s_sel[k] & 1) ? 1 : -1);
        bool first = true;          // the lowest rank that targets this destination does the work
        int other = -1;             // a second source of the same destination, if any
        for (int q = 0; q < a.m; ++q) {
            if (q == k) continue;
            const int qpos = s_sel[q] >> 1, qdst = qpos + ((s_sel[q] & 1) ? 1 : -1);
            if (qdst == dst) { if (q < k) first = false; else other = qpos; }
        }
        if (!first) continue;
        const unsigned rd = s_root[dst], ra = s_root[pos], rb = other >= 0 ? s_root[other] : 0u;
        const size_t od = (size_t)(rd & ~kMergedBit) * D, oa = (size_t)(ra & ~kMergedBit) * D,
                     ob = (size_t)(rb & ~kMergedBit) * D;
        for (int e = lane * V; e < D; e += 32 * V) {
            float x[V], y[V];
            load_vec<T>(tokens + od, acc + od, rd & kMergedBit, e, x);
            load_vec<T>(tokens + oa, acc + oa, ra & kMergedBit, e, y);
#pragma unroll
            for (int q = 0; q < V; ++q) x[q] += y[q];
            if (other >= 0) {
                load_vec<T>(tokens + ob, acc + ob, rb & kMergedBit, e, y);
#pragma unroll
                for (int q = 0; q < V; ++q) x[q] += y[q];
            }
#pragma unroll
            for (int q = 0; q < V; q += 4)
                *reinterpret_cast<float4*>(acc + od + e + q) = make_float4(x[q], x[q + 1], x[q + 2], x[q + 3]);
        }
        if (lane == 0) {
            const int id = rd & ~kMergedBit, ia = ra & ~kMergedBit;
            int s = size[id] + size[ia];
            a.parent[img + ia] = id;
            if (other >= 0) {
                const int ib = rb & ~kMergedBit;
                s += size[ib];
                a.parent[img + ib] = id;
            }
            size[id] = s;
        }
    }
}

// One warp per final cell: the mean of its sources in the caller's element type,
// its size, and the root -> cell table the map kernel needs.
template <typename T>
__global__ void __launch_bounds__(256) oim_emit_kernel(const void* tokens_v, const float* acc, const int32_t* cell,
                                                       const int32_t* size, int32_t* cellpos, void* out_v,
                                                       int32_t* out_sizes, int HW, int target, int D,
                                                       long long total_cells) {
    constexpr int V = Elem<T>::kVec;
    const long long gw = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (gw >= total_cells) return;
    const int b = (int)(gw / target), c = (int)(gw % target);
    const size_t img = (size_t)b * HW;
    const int root = cell[img + c];
    const int s = size[img + root];
    const T* tok = reinterpret_cast<const T*>(tokens_v) + (img + root) * D;
    const float* arow = acc + (img + root) * D;
    T* out = reinterpret_cast<T*>(out_v) + ((size_t)b * target + c) * D;
    if (lane == 0) { out_sizes[(size_t)b * target + c] = s; cellpos[img + root] = c; }
    if (s == 1) {
        for (int e = lane * V; e < D; e += 32 * V)
            *reinterpret_cast<uint4*>(out + e) = __ldg(reinterpret_cast<const uint4*>(tok + e));
        return;
    }
    const float fs = (float)s;
    for (int e = lane * V; e < D; e += 32 * V) {
        float x[V];
        load_vec<T>(tok, arow, true, e, x);
#pragma unroll
        for (int q = 0; q < V; ++q) x[q] = x[q] / fs;
        if constexpr (sizeof(T) == 4) {
            *reinterpret_cast<float4*>(out + e) = make_float4(x[0], x[1], x[2], x[3]);
        } else {
            uint4 u;
            __nv_bfloat162 p;
            p = __floats2bfloat162_rn(x[0], x[1]); u.x = *reinterpret_cast<unsigned*>(&p);
            p = __floats2bfloat162_rn(x[2], x[3]); u.y = *reinterpret_cast<unsigned*>(&p);
            p = __floats2bfloat162_rn(x[4], x[5]); u.z = *reinterpret_cast<unsigned*>(&p);
            p = __floats2bfloat162_rn(x[6], x[7]); u.w = *reinterpret_cast<unsigned*>(&p);
            *reinterpret_cast<uint4*>(out + e) = u;
        }
    }
}

// Every source token follows its chain of merges to the root that survived.
__global__ void oim_map_kernel(const int32_t* parent, const int32_t* cellpos, int32_t* out_map, int HW,
                               long long total) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const size_t img = (size_t)(i / HW) * HW;
    int r = (int)(i % HW);
    for (int hop = 0; hop < HW; ++hop) {   // a chain is shorter than the number of tokens
        const int p = parent[img + r];
        if (p < 0) break;
        r = p;
    }
    out_map[i] = cellpos[img + r];
}

struct Workspace {
    float* acc;
    int32_t *cell_a, *cell_b, *size, *parent, *cellpos;
};

Workspace carve(void* ws, int B, int HW, int D) {
    unsigned char* p = static_cast<unsigned char*>(ws);
    Workspace w;
    const size_t n = (size_t)B * HW;
    w.acc = reinterpret_cast<float*>(p); p += align_up(n * D * sizeof(float));
    w.cell_a = reinterpret_cast<int32_t*>(p); p += align_up(n * 4);
    w.cell_b = reinterpret_cast<int32_t*>(p); p += align_up(n * 4);
    w.size = reinterpret_cast<int32_t*>(p); p += align_up(n * 4);
    w.parent = reinterpret_cast<int32_t*>(p); p += align_up(n * 4);
    w.cellpos = reinterpret_cast<int32_t*>(p);
    return w;
}

}  // namespace

bool oim_final_dims(int H, int W, int target, int* Hf, int* Wf) {
    if (H < 1 || W < 1 || target < 1 || (long long)target > (long long)H * W) return false;
    // the admissible factor pair whose shape is nearest to the input's, compared as
    // cross products so that no logarithm is needed: |ln(hf/wf) - ln(H/W)| is monotone
    // in max(hf*W, wf*H) / min(hf*W, wf*H)
    int bh = 0, bw = 0;
    double best = 0;
    for (int hf = H; hf >= 1; --hf) {   // descending: on a tie the larger height is met first
        if (target % hf) continue;
        const int wf = target / hf;
        if (wf > W) continue;
        const double x = (double)hf * W, y = (double)wf * H;
        const double ratio = x > y ? x / y : y / x;
        if (!bh || ratio < best * (1.0 - 1e-12)) { best = ratio; bh = hf; bw = wf; }
    }
    if (!bh) return false;
    *Hf = bh; *Wf = bw;
    return true;
}

bool oim_schedule(int H, int W, int Hf, int Wf, int r, int height_first, OimStep* steps, int cap, int* n_steps) {
    if (Hf < 1 || Wf < 1 || Hf > H || Wf > W || r < 1) return false;
    int h = H, w = W, n = 0;
    while (h != Hf || w != Wf) {
        bool moved = false;
        for (int turn = 0; turn < 2; ++turn) {
            const int axis = height_first ? 1 - turn : turn;
            const int len = axis == 0 ? w : h, goal = axis == 0 ? Wf : Hf;
            int m = len - goal < r ? len - goal : r;
            if (m > (len + 1) / 2) m = (len + 1) / 2;   // only even-position cells can be merged away
            if (len < 2 || m <= 0) continue;
            if (steps && n < cap) steps[n] = OimStep{axis, m, h, w};
            ++n;
            if (axis == 0) w -= m; else h -= m;
            moved = true;
        }
        if (!moved) return false;
    }
    *n_steps = n;
    return true;
}

size_t oim_workspace_bytes(int B, int H, int W, int D, int /*dtype*/) {
    const size_t n = (size_t)B * H * W;
    return align_up(n * D * sizeof(float)) + 5 * align_up(n * 4);
}

template <typename T>
static int oim_run_typed(const OimProblem& p) {
    const int HW = p.H * p.W, target = p.Hf * p.Wf;
    const long long n = (long long)p.B * HW;
    Workspace ws = carve(p.workspace, p.B, HW, p.D);
    int n_steps = 0;
    const int cap = 2 * (p.H + p.W) + 4;
    OimStep* steps = new OimStep[cap];
    if (!oim_schedule(p.H, p.W, p.Hf, p.Wf, p.r, p.height_first, steps, cap, &n_steps)) {
        delete[] steps;
        return LUVC_ERR_TARGET;
    }
    phase_begin(LUVC_PHASE_OIM_TOTAL, p.stream);
    oim_init_kernel<<<(unsigned)((n + 255) / 256), 256, 0, p.stream>>>(ws.cell_a, ws.size, ws.parent, HW, n);
    count_launch();
    phase_begin(LUVC_PHASE_OIM_STEPS, p.stream);
    int32_t *cin = ws.cell_a, *cout = ws.cell_b;
    long long trace_off = 0;
    for (int s = 0; s < n_steps; ++s) {
        const OimStep& st = steps[s];
        const int len = st.axis == 0 ? st.w : st.h, lines = st.axis == 0 ? st.h : st.w;
        StepArgs a;
        a.tokens = p.tokens; a.acc = ws.acc; a.cell_in = cin; a.cell_out = cout;
        a.size = ws.size; a.parent = ws.parent;
        a.trace = p.trace ? p.trace + trace_off : nullptr;
        a.trace_stride = (long long)HW - target;
        a.h = st.h; a.w = st.w; a.axis = st.axis; a.m = st.m; a.D = p.D; a.HW = HW;
        const size_t smem = (size_t)(3 * len + 2 * ((len + 1) / 2) + st.m + 8) * 4;
        const int chunk = 32 * Elem<T>::kVec;
        const int nchunk = p.D % chunk == 0 ? p.D / chunk : 0;
        const dim3 grid(lines, p.B);
        switch (nchunk) {
            case 4: oim_step_kernel<T, 4><<<grid, kStepThreads, smem, p.stream>>>(a); break;
            case 5: oim_step_kernel<T, 5><<<grid, kStepThreads, smem, p.stream>>>(a); break;
            case 8: oim_step_kernel<T, 8><<<grid, kStepThreads, smem, p.stream>>>(a); break;
            default: oim_step_kernel<T, 0><<<grid, kStepThreads, smem, p.stream>>>(a); break;
        }
        count_launch();
        trace_off += (long long)lines * st.m;
        int32_t* t = cin; cin = cout; cout = t;
    }
    delete[] steps;
    phase_end(LUVC_PHASE_OIM_STEPS, p.stream);
    const long long cells = (long long)p.B * target;
    oim_emit_kernel<T><<<(unsigned)((cells * 32 + 255) / 256), 256, 0, p.stream>>>(
        p.tokens, ws.acc, cin, ws.size, ws.cellpos, p.out_tokens, p.out_sizes, HW, target, p.D, cells);
    count_launch();
    oim_map_kernel<<<(unsigned)((n + 255) / 256), 256, 0, p.stream>>>(ws.parent, ws.cellpos, p.out_map, HW, n);
    count_launch();
    phase_end(LUVC_PHASE_OIM_TOTAL, p.stream);
    return cudaGetLastError() == cudaSuccess ? LUVC_OK : LUVC_ERR_CUDA;
}

int oim_run(const OimProblem& p) {
    return p.dtype == LUVC_F32 ? oim_run_typed<float>(p) : oim_run_typed<__nv_bfloat16>(p);
}

}  // namespace luvc
