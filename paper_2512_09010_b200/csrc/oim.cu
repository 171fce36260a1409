// Orthogonal Iterative Merger (Section 3.2 of the paper) for sm_100a.
//
// Data layout.  The token vectors never move.  A cell of the current grid is
// named by its root: the index (0 .. H*W-1) of one of its source tokens.  A
// cell that has absorbed nothing reads its vector straight from the caller's
// input row; a cell that has absorbed others keeps the fp32 SUM of its sources
// in row `root` of a scratch matrix acc[B][H*W][D] (cosines are scale-free, so
// sums serve for the similarity; the mean is formed once, at the end).  The
// grid itself is a small int32 matrix of (root | merged-bit) that is compacted
// every step.  A step therefore reads every live vector once (that is the
// algorithm: all neighbour similarities along the axis change when the
// orthogonal axis was compacted) and writes only the merged rows.
//
// Execution.  The whole chain of steps of one call is ONE persistent kernel.
// Its work items are the lines (rows or columns) of every image at every step,
// numbered step-major, and handed out through an atomic counter.  A line of
// image b at step s needs only image b's lines of step s-1, so each image has a
// counter of finished lines per step and an item waits (bounded spin) on its
// image's previous counter: images drift apart and one image's ranking and
// merging overlaps another's streaming; there is no grid-wide barrier and no
// launch between steps.  Items are claimed only by running CTAs and depend
// only on lower-numbered items, so the lowest unfinished item can always run
// and no co-residency guarantee is needed.
//
// One CTA owns one line: its warps stream the line's vectors with 128-bit
// loads and fp32 accumulation (norm of each cell and dot with its successor),
// warp 0 ranks the even-position cells, then the warps apply the merges and
// close the line up.  Data written inside the kernel by other CTAs (grid,
// sizes, fp32 sums) is read with L1-bypassing loads.

#include <cuda_bf16.h>
#include <float.h>

#include "luvc_internal.h"
#include "oim_common.cuh"

namespace luvc {
namespace {

// Asks L2 for `bytes` (a multiple of 16) starting at the 16-byte aligned address p; nothing waits for it.
__device__ __forceinline__ void prefetch_l2(const void* p, unsigned bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// |x|^2 and <x, y> over one lane's share of two vectors.  NCHUNK > 0: D == NCHUNK * 32 * kVec and
// the loop is fully unrolled so that all of a lane's loads are in flight together.
template <typename T, int NCHUNK>
__device__ __forceinline__ void pair_stats(const T* __restrict__ t0, const float* a0, bool m0,
                                           const T* __restrict__ t1, const float* a1, bool m1, bool has_next,
                                           int lane, int D, float& nn, float& dd) {
    constexpr int V = Elem<T>::kVec;
    if (has_next) {
        if constexpr (NCHUNK > 0) {
#pragma unroll
            float2 nn2 = make_float2(0.f, 0.f), dd2 = make_float2(0.f, 0.f);   // packed FMAs: even and odd elements apart
#pragma unroll
            for (int c = 0; c < NCHUNK; ++c) {
                float x[V], y[V];
                load_vec<T>(t0, a0, m0, (c * 32 + lane) * V, x);
                load_vec<T>(t1, a1, m1, (c * 32 + lane) * V, y);
#pragma unroll
                for (int q = 0; q < V; q += 2) {
                    const float2 xx = make_float2(x[q], x[q + 1]);
                    nn2 = __ffma2_rn(xx, xx, nn2);
                    dd2 = __ffma2_rn(xx, make_float2(y[q], y[q + 1]), dd2);
                }
            }
            nn += nn2.x + nn2.y;
            dd += dd2.x + dd2.y;
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

// Set-up: identity grid, unit sizes, no parents, zeroed counters, and the step table
// (the same rule the host uses to validate the request).
__global__ void oim_setup_kernel(int32_t* cell, int32_t* cell_b, int32_t* size, int32_t* parent, int32_t* cellpos,
                                 int HW, long long total, StepDesc* steps, int* done, int* next_item,
                                 const int* status, int B, int H, int W, int Hf, int Wf, int r_w, int r_h,
                                 int height_first, int n_steps) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < total) {
        cell[i] = (int32_t)(i % HW);
        cell_b[i] = (int32_t)(i % HW);     // never read before a step writes it; valid all the same
        size[i] = 1;
        parent[i] = -1;
        cellpos[i] = 0;
    }
    // the first counter starts below zero only when a test holds it back (its waits then run out)
    if (i < (long long)n_steps * B) done[i] = i == 0 ? -status[kStatusHoldBack] : 0;
    if (i == 0) {
        int h = H, w = W, n = 0, item = 0, toff = 0;
        while ((h != Hf || w != Wf) && n < n_steps) {
            for (int turn = 0; turn < 2 && n < n_steps; ++turn) {
                const int axis = height_first ? 1 - turn : turn;
                const int len = axis == 0 ? w : h, goal = axis == 0 ? Wf : Hf, r = axis == 0 ? r_w : r_h;
                int m = len - goal < r ? len - goal : r;
                if (m > (len + 1) / 2) m = (len + 1) / 2;
                if (len < 2 || m <= 0) continue;
                const int lines = axis == 0 ? h : w;
                steps[n] = StepDesc{axis, m, h, w, item, toff};
                item += lines * B;
                toff += lines * m;
                ++n;
                if (axis == 0) w -= m; else h -= m;
            }
        }
        // A status word that is already set (an earlier call's failure that nobody has read yet) stops
        // this call before it starts: the work counter begins past the last item, so the chain's CTAs
        // find nothing to claim (and the emit and map kernels look at the word themselves).
        *next_item = status[kStatusWord] != 0 ? item : 0;
    }
}

// MINB: CTAs per SM the register budget is cut for.
template <typename T, int NCHUNK, int MINB, int THREADS>
__global__ void __launch_bounds__(THREADS, MINB) oim_chain_kernel(const ChainArgs a) {
    constexpr int kThreads = THREADS, kWarps = THREADS / 32;
    constexpr int V = Elem<T>::kVec;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ int s_item;
    __shared__ int s_ok;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int D = a.D, B = a.B;
    int step = 0;
    StepDesc st = a.steps[0];
    int step_end = a.n_steps > 1 ? a.steps[1].item_begin : a.total_items;

    for (;;) {
        __syncthreads();                       // the previous item's shared memory is no longer read
        if (tid == 0) s_item = atomicAdd(a.next_item, 1);
        __syncthreads();
        const int item = s_item;
        if (item >= a.total_items) break;
        while (item >= step_end) {             // items only grow: walk the step table forward
            ++step;
            st = a.steps[step];
            step_end = step + 1 < a.n_steps ? a.steps[step + 1].item_begin : a.total_items;
        }
        const int len = st.axis == 0 ? st.w : st.h;
        const int lines = st.axis == 0 ? st.h : st.w;
        const int local = item - st.item_begin;
        const int b = local / lines, line = local - b * lines;

        if (step > 0) {                        // every line of this image's previous step must be finished
            if (tid == 0) {
                const StepDesc prev = a.steps[step - 1];
                const int need = prev.axis == 0 ? prev.h : prev.w;
                s_ok = wait_for_count(a.done + (size_t)(step - 1) * B + b, need, a.status) ? 1 : 0;
            }
            __syncthreads();
            if (!s_ok) break;
        }

        const int ncand = (len + 1) >> 1;
        float* s_dot = reinterpret_cast<float*>(smem_raw);          // <v_j, v_{j+1}>
        float* s_nrm = s_dot + len;                                  // 1 / |v_j| (0 for a zero vector)
        float* s_score = s_nrm + len;                                // best cosine of even cell 2c
        unsigned* s_root = reinterpret_cast<unsigned*>(s_score + ncand);   // root | merged bit
        int* s_dir = reinterpret_cast<int*>(s_root + len);           // best direction of even cell 2c
        int* s_sel = s_dir + ncand;                                  // chosen (pos * 2 + dir), m entries

        const int base = st.axis == 0 ? line * st.w : line;
        const int stride = st.axis == 0 ? 1 : st.w;
        const size_t img = (size_t)b * a.HW;
        const int32_t* cell_in = a.cell[step & 1] + img;
        int32_t* cell_out = a.cell[(step + 1) & 1] + img;
        int32_t* size = a.size + img;
        const T* tokens = reinterpret_cast<const T*>(a.tokens) + img * D;
        float* acc = a.acc + img * D;

        // Every row of the line is asked for at once (one bulk prefetch into L2 per cell, no register
        // held): the similarity pass below walks the cells a few at a time, and without this only its
        // first loads would overlap the memory latency.
        for (int j = tid; j < len; j += kThreads) {
            const unsigned r = (unsigned)__ldcg(cell_in + base + j * stride);
            s_root[j] = r;
            const size_t o = (size_t)(r & ~kMergedBit) * D;
            if (r & kMergedBit) prefetch_l2(acc + o, (unsigned)(D * sizeof(float)));
            else prefetch_l2(tokens + o, (unsigned)(D * sizeof(T)));
        }
        __syncthreads();

        // ---- similarity pass: one warp per cell, norm of v_j and dot with its successor
        for (int j = warp; j < len; j += kWarps) {
            const unsigned r0 = s_root[j];
            const bool has_next = j + 1 < len;
            const unsigned r1 = has_next ? s_root[j + 1] : r0;
            const size_t o0 = (size_t)(r0 & ~kMergedBit) * D, o1 = (size_t)(r1 & ~kMergedBit) * D;
            float nn = 0.f, dd = 0.f;
            pair_stats<T, NCHUNK>(tokens + o0, acc + o0, r0 & kMergedBit, tokens + o1, acc + o1, r1 & kMergedBit,
                                  has_next, lane, D, nn, dd);
            nn = warp_sum(nn);
            dd = warp_sum(dd);
            if (lane == 0) { s_nrm[j] = nn > 0.f ? 1.0f / sqrtf(nn) : 0.f; s_dot[j] = dd; }
        }
        __syncthreads();

        // ---- ranking: warp 0 scores the even cells and takes the m best
        if (warp == 0) {
            for (int c = lane; c < ncand; c += 32) {
                const int j = 2 * c;
                const float ij = s_nrm[j];                       // a zero vector has similarity 0 with everything
                float cl = -FLT_MAX, cr = -FLT_MAX;
                if (j >= 1) {
                    cl = s_dot[j - 1] * (ij * s_nrm[j - 1]);
                    if (!(cl == cl)) cl = -FLT_MAX;
                }
                if (j + 1 < len) {
                    cr = s_dot[j] * (ij * s_nrm[j + 1]);
                    if (!(cr == cr)) cr = -FLT_MAX;
                }
                const bool right = (j < 1) || (j + 1 < len && cr > cl);   // ties stay with the previous cell
                s_dir[c] = right ? 1 : 0;
                s_score[c] = right ? cr : cl;
            }
            __syncwarp();
            for (int k = 0; k < st.m; ++k) {
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
                for (int k = lane; k < st.m; k += 32)
                    a.trace[(size_t)b * a.trace_stride + st.trace_off + (size_t)line * st.m + k] = s_sel[k];
        }
        __syncthreads();

        // ---- close the line up: surviving cells keep their order; receivers get the merged bit
        {
            const int out_w = st.axis == 0 ? st.w - st.m : st.w;
            for (int j = tid; j < len; j += kThreads) {
                int before = 0;
                bool removed = false, receives = false;
                for (int k = 0; k < st.m; ++k) {
                    const int p = s_sel[k] >> 1;   // position of the merged cell
                    removed |= p == j;
                    before += p < j;
                    receives |= p + ((s_sel[k] & 1) ? 1 : -1) == j;
                }
                if (!removed) {
                    const int nj = j - before;
                    const int dst = st.axis == 0 ? line * out_w + nj : nj * out_w + line;
                    cell_out[dst] = (int32_t)(s_root[j] | (receives ? kMergedBit : 0u));
                }
            }
        }

        // ---- merges: the warps are dealt out over (destination cell, slice of D); new sums are written as fp32
        {
            const int m = st.m;
            const int nsl = m < kWarps ? kWarps / m : 1;        // slices of D per merge
            for (int idx = warp; idx < m * nsl; idx += kWarps) {
                const int k = idx % m, sl = idx / m;
                const int pos = s_sel[k] >> 1, dst = pos + ((s_sel[k] & 1) ? 1 : -1);
                bool first = true;          // the lowest rank that targets this destination does the work
                int other = -1;             // a second source of the same destination, if any
                for (int q = 0; q < m; ++q) {
                    if (q == k) continue;
                    const int qpos = s_sel[q] >> 1, qdst = qpos + ((s_sel[q] & 1) ? 1 : -1);
                    if (qdst == dst) { if (q < k) first = false; else other = qpos; }
                }
                if (!first) continue;
                const unsigned rd = s_root[dst], ra = s_root[pos], rb = other >= 0 ? s_root[other] : 0u;
                const size_t od = (size_t)(rd & ~kMergedBit) * D, oa = (size_t)(ra & ~kMergedBit) * D,
                             ob = (size_t)(rb & ~kMergedBit) * D;
                for (int e = (sl * 32 + lane) * V; e < D; e += nsl * 32 * V) {
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
                if (sl == 0 && lane == 0) {
                    const int id = rd & ~kMergedBit, ia = ra & ~kMergedBit;
                    int sz = __ldcg(size + id) + __ldcg(size + ia);
                    a.parent[img + ia] = id;
                    if (other >= 0) {
                        const int ib = rb & ~kMergedBit;
                        sz += __ldcg(size + ib);
                        a.parent[img + ib] = id;
                    }
                    size[id] = sz;
                }
            }
        }

        // ---- publish: every write of this line is ordered before the counter increment
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            atomicAdd(a.done + (size_t)step * B + b, 1);
        }
    }
}

// One warp per final cell: the mean of its sources in the caller's element type,
// its size, and the root -> cell table the map kernel needs.
template <typename T>
__global__ void __launch_bounds__(256) oim_emit_kernel(const void* tokens_v, const float* acc, const int32_t* cell,
                                                       const int32_t* size, int32_t* cellpos, void* out_v,
                                                       int32_t* out_sizes, float* out_log_sizes, int HW, int target,
                                                       int D, long long total_cells, const int* status) {
    constexpr int V = Elem<T>::kVec;
    const long long gw = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (gw >= total_cells) return;
    if (__ldcg(status) != 0) return;       // the chain gave up: its grids are unfinished, nothing is emitted
    const int b = (int)(gw / target), c = (int)(gw % target);
    const size_t img = (size_t)b * HW;
    const int root = (int)((unsigned)cell[img + c] & ~kMergedBit);
    if (root >= HW) return;                // cannot happen after a finished chain; keeps every index in range
    const int s = size[img + root];
    const T* tok = reinterpret_cast<const T*>(tokens_v) + (img + root) * D;
    const float* arow = acc + (img + root) * D;
    T* out = reinterpret_cast<T*>(out_v) + ((size_t)b * target + c) * D;
    if (lane == 0) {
        out_sizes[(size_t)b * target + c] = s;
        cellpos[img + root] = c;
        if (out_log_sizes != nullptr) out_log_sizes[(size_t)b * target + c] = logf((float)s);   // Eq. 2's log s
    }
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
                               long long total, const int* status) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    if (__ldcg(status) != 0) return;
    const size_t img = (size_t)(i / HW) * HW;
    int r = (int)(i % HW);
    for (int hop = 0; hop < HW; ++hop) {   // a chain is shorter than the number of tokens
        const int p = parent[img + r];
        if (p < 0 || p >= HW) break;
        r = p;
    }
    out_map[i] = cellpos[img + r];
}

struct Workspace {
    float* acc;
    int32_t *cell_a, *cell_b, *size, *parent, *cellpos;
    StepDesc* steps;
    int* done;
    int* counters;   // [0] next item, [1] status
    __nv_bfloat16* split;   // bipartite matching only
    float* nrm2;            // bipartite matching only
};

size_t max_steps(int H, int W) { return (size_t)H + W + 2; }

Workspace carve(void* ws, int B, int H, int W, int D, int matching) {
    unsigned char* p = static_cast<unsigned char*>(ws);
    Workspace w;
    const size_t n = (size_t)B * H * W;
    w.acc = reinterpret_cast<float*>(p); p += align_up(n * D * sizeof(float));
    w.cell_a = reinterpret_cast<int32_t*>(p); p += align_up(n * 4);
    w.cell_b = reinterpret_cast<int32_t*>(p); p += align_up(n * 4);
    w.size = reinterpret_cast<int32_t*>(p); p += align_up(n * 4);
    w.parent = reinterpret_cast<int32_t*>(p); p += align_up(n * 4);
    w.cellpos = reinterpret_cast<int32_t*>(p); p += align_up(n * 4);
    w.steps = reinterpret_cast<StepDesc*>(p); p += align_up(max_steps(H, W) * sizeof(StepDesc));
    w.done = reinterpret_cast<int*>(p); p += align_up(max_steps(H, W) * B * sizeof(int));
    w.counters = reinterpret_cast<int*>(p); p += 256;
    w.split = nullptr;
    w.nrm2 = nullptr;
    if (matching == LUVC_OIM_MATCH_BIPARTITE) {
        w.split = reinterpret_cast<__nv_bfloat16*>(p); p += align_up(n * D * 2 * sizeof(__nv_bfloat16));
        w.nrm2 = reinterpret_cast<float*>(p);
    }
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

bool oim_schedule(int H, int W, int Hf, int Wf, int r_w, int r_h, int height_first, OimStep* steps, int cap,
                  int* n_steps) {
    if (Hf < 1 || Wf < 1 || Hf > H || Wf > W || r_w < 1 || r_h < 1) return false;
    int h = H, w = W, n = 0;
    while (h != Hf || w != Wf) {
        bool moved = false;
        for (int turn = 0; turn < 2; ++turn) {
            const int axis = height_first ? 1 - turn : turn;
            const int len = axis == 0 ? w : h, goal = axis == 0 ? Wf : Hf, r = axis == 0 ? r_w : r_h;
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

size_t oim_workspace_bytes(int B, int H, int W, int D, int /*dtype*/, int matching) {
    const size_t n = (size_t)B * H * W;
    size_t bytes = align_up(n * D * sizeof(float)) + 5 * align_up(n * 4) + align_up(max_steps(H, W) * sizeof(StepDesc)) +
                   align_up(max_steps(H, W) * B * sizeof(int)) + 256;
    if (matching == LUVC_OIM_MATCH_BIPARTITE) bytes += align_up(n * D * 2 * sizeof(__nv_bfloat16)) + align_up(n * 4);
    return bytes;
}

template <typename T, int NCHUNK, int MINB, int THREADS = 256>
static cudaError_t launch_chain_b(const ChainArgs& a, int max_len, int r, cudaStream_t stream) {
    static int sms = 0;      // per kernel instantiation
    int blocks_per_sm = 0;
    const size_t smem = (size_t)(3 * max_len + 2 * ((max_len + 1) / 2) + r + 8) * 4;
    if (smem > 48 * 1024)
        cudaFuncSetAttribute(oim_chain_kernel<T, NCHUNK, MINB, THREADS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks_per_sm, oim_chain_kernel<T, NCHUNK, MINB, THREADS>, THREADS, smem);
    if (blocks_per_sm < 1) blocks_per_sm = 1;
    int grid = blocks_per_sm * sms;
    if (grid > a.total_items) grid = a.total_items;
    oim_chain_kernel<T, NCHUNK, MINB, THREADS><<<grid, THREADS, smem, stream>>>(a);
    return cudaGetLastError();
}

// Short lines leave a CTA mostly in its serial phases (ranking, merging, waiting for the image's
// previous step): more resident CTAs overlap them.  Longer lines are dominated by the streaming
// pass: three CTAs of ten warps per SM (64 registers) do best at 72 cells, and beyond about a
// hundred cells a line keeps sixteen warps busy, so two CTAs of 512 threads finish each line sooner
// (a batch of few large images has fewer lines per step than the GPU has CTA slots, so the time per
// line is what counts).  The switch points are measured (36-, 72- and 128-cell lines).
template <typename T, int NCHUNK>
static cudaError_t launch_chain(const ChainArgs& a, int max_len, int r, cudaStream_t stream) {
    if (max_len <= 48) return launch_chain_b<T, NCHUNK, 4>(a, max_len, r, stream);
    if (max_len <= 96) return launch_chain_b<T, NCHUNK, 3, 320>(a, max_len, r, stream);
    return launch_chain_b<T, NCHUNK, 2, 512>(a, max_len, r, stream);
}

template <typename T>
static int oim_run_typed(const OimProblem& p) {
    const int HW = p.H * p.W, target = p.Hf * p.Wf;
    const long long n = (long long)p.B * HW;
    Workspace ws = carve(p.workspace, p.B, p.H, p.W, p.D, p.matching);
    const int cap = (int)max_steps(p.H, p.W);
    OimStep* steps = new OimStep[cap];
    int n_steps = 0;
    if (!oim_schedule(p.H, p.W, p.Hf, p.Wf, p.r_w, p.r_h, p.height_first, steps, cap, &n_steps) || n_steps > cap) {
        delete[] steps;
        return LUVC_ERR_TARGET;
    }
    long long total_items = 0;
    for (int s = 0; s < n_steps; ++s) total_items += (long long)p.B * (steps[s].axis == 0 ? steps[s].h : steps[s].w);
    delete[] steps;
    if (total_items > 0x7fffffffll) return LUVC_ERR_SHAPE;

    phase_begin(LUVC_PHASE_OIM_TOTAL, p.stream);
    long long setup_threads = n > (long long)n_steps * p.B ? n : (long long)n_steps * p.B;
    oim_setup_kernel<<<(unsigned)((setup_threads + 255) / 256), 256, 0, p.stream>>>(
        ws.cell_a, ws.cell_b, ws.size, ws.parent, ws.cellpos, HW, n, ws.steps, ws.done, ws.counters, p.status, p.B, p.H,
        p.W, p.Hf, p.Wf, p.r_w, p.r_h, p.height_first, n_steps);
    count_launch();
    phase_begin(LUVC_PHASE_OIM_STEPS, p.stream);
    if (n_steps > 0) {
        ChainArgs a;
        a.tokens = p.tokens; a.acc = ws.acc; a.cell[0] = ws.cell_a; a.cell[1] = ws.cell_b;
        a.size = ws.size; a.parent = ws.parent; a.trace = p.trace; a.steps = ws.steps; a.done = ws.done;
        a.next_item = ws.counters; a.status = p.status;
        a.B = p.B; a.HW = HW; a.D = p.D; a.n_steps = n_steps; a.total_items = (int)total_items;
        a.trace_stride = HW - target;
        const int chunk = 32 * Elem<T>::kVec;
        const int nchunk = p.D % chunk == 0 ? p.D / chunk : 0;
        const int max_len = p.H > p.W ? p.H : p.W;
        const int r_max = p.r_w > p.r_h ? p.r_w : p.r_h;
        cudaError_t err;
        if (p.matching == LUVC_OIM_MATCH_BIPARTITE) {
            err = oim_bipartite_prepare(a, ws.split, ws.nrm2, p.dtype, p.stream);
            count_launch();
            if (err == cudaSuccess) err = oim_bipartite_launch(a, ws.split, ws.nrm2, p.dtype, max_len, r_max, p.stream);
        } else
        switch (nchunk) {
            case 4: err = launch_chain<T, 4>(a, max_len, r_max, p.stream); break;
            case 5: err = launch_chain<T, 5>(a, max_len, r_max, p.stream); break;
            case 8: err = launch_chain<T, 8>(a, max_len, r_max, p.stream); break;
            default: err = launch_chain<T, 0>(a, max_len, r_max, p.stream); break;
        }
        count_launch();
        if (err != cudaSuccess) return LUVC_ERR_CUDA;
    }
    phase_end(LUVC_PHASE_OIM_STEPS, p.stream);
    const int32_t* final_cell = (n_steps & 1) ? ws.cell_b : ws.cell_a;
    const long long cells = (long long)p.B * target;
    oim_emit_kernel<T><<<(unsigned)((cells * 32 + 255) / 256), 256, 0, p.stream>>>(
        p.tokens, ws.acc, final_cell, ws.size, ws.cellpos, p.out_tokens, p.out_sizes, p.out_log_sizes, HW, target, p.D,
        cells, p.status);
    count_launch();
    oim_map_kernel<<<(unsigned)((n + 255) / 256), 256, 0, p.stream>>>(ws.parent, ws.cellpos, p.out_map, HW, n, p.status);
    count_launch();
    phase_end(LUVC_PHASE_OIM_TOTAL, p.stream);
    return cudaGetLastError() == cudaSuccess ? LUVC_OK : LUVC_ERR_CUDA;
}

// Value enhancement of Eq. 2: one warp per token row, 16 bytes per lane per trip.
template <typename T>
__global__ void __launch_bounds__(256) oim_value_enhance_kernel(const T* __restrict__ v, const int32_t* __restrict__ sizes,
                                                                T* __restrict__ out, long long rows, int D) {
    constexpr int V = 16 / sizeof(T);
    const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    const float bias = logf((float)sizes[row]);
    const T* src = v + row * D;
    T* dst = out + row * D;
    for (int e = lane * V; e < D; e += 32 * V) {
        if constexpr (sizeof(T) == 4) {
            float4 f = *reinterpret_cast<const float4*>(src + e);
            f.x += bias; f.y += bias; f.z += bias; f.w += bias;
            *reinterpret_cast<float4*>(dst + e) = f;
        } else {
            const uint4 u = *reinterpret_cast<const uint4*>(src + e);
            const unsigned w[4] = {u.x, u.y, u.z, u.w};
            unsigned r[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const __nv_bfloat162 pr = __floats2bfloat162_rn(__uint_as_float(w[q] << 16) + bias,
                                                                __uint_as_float(w[q] & 0xffff0000u) + bias);
                r[q] = *reinterpret_cast<const unsigned*>(&pr);
            }
            *reinterpret_cast<uint4*>(dst + e) = make_uint4(r[0], r[1], r[2], r[3]);
        }
    }
}

int oim_value_enhance(const void* values, const int32_t* sizes, long long rows, int D, int dtype, void* out,
                      cudaStream_t stream) {
    const unsigned grid = (unsigned)((rows * 32 + 255) / 256);
    if (dtype == LUVC_F32)
        oim_value_enhance_kernel<float><<<grid, 256, 0, stream>>>(static_cast<const float*>(values), sizes,
                                                                  static_cast<float*>(out), rows, D);
    else
        oim_value_enhance_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(values), sizes,
                                                                          static_cast<__nv_bfloat16*>(out), rows, D);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LUVC_OK : LUVC_ERR_CUDA;
}

int oim_run(const OimProblem& p) {
    return p.dtype == LUVC_F32 ? oim_run_typed<float>(p) : oim_run_typed<__nv_bfloat16>(p);
}

}  // namespace luvc
