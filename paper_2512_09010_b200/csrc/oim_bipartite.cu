// Orthogonal Iterative Merger with full-line bipartite matching (Section 3.2 of the paper: the
// O(n_v^1.5 k) cost it states for OIM is that of one similarity matrix per line).
//
// A line of `len` cells is split into set A (even positions) and set B (odd positions); every
// A cell proposes the most similar B cell of its line and the m best proposals are merged.  The
// similarity matrix S = A B^T (ceil(len/2) x floor(len/2), contraction over D) is a dense
// contraction and runs on the tensor cores:
//
//   * every vector the chain can meet exists in global memory as bf16 hi + lo parts with its
//     squared norm: bf16 input rows are their own hi part (lo = 0), fp32 input rows are split
//     by a preparation kernel, and the merge phase writes the parts and the norm of every sum
//     it forms (next to the fp32 sum itself);
//   * eight loader warps gather the line's rows through the cell grid with cp.async, 16 bytes
//     at a time, straight into K-major operand tiles of 64 channels, several tiles in flight;
//     the lo rows of an operand sit below its hi rows in the same tile;
//   * a ninth warp issues tcgen05.mma (fp32 accumulation in TMEM), per 16 channels A hi x B hi^T and,
//     into the same accumulator, A lo x B hi^T and A hi x B lo^T; a part that is zero for the whole
//     line is left out.  (One instruction on stacked operands, [A hi; A lo] x [B hi; B lo]^T, was
//     slower: its blocks have to be added after the read-back, across TMEM lanes.)
//   * the rows of the product are read back with tcgen05.ld by the two warps of each lane quadrant,
//     scaled to cosines, and each A row keeps its first maximum.
// Loaders and the issuing warp meet only through mbarriers (tile landed / tile consumed).
//
// Ranking, the size-weighted merge and the compaction of the line follow; the data layout, the
// work distribution (one persistent kernel, lines claimed through an atomic counter, bounded
// waits on the image's previous step) and the emit / map kernels are those of the adjacent-pair
// chain.  A line's phases are latency-bound, so several CTAs share an SM.  Every wait has an
// iteration limit and reports through the status word.

#include <cuda_bf16.h>
#include <float.h>

#include "luvc_internal.h"
#include "oim_common.cuh"
#include "sm100_ptx.cuh"

namespace luvc {
namespace {

using namespace ptx;

constexpr int kLoaders = 256;            // threads that gather operand tiles (and do everything else)
constexpr int kThreads = kLoaders + 32;  // plus the warp that issues the MMAs
constexpr int kWarps = kLoaders / 32;
constexpr int kIssueWarp = kWarps;
constexpr int kKC = 64;                  // channels per operand tile
constexpr int kPieces = kKC / 8;         // 16-byte pieces (8 bf16) per row and tile
constexpr int kSlack = 4096;             // the M = 128 operand read may run this far past the last tile
constexpr int kMaxLen = 256;             // 128 A rows (the MMA's M) and 128 B rows
constexpr int kMaxStages = 7;
constexpr int kWaitLimit = 1 << 22;

// Operand tile of R rows (R a multiple of 8): piece p of row r sits at
//   p * lbo(R) + (r / 8) * 128 + (r % 8) * 16,   lbo(R) = R * 16 + 16
// i.e. core matrices of 8 rows x 16 bytes, 8-row groups contiguous (stride 128), K pieces lbo
// apart; the extra 16 bytes spread a warp's stores over all banks.
__host__ __device__ constexpr int tile_lbo(int rows) { return rows * 16 + 16; }

struct LineGeom {
    int na, nb;          // cells in A and B
    int ra, rb;          // rows of one half (hi or lo) of the A and B tiles: na, nb rounded up to 8 and 16
    int lbo_a, lbo_b;    // tiles hold 2 * ra and 2 * rb rows: hi rows, then lo rows
    int off_b;           // byte offset of the B tile inside one stage (the A tile is at 0)
    int stage_bytes;
};

__host__ __device__ inline LineGeom line_geom(int len) {
    LineGeom g;
    g.na = (len + 1) >> 1;
    g.nb = len >> 1;
    g.ra = (g.na + 7) & ~7;
    g.rb = (g.nb + 15) & ~15;
    if (g.rb < 16) g.rb = 16;
    g.lbo_a = tile_lbo(2 * g.ra);
    g.lbo_b = tile_lbo(2 * g.rb);
    g.off_b = kPieces * g.lbo_a;
    g.stage_bytes = g.off_b + kPieces * g.lbo_b;
    return g;
}

// Bounded wait on an mbarrier phase.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, int parity, int* status) {
    for (int it = 0; it < kWaitLimit; ++it) {
        if (mbar_test_wait(bar, parity)) return true;
        __nanosleep(it < 4096 ? 32 : 256);         // a spinning warp would take issue slots from the working ones
    }
    atomicCAS(status, 0, (int)LUVC_ERR_TIMEOUT);
    return false;
}

__device__ __forceinline__ unsigned pack_bf16(float a, float b) {
    const __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<const unsigned*>(&p);
}

// Writes the bf16 hi parts of x[0..V) and the bf16 lo parts (x - hi) to the two planes of a row, at channel e.
template <int V>
__device__ __forceinline__ void store_parts(__nv_bfloat16* hi_row, __nv_bfloat16* lo_row, int e, const float (&x)[V]) {
    unsigned h[V / 2], l[V / 2];
#pragma unroll
    for (int q = 0; q < V / 2; ++q) {
        h[q] = pack_bf16(x[2 * q], x[2 * q + 1]);
        l[q] = pack_bf16(x[2 * q] - bf16lo(h[q]), x[2 * q + 1] - bf16hi(h[q]));
    }
    if constexpr (V == 8) {
        *reinterpret_cast<uint4*>(hi_row + e) = make_uint4(h[0], h[1], h[2], h[3]);
        *reinterpret_cast<uint4*>(lo_row + e) = make_uint4(l[0], l[1], l[2], l[3]);
    } else {
        *reinterpret_cast<uint2*>(hi_row + e) = make_uint2(h[0], h[1]);
        *reinterpret_cast<uint2*>(lo_row + e) = make_uint2(l[0], l[1]);
    }
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// cp.async.wait_group with a run-time count (0 .. 6 groups may stay pending).
__device__ __forceinline__ void cp_async_wait_dyn(int n) {
    switch (n) {
        case 0: cp_async_wait<0>(); break;
        case 1: cp_async_wait<1>(); break;
        case 2: cp_async_wait<2>(); break;
        case 3: cp_async_wait<3>(); break;
        case 4: cp_async_wait<4>(); break;
        case 5: cp_async_wait<5>(); break;
        default: cp_async_wait<6>(); break;
    }
}

// Preparation: squared norm of every input token and, for fp32 input, its bf16 hi + lo parts.
template <typename T>
__global__ void __launch_bounds__(256) oim_bipartite_prepare_kernel(const T* __restrict__ tokens, __nv_bfloat16* split,
                                                                    float* nrm2, long long rows, int D) {
    constexpr int V = Elem<T>::kVec;
    const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    const T* src = tokens + row * D;
    float nn = 0.f;
    for (int e = lane * V; e < D; e += 32 * V) {
        float x[V];
        load_vec<T>(src, nullptr, false, e, x);
#pragma unroll
        for (int q = 0; q < V; ++q) nn = fmaf(x[q], x[q], nn);
        if constexpr (sizeof(T) == 4) store_parts<V>(split + row * 2 * D, split + row * 2 * D + D, e, x);
    }
    nn = warp_sum(nn);
    if (lane == 0) nrm2[row] = nn;
}

struct BipartiteLaunch {
    int n_stages;       // operand stages in shared memory (1 .. kMaxStages)
    int ahead;          // tiles requested ahead of the one whose arrival is awaited (0 .. n_stages - 1)
    int stage_stride;   // bytes between stages (the geometry of the longest line)
    int tmem_cols;      // power of two >= 32 covering the widest similarity matrix
    int max_len, r;
    __nv_bfloat16* split;   // [B][HW][2][D] bf16 hi and lo parts of fp32 rows
    float* nrm2;            // [B][HW] squared norm by root
};

template <typename T>
__global__ void __launch_bounds__(kThreads, 3) oim_bipartite_kernel(const ChainArgs a, const BipartiteLaunch cfg) {
    constexpr int V = Elem<T>::kVec;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    // [0 .. 6] tile landed (one arrival per loader warp), [7 .. 13] tile consumed by the MMAs,
    // [14] product complete
    __shared__ __align__(8) unsigned long long s_bar[2 * kMaxStages + 1];
    __shared__ uint32_t s_tmem;
    __shared__ int s_item, s_ok, s_fail;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int D = a.D, B = a.B;

    // shared memory: operand stages, slack for the M = 128 over-read, then the per-line arrays
    const uint32_t stages_base = smem_u32(smem_raw);
    unsigned char* tail = smem_raw + (size_t)cfg.n_stages * cfg.stage_stride + kSlack;
    const __nv_bfloat16** s_hi = reinterpret_cast<const __nv_bfloat16**>(tail);   // [len] hi part of tile row
    // [len] where the row's first piece goes inside a stage (| 1: the row has a lo part, behind its hi part;
    // | 2: A row) and the byte distance between its pieces
    uint2* s_where = reinterpret_cast<uint2*>(s_hi + cfg.max_len);
    float* s_rn = reinterpret_cast<float*>(s_where + cfg.max_len);                   // [len] 1 / |v| by tile row (A rows, then B rows)
    unsigned* s_root = reinterpret_cast<unsigned*>(s_rn + cfg.max_len);           // [len] root | merged bit by position
    float* s_score = reinterpret_cast<float*>(s_root + cfg.max_len);              // [na] best cosine of A cell i
    int* s_dst = reinterpret_cast<int*>(s_score + (cfg.max_len + 1) / 2);         // [na] position of its best B cell
    int* s_sel = s_dst + (cfg.max_len + 1) / 2;                                   // [m] (A position << 16) | B position
    float* s_part = reinterpret_cast<float*>(s_sel + cfg.r + 8);                  // partial squared norms of the new sums
    float* s_score2 = s_part + cfg.r + 8 + kWarps;                                // [na] candidate of the second warp of a quadrant
    int* s_dst2 = reinterpret_cast<int*>(s_score2 + (cfg.max_len + 1) / 2);

    const uint32_t bar0 = smem_u32(&s_bar[0]);
    const uint32_t bar_acc = bar0 + 8 * (2 * kMaxStages);
    if (tid == 0) {
        for (int i = 0; i < kMaxStages; ++i) {
            mbar_init(bar0 + 8 * i, kWarps);
            mbar_init(bar0 + 8 * (kMaxStages + i), 1);
        }
        mbar_init(bar_acc, 1);
        mbar_fence_init();
        s_fail = 0;
    }
    if (warp == 0) tmem_alloc(smem_u32(&s_tmem), cfg.tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;

    int step = 0;
    StepDesc st = a.steps[0];
    int step_end = a.n_steps > 1 ? a.steps[1].item_begin : a.total_items;
    unsigned fills = 0;        // operand tiles consumed so far by this CTA (all items)
    unsigned items_done = 0;   // products completed so far by this CTA
    bool mma_pending = false;  // an item was abandoned with MMAs possibly in flight
    const unsigned S = (unsigned)cfg.n_stages;

    for (;;) {
        __syncthreads();                       // the previous item's shared memory is no longer read
        if (tid == 0) s_item = atomicAdd(a.next_item, 1);
        __syncthreads();
        const int item = s_item;
        if (item >= a.total_items) break;
        while (item >= step_end) {
            ++step;
            st = a.steps[step];
            step_end = step + 1 < a.n_steps ? a.steps[step + 1].item_begin : a.total_items;
        }
        const int len = st.axis == 0 ? st.w : st.h;
        const int lines = st.axis == 0 ? st.h : st.w;
        const int local = item - st.item_begin;
        const int b = local / lines, line = local - b * lines;
        const LineGeom g = line_geom(len);

        if (step > 0) {                        // every line of this image's previous step must be finished
            if (tid == 0) {
                const StepDesc prev = a.steps[step - 1];
                const int need = prev.axis == 0 ? prev.h : prev.w;
                s_ok = wait_for_count(a.done + (size_t)(step - 1) * B + b, need, a.status) ? 1 : 0;
            }
            __syncthreads();
            if (!s_ok) break;
        }

        const int base = st.axis == 0 ? line * st.w : line;
        const int stride = st.axis == 0 ? 1 : st.w;
        const size_t img = (size_t)b * a.HW;
        const int32_t* cell_in = a.cell[step & 1] + img;
        int32_t* cell_out = a.cell[(step + 1) & 1] + img;
        int32_t* size = a.size + img;
        const T* tokens = reinterpret_cast<const T*>(a.tokens) + img * D;
        float* acc = a.acc + img * D;
        __nv_bfloat16* split = cfg.split + img * 2 * D;
        float* nrm2 = cfg.nrm2 + img;

        // ---- the line's cells: where the parts of each row live, and its norm.  A lo part exists
        // for fp32 input and for every cell that holds a sum.
        bool m_a = false, m_b = false;
        for (int j = tid; j < len; j += kThreads) {
            const unsigned r = (unsigned)__ldcg(cell_in + base + j * stride);
            s_root[j] = r;
            const int id = (int)(r & ~kMergedBit);
            const bool parts = sizeof(T) == 4 || (r & kMergedBit) != 0;
            const bool is_a = !(j & 1);
            const int rr = j >> 1, row = is_a ? rr : g.na + rr;
            s_hi[row] = parts ? split + (size_t)id * 2 * D : reinterpret_cast<const __nv_bfloat16*>(tokens + (size_t)id * D);
            s_where[row] = make_uint2((uint32_t)((is_a ? 0 : g.off_b) + (rr >> 3) * 128 + (rr & 7) * 16) | (parts ? 1u : 0u) |
                                          (is_a ? 2u : 0u),
                                      (uint32_t)(is_a ? g.lbo_a : g.lbo_b));
            const float nn = __ldcg(nrm2 + id);
            s_rn[row] = nn > 0.f ? 1.0f / sqrtf(nn) : 0.f;          // a zero vector has similarity 0 with everything
            if (parts) { if (is_a) m_a = true; else m_b = true; }
        }
        const bool lo_a = __syncthreads_or(m_a) != 0;
        const bool lo_b = __syncthreads_or(m_b) != 0;

        // ---- the similarity matrix A B^T (hi and lo parts) over tiles of 64 channels
        const int nkc = (D + kKC - 1) / kKC;
        const unsigned fill0 = fills;

        if (warp < kWarps) {
            // loaders: tile c of this line goes to stage (fill0 + c) % S once the MMAs that last read it are done
            const int total_q = len * kPieces;
            const uint32_t lo_off_a = lo_a ? (uint32_t)(g.ra >> 3) * 128 : 0u;   // the lo row sits ra (rb) rows below the hi row;
            const uint32_t lo_off_b = lo_b ? (uint32_t)(g.rb >> 3) * 128 : 0u;   // 0: that operand has no lo half in this line
            int issued = 0;
            for (int kc = 0; kc < nkc; ++kc) {
                while (issued < nkc && issued <= kc + cfg.ahead) {
                    const unsigned f = fill0 + (unsigned)issued;
                    const unsigned stage = f % S, use = f / S;
                    if (use >= 1) {                                // lane 0 watches the barrier for its warp
                        if (lane == 0 && !mbar_wait(bar0 + 8 * (kMaxStages + stage), (int)((use - 1) & 1), a.status)) s_fail = 1;
                        __syncwarp();
                    }
                    const uint32_t sb = stages_base + stage * (uint32_t)cfg.stage_stride;
                    for (int q = tid; q < total_q; q += kLoaders) {
                        const int row = q >> 3, piece = q & 7;
                        const bool valid = issued * kKC + piece * 8 < D;
                        const uint2 w = s_where[row];
                        const __nv_bfloat16* hi = s_hi[row];
                        const __nv_bfloat16* src = hi + (issued * kKC + piece * 8);
                        const uint32_t dst = sb + (w.x & ~15u) + piece * w.y;
                        cp_async16(dst, valid ? src : hi, valid);
                        const uint32_t lo_off = (w.x & 2u) ? lo_off_a : lo_off_b;
                        if (lo_off) {
                            const bool have = valid && (w.x & 1u);
                            cp_async16(dst + lo_off, have ? src + D : hi, have);
                        }
                    }
                    cp_async_commit();
                    ++issued;
                }
                cp_async_wait_dyn(issued - kc - 1);        // this thread's share of tile kc has landed
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar0 + 8 * ((fill0 + (unsigned)kc) % S));
            }
        } else {
            // issuing warp: lane 0 works, the others wait at the warp barriers (a lane that spun on the
            // product barrier beside the issuing lane would take its issue slots)
            // hi x hi, then lo x hi and hi x lo where the line has lo parts: all into the same columns
            const uint32_t idesc = make_idesc_bf16(128, g.rb, false, false);
            for (int kc = 0; kc < nkc; ++kc) {
                const unsigned f = fill0 + (unsigned)kc;
                const unsigned stage = f % S, use = f / S;
                if (lane == 0) {
                    if (!mbar_wait(bar0 + 8 * stage, (int)(use & 1), a.status)) s_fail = 1;
                    tc_fence_after();
                    const uint32_t sb = stages_base + stage * (uint32_t)cfg.stage_stride;
                    if (!s_fail) {
#pragma unroll
                        for (int ks = 0; ks < kKC / 16; ++ks) {
                            const uint64_t a_hi = make_desc(sb + ks * 2 * g.lbo_a, g.lbo_a, 128);
                            const uint64_t b_hi = make_desc(sb + g.off_b + ks * 2 * g.lbo_b, g.lbo_b, 128);
                            umma_bf16(tmem, a_hi, b_hi, idesc, (kc | ks) ? 1u : 0u);
                            if (lo_a)
                                umma_bf16(tmem, make_desc(sb + ks * 2 * g.lbo_a + (g.ra >> 3) * 128, g.lbo_a, 128), b_hi, idesc, 1u);
                            if (lo_b)
                                umma_bf16(tmem, a_hi, make_desc(sb + g.off_b + ks * 2 * g.lbo_b + (g.rb >> 3) * 128, g.lbo_b, 128),
                                          idesc, 1u);
                        }
                    }
                    umma_commit(bar0 + 8 * (kMaxStages + stage));
                }
                __syncwarp();
            }
            if (lane == 0) umma_commit(bar_acc);
            __syncwarp();
        }
        fills += (unsigned)nkc;
        if (lane == 0 && !mbar_wait(bar_acc, (int)(items_done & 1), a.status)) s_fail = 1;   // one watcher per warp
        __syncthreads();
        if (s_fail) { mma_pending = true; break; }
        ++items_done;
        tc_fence_after();

        // Two warps share each quadrant of TMEM lanes (warp & 3) and take alternate 16-column chunks (warp >> 2).
        const int quad = warp & 3, half = (warp >> 2) & 1;

        // ---- proposals: A row i (TMEM lane i) keeps the first maximum of its cosines
        if (warp < kWarps && quad * 32 < g.na) {
            const int i = quad * 32 + lane;
            const float rn_i = i < g.na ? s_rn[i] : 0.f;
            float best = -INFINITY;
            int best_j = 0;
            for (int c0 = half * 16; c0 < g.rb; c0 += 32) {
                uint32_t v[16];
                tmem_ld16(tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)c0, v);
                tmem_ld_wait_for(v);
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) {
                    const int j = c0 + jj;
                    if (j < g.nb) {
                        float c = __uint_as_float(v[jj]) * (rn_i * s_rn[g.na + j]);
                        if (!(c == c)) c = -FLT_MAX;
                        if (c > best) { best = c; best_j = j; }
                    }
                }
            }
            if (i < g.na) {                     // this warp's candidate; warp 0 joins the two halves below
                (half ? s_score2 : s_score)[i] = best;
                (half ? s_dst2 : s_dst)[i] = 2 * best_j + 1;
            }
        }
        tc_fence_before();
        __syncthreads();

        // ---- ranking: warp 0 takes the m best proposals (ties: the lowest A position)
        if (warp == 0) {
            for (int c = lane; c < g.na; c += 32) {      // first maximum over both halves: the larger cosine, then the lower position
                const float s2 = s_score2[c];
                const int d2 = s_dst2[c];
                if (s2 > s_score[c] || (s2 == s_score[c] && d2 < s_dst[c])) { s_score[c] = s2; s_dst[c] = d2; }
            }
            __syncwarp();
            for (int k = 0; k < st.m; ++k) {
                float best = -INFINITY;
                int best_c = 0x7fffffff;
                for (int c = lane; c < g.na; c += 32) {
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
                    if (best_c >= g.na) best_c = 0;              // cannot happen: m <= na and every score is finite
                    s_sel[k] = ((2 * best_c) << 16) | s_dst[best_c];
                    s_score[best_c] = -INFINITY;                 // taken
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
                    const int p = s_sel[k] >> 16, d = s_sel[k] & 0xffff;
                    removed |= p == j;
                    before += p < j;
                    receives |= d == j;
                }
                if (!removed) {
                    const int nj = j - before;
                    const int dst = st.axis == 0 ? line * out_w + nj : nj * out_w + line;
                    cell_out[dst] = (int32_t)(s_root[j] | (receives ? kMergedBit : 0u));
                }
            }
        }

        // ---- merges: the loader warps are dealt out over (destination cell, slice of D).  The lowest
        // rank that targets a destination adds every source of that destination, in rank order, and
        // writes the fp32 sum, its bf16 parts and its share of the squared norm.
        const int m = st.m;
        const int nsl = m < kWarps ? kWarps / m : 1;
        for (int idx = warp; idx < m * nsl && warp < kWarps; idx += kWarps) {
            const int k = idx % m, sl = idx / m;
            const int dst = s_sel[k] & 0xffff;
            bool first = true;
            for (int q = 0; q < k; ++q) first &= (s_sel[q] & 0xffff) != dst;
            if (!first) continue;
            const unsigned rd = s_root[dst];
            const int id = (int)(rd & ~kMergedBit);
            const size_t od = (size_t)id * D;
            __nv_bfloat16* hi_row = split + (size_t)id * 2 * D;
            float nn = 0.f;
            for (int e = (sl * 32 + lane) * V; e < D; e += nsl * 32 * V) {
                float x[V], y[V];
                load_vec<T>(tokens + od, acc + od, rd & kMergedBit, e, x);
                for (int q = k; q < m; ++q) {
                    if ((s_sel[q] & 0xffff) != dst) continue;
                    const unsigned ra = s_root[s_sel[q] >> 16];
                    const size_t oa = (size_t)(ra & ~kMergedBit) * D;
                    load_vec<T>(tokens + oa, acc + oa, ra & kMergedBit, e, y);
#pragma unroll
                    for (int i = 0; i < V; ++i) x[i] += y[i];
                }
#pragma unroll
                for (int i = 0; i < V; i += 4)
                    *reinterpret_cast<float4*>(acc + od + e + i) = make_float4(x[i], x[i + 1], x[i + 2], x[i + 3]);
                store_parts<V>(hi_row, hi_row + D, e, x);
#pragma unroll
                for (int i = 0; i < V; ++i) nn = fmaf(x[i], x[i], nn);
            }
            nn = warp_sum(nn);
            if (lane == 0) {
                s_part[k * nsl + sl] = nn;
                if (sl == 0) {
                    int sz = __ldcg(size + id);
                    for (int q = k; q < m; ++q) {
                        if ((s_sel[q] & 0xffff) != dst) continue;
                        const int ia = s_root[s_sel[q] >> 16] & ~kMergedBit;
                        sz += __ldcg(size + ia);
                        a.parent[img + ia] = id;
                    }
                    size[id] = sz;
                }
            }
        }
        __syncthreads();
        for (int k = tid; k < m; k += kThreads) {          // norms of the new sums, slices added in order
            const int dst = s_sel[k] & 0xffff;
            bool first = true;
            for (int q = 0; q < k; ++q) first &= (s_sel[q] & 0xffff) != dst;
            if (!first) continue;
            float nn = 0.f;
            for (int sl = 0; sl < nsl; ++sl) nn += s_part[k * nsl + sl];
            nrm2[s_root[dst] & ~kMergedBit] = nn;
        }

        // ---- publish: every write of this line is ordered before the counter increment
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            atomicAdd(a.done + (size_t)step * B + b, 1);
        }
    }

    // ---- exit: no copy and no MMA may be in flight when the CTA ends and its accumulator columns are returned
    cp_async_wait<0>();
    if (mma_pending && warp == kIssueWarp && lane == 0) {
        umma_commit(bar_acc);
        mbar_wait(bar_acc, (int)(items_done & 1), a.status);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, cfg.tmem_cols);
}

size_t tail_bytes(int max_len, int r) {
    return (size_t)max_len * (8 + 8 + 4 + 4) + (size_t)((max_len + 1) / 2) * 8 + (size_t)(r + 8) * 4 +
           (size_t)(r + 8 + kWarps) * 4 + (size_t)((max_len + 1) / 2) * 8;
}

template <typename T>
cudaError_t launch_typed(const ChainArgs& a, __nv_bfloat16* split, float* nrm2, int max_len, int r, cudaStream_t stream) {
    static int sms = 0, smem_cap = 0, regs_per_cta = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&smem_cap, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
        cudaFuncAttributes fa;
        if (cudaFuncGetAttributes(&fa, oim_bipartite_kernel<T>) != cudaSuccess) return cudaGetLastError();
        regs_per_cta = (kThreads / 32) * ((fa.numRegs * 32 + 255) / 256 * 256);   // registers are granted per warp, in units of 256
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    BipartiteLaunch cfg;
    cfg.max_len = max_len;
    cfg.r = r;
    cfg.split = split;
    cfg.nrm2 = nrm2;
    cfg.stage_stride = (line_geom(max_len).stage_bytes + 127) & ~127;
    int cols = 32;
    while (cols < line_geom(max_len).rb) cols <<= 1;
    cfg.tmem_cols = cols;
    const size_t fixed = kSlack + tail_bytes(max_len, r) + 128;
    // CTAs per SM: the occupancy query of the runtime answers 1 for a kernel that allocates tensor
    // memory, although such CTAs do share an SM; so the limits are counted here: registers, the
    // 512 TMEM columns of an SM, and shared memory with at least three operand stages per CTA.
    const size_t per_sm = (size_t)smem_cap + 1024;
    int ctas = 65536 / regs_per_cta;
    if (ctas > 512 / cols) ctas = 512 / cols;
    if (ctas > 3) ctas = 3;
    if (ctas < 1) ctas = 1;
    int stages = 0;
    for (; ctas >= 1; --ctas) {
        const size_t budget = per_sm / ctas - 1024 /* reserved per CTA */ - 1024 /* static shared variables */;
        stages = budget > fixed ? (int)((budget - fixed) / (size_t)cfg.stage_stride) : 0;
        if (stages >= 3 || ctas == 1) break;
    }
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 1) return cudaErrorInvalidConfiguration;
    const int ahead = stages >= 3 ? stages - 2 : stages - 1;     // from three stages on, a refill never waits for the MMAs just issued
    cfg.n_stages = stages;
    cfg.ahead = ahead;
    const size_t smem = (size_t)stages * cfg.stage_stride + fixed;
    cudaError_t err = cudaFuncSetAttribute(oim_bipartite_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    cudaFuncSetAttribute(oim_bipartite_kernel<T>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    int grid = ctas * sms;
    if (grid > a.total_items) grid = a.total_items;
    oim_bipartite_kernel<T><<<grid, kThreads, smem, stream>>>(a, cfg);
    return cudaGetLastError();
}

}  // namespace

cudaError_t oim_bipartite_prepare(const ChainArgs& a, __nv_bfloat16* split, float* nrm2, int dtype, cudaStream_t stream) {
    const long long rows = (long long)a.B * a.HW;
    const unsigned grid = (unsigned)((rows * 32 + 255) / 256);
    if (dtype == LUVC_F32)
        oim_bipartite_prepare_kernel<float><<<grid, 256, 0, stream>>>(static_cast<const float*>(a.tokens), split, nrm2,
                                                                      rows, a.D);
    else
        oim_bipartite_prepare_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(
            static_cast<const __nv_bfloat16*>(a.tokens), split, nrm2, rows, a.D);
    return cudaGetLastError();
}

cudaError_t oim_bipartite_launch(const ChainArgs& a, __nv_bfloat16* split, float* nrm2, int dtype, int max_len, int r,
                                 cudaStream_t stream) {
    if (max_len > kMaxLen) return cudaErrorInvalidValue;
    return dtype == LUVC_F32 ? launch_typed<float>(a, split, nrm2, max_len, r, stream)
                             : launch_typed<__nv_bfloat16>(a, split, nrm2, max_len, r, stream);
}

}  // namespace luvc
