// Orthogonal Iterative Merger with full-line bipartite matching (Section 3.2 of the paper: the
// O(n_v^1.5 k) cost it states for OIM is that of one similarity matrix per line).
//
// A line of `len` cells is split into set A (even positions) and set B (odd positions); every
// A cell proposes the most similar B cell of its line and the m best proposals are merged.  The
// similarity matrix S = A B^T (ceil(len/2) x floor(len/2), contraction over D) is a dense
// contraction and runs on the tensor cores:
//
//   * the line's vectors are gathered through the cell grid (bf16 input rows, or fp32 sums of
//     merged cells), split into bf16 hi + lo parts and written to shared memory as K-major
//     operand tiles, 128 channels at a time, while each thread also accumulates the squared
//     norms of the rows it handles;
//   * one thread issues tcgen05.mma for hi*hi, lo*hi and hi*lo (fp32 accumulation in TMEM;
//     a part that is zero for the whole line is skipped);
//   * the rows of S are read back with tcgen05.ld, scaled to cosines, and each A row keeps its
//     first maximum.
//
// Ranking, the size-weighted merge and the compaction of the line follow; the data layout, the
// work distribution (one persistent kernel, lines claimed through an atomic counter, bounded
// waits on the image's previous step) and the emit / map kernels are those of the adjacent-pair
// chain.  Every wait has an iteration limit and reports through the status word.

#include <cuda_bf16.h>
#include <float.h>

#include "luvc_internal.h"
#include "oim_common.cuh"
#include "sm100_ptx.cuh"

namespace luvc {
namespace {

using namespace ptx;

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kKC = 128;                 // channels per operand tile
constexpr int kPieces = kKC / 8;         // 16-byte pieces (8 bf16) per row and tile
constexpr int kSlack = 2048;             // the M = 128 operand read may run this far past the last tile
constexpr int kMaxLen = 256;             // 128 A rows (the MMA's M) and 128 B rows
constexpr int kWaitLimit = 1 << 22;

// Operand tile of R rows (R a multiple of 8): piece p of row r sits at
//   p * lbo(R) + (r / 8) * 128 + (r % 8) * 16,   lbo(R) = R * 16 + 16
// i.e. core matrices of 8 rows x 16 bytes, 8-row groups contiguous (stride 128), K pieces lbo
// apart; the extra 16 bytes spread a warp's stores over all banks.
__host__ __device__ constexpr int tile_lbo(int rows) { return rows * 16 + 16; }

struct LineGeom {
    int na, nb;          // cells in A and B
    int ra, rb;          // rows of the A and B tiles (na, nb rounded up to 8 and 16)
    int lbo_a, lbo_b;
    int off_alo, off_bhi, off_blo;   // byte offsets of the planes inside one stage (A hi at 0)
    int stage_bytes;
};

__host__ __device__ inline LineGeom line_geom(int len) {
    LineGeom g;
    g.na = (len + 1) >> 1;
    g.nb = len >> 1;
    g.ra = (g.na + 7) & ~7;
    g.rb = (g.nb + 15) & ~15;
    if (g.rb < 16) g.rb = 16;
    g.lbo_a = tile_lbo(g.ra);
    g.lbo_b = tile_lbo(g.rb);
    g.off_alo = kPieces * g.lbo_a;
    g.off_bhi = 2 * kPieces * g.lbo_a;
    g.off_blo = g.off_bhi + kPieces * g.lbo_b;
    g.stage_bytes = g.off_blo + kPieces * g.lbo_b;
    return g;
}

// Bounded wait on an mbarrier phase.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, int parity, int* status) {
    for (int it = 0; it < kWaitLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it > 1024) __nanosleep(64);
    }
    atomicCAS(status, 0, (int)LUVC_ERR_TIMEOUT);
    return false;
}

__device__ __forceinline__ unsigned pack_bf16(float a, float b) {
    const __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<const unsigned*>(&p);
}

// x[0..7] -> bf16 hi parts and bf16 lo parts (x - hi), packed as 16 bytes each.
__device__ __forceinline__ void split8(const float (&x)[8], uint4& hi, uint4& lo) {
    unsigned h[4], l[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        h[q] = pack_bf16(x[2 * q], x[2 * q + 1]);
        l[q] = pack_bf16(x[2 * q] - bf16lo(h[q]), x[2 * q + 1] - bf16hi(h[q]));
    }
    hi = make_uint4(h[0], h[1], h[2], h[3]);
    lo = make_uint4(l[0], l[1], l[2], l[3]);
}

__device__ __forceinline__ void st_shared16(uint32_t addr, const uint4& v) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// Eight consecutive channels of a cell, starting at channel e, as fp32 (zeros past D).
template <typename T>
__device__ __forceinline__ void load_piece(const T* __restrict__ tok_row, const float* acc_row, bool merged, int e, int D,
                                           float (&x)[8]) {
    if (e >= D) {
#pragma unroll
        for (int q = 0; q < 8; ++q) x[q] = 0.f;
        return;
    }
    if (merged || sizeof(T) == 4) {
        const float* src = merged ? acc_row : reinterpret_cast<const float*>(tok_row);
        float4 f0, f1 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (merged) {
            f0 = __ldcg(reinterpret_cast<const float4*>(src + e));
            if (e + 4 < D) f1 = __ldcg(reinterpret_cast<const float4*>(src + e + 4));
        } else {
            f0 = __ldg(reinterpret_cast<const float4*>(src + e));
            if (e + 4 < D) f1 = __ldg(reinterpret_cast<const float4*>(src + e + 4));
        }
        x[0] = f0.x; x[1] = f0.y; x[2] = f0.z; x[3] = f0.w;
        x[4] = f1.x; x[5] = f1.y; x[6] = f1.z; x[7] = f1.w;
    } else {
        const uint4 u = __ldg(reinterpret_cast<const uint4*>(tok_row + e));
        x[0] = bf16lo(u.x); x[1] = bf16hi(u.x); x[2] = bf16lo(u.y); x[3] = bf16hi(u.y);
        x[4] = bf16lo(u.z); x[5] = bf16hi(u.z); x[6] = bf16lo(u.w); x[7] = bf16hi(u.w);
    }
}

struct BipartiteLaunch {
    int n_stages;       // operand stages in shared memory
    int stage_stride;   // bytes between stages (the geometry of the longest line)
    int tmem_cols;      // power of two >= 32 covering the widest similarity matrix
    int max_len, r;
};

template <typename T>
__global__ void __launch_bounds__(kThreads) oim_bipartite_kernel(const ChainArgs a, const BipartiteLaunch cfg) {
    constexpr int V = Elem<T>::kVec;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long s_bar[9];   // [0..7] stage consumed, [8] similarity matrix complete
    __shared__ uint32_t s_tmem;
    __shared__ int s_item, s_ok, s_fail;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int D = a.D, B = a.B;

    // shared memory: operand stages, slack for the M = 128 over-read, then the per-line arrays
    const uint32_t stages_base = smem_u32(smem_raw);
    unsigned char* tail = smem_raw + (size_t)cfg.n_stages * cfg.stage_stride + kSlack;
    float* s_nn = reinterpret_cast<float*>(tail);                         // [len][16] partial squared norms
    float* s_rn = s_nn + (size_t)cfg.max_len * kPieces;                   // [len] 1 / |v| by tile row (A rows, then B rows)
    unsigned* s_root = reinterpret_cast<unsigned*>(s_rn + cfg.max_len);   // [len] root | merged bit by position
    float* s_score = reinterpret_cast<float*>(s_root + cfg.max_len);      // [na] best cosine of A cell i
    int* s_dst = reinterpret_cast<int*>(s_score + (cfg.max_len + 1) / 2); // [na] position of its best B cell
    int* s_sel = s_dst + (cfg.max_len + 1) / 2;                           // [m] (A position << 16) | B position

    const uint32_t bar0 = smem_u32(&s_bar[0]);
    const uint32_t bar_acc = bar0 + 8 * 8;
    if (tid == 0) {
        for (int i = 0; i < 9; ++i) mbar_init(bar0 + 8 * i, 1);
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
    unsigned fills = 0;        // operand tiles written so far by this CTA (all items)
    unsigned items_done = 0;   // similarity matrices completed so far by this CTA
    bool mma_pending = false;  // an item was abandoned with MMAs possibly in flight

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

        // ---- the line's cells; a lo part is needed only where some cell holds an fp32 sum
        bool m_a = sizeof(T) == 4, m_b = sizeof(T) == 4;
        for (int j = tid; j < len; j += kThreads) {
            const unsigned r = (unsigned)__ldcg(cell_in + base + j * stride);
            s_root[j] = r;
            if (r & kMergedBit) { if (j & 1) m_b = true; else m_a = true; }
        }
        const bool lo_a = __syncthreads_or(m_a) != 0;
        const bool lo_b = __syncthreads_or(m_b) != 0;

        // ---- similarity matrix: operand tiles of 128 channels, MMAs issued behind them
        const int nkc = (D + kKC - 1) / kKC;
        const int total_q = len * kPieces;
        const uint32_t idesc = make_idesc_bf16(128, g.rb, false, false);
        bool alive = true;
        for (int kc = 0; kc < nkc; ++kc) {
            const int stage = (int)(fills % (unsigned)cfg.n_stages);
            const unsigned use = fills / (unsigned)cfg.n_stages;
            if (use >= 1 && !mbar_wait(bar0 + 8 * stage, (int)((use - 1) & 1), a.status)) s_fail = 1;
            const uint32_t sb = stages_base + (uint32_t)stage * (uint32_t)cfg.stage_stride;
            for (int q0 = tid; q0 < total_q; q0 += 4 * kThreads) {
                float x[4][8];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int q = q0 + u * kThreads;
                    if (q < total_q) {
                        const int row = q >> 4, piece = q & 15;
                        const int pos = row < g.na ? 2 * row : 2 * (row - g.na) + 1;
                        const unsigned r = s_root[pos];
                        const size_t o = (size_t)(r & ~kMergedBit) * D;
                        load_piece<T>(tokens + o, acc + o, (r & kMergedBit) != 0, kc * kKC + piece * 8, D, x[u]);
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int q = q0 + u * kThreads;
                    if (q < total_q) {
                        const int row = q >> 4, piece = q & 15;
                        float nn = kc == 0 ? 0.f : s_nn[q];
#pragma unroll
                        for (int e = 0; e < 8; ++e) nn = fmaf(x[u][e], x[u][e], nn);
                        s_nn[q] = nn;
                        uint4 hi, lo;
                        split8(x[u], hi, lo);
                        const bool is_a = row < g.na;
                        const int rr = is_a ? row : row - g.na;
                        const uint32_t addr = sb + (is_a ? 0 : g.off_bhi) + piece * (is_a ? g.lbo_a : g.lbo_b) +
                                              (rr >> 3) * 128 + (rr & 7) * 16;
                        st_shared16(addr, hi);
                        if (is_a ? lo_a : lo_b) st_shared16(addr + (is_a ? g.off_alo : g.off_blo - g.off_bhi), lo);
                    }
                }
            }
            fence_proxy_async();
            __syncthreads();
            if (s_fail) { alive = false; break; }
            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < kKC / 16; ++ks) {
                    const uint64_t a_hi = make_desc(sb + ks * 2 * g.lbo_a, g.lbo_a, 128);
                    const uint64_t b_hi = make_desc(sb + g.off_bhi + ks * 2 * g.lbo_b, g.lbo_b, 128);
                    umma_bf16(tmem, a_hi, b_hi, idesc, (kc | ks) ? 1u : 0u);
                    if (lo_a) umma_bf16(tmem, make_desc(sb + g.off_alo + ks * 2 * g.lbo_a, g.lbo_a, 128), b_hi, idesc, 1u);
                    if (lo_b) umma_bf16(tmem, a_hi, make_desc(sb + g.off_blo + ks * 2 * g.lbo_b, g.lbo_b, 128), idesc, 1u);
                }
                umma_commit(bar0 + 8 * stage);
            }
            ++fills;
        }
        if (!alive) { mma_pending = true; break; }
        if (tid == 0) umma_commit(bar_acc);

        // ---- norms (fixed summation order), while the last MMAs finish
        for (int j = tid; j < len; j += kThreads) {
            float nn = 0.f;
#pragma unroll
            for (int p = 0; p < kPieces; ++p) nn += s_nn[j * kPieces + p];
            s_rn[j] = nn > 0.f ? 1.0f / sqrtf(nn) : 0.f;           // a zero vector has similarity 0 with everything
        }
        if (!mbar_wait(bar_acc, (int)(items_done & 1), a.status)) s_fail = 1;
        __syncthreads();
        if (s_fail) { mma_pending = true; break; }
        ++items_done;
        tc_fence_after();

        // ---- proposals: A row i (TMEM lane i) keeps the first maximum of its cosines
        if (warp < 4 && warp * 32 < g.na) {
            const int i = warp * 32 + lane;
            const float rn_i = i < g.na ? s_rn[i] : 0.f;
            float best = -INFINITY;
            int best_j = 0;
            for (int c0 = 0; c0 < g.rb; c0 += 16) {
                uint32_t v[16];
                tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
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
            if (i < g.na) { s_score[i] = best; s_dst[i] = 2 * best_j + 1; }
        }
        tc_fence_before();
        __syncthreads();

        // ---- ranking: warp 0 takes the m best proposals (ties: the lowest A position)
        if (warp == 0) {
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

        // ---- merges: the warps are dealt out over (destination cell, slice of D).  The lowest rank
        // that targets a destination adds every source of that destination, in rank order.
        {
            const int m = st.m;
            const int nsl = m < kWarps ? kWarps / m : 1;
            for (int idx = warp; idx < m * nsl; idx += kWarps) {
                const int k = idx % m, sl = idx / m;
                const int dst = s_sel[k] & 0xffff;
                bool first = true;
                for (int q = 0; q < k; ++q) first &= (s_sel[q] & 0xffff) != dst;
                if (!first) continue;
                const unsigned rd = s_root[dst];
                const size_t od = (size_t)(rd & ~kMergedBit) * D;
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
                }
                if (sl == 0 && lane == 0) {
                    const int id = rd & ~kMergedBit;
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

        // ---- publish: every write of this line is ordered before the counter increment
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            atomicAdd(a.done + (size_t)step * B + b, 1);
        }
    }

    // ---- exit: no MMA may be in flight when the accumulator columns are returned
    if (mma_pending && tid == 0) {
        umma_commit(bar_acc);
        mbar_wait(bar_acc, (int)(items_done & 1), a.status);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, cfg.tmem_cols);
}

template <typename T>
cudaError_t launch_typed(const ChainArgs& a, int max_len, int r, cudaStream_t stream) {
    static int sms = 0, smem_cap = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&smem_cap, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    BipartiteLaunch cfg;
    cfg.max_len = max_len;
    cfg.r = r;
    cfg.stage_stride = (line_geom(max_len).stage_bytes + 127) & ~127;
    const size_t tail = (size_t)max_len * kPieces * 4 + (size_t)max_len * 8 + (size_t)((max_len + 1) / 2) * 8 +
                        (size_t)(r + 8) * 4;
    // two stages and two CTAs per SM where that fits, else as many stages (up to 4) as one CTA can hold
    const size_t budget = (size_t)smem_cap - 1024;            // the static shared variables
    const size_t fixed = kSlack + tail + 128;
    int stages = 2;
    if (2 * (2 * (size_t)cfg.stage_stride + fixed + 1024) > (size_t)smem_cap + 1024) {
        stages = (int)((budget - fixed) / (size_t)cfg.stage_stride);
        if (stages > 4) stages = 4;
        if (stages < 1) return cudaErrorInvalidConfiguration;
    }
    cfg.n_stages = stages;
    int cols = 32;
    while (cols < line_geom(max_len).rb) cols <<= 1;
    cfg.tmem_cols = cols;
    const size_t smem = (size_t)stages * cfg.stage_stride + fixed;
    cudaError_t err = cudaFuncSetAttribute(oim_bipartite_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    int blocks_per_sm = 0;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks_per_sm, oim_bipartite_kernel<T>, kThreads, smem);
    if (blocks_per_sm < 1) blocks_per_sm = 1;
    if (blocks_per_sm * cols > 512) blocks_per_sm = 512 / cols;     // TMEM columns of an SM
    int grid = blocks_per_sm * sms;
    if (grid > a.total_items) grid = a.total_items;
    oim_bipartite_kernel<T><<<grid, kThreads, smem, stream>>>(a, cfg);
    return cudaGetLastError();
}

}  // namespace

cudaError_t oim_bipartite_launch(const ChainArgs& a, int dtype, int max_len, int r, cudaStream_t stream) {
    if (max_len > kMaxLen) return cudaErrorInvalidValue;
    return dtype == LUVC_F32 ? launch_typed<float>(a, max_len, r, stream)
                             : launch_typed<__nv_bfloat16>(a, max_len, r, stream);
}

}  // namespace luvc
