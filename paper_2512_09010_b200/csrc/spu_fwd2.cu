// Two-stage forward transform of the Spectrum Pruning Unit for bf16 tokens (Eq. 4, restricted to
// the pass band |f| <= sigma of Eq. 5), for sequence lengths N = P * Q with P a multiple of 16.
//
// Token n = p Q + q, frequency k = k1 + P k2:
//   stage 1   A_q[k1] = sum_p x[p Q + q] e^{-2 pi i k1 p / P}        all k1: a dense P-point DFT over
//                                                                    tokens that are Q apart
//   stage 2   X[k]    = sum_q e^{-2 pi i q k / N} A_q[k mod P]       only the bins 0 <= k <= sigma
// Stage 1 is a real P x P matrix (rows: A[0], A[P/2], then Re / Im of A[1 .. P/2-1]; the other half
// follows from A[P-k1] = conj A[k1] because x is real) applied to a tile of Q-strided tokens: one
// tcgen05 contraction per tile, the matrix held in shared memory as a bf16 pair (hi + lo) built
// once per CTA, the token tile brought in by TMA (one 4-D box {channels, P strided tokens, tile
// tokens} per channel block, swizzled so that it is a legal MN-major operand as it lands), fp32
// accumulators in TMEM (two buffers).  Stage 2 runs on the CUDA
// cores straight out of TMEM: the thread that owns TMEM lane j owns the frequency pair
// (k1, P - k1) of that row and keeps its band bins for a few channels in registers for the whole
// sequence, so the input is read exactly once and nothing but the band spectrum is written:
//   Y[b][r][d], r = k (cos rows, 0..sigma) and r = sigma + k (sin rows, k >= 1), times the row
//   constants c[r] (mask of Eq. 5/6, 1/N and the weight of the conjugate half).
//
// A CTA is persistent over work items (sequence x channel tile x bin slice) and runs 16 warps, all
// of them doing stage 2.  Thread 0 is also the producer: when the accumulator of tile u has
// arrived (so the MMAs of tile u are done and their shared-memory stage is free) it issues the TMA
// copies of tile u + 2 into that stage and the MMAs of tile u + 1 into the other accumulator, which
// then run underneath stage 2 of tile u.  Every mbarrier wait is bounded (on expiry: status word,
// free TMEM, return).

#include <cuda.h>
#include <cuda_bf16.h>

#include "luvc_internal.h"
#include "sm100_ptx.cuh"
#include "spu_images.cuh"

namespace luvc {
namespace {

using namespace ptx;

constexpr int kEpiWarps = 16;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kThreads = kEpiThreads;         // no producer warps: thread 0 also issues the TMA copies and the MMAs
constexpr int kNmma = 256;                    // columns of a tile: QT tokens x C channels
constexpr int kTmemCols = 512;                // two accumulator buffers
constexpr int kSpin = 1 << 22;
constexpr int kProducer = 96;                 // its warp issues TMA and MMA (one elected lane): a warp with the fewest bins
constexpr int kStaticTabBytes = 24 * 1024;

struct FwdArgs {
    const __nv_bfloat16* x;   // [B][N][D]
    float* Y;                 // [B][R][D]
    const float* scale;       // c[r], r < R
    int* status;
    int B, N, D, P, Q, sigma, R;
    int nblk;                 // copies of the P x P matrix on the diagonal of the 128-row operand: each
                              // serves its own block of channels of the same tokens (P <= 64)
    int n_ctiles, n_slices, n_items;
    int static_tab;           // 1: the table of e^{-2 pi i q k2 / Q} for all q is built once per CTA (one slice only)
    const unsigned char* f_img;   // both parts of the stage-1 matrix as they sit in shared memory (built once per call)
    int n_stages;             // input stages in shared memory: 3 where they fit (copies run two tiles ahead), else 2
};

// barriers: 0-2 stage full | 3,4 accumulator full | 5,6 accumulator empty | 7,8 table ready | 9 operand image landed
enum { kBarFull = 0, kBarAccFull = 3, kBarAccEmpty = 5, kBarTab = 7, kBarImg = 9, kBars = 10 };
constexpr int kMaxStages = 3;

__device__ __forceinline__ bool wait_bar(uint32_t bar, int parity, volatile int* s_fail, int* status) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer();
    for (int it = 0; it < kSpin; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*s_fail) return false;
        if ((it & 63) == 63 && global_timer() - t0 > 1000000000ull) break;   // one second
    }
    atomicCAS(status, 0, (int)LUVC_ERR_TIMEOUT);
    *s_fail = 1;
    return false;
}

__device__ __forceinline__ float2 cmul(float2 a, float2 b) {
    return make_float2(a.x * b.x - a.y * b.y, fmaf(a.x, b.y, a.y * b.x));
}
// e^{-2 pi i num / den}, 0 <= num < den
__device__ __forceinline__ float2 root_neg(unsigned num, unsigned den) {
    float s, c;
    sincospif(2.0f * (float)num / (float)den, &s, &c);
    return make_float2(c, -s);
}
// A table entry g = e^{-2 pi i num / den} in the form the packed complex multiply-add wants:
// (g.x, g.x, -g.y, g.y), so that y += g w is two packed FMAs, (g.x, g.x) * (w.x, w.y) and (-g.y, g.y) * (w.y, w.x).
__device__ __forceinline__ float4 root_neg_packed(unsigned num, unsigned den) {
    const float2 g = root_neg(num, den);
    return make_float4(g.x, g.x, -g.y, g.y);
}

template <int NCOL> __device__ __forceinline__ void tmem_load(uint32_t addr, uint32_t (&v)[NCOL]) {
    if constexpr (NCOL == 2) tmem_ld2(addr, v);
    else if constexpr (NCOL == 4) tmem_ld4(addr, v);
    else if constexpr (NCOL == 8) tmem_ld8(addr, v);
    else tmem_ld16(addr, v);
}

template <int CH> __device__ __forceinline__ void store_row(float* dst, const float (&v)[CH]) {
    if constexpr (CH >= 4) {
#pragma unroll
        for (int c = 0; c < CH; c += 4) *reinterpret_cast<float4*>(dst + c) = make_float4(v[c], v[c + 1], v[c + 2], v[c + 3]);
    } else if constexpr (CH == 2) {
        *reinterpret_cast<float2*>(dst) = make_float2(v[0], v[1]);
    } else {
        dst[0] = v[0];
    }
}

// Stage 2 of one tile for one thread: NB bins (compile time, so that the loops carry no branches) of
// the thread's frequency for the 2 CH channels of its warp.  The even lane of a pair owns the row
// of real parts and the frequency k1, the odd lane the imaginary parts and the frequency P - k1,
// whose stage-1 value is the conjugate: each sends its row to the other, and with e = own + i c other
// the even lane holds A[k1] (c = 1) while the odd lane holds i conj(A[k1]) (c = 1), so the factor
// -i is folded into its rotation; the pair of rows 0 / 1 holds the two real values A[0], A[P/2] (c = 0).
// `tab` holds e^{-2 pi i q k2 / Q} for the tile's tokens.
template <int KB, int CH, int NB>
__device__ __forceinline__ void stage2_tile(uint32_t taddr, int nq, const float4* __restrict__ tab, float2& rot,
                                            float2 step, float cg, bool warp_active, uint32_t acc_empty_bar,
                                            int lane, float2 (&y)[KB][2 * CH]) {
    constexpr int C = 8 * CH, W = 2 * CH;
    uint32_t v[W], vn[W];
    tmem_load<W>(taddr, vn);
    for (int ql = 0; ql < nq; ++ql) {
        tmem_ld_wait_for(vn);
#pragma unroll
        for (int c = 0; c < W; ++c) v[c] = vn[c];
        if (ql + 1 < nq) {
            tmem_load<W>(taddr + (uint32_t)((ql + 1) * C), vn);   // in flight under this token's arithmetic
        } else {                     // this warp has read all it needs of the buffer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty_bar);
        }
        if (!warp_active) continue;
        // packed fp32 arithmetic (two FMAs per instruction): a complex product a b is
        // (a.x, a.x) * (b.x, b.y) + (-a.y, a.y) * (b.y, b.x)
        const float2 rxx = make_float2(rot.x, rot.x), ryy = make_float2(-rot.y, rot.y);
        if constexpr (NB <= 6) {            // few bins: the table row stays in registers across the channels
            float4 g[NB];
#pragma unroll
            for (int t = 0; t < NB; ++t) g[t] = tab[ql * KB + t];
#pragma unroll
            for (int c = 0; c < W; ++c) {
                const float own = __uint_as_float(v[c]);
                const float other = cg * __shfl_xor_sync(0xffffffffu, own, 1);
                const float2 w = __ffma2_rn(rxx, make_float2(own, other), __fmul2_rn(ryy, make_float2(other, own)));
                const float2 ws = make_float2(w.y, w.x);
#pragma unroll
                for (int t = 0; t < NB; ++t) {
                    y[t][c] = __ffma2_rn(make_float2(g[t].x, g[t].y), w, y[t][c]);
                    y[t][c] = __ffma2_rn(make_float2(g[t].z, g[t].w), ws, y[t][c]);
                }
            }
        } else {                            // many bins, few channels: the rotated values stay, the table streams
            float2 w[W], ws[W];
#pragma unroll
            for (int c = 0; c < W; ++c) {
                const float own = __uint_as_float(v[c]);
                const float other = cg * __shfl_xor_sync(0xffffffffu, own, 1);
                w[c] = __ffma2_rn(rxx, make_float2(own, other), __fmul2_rn(ryy, make_float2(other, own)));
                ws[c] = make_float2(w[c].y, w[c].x);
            }
#pragma unroll
            for (int t = 0; t < NB; ++t) {
                const float4 g = tab[ql * KB + t];
#pragma unroll
                for (int c = 0; c < W; ++c) {
                    y[t][c] = __ffma2_rn(make_float2(g.x, g.y), w[c], y[t][c]);
                    y[t][c] = __ffma2_rn(make_float2(g.z, g.w), ws[c], y[t][c]);
                }
            }
        }
        rot = cmul(rot, step);
    }
}

// The same for few bins per thread (KB <= 4): instead of rotating every stage-1 value by e^{-2 pi i q k1 / N} and
// then multiplying it by a table entry per bin, the thread carries the whole factor g[t] = e^{-2 pi i q k_t / N} of
// each of its bins from token to token (one complex product per bin and token, whatever the number of channels)
// and a value costs two packed FMAs per bin: y += g (own + i c other) = (g.x, g.y) own + (-g.y, g.x) c other.
// On the odd lane of a pair g carries the factor -i (see stage2_tile).
template <int KB, int CH, int NB>
__device__ __forceinline__ void stage2_tile_few(uint32_t taddr, int nq, float2 (&g)[KB], const float2 (&gstep)[KB], float cg,
                                                bool warp_active, uint32_t acc_empty_bar, int lane, float2 (&y)[KB][2 * CH]) {
    constexpr int C = 8 * CH, W = 2 * CH;
    uint32_t v[W], vn[W];
    tmem_load<W>(taddr, vn);
    for (int ql = 0; ql < nq; ++ql) {
        tmem_ld_wait_for(vn);
#pragma unroll
        for (int c = 0; c < W; ++c) v[c] = vn[c];
        if (ql + 1 < nq) {
            tmem_load<W>(taddr + (uint32_t)((ql + 1) * C), vn);   // in flight under this token's arithmetic
        } else {                     // this warp has read all it needs of the buffer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty_bar);
        }
        if (!warp_active) continue;
        float2 gp[NB], gq[NB];
#pragma unroll
        for (int t = 0; t < NB; ++t) { gp[t] = g[t]; gq[t] = make_float2(-g[t].y, g[t].x); }
#pragma unroll
        for (int c = 0; c < W; ++c) {
            const float own = __uint_as_float(v[c]);
            const float other = cg * __shfl_xor_sync(0xffffffffu, own, 1);
            const float2 oo = make_float2(own, own), cc = make_float2(other, other);
#pragma unroll
            for (int t = 0; t < NB; ++t) {
                y[t][c] = __ffma2_rn(gp[t], oo, y[t][c]);
                y[t][c] = __ffma2_rn(gq[t], cc, y[t][c]);
            }
        }
#pragma unroll
        for (int t = 0; t < KB; ++t) g[t] = cmul(g[t], gstep[t]);
    }
}

// KB: band bins per frequency class held by a thread; CH: channels per thread (C = 8 CH per block).
template <int KB, int CH>
__global__ void __launch_bounds__(kThreads, 1) spu_fwd2_kernel(const __grid_constant__ CUtensorMap tmap, const FwdArgs a) {
    constexpr int C = 8 * CH;
    constexpr int QT = kNmma / C;
    constexpr int LOG_CC = CH == 8 ? 3 : (CH == 4 ? 2 : (CH == 2 ? 1 : 0));   // log2(C / 8)
    constexpr int ROWB = 2 * C;                  // bytes of one token row of a tile: 16 (no swizzle), 32, 64 or 128
    constexpr uint32_t LAYOUT = CH == 8 ? 2u : (CH == 4 ? 4u : (CH == 2 ? 6u : 0u));
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long s_bar[kBars];
    __shared__ uint32_t s_tmem;
    __shared__ int s_fail;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int P = a.P, Q = a.Q, N = a.N, D = a.D, sigma = a.sigma;
    const int KT = a.nblk * P;                   // K extent of a tile: nblk channel blocks x P tokens
    const int f_bytes = KT * 256;                // one part of the stage-1 matrix: KT/8 K chunks x 128 rows x 16 B
    const int blk_bytes = QT * P * ROWB;         // one channel block of a tile: [tile token][P tokens][C channels]
    const int stage_bytes = a.nblk * blk_bytes;  // = 256 columns x KT rows x 2 bytes
    // swizzled tiles need their 1024-byte atoms on 1024-byte boundaries (1 KB of slack is requested for this)
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* s_fhi = smem;
    unsigned char* s_flo = smem + f_bytes;
    unsigned char* s_x = smem + 2 * f_bytes;
    const int nst = a.n_stages;
    float4* s_tab = reinterpret_cast<float4*>(s_x + nst * stage_bytes);   // [Q * KB] or [2][QT * KB]
    const uint32_t bar0 = smem_u32(&s_bar[0]);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    if (tid == 0) {
        for (int s = 0; s < kMaxStages; ++s) mbar_init(bar(kBarFull + s), 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kBarAccFull + s), 1);
            mbar_init(bar(kBarAccEmpty + s), kEpiWarps);
            mbar_init(bar(kBarTab + s), kEpiWarps);
        }
        mbar_init(bar(kBarImg), 1);
        s_fail = 0;
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc(smem_u32(&s_tmem), kTmemCols);

    // the stage-1 matrix (both parts) was built once per call in global memory, in its shared-memory layout
    if (tid == 0) {
        mbar_arrive_expect_tx(bar(kBarImg), (uint32_t)(2 * f_bytes));
        bulk_load(smem_u32(s_fhi), a.f_img, (uint32_t)(2 * f_bytes), bar(kBarImg));
    }
    constexpr bool kFew = KB <= 4;               // few bins: the per-bin factors are carried in registers, no table
    if (!kFew && a.static_tab)
        for (int e = tid; e < Q * KB; e += kThreads) {
            const int q = e / KB, k2 = e - q * KB;
            s_tab[e] = root_neg_packed(((unsigned)q * (unsigned)k2) % (unsigned)Q, Q);
        }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    volatile int* fail = &s_fail;
    if (!__all_sync(0xffffffffu, wait_bar(bar(kBarImg), 0, fail, a.status))) {     // the matrix has landed
        __syncthreads();
        if (warp == 0) tmem_dealloc(tmem, kTmemCols);
        return;
    }
    const int tiles_per_item = (Q + QT - 1) / QT;
    const int item_channels = a.nblk * C;

    const uint32_t xs = smem_u32(s_x), fhi = smem_u32(s_fhi), flo = smem_u32(s_flo);
    const uint32_t idesc = make_idesc_bf16(128, kNmma, false, true);
    int n_my_items = 0;
    for (int item = blockIdx.x; item < a.n_items; item += gridDim.x) ++n_my_items;
    const int total_tiles = n_my_items * tiles_per_item;

    const uint64_t a_hi0 = make_desc(fhi, 2048, 128), a_lo0 = make_desc(flo, 2048, 128);
    const uint64_t b0 = LAYOUT ? make_desc_layout(xs, P * ROWB, 8 * ROWB, LAYOUT) : make_desc(xs, 128, P * 16);

    // producer steps (one thread only)
    auto issue_tma = [&](int v) {           // tile v of this CTA's sequence of tiles -> stage v % nst
        const int item = blockIdx.x + (v / tiles_per_item) * gridDim.x, tile = v % tiles_per_item;
        const int rest = item / a.n_slices;
        const int ctile = rest % a.n_ctiles, b = rest / a.n_ctiles;
        const int c0 = ctile * item_channels, buf = v % nst;
        // boxes that reach past Q or D are filled with zeros there and still count in full
        if (elect_one()) {
            mbar_arrive_expect_tx(bar(kBarFull + buf), (uint32_t)stage_bytes);
            for (int jb = 0; jb < a.nblk; ++jb)
                tma_load_4d(xs + buf * stage_bytes + jb * blk_bytes, &tmap, bar(kBarFull + buf), c0 + jb * C, 0, tile * QT, b);
        }
        __syncwarp();
    };
    auto issue_mma = [&](int v) -> bool {   // needs tile v in its stage and accumulator v & 1 drained
        const int buf = v & 1, st = v % nst;
        if (!__all_sync(0xffffffffu, wait_bar(bar(kBarFull + st), (v / nst) & 1, fail, a.status))) return false;
        if (v >= 2 && !__all_sync(0xffffffffu, wait_bar(bar(kBarAccEmpty + buf), ((v - 2) >> 1) & 1, fail, a.status))) return false;
        tc_fence_after();
        const uint32_t acc = tmem + (uint32_t)(buf * kNmma);
        if (elect_one()) {
            uint64_t ah = a_hi0, al = a_lo0;             // descriptors advance by adding to the address field
            for (int jb = 0; jb < a.nblk; ++jb) {        // K rows of channel block jb
                uint64_t bd = b0 + (uint64_t)((st * stage_bytes + jb * blk_bytes) >> 4);
                for (int kl = 0; kl < P / 16; ++kl) {
                    umma_bf16(acc, ah, bd, idesc, (jb | kl) ? 1u : 0u);
                    umma_bf16(acc, al, bd, idesc, 1u);
                    ah += 4096 >> 4; al += 4096 >> 4; bd += (16 * ROWB) >> 4;
                }
            }
            umma_commit(bar(kBarAccFull + buf));
        }
        __syncwarp();
        return true;
    };
    // The producer is a whole warp running warp-uniform code, with one elected lane issuing: the descriptors
    // then stay in uniform registers (a tcgen05.mma issued from divergent code costs its thread twice as long).
    const int warp_u = __shfl_sync(0xffffffffu, warp, 0);
    const bool producer = warp_u == kProducer / 32;
    if (producer && total_tiles > 0) {
        for (int v = 0; v < nst && v < total_tiles; ++v) issue_tma(v);
        issue_mma(0);
    }
    __syncwarp();

    {
        // ------------------------------------------------------------------ stage 2 (all warps)
        const int quarter = warp & 3, grp = warp >> 2;
        const int j = quarter * 32 + lane;
        const int jb = j / P, jr = j - jb * P;
        const bool active = j < KT;
        const int i = jr >> 1;
        const bool odd = jr & 1, special = i == 0;
        const bool warp_active = quarter * 32 < KT;
        // this lane's frequency: k1 = i on the even lane, P - i on the odd lane (0 and P/2 for the first pair)
        const int kf = special ? (odd ? P / 2 : 0) : (odd ? P - i : i);
        const float cg = special ? 0.f : 1.f;
        const int my_c = jb * C + grp * 2 * CH;                    // first of this thread's channels in the item
        const float2 step = root_neg(kf % N, N);
        const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
        int u = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < a.n_items && ok; item += gridDim.x) {
            const int slice = item % a.n_slices, rest = item / a.n_slices;
            const int ctile = rest % a.n_ctiles, b = rest / a.n_ctiles;
            const int k2_lo = slice * KB;
            // bins of this thread in this slice: k = kf + P (k2_lo + t) <= sigma
            int nb = (active && kf <= sigma) ? (sigma - kf) / P + 1 - k2_lo : 0;
            nb = max(0, min(KB, nb));
            const int nb_w = __reduce_max_sync(0xffffffffu, nb);
            float2 y[KB][2 * CH];
#pragma unroll
            for (int t = 0; t < KB; ++t)
#pragma unroll
                for (int c = 0; c < 2 * CH; ++c) y[t][c] = make_float2(0.f, 0.f);

            float2 rot = make_float2(1.f, 0.f);
            float2 gk[KB], gstep[KB];                    // few bins: e^{-2 pi i q k_t / N} and its step from token to token
#pragma unroll
            for (int t = 0; t < KB; ++t) {
                gk[t] = make_float2(1.f, 0.f);
                gstep[t] = kFew ? root_neg((unsigned)((kf + P * (k2_lo + t)) % N), N) : make_float2(1.f, 0.f);
            }
            for (int tile = 0; tile < tiles_per_item; ++tile, ++u) {
                const int q0 = tile * QT, nq = min(QT, Q - q0), buf = u & 1, par = (u >> 1) & 1;
                // table of e^{-2 pi i q k2 / Q} for the tile's tokens and the slice's k2
                const float4* tab = s_tab + q0 * KB;
                if (!kFew && !a.static_tab) {
                    float4* tw = s_tab + buf * (QT * KB);
                    for (int e = tid; e < QT * KB; e += kEpiThreads) {
                        const int ql = e / KB, k2 = k2_lo + (e - ql * KB);
                        tw[e] = root_neg_packed(((unsigned)(q0 + ql) * (unsigned)k2) % (unsigned)Q, Q);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(kBarTab + buf));
                    ok = wait_bar(bar(kBarTab + buf), par, fail, a.status);
                    tab = tw;
                }
                ok = wait_bar(bar(kBarAccFull + buf), par, fail, a.status) && ok;
                ok = __all_sync(0xffffffffu, ok);
                if (producer && ok) {
                    // the MMAs of tile u are done: refill their stage, and start tile u + 1
                    if (u + nst < total_tiles) issue_tma(u + nst);
                    if (u + 1 < total_tiles) ok = issue_mma(u + 1);
                }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                if ((tile & 15) == 0) {     // exact restart of e^{-2 pi i q k / N}; in between it is carried along
                    if constexpr (kFew) {
#pragma unroll
                        for (int t = 0; t < KB; ++t) {
                            const unsigned long long m = (unsigned long long)q0 * (unsigned)(kf + P * (k2_lo + t));
                            gk[t] = root_neg((unsigned)(m % (unsigned)N), N);
                            if (odd && !special) gk[t] = make_float2(gk[t].y, -gk[t].x);      // times -i (see stage2_tile)
                        }
                    } else {
                        rot = root_neg(((unsigned)q0 * (unsigned)kf) % (unsigned)N, N);   // q0 kf < Q P = N
                        if (odd && !special) rot = make_float2(rot.y, -rot.x);           // times -i (see stage2_tile)
                    }
                }
                const uint32_t taddr = lane_addr + (uint32_t)(buf * kNmma + grp * 2 * CH);
                const uint32_t eb = bar(kBarAccEmpty + buf);
                if constexpr (kFew) {
                    if (nb_w == KB)
                        stage2_tile_few<KB, CH, KB>(taddr, nq, gk, gstep, cg, warp_active, eb, lane, y);
                    else if (nb_w == KB - 1 || KB == 2)
                        stage2_tile_few<KB, CH, (KB > 1 ? KB - 1 : 1)>(taddr, nq, gk, gstep, cg, warp_active, eb, lane, y);
                    else
                        stage2_tile_few<KB, CH, (KB >= 4 ? KB / 2 : KB)>(taddr, nq, gk, gstep, cg, warp_active, eb, lane, y);
                } else if (nb_w == KB)
                    stage2_tile<KB, CH, KB>(taddr, nq, tab, rot, step, cg, warp_active, eb, lane, y);
                else if (nb_w == KB - 1 || KB == 2)
                    stage2_tile<KB, CH, (KB > 1 ? KB - 1 : 1)>(taddr, nq, tab, rot, step, cg, warp_active, eb, lane, y);
                else if (KB >= 4 && nb_w <= KB / 2)
                    stage2_tile<KB, CH, (KB >= 4 ? KB / 2 : KB)>(taddr, nq, tab, rot, step, cg, warp_active, eb, lane, y);
                else
                    stage2_tile<KB, CH, KB>(taddr, nq, tab, rot, step, cg, warp_active, eb, lane, y);
            }
            if (!ok) break;
            // band spectrum of this thread's channels: cos row k, sin row sigma + k
            const int ch0 = ctile * item_channels + my_c;
            if (active && ch0 < D) {
                float* Yb = a.Y + (size_t)b * a.R * D + ch0;
                const bool second = ch0 + CH < D;      // D is a multiple of 8 and ch0 of CH: each half is whole or absent
#pragma unroll
                for (int t = 0; t < KB; ++t) {
                    if (t >= nb) continue;
                    const int k = kf + P * (k2_lo + t);
                    const float cr = __ldg(a.scale + k);
                    const float ci = k >= 1 ? __ldg(a.scale + sigma + k) : 0.f;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (h == 1 && !second) continue;
                        float vr[CH], vi[CH];
#pragma unroll
                        for (int c = 0; c < CH; ++c) { vr[c] = cr * y[t][h * CH + c].x; vi[c] = ci * y[t][h * CH + c].y; }
                        store_row<CH>(Yb + (size_t)k * D + h * CH, vr);          // aligned vector stores
                        if (k >= 1) store_row<CH>(Yb + (size_t)(sigma + k) * D + h * CH, vi);
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// The stage-1 matrix image (spu_images.cuh), built once per call instead of once per CTA.
__global__ void __launch_bounds__(256) spu_fwd2_img_kernel(unsigned char* __restrict__ img, int P, int KT) {
    const int idx = blockIdx.x * 256 + threadIdx.x;
    if (idx < 128 * KT) spu_fwd2_img_element(img, P, KT, idx);
}

// YT[b][d][r] (bf16 pair, r padded with zeros to r_pad) from Y[b][r][d]
__global__ void __launch_bounds__(256) spu_y_transpose_kernel(const float* __restrict__ Y, __nv_bfloat16* __restrict__ hi,
                                                              __nv_bfloat16* __restrict__ lo, int R, int r_pad, int D) {
    __shared__ float tile[32][33];
    const int b = blockIdx.z, r0 = blockIdx.x * 32, d0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int rr = ty; rr < 32; rr += 8) {
        const int r = r0 + rr, d = d0 + tx;
        tile[rr][tx] = (r < R && d < D) ? Y[((size_t)b * R + r) * D + d] : 0.f;
    }
    __syncthreads();
    for (int dd = ty; dd < 32; dd += 8) {
        const int d = d0 + dd, r = r0 + tx;
        if (d < D && r < r_pad) {
            const float v = tile[tx][dd];
            const __nv_bfloat16 h = __float2bfloat16_rn(v);
            const size_t o = ((size_t)b * D + d) * r_pad + r;
            hi[o] = h;
            lo[o] = __float2bfloat16_rn(v - __bfloat162float(h));
        }
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

template <int KB, int CH>
cudaError_t launch_fwd2(const FwdArgs& a_in, const SpuFwd2Plan& pl, cudaStream_t stream) {
    constexpr int C = 8 * CH, QT = kNmma / C;
    const int KT = a_in.nblk * a_in.P;
    FwdArgs a = a_in;
    // the tokens of one sequence as [q][p][channel]: token p Q + q sits P-strided in memory
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return cudaErrorNotSupported;
    CUtensorMap tmap;
    const cuuint64_t dims[4] = {(cuuint64_t)a.D, (cuuint64_t)a.P, (cuuint64_t)a.Q, (cuuint64_t)a.B};
    const cuuint64_t strides[3] = {(cuuint64_t)a.Q * a.D * 2, (cuuint64_t)a.D * 2, (cuuint64_t)a.N * a.D * 2};
    const cuuint32_t box[4] = {(cuuint32_t)C, (cuuint32_t)a.P, (cuuint32_t)QT, 1u};
    const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    const CUtensorMapSwizzle swz = CH == 8 ? CU_TENSOR_MAP_SWIZZLE_128B
                                 : CH == 4 ? CU_TENSOR_MAP_SWIZZLE_64B
                                 : CH == 2 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE;
    if (encode(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<__nv_bfloat16*>(a.x), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    const size_t tab_bytes = a.static_tab ? (size_t)a.Q * KB * sizeof(float4) : (size_t)2 * QT * KB * sizeof(float4);
    const size_t fixed = 1024 + (size_t)2 * KT * 256 + tab_bytes, stage = (size_t)kNmma * KT * 2;
    a.n_stages = fixed + kMaxStages * stage <= (size_t)226 * 1024 ? kMaxStages : 2;
    const size_t smem = fixed + a.n_stages * stage;
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    cudaFuncSetAttribute(spu_fwd2_kernel<KB, CH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    const int grid = pl.n_items < sms ? pl.n_items : sms;
    spu_fwd2_kernel<KB, CH><<<grid, kThreads, smem, stream>>>(tmap, a);
    return cudaGetLastError();
}

}  // namespace

SpuFwd2Plan spu_fwd2_plan(int B, int N, int D, int sigma) {
    SpuFwd2Plan pl = {};
    for (int p = 128; p >= 16; p -= 16)
        if (N % p == 0) { pl.P = p; break; }
    if (!pl.P) return pl;
    pl.Q = N / pl.P;
    if (pl.Q > 32768) return pl;                       // keeps q * k2 inside 32 bits
    pl.nblk = 128 / pl.P;
    const int nk2 = sigma / pl.P + 1;                  // values of k2 that reach into the band
    const int kbs[4] = {2, 4, 9, 17}, chs[4] = {8, 4, 2, 1};
    int best = -1;
    for (int v = 0; v < 4; ++v) {
        const int slices = (nk2 + kbs[v] - 1) / kbs[v];
        if (best < 0 || slices < pl.slices) { best = v; pl.slices = slices; }
    }
    // A small batch in wide channel tiles leaves most SMs without a work item: with up to two bins per class the
    // four-bin variant does the same arithmetic on tiles of half the channels, which doubles the items.
    if (best == 0 && (long long)B * ((D + 64 * pl.nblk - 1) / (64 * pl.nblk)) * pl.slices <= 74) best = 1;
    pl.KB = kbs[best];
    pl.CH = chs[best];
    const int C = 8 * pl.CH * pl.nblk;                 // channels of one work item
    pl.n_ctiles = (D + C - 1) / C;
    const long long items = (long long)B * pl.n_ctiles * pl.slices;
    if (items > 0x7fffffffll) return pl;
    pl.n_items = (int)items;
    pl.ok = 1;
    return pl;
}

int spu_fwd2_run(const void* hidden, float* Y, const float* scale, void* yt_hi, void* yt_lo, int r_pad, int B, int N,
                 int D, int sigma, int* status, cudaStream_t stream, void* img, bool img_ready) {
    const SpuFwd2Plan pl = spu_fwd2_plan(B, N, D, sigma);
    if (!pl.ok) return LUVC_ERR_INTERNAL;
    if (!img_ready) {
        const int KT = pl.nblk * pl.P;
        spu_fwd2_img_kernel<<<(128 * KT + 255) / 256, 256, 0, stream>>>(static_cast<unsigned char*>(img), pl.P, KT);
        count_launch();
    }
    FwdArgs a;
    a.x = reinterpret_cast<const __nv_bfloat16*>(hidden);
    a.Y = Y; a.scale = scale; a.status = status;
    a.B = B; a.N = N; a.D = D; a.P = pl.P; a.Q = pl.Q; a.sigma = sigma; a.R = 2 * sigma + 1;
    a.nblk = pl.nblk;
    a.n_ctiles = pl.n_ctiles; a.n_slices = pl.slices; a.n_items = pl.n_items;
    a.f_img = static_cast<const unsigned char*>(img);
    a.static_tab = (pl.slices == 1 && (size_t)pl.Q * pl.KB * sizeof(float4) <= (size_t)kStaticTabBytes) ? 1 : 0;
    cudaError_t err;
    if (pl.KB == 2) err = launch_fwd2<2, 8>(a, pl, stream);
    else if (pl.KB == 4) err = launch_fwd2<4, 4>(a, pl, stream);
    else if (pl.KB == 9) err = launch_fwd2<9, 2>(a, pl, stream);
    else err = launch_fwd2<17, 1>(a, pl, stream);
    count_launch();
    if (err != cudaSuccess) return LUVC_ERR_CUDA;
    if (yt_hi != nullptr) {
        const int R = 2 * sigma + 1;
        spu_y_transpose_kernel<<<dim3((r_pad + 31) / 32, (D + 31) / 32, B), 256, 0, stream>>>(
            Y, reinterpret_cast<__nv_bfloat16*>(yt_hi), reinterpret_cast<__nv_bfloat16*>(yt_lo), R, r_pad, D);
        count_launch();
    }
    return cudaGetLastError() == cudaSuccess ? LUVC_OK : LUVC_ERR_CUDA;
}

}  // namespace luvc
