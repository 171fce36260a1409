// Forward transform of the Spectrum Pruning Unit for bf16 tokens with BOTH stages on the tensor
// cores (Eq. 4, restricted to the pass band |f| <= sigma of Eq. 5), for sequence lengths
// N = 128 Q, Q <= 128.
//
// Token n = p Q + q (p < 128), frequency k = k1 + 128 k2:
//   stage 1   A_q[k1] = sum_p x[p Q + q] e^{-2 pi i k1 p / 128}       dense 128-point DFT over tokens Q apart
//   twiddle   B_q[k1] = e^{-2 pi i q k1 / N} A_q[k1]                   CUDA cores, fp32
//   stage 2   X[k1 + 128 k2] = sum_q e^{-2 pi i q k2 / Q} B_q[k1]      a Q-point DFT of which only the
//                                                                      k2 < K2 bins inside the band are formed
// Stage 1 is the contraction of spu_fwd2.cu: a real 128 x 128 matrix (bf16 hi + lo) times a tile of
// Q-strided tokens that TMA lands as a legal MN-major operand, fp32 accumulators in TMEM (lane =
// row = real or imaginary part of one k1).  Stage 2 is a second contraction, over the tokens q of
// a sequence, with the same small matrix for every k1 and every channel (that is what the twiddle
// buys): out[lane, (channel, k2, re/im)] += sum over (q, re/im) of B[lane, (channel, q, re/im)]
// W[(q, re/im), (k2, re/im)].  Its A operand is B itself, which the threads that own the TMEM lanes
// write back into tensor memory as bf16 hi + lo pairs (row = lane, K along the columns); its B
// operand comes from a table in shared memory (per group of tokens a 16 x N2 matrix, bf16 hi and lo
// parts; block-diagonal over two channels in the narrow-band variant); the band spectrum accumulates
// in TMEM over the whole sequence and is written out once per work item, times the row constants
// (mask of Eq. 5/6, 1/N and the weight of the conjugate half), in the "operand form" that the
// inverse kernel of spu_inv3.cu multiplies from: per sequence and channel, for every TMEM lane its
// bins k2 = 0, 1, .. as four bf16 each (Re hi, Im hi, Re lo, Im lo), 16 bytes per lane and pair of
// bins, the 128 lanes side by side.
// What is left on the CUDA cores per stage-1 value is one TMEM read, one lane exchange, the twiddle
// and the split into two bf16 pairs: the same for every band width.
//
// Three geometries share the 512 TMEM columns (two stage-1 accumulators, one operand slot, 64 result
// columns per converter thread): 32 channels x 4 bins per frequency class, 16 x 8 and 8 x 16.  One
// value of k2 more than the geometry holds still costs no second pass: the lanes that reach it keep
// that bin on the CUDA cores (EXTRA = 1), and when only k1 = 0 reaches it (sigma a multiple of 128)
// the stage-2 issuing warps form it from the lane-0 values of each tile (EXTRA = 2).
//
// A CTA is persistent over work items (sequence x channel tile x slice of k2 values) and runs
// sixteen converter warps (four per TMEM lane quadrant: a group of four warps, one per quadrant,
// shares the same channels of a tile), one warp that issues the TMA copies and stage 1, and one
// warp per converter group that issues that group's stage-2 MMAs: a tcgen05.mma costs its issuing
// thread some fifty cycles whatever its size, and the many small MMAs of stage 2 only keep up when
// several warps issue them side by side.  Every mbarrier wait is bounded (on expiry: status word,
// free TMEM, return).

#include <cuda.h>
#include <cuda_bf16.h>

#include "luvc_internal.h"
#include "sm100_ptx.cuh"

namespace luvc {
namespace {

using namespace ptx;

constexpr int kConvWarps = 16;
constexpr int kConvThreads = kConvWarps * 32;
constexpr int kIssueWarps = 5;                // one for TMA copies and stage 1, one per converter group for stage 2
constexpr int kThreads = kConvThreads + kIssueWarps * 32;
constexpr int kP = 128;
constexpr int kSpin = 1 << 22;
constexpr int kTN = 64;                       // columns of a tile = QT tokens x C channels
constexpr int kSlotCols = 2 * kTN;            // TMEM columns of the stage-2 operand of one tile (16 units of 8)
constexpr int kUnits = 16;                    // stage-2 units of a tile: four per converter thread
constexpr int kStages = 4;                    // input stages in shared memory

struct Fwd3Args {
    const __nv_bfloat16* x;   // [B][N][D]
    unsigned char* yop;       // band spectrum in operand form: [B][D][ks_out][2 K chunks][128 lanes][16 B]
    float* yx;                // [2][B][D]: cos and sin value of the bin 128 * extra_k2 (written only if extra_k2 > 0)
    const float* scale;       // c[r], r < R
    int* status;
    int B, N, D, Q, sigma, ks_out;
    int n_ctiles, n_slices, n_items;
    const unsigned char* img; // stage-1 matrix, stage-2 matrices and root tables in their shared-memory layouts (built once per call)
    int extra_in_op;          // 1: that extra bin goes into the operand form (one more K step) instead of yx
    int extra_k2;             // > 0: one more value of k2 (= K2MAX) reaches into the band, for a few lanes only; those
                              // bins are accumulated on the CUDA cores instead of costing a second pass over the input
};

// barriers
enum {
    kBarFull = 0,                       // [kStages] TMA landed in stage s
    kBarAccFull = kBarFull + kStages,   // [2] stage-1 accumulator s complete (and its input stage free)
    kBarAccEmpty = kBarAccFull + 2,     // [2] every converter warp has read accumulator s
    kBarGrpFull = kBarAccEmpty + 2,     // [4 groups][2] the four warps of a converter group have written their units of slot s
    kBarGrpEmpty = kBarGrpFull + 8,     // [4 groups][2] the MMAs that read those units are done
    kBarOutFull = kBarGrpEmpty + 8,     // the band spectrum of the work item is complete (four issuers)
    kBarOutEmpty = kBarOutFull + 1,     // every converter warp has read it
    kBarImg = kBarOutEmpty + 1,         // the operand images have landed
    kBars = kBarImg + 1
};

__device__ __forceinline__ bool wait_bar(uint32_t bar, int parity, volatile int* s_fail, int* status) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer();
    // a probe suspends the thread for a while by itself; the failure flag and the clock are looked at now and then
    for (int it = 0; it < kSpin; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 15) == 15) {
            if (*s_fail) return false;
            if (global_timer() - t0 > 1000000000ull) break;   // one second
        }
    }
    atomicCAS(status, 0, (int)LUVC_ERR_TIMEOUT);
    *s_fail = 1;
    return false;
}

// The same wait for a whole warp: every lane gets the same answer (the issuing warps stay converged).
__device__ __forceinline__ bool wait_bar_warp(uint32_t bar, int parity, volatile int* s_fail, int* status) {
    return __all_sync(0xffffffffu, wait_bar(bar, parity, s_fail, status));
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

__device__ __forceinline__ uint32_t bf16x2_bits(float lo_half, float hi_half) {
    const __nv_bfloat162 p = __floats2bfloat162_rn(lo_half, hi_half);
    return *reinterpret_cast<const uint32_t*>(&p);
}

template <int NCOL> __device__ __forceinline__ void tmem_load(uint32_t addr, uint32_t (&v)[NCOL]) {
    if constexpr (NCOL == 2) tmem_ld2(addr, v);
    else if constexpr (NCOL == 4) tmem_ld4(addr, v);
    else tmem_ld8(addr, v);
}

// Geometry of a variant.  A tile is 64 columns (QT tokens x C channels); a converter thread owns W
// channels of every token of the tile, 16 values, which are 4 units; a unit is one stage-2 MMA's
// worth of rows (four complex values per lane = 16 bf16 along K, 8 TMEM columns).
//   C     channels of a work item
//   N2    columns of the stage-2 result per unit
//   QPU   tokens per unit: 2 (two channels x two tokens, block-diagonal over the channels: up to 4 bins
//         per frequency class) or 4 (one channel x four tokens: up to 16)
//   RING  operand slots (tiles) in tensor memory
template <int C_, int N2_, int QPU_, int RING_>
struct Geo {
    static constexpr int C = C_, N2 = N2_, QPU = QPU_, RING = RING_;
    static constexpr int QT = kTN / C;                        // tokens per tile: 2, 4 or 8
    static constexpr int W = C / 4;                           // channels per converter thread: 8, 4 or 2
    static constexpr int CPU_ = 4 / QPU;                      // channels per unit: 2 or 1
    static constexpr int K2MAX = N2 / (2 * CPU_);             // bins of k2 per lane and channel
    static constexpr int GQ = QT / QPU;                       // token groups per tile: 1 or 2
    static constexpr int UC = C / CPU_;                       // result units (column groups of the spectrum): 16 or 8
    static constexpr int UT = W / CPU_;                       // result units of one converter thread: 4 or 2
    static constexpr int OUT_COLS = UC * N2;                  // columns of the band spectrum in TMEM
    static constexpr int ACC0 = 0;                            // two stage-1 accumulators
    static constexpr int RING0 = 2 * kTN;
    static constexpr int OUT0 = RING0 + RING * kSlotCols;
    static constexpr int TMEM_COLS = 512;
    static constexpr int ROWB = 2 * C;                        // bytes of one token row of a tile: 64, 32 or 16
    static constexpr uint32_t LAYOUT = C == 32 ? 4u : (C == 16 ? 6u : 0u);   // 64-byte or 32-byte swizzle, or none
    static constexpr int STAGE_BYTES = kTN * kP * 2;
    static constexpr int W_BYTES = 16 * N2 * 2;               // one part (hi or lo) of one token group's matrix
    static_assert(OUT0 + OUT_COLS <= TMEM_COLS, "tensor memory budget");
    static_assert(W * QT == 16 && GQ * UT == 4 && GQ * UC == kUnits && kUnits * 8 == kSlotCols,
                  "a tile is sixteen units, four per converter thread");
};

template <typename G, int EXTRA>          // EXTRA: 0 none; 1 the extra bin on the converters; 2 on the issuing warps (k1 = 0 only)
__global__ void __launch_bounds__(kThreads, 1) spu_fwd3_kernel(const __grid_constant__ CUtensorMap tmap, const Fwd3Args a) {
    constexpr int C = G::C, N2 = G::N2, QPU = G::QPU, QT = G::QT, W = G::W;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long s_bar[kBars];
    __shared__ uint32_t s_tmem;
    __shared__ int s_fail;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Q = a.Q, N = a.N, D = a.D, sigma = a.sigma;
    const int tiles_per_item = (Q + QT - 1) / QT;
    const int n_groups = tiles_per_item * G::GQ;                    // token groups of a sequence (padded)
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* s_fhi = smem;                                        // stage-1 matrix, 32 KB per part
    unsigned char* s_flo = smem + 32768;
    unsigned char* s_x = smem + 65536;                                  // input stages
    unsigned char* s_w = s_x + kStages * G::STAGE_BYTES;                // [n_groups][hi, lo][16 x N2] stage-2 matrices
    float2* s_root = reinterpret_cast<float2*>(s_w + (size_t)n_groups * 2 * G::W_BYTES);   // e^{-2 pi i m / Q}, m < Q
    float2* s_fine = s_root + ((Q + 1) & ~1);                                              // e^{-2 pi i m / N}, m < 128
    uint32_t* s_dc = reinterpret_cast<uint32_t*>(s_fine + kP);                             // [4 groups][3][16] stage-1 values of k1 = 0
    const uint32_t bar0 = smem_u32(&s_bar[0]);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(bar(kBarFull + s), 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kBarAccFull + s), 1);
            mbar_init(bar(kBarAccEmpty + s), kConvWarps);
        }
        for (int s = 0; s < 8; ++s) {
            mbar_init(bar(kBarGrpFull + s), 4);
            mbar_init(bar(kBarGrpEmpty + s), 1);
        }
        mbar_init(bar(kBarOutFull), 4);
        mbar_init(bar(kBarOutEmpty), kConvWarps);
        mbar_init(bar(kBarImg), 1);
        s_fail = 0;
        mbar_fence_init();
    }
    if (warp == kConvWarps) tmem_alloc(smem_u32(&s_tmem), G::TMEM_COLS);

    // The stage-1 matrix, the stage-2 matrices and the two root tables were built once per call in global
    // memory, in the layouts used here: two bulk copies fetch them.
    const int tab_bytes = n_groups * 2 * G::W_BYTES + (((Q + 1) & ~1) + kP) * (int)sizeof(float2);
    if (tid == 0) {
        mbar_arrive_expect_tx(bar(kBarImg), (uint32_t)(65536 + tab_bytes));
        bulk_load(smem_u32(s_fhi), a.img, 65536u, bar(kBarImg));
        bulk_load(smem_u32(s_w), a.img + 65536, (uint32_t)tab_bytes, bar(kBarImg));
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    volatile int* fail = &s_fail;
    if (!__all_sync(0xffffffffu, wait_bar(bar(kBarImg), 0, fail, a.status))) {
        __syncthreads();
        if (warp == kConvWarps) tmem_dealloc(tmem, G::TMEM_COLS);
        return;
    }

    int n_my_items = 0;
    for (int item = blockIdx.x; item < a.n_items; item += gridDim.x) ++n_my_items;
    const int total_tiles = n_my_items * tiles_per_item;

    // warp index as the compiler can see it to be the same in every lane: the issuing warps then run
    // warp-uniform code and their descriptors live in uniform registers
    const int warp_u = __shfl_sync(0xffffffffu, warp, 0);
    if (warp_u == kConvWarps) {
        // ------------------------------------------------------------------ TMA copies and stage 1
        if (total_tiles > 0) {
            const uint32_t xs = smem_u32(s_x);
            const uint32_t idesc1 = make_idesc_bf16(128, kTN, false, true);
            const uint64_t a_hi0 = make_desc(smem_u32(s_fhi), 2048, 128), a_lo0 = make_desc(smem_u32(s_flo), 2048, 128);
            const uint64_t b0 = G::LAYOUT ? make_desc_layout(xs, kP * G::ROWB, 8 * G::ROWB, G::LAYOUT)
                                          : make_desc(xs, 128, kP * 16);
            auto issue_tma = [&](int v) {                               // tile v of this CTA's sequence of tiles
                const int item = blockIdx.x + (v / tiles_per_item) * gridDim.x;
                const int rest = item / a.n_slices;
                const int c0 = (rest % a.n_ctiles) * C, b = rest / a.n_ctiles, q0 = (v % tiles_per_item) * QT;
                const int st = v % kStages;
                if (elect_one()) {
                    // a box that reaches past Q or D is filled with zeros there and still counts in full
                    mbar_arrive_expect_tx(bar(kBarFull + st), (uint32_t)G::STAGE_BYTES);
                    tma_load_4d(xs + st * G::STAGE_BYTES, &tmap, bar(kBarFull + st), c0, 0, q0, b);
                }
                __syncwarp();
            };
            auto issue_stage1 = [&](int v) {                           // needs tile v in its stage and accumulator v & 1 read
                const uint32_t acc = tmem + (uint32_t)(G::ACC0 + (v & 1) * kTN);
                const uint64_t bd0 = b0 + (uint64_t)(((v % kStages) * G::STAGE_BYTES) >> 4);
                if (elect_one()) {
#pragma unroll
                    for (int kl = 0; kl < kP / 16; ++kl) {
                        const uint64_t bd = bd0 + (uint64_t)((kl * 16 * G::ROWB) >> 4);
                        umma_bf16(acc, a_hi0 + (uint64_t)((kl * 4096) >> 4), bd, idesc1, kl ? 1u : 0u);
                        umma_bf16(acc, a_lo0 + (uint64_t)((kl * 4096) >> 4), bd, idesc1, 1u);
                    }
                    umma_commit(bar(kBarAccFull + (v & 1)));
                }
                __syncwarp();
            };
            bool ok = true;
            for (int v = 0; v < kStages && v < total_tiles; ++v) issue_tma(v);
            ok = wait_bar_warp(bar(kBarFull), 0, fail, a.status);
            if (ok) {
                tc_fence_after();
                issue_stage1(0);
            }
            for (int v = 1; v < total_tiles && ok; ++v) {
                // tile v: its copy has landed, and the converters have read the accumulator it reuses
                ok = wait_bar_warp(bar(kBarFull + v % kStages), (v / kStages) & 1, fail, a.status);
                if (ok && v >= 2) ok = wait_bar_warp(bar(kBarAccEmpty + (v & 1)), ((v - 2) >> 1) & 1, fail, a.status);
                if (!ok) break;
                tc_fence_after();
                issue_stage1(v);
                if (v - 1 + kStages < total_tiles) {
                    // the stage that held tile v - 1 is free once its stage-1 MMAs are done (issued one tile ago)
                    ok = wait_bar_warp(bar(kBarAccFull + ((v - 1) & 1)), ((v - 1) >> 1) & 1, fail, a.status);
                    if (!ok) break;
                    issue_tma(v - 1 + kStages);
                }
            }
        }
    } else if (warp_u > kConvWarps) {
        // ------------------------------------------------------------------ stage 2 of one converter group
        const int g = warp_u - kConvWarps - 1;
        const uint32_t idesc2 = make_idesc_bf16(128, N2, false, false);
        const uint64_t w0 = make_desc(smem_u32(s_w), N2 * 16, 128);
        // the extra bin of k1 = 0 (extra_dc): lane i < 16 takes value i = ql W + c of a tile, token q = tile QT + ql
        constexpr bool dc = EXTRA == 2;
        const int dc_ql = (lane & 15) / W, dc_c = (lane & 15) % W;
        const int dc_step = dc ? (QT * a.extra_k2) % Q : 0;
        int dc_angle = 0;
        float2 dc_acc = make_float2(0.f, 0.f);
        bool ok = true;
        for (int u = 0; u < total_tiles && ok; ++u) {
            const int tile = u % tiles_per_item, item_seq = u / tiles_per_item;
            if (tile == 0 && item_seq > 0) {
                // the converters have read the previous item's band spectrum out of tensor memory
                ok = wait_bar_warp(bar(kBarOutEmpty), (item_seq - 1) & 1, fail, a.status);
                if (!ok) break;
            }
            const int slot = u % G::RING, use = u / G::RING;
            ok = wait_bar_warp(bar(kBarGrpFull + g * 2 + slot), use & 1, fail, a.status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t ring = tmem + (uint32_t)(G::RING0 + slot * kSlotCols + g * G::UT * 8);
            const uint32_t out = tmem + (uint32_t)(G::OUT0 + g * G::UT * N2);
            const uint64_t wg = w0 + (uint64_t)((tile * G::GQ * 2 * G::W_BYTES) >> 4);
            const uint32_t first = tile == 0 ? 0u : 1u;
            if (elect_one()) {
                // unit (token group gq, result unit cu of this group's threads): operand columns
                // (gq UC + g UT + cu) * 8, result columns (g UT + cu) * N2, matrix of token group tile * GQ + gq
#pragma unroll
                for (int gq = 0; gq < G::GQ; ++gq)
#pragma unroll
                    for (int cu = 0; cu < G::UT; ++cu) {
                        const uint64_t whi = wg + (uint64_t)((gq * 2 * G::W_BYTES) >> 4), wlo = whi + (uint64_t)(G::W_BYTES >> 4);
                        const uint32_t opnd = ring + (uint32_t)((gq * G::UC + cu) * 8), res = out + (uint32_t)(cu * N2);
                        umma_bf16_ts(res, opnd, whi, idesc2, gq ? 1u : first);
                        umma_bf16_ts(res, opnd, wlo, idesc2, 1u);
                    }
                umma_commit(bar(kBarGrpEmpty + g * 2 + slot));
                if (tile == tiles_per_item - 1) umma_commit(bar(kBarOutFull));
            }
            __syncwarp();
            if constexpr (dc) {
                if (tile == 0) {
                    dc_angle = (dc_ql * a.extra_k2) % Q;
                    dc_acc = make_float2(0.f, 0.f);
                }
                if (lane < 16) {
                    const float val = __uint_as_float(s_dc[(g * 3 + u % 3) * 16 + lane]);
                    const float2 wex = s_root[dc_angle];             // e^{-2 pi i q extra_k2 / Q}
                    dc_acc.x = fmaf(val, wex.x, dc_acc.x);
                    dc_acc.y = fmaf(val, wex.y, dc_acc.y);
                }
                dc_angle += dc_step;
                if (dc_angle >= Q) dc_angle -= Q;
                if (tile == tiles_per_item - 1) {
                    // sum over the tokens of a tile, then lane c holds channel c of this group
                    float2 t = lane < 16 ? dc_acc : make_float2(0.f, 0.f);
#pragma unroll
                    for (int off = W; off < 16; off <<= 1) {
                        t.x += __shfl_xor_sync(0xffffffffu, t.x, off);
                        t.y += __shfl_xor_sync(0xffffffffu, t.y, off);
                    }
                    const int item = blockIdx.x + item_seq * gridDim.x, rest = item / a.n_slices;
                    const int ctile = rest % a.n_ctiles, b = rest / a.n_ctiles;
                    const int ch = ctile * C + g * W + lane;
                    if (lane < W && ch < D) {
                        const int k = kP * a.extra_k2;
                        const float re = __ldg(a.scale + k) * t.x, im = __ldg(a.scale + sigma + k) * t.y;
                        if (a.extra_in_op) {
                            const uint32_t hi = bf16x2_bits(re, im);
                            const uint32_t lo = bf16x2_bits(re - __uint_as_float(hi << 16), im - __uint_as_float(hi & 0xffff0000u));
                            unsigned char* yc = a.yop + ((size_t)b * D + ch) * ((size_t)a.ks_out * 4096) + (size_t)(a.extra_k2 / 4) * 4096;
                            *reinterpret_cast<uint4*>(yc) = make_uint4(hi, lo, 0u, 0u);                 // TMEM lane 0 = k1 = 0
                            *reinterpret_cast<uint4*>(yc + 2048) = make_uint4(0u, 0u, 0u, 0u);
                        } else {
                            a.yx[(size_t)b * D + ch] = re;
                            a.yx[(size_t)a.B * D + (size_t)b * D + ch] = im;
                        }
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ converters
        const int quarter = warp & 3, g = warp >> 2;
        const int j = quarter * 32 + lane;                           // TMEM lane = row of the stage-1 matrix
        const int i = j >> 1;
        const bool odd = j & 1, special = i == 0;
        // this lane's frequency: k1 = i on the even lane, 128 - i on the odd lane (0 and 64 for the first pair)
        const int kf = special ? (odd ? kP / 2 : 0) : (odd ? kP - i : i);
        const float cg = special ? 0.f : 1.f;
        const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
        int u = 0, item_seq = 0;
        bool ok = true;
        float2 within[QT];
        int within_kfe = -1;
        for (int item = blockIdx.x; item < a.n_items && ok; item += gridDim.x, ++item_seq) {
            const int slice = item % a.n_slices, rest = item / a.n_slices;
            const int ctile = rest % a.n_ctiles, b = rest / a.n_ctiles;
            const int k2_lo = slice * G::K2MAX;
            const int kfe = kf + kP * k2_lo;                         // the slice's first bin of this lane
            // twiddle of token q0 + ql: e^{-2 pi i q0 kfe / N}, exact per tile, times e^{-2 pi i ql kfe / N},
            // exact per item: two roundings per value however long the sequence is
            // (the same for every work item of a slice, so with one slice they are computed once per kernel)
            if (kfe != within_kfe) {
#pragma unroll
                for (int ql = 0; ql < QT; ++ql)
                    within[ql] = root_neg((unsigned)(((unsigned long long)ql * (unsigned)kfe) % (unsigned)N), (unsigned)N);
                within_kfe = kfe;
            }
            // angle of the tile's first token, q0 kfe mod N, carried in integers (exact); N = 128 Q, so
            // e^{-2 pi i m / N} = e^{-2 pi i (m >> 7) / Q} e^{-2 pi i (m & 127) / N}: two table entries
            const int d_angle = (int)(((unsigned long long)QT * (unsigned)kfe) % (unsigned)N);
            int angle = 0;
            float2 extra[W];                                         // bin kfe + 128 extra_k2 of this lane's channels
#pragma unroll
            for (int c = 0; c < W; ++c) extra[c] = make_float2(0.f, 0.f);
            // only the warps with a lane that reaches that bin accumulate it; the angle q extra_k2 mod Q is carried
            // along in integers from token to token
            const bool need_x = EXTRA == 1 && __any_sync(0xffffffffu, kfe + kP * a.extra_k2 <= sigma);
            int x_angle = 0;
            const int x_step = EXTRA == 1 ? a.extra_k2 % Q : 0;
            // The TMEM round trips are long (a load or a store takes several hundred cycles), so the loop is
            // software-pipelined: the next tile's values are requested before this tile's arithmetic, and
            // a tile's stores are only waited for (and its units handed to the MMA warp) one tile later.
            const uint32_t acc_addr = lane_addr + (uint32_t)(G::ACC0 + g * W);
            uint32_t v[QT][W], vn[QT][W];
            ok = wait_bar(bar(kBarAccFull + (u & 1)), (u >> 1) & 1, fail, a.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int ql = 0; ql < QT; ++ql) tmem_load<W>(acc_addr + (uint32_t)((u & 1) * kTN + ql * C), vn[ql]);
            int pending_slot = -1;                                   // slot whose stores are in flight
            for (int tile = 0; tile < tiles_per_item && ok; ++tile, ++u) {
                const int buf = u & 1;
                float2 base = cmul(s_root[angle >> 7], s_fine[angle & 127]);
                if (odd && !special) base = make_float2(base.y, -base.x);    // times -i: the odd lane holds i conj(A)
                angle += d_angle;
                if (angle >= N) angle -= N;
                // every value of this thread in the tile: W channels of QT tokens
                tmem_ld_wait_for(reinterpret_cast<uint32_t(&)[QT * W]>(vn));
#pragma unroll
                for (int ql = 0; ql < QT; ++ql)
#pragma unroll
                    for (int c = 0; c < W; ++c) v[ql][c] = vn[ql][c];
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarAccEmpty + buf));  // the accumulator may be overwritten
                if constexpr (EXTRA == 2) {
                    // k1 = 0 (TMEM lane 0): its stage-1 values of this tile for the warp that forms the extra bin.  Three
                    // buffers: the one of tile u - 3 was read before the MMAs of tile u - 2 were issued, and their
                    // completion was waited for at the end of tile u - 1
                    if (j == 0) {
                        uint4* dst = reinterpret_cast<uint4*>(s_dc + (g * 3 + u % 3) * 16);
#pragma unroll
                        for (int i4 = 0; i4 < 4; ++i4) {
                            const int i = i4 * 4;
                            dst[i4] = make_uint4(v[i / W][i % W], v[(i + 1) / W][(i + 1) % W], v[(i + 2) / W][(i + 2) % W],
                                                 v[(i + 3) / W][(i + 3) % W]);
                        }
                    }
                }
                if (tile + 1 < tiles_per_item) {                     // request the next tile's values
                    ok = wait_bar(bar(kBarAccFull + ((u + 1) & 1)), ((u + 1) >> 1) & 1, fail, a.status);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int ql = 0; ql < QT; ++ql)
                        tmem_load<W>(acc_addr + (uint32_t)(((u + 1) & 1) * kTN + ql * C), vn[ql]);
                }

                uint32_t op[4][8];                                   // four units of four complex values: (hi pair, lo pair) each
#pragma unroll
                for (int ql = 0; ql < QT; ++ql) {
                    if (ql == QT / 2 && pending_slot >= 0) {
                        // half way through the arithmetic the previous tile's stores have long landed: hand its
                        // units to the MMA warp now, which then has the other half to finish with them before
                        // this tile's units go into the same columns
                        tmem_st_wait();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(kBarGrpFull + g * 2 + pending_slot));
                        pending_slot = -1;
                    }
                    const float2 rot = cmul(base, within[ql]);
                    // B = rot * (own + i cg other):  Re = rot.x own - cg rot.y other,  Im = rot.y own + cg rot.x other
                    const float ox = -cg * rot.y, oy = cg * rot.x;
                    float2 wex = make_float2(0.f, 0.f);              // e^{-2 pi i q extra_k2 / Q} of this token
                    if constexpr (EXTRA == 1) {
                        if (need_x) {
                            wex = s_root[x_angle];
                            x_angle += x_step;
                            if (x_angle >= Q) x_angle -= Q;
                        }
                    }
#pragma unroll
                    for (int c = 0; c < W; ++c) {
                        const float own = __uint_as_float(v[ql][c]);
                        const float other = __shfl_xor_sync(0xffffffffu, own, 1);
                        const float wx = fmaf(rot.x, own, ox * other), wy = fmaf(rot.y, own, oy * other);
                        if constexpr (EXTRA == 1) {
                            if (need_x) {
                                extra[c].x = fmaf(wx, wex.x, fmaf(-wy, wex.y, extra[c].x));
                                extra[c].y = fmaf(wx, wex.y, fmaf(wy, wex.x, extra[c].y));
                            }
                        }
                        const uint32_t hi = bf16x2_bits(wx, wy);
                        const uint32_t lo = bf16x2_bits(wx - __uint_as_float(hi << 16), wy - __uint_as_float(hi & 0xffff0000u));
                        // unit and position of this value: two channels x two tokens, or one channel x four tokens
                        const int unit = QPU == 2 ? ((ql >> 1) * G::UT + (c >> 1)) : ((ql >> 2) * G::UT + c);
                        const int z = QPU == 2 ? ((ql & 1) * 2 + (c & 1)) : (ql & 3);
                        op[unit][2 * z] = hi;
                        op[unit][2 * z + 1] = lo;
                    }
                }
                // the MMAs that read this slot a ring ago are done
                const int slot = u % G::RING, use = u / G::RING;
                if (use >= 1) {
                    ok = wait_bar(bar(kBarGrpEmpty + g * 2 + slot), (use - 1) & 1, fail, a.status);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
                }
                // unit (token group gq, this thread's result unit cu) sits at columns (gq UC + g UT + cu) * 8 of the slot
                const uint32_t ring = lane_addr + (uint32_t)(G::RING0 + slot * kSlotCols + g * G::UT * 8);
#pragma unroll
                for (int gq = 0; gq < G::GQ; ++gq)
#pragma unroll
                    for (int cu = 0; cu < G::UT; ++cu) tmem_st8(ring + (uint32_t)((gq * G::UC + cu) * 8), op[gq * G::UT + cu]);
                pending_slot = slot;
            }
            if (!ok) break;
            if (pending_slot >= 0) {                                 // the item's last tile
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarGrpFull + g * 2 + pending_slot));
            }
            if (!ok) break;
            // ---- the item's band spectrum: out of tensor memory, times the row constants, split into bf16 pairs and
            // stored in operand form: per channel and K chunk (two bins) the 128 lanes write 16 bytes each, side by side
            ok = wait_bar(bar(kBarOutFull), item_seq & 1, fail, a.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            {
                const int ch0 = ctile * C + g * W;                   // first of this thread's channels
                const size_t chan_bytes = (size_t)a.ks_out * 4096;
                unsigned char* yb = a.yop + ((size_t)b * D + ch0) * chan_bytes + (size_t)j * 16;
                // two bins (k2, k2 + 1) of one channel: (Re hi, Im hi, Re lo, Im lo) each; bins past the band are zero
                auto chunk = [&](const uint32_t* o, int k2) {
                    uint32_t w[4];
#pragma unroll
                    for (int z = 0; z < 2; ++z) {
                        const int k = kfe + kP * (k2 + z);
                        const bool in = k <= sigma;
                        const float cr = in ? __ldg(a.scale + k) : 0.f, ci = (in && k >= 1) ? __ldg(a.scale + sigma + k) : 0.f;
                        const float re = cr * __uint_as_float(o[2 * z]), im = ci * __uint_as_float(o[2 * z + 1]);
                        const uint32_t hi = bf16x2_bits(re, im);
                        w[2 * z] = hi;
                        w[2 * z + 1] = bf16x2_bits(re - __uint_as_float(hi << 16), im - __uint_as_float(hi & 0xffff0000u));
                    }
                    return make_uint4(w[0], w[1], w[2], w[3]);
                };
                // All of this thread's result columns at once (UT N2 = 64 in every geometry), then the accumulators are
                // free for the next work item while the values are scaled, split and stored.
                static_assert(G::UT * N2 == 64, "a converter thread owns 64 result columns");
                uint32_t o[4][16];
#pragma unroll
                for (int h = 0; h < 4; ++h) tmem_ld16(lane_addr + (uint32_t)(G::OUT0 + g * 64 + h * 16), o[h]);
#pragma unroll
                for (int h = 0; h < 4; ++h) tmem_ld_wait_for(o[h]);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarOutEmpty));
                if constexpr (QPU == 2) {
                    // unit h: channels 2h, 2h+1 of the thread; column = cc * 8 + k2 * 2 + ri: one K step of four bins
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
#pragma unroll
                        for (int cc = 0; cc < 2; ++cc) {
                            if (ch0 + 2 * h + cc >= D) continue;
                            unsigned char* yc = yb + (size_t)(2 * h + cc) * chan_bytes;
                            *reinterpret_cast<uint4*>(yc) = chunk(o[h] + cc * 8, 0);
                            *reinterpret_cast<uint4*>(yc + 2048) = chunk(o[h] + cc * 8 + 4, 2);
                        }
                    }
                } else {
                    // channel cc of the thread: N2 columns, k2 * 2 + ri: K step s holds bins 4 s .. 4 s + 3
                    const int ks_held = min(a.ks_out, N2 / 8);       // K steps whose bins were accumulated in tensor memory
#pragma unroll
                    for (int cc = 0; cc < W; ++cc) {
#pragma unroll
                        for (int s2 = 0; s2 < N2 / 8; ++s2) {
                            if (s2 >= ks_held || ch0 + cc >= D) continue;
                            const int col = cc * N2 + s2 * 8;        // compile-time after unrolling
                            unsigned char* yc = yb + (size_t)cc * chan_bytes + (size_t)s2 * 4096;
                            *reinterpret_cast<uint4*>(yc) = chunk(o[col / 16] + (col % 16), 4 * s2);
                            *reinterpret_cast<uint4*>(yc + 2048) = chunk(o[col / 16] + (col % 16) + 4, 4 * s2 + 2);
                        }
                    }
                }
                if (EXTRA == 2 && a.extra_in_op) {
                    // one more K step of the operand form: zeros on every lane but TMEM lane 0, whose bin the issuing warp writes
                    if (j != 0) {
#pragma unroll
                        for (int c = 0; c < W; ++c) {
                            if (ch0 + c >= D) continue;
                            unsigned char* yc = yb + (size_t)c * chan_bytes + (size_t)(a.extra_k2 / 4) * 4096;
                            *reinterpret_cast<uint4*>(yc) = make_uint4(0u, 0u, 0u, 0u);
                            *reinterpret_cast<uint4*>(yc + 2048) = make_uint4(0u, 0u, 0u, 0u);
                        }
                    }
                } else if (EXTRA == 1 && a.extra_in_op) {
                    // the extra bin opens one more K step of the operand form: its first bin on the lanes that reach it,
                    // zeros everywhere else
                    const int k = kfe + kP * a.extra_k2;
                    const bool in = k <= sigma;
                    const float cr = in ? __ldg(a.scale + k) : 0.f, ci = in ? __ldg(a.scale + sigma + k) : 0.f;
#pragma unroll
                    for (int c = 0; c < W; ++c) {
                        if (ch0 + c >= D) continue;
                        const float re = cr * extra[c].x, im = ci * extra[c].y;
                        const uint32_t hi = bf16x2_bits(re, im);
                        const uint32_t lo = bf16x2_bits(re - __uint_as_float(hi << 16), im - __uint_as_float(hi & 0xffff0000u));
                        unsigned char* yc = yb + (size_t)c * chan_bytes + (size_t)(a.extra_k2 / 4) * 4096;
                        *reinterpret_cast<uint4*>(yc) = make_uint4(hi, lo, 0u, 0u);
                        *reinterpret_cast<uint4*>(yc + 2048) = make_uint4(0u, 0u, 0u, 0u);
                    }
                }                                        // (EXTRA == 1 always goes into the operand form)
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kConvWarps) tmem_dealloc(tmem, G::TMEM_COLS);
}

// The operand images of one call, as the kernel's shared memory holds them:
//   [0, 64 KB)   stage-1 matrix, hi part then lo part, K-major: element (row j, column p) at
//                (j/8)*128 + (p/8)*2048 + (j%8)*16 + (p%8)*2; rows 0 / 1: A[0] and A[64] (real), rows 2i / 2i+1: Re and Im of A[i]
//   then         the stage-2 matrices [n_groups][hi, lo][16 x N2], K-major [n][k]: element at
//                (n/8)*128 + (k/8)*(N2*16) + (n%8)*16 + (k%8)*2;  k = z*4 + t: complex value z of the unit, t = Re hi,
//                Im hi, Re lo, Im lo (the lo rows of the hi-part matrix repeat the hi rows; the lo-part matrix has zeros
//                there);  n = (channel of the unit, k2, re/im), block-diagonal over the channels of a unit
//   then         e^{-2 pi i m / Q}, m < Q (padded to an even count), and e^{-2 pi i m / N}, m < 128
template <typename G>
__global__ void __launch_bounds__(256) spu_fwd3_img_kernel(unsigned char* __restrict__ img, int Q, int N, int n_groups) {
    constexpr int N2 = G::N2, QPU = G::QPU;
    const int idx = blockIdx.x * 256 + threadIdx.x;
    if (idx < kP * kP) {
        const int j = idx >> 7, p = idx & 127;
        float v;
        if (j == 0) v = 1.f;
        else if (j == 1) v = (p & 1) ? -1.f : 1.f;
        else {
            const int m = ((j >> 1) * p) & 127;
            float s, c;
            sincospif((float)m * (1.0f / 64.0f), &s, &c);
            v = (j & 1) ? -s : c;
        }
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        const int off = (j >> 3) * 128 + (p >> 3) * 2048 + (j & 7) * 16 + (p & 7) * 2;
        *reinterpret_cast<__nv_bfloat16*>(img + off) = h;
        *reinterpret_cast<__nv_bfloat16*>(img + 32768 + off) = __float2bfloat16_rn(v - __bfloat162float(h));
    }
    unsigned char* tabs = img + 65536;
    if (idx < n_groups * 16 * N2) {
        const int grp = idx / (16 * N2), rem = idx - grp * 16 * N2;
        const int n = rem >> 4, k = rem & 15;
        const int z = k >> 2, t = k & 3;
        int qq, zc;
        if constexpr (QPU == 2) { qq = z >> 1; zc = z & 1; } else { qq = z; zc = 0; }
        const int per_ch = N2 / G::CPU_;
        const int nc = n / per_ch, nr = n - nc * per_ch, k2 = nr >> 1, ri = nr & 1;
        const int q = grp * QPU + qq;
        float v = 0.f;
        if (nc == zc && q < Q) {
            const float2 w = root_neg((unsigned)(((long long)q * k2) % Q), (unsigned)Q);    // e^{-2 pi i q k2 / Q}
            // (Re, Im) of B times w: Re out = Re B w.x - Im B w.y, Im out = Re B w.y + Im B w.x
            v = (t & 1) == 0 ? (ri == 0 ? w.x : w.y) : (ri == 0 ? -w.y : w.x);
        }
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        const __nv_bfloat16 l = __float2bfloat16_rn(v - __bfloat162float(h));
        const int off = (n >> 3) * 128 + (k >> 3) * (N2 * 16) + (n & 7) * 16 + (k & 7) * 2;
        unsigned char* base = tabs + (size_t)grp * 2 * G::W_BYTES;
        *reinterpret_cast<__nv_bfloat16*>(base + off) = h;
        *reinterpret_cast<__nv_bfloat16*>(base + G::W_BYTES + off) = t < 2 ? l : __float2bfloat16_rn(0.f);
    }
    float2* roots = reinterpret_cast<float2*>(tabs + (size_t)n_groups * 2 * G::W_BYTES);
    const int q_even = (Q + 1) & ~1;
    if (idx < q_even) roots[idx] = idx < Q ? root_neg((unsigned)idx, (unsigned)Q) : make_float2(0.f, 0.f);
    if (idx < kP) roots[q_even + idx] = root_neg((unsigned)idx, (unsigned)N);
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

template <typename G>
size_t fwd3_smem(int Q) {
    const int tiles = (Q + G::QT - 1) / G::QT, groups = tiles * G::GQ;
    return 1024 + 65536 + (size_t)kStages * G::STAGE_BYTES + (size_t)groups * 2 * G::W_BYTES + (size_t)(((Q + 1) & ~1) + kP) * sizeof(float2) + 4 * 3 * 16 * sizeof(uint32_t);
}

template <typename G, int EXTRA>
cudaError_t launch_fwd3(const Fwd3Args& a, cudaStream_t stream) {
    // the tokens of one sequence as [q][p][channel]: token p Q + q sits 128-strided in memory
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return cudaErrorNotSupported;
    CUtensorMap tmap;
    const cuuint64_t dims[4] = {(cuuint64_t)a.D, (cuuint64_t)kP, (cuuint64_t)a.Q, (cuuint64_t)a.B};
    const cuuint64_t strides[3] = {(cuuint64_t)a.Q * a.D * 2, (cuuint64_t)a.D * 2, (cuuint64_t)a.N * a.D * 2};
    const cuuint32_t box[4] = {(cuuint32_t)G::C, (cuuint32_t)kP, (cuuint32_t)G::QT, 1u};
    const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    const CUtensorMapSwizzle swz = G::C == 32 ? CU_TENSOR_MAP_SWIZZLE_64B
                                 : G::C == 16 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE;
    if (encode(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<__nv_bfloat16*>(a.x), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    {
        const int tiles = (a.Q + G::QT - 1) / G::QT, groups = tiles * G::GQ;
        const int n = kP * kP > groups * 16 * G::N2 ? kP * kP : groups * 16 * G::N2;
        spu_fwd3_img_kernel<G><<<(n + 255) / 256, 256, 0, stream>>>(const_cast<unsigned char*>(a.img), a.Q, a.N, groups);
    }
    const size_t smem = fwd3_smem<G>(a.Q);
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    cudaFuncSetAttribute(spu_fwd3_kernel<G, EXTRA>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    const int grid = a.n_items < sms ? a.n_items : sms;
    spu_fwd3_kernel<G, EXTRA><<<grid, kThreads, smem, stream>>>(tmap, a);
    return cudaGetLastError();
}

using GeoNarrow = Geo<32, 16, 2, 1>;     // up to 4 bins per frequency class; 64-byte token rows keep TMA at full rate
using GeoMid = Geo<16, 16, 4, 1>;        // up to 8 bins per frequency class; 32-byte token rows
using GeoWide = Geo<8, 32, 4, 1>;        // up to 16 bins per frequency class (per slice); 16-byte token rows cap the TMA feed
                                         // near 1.5 TB/s, which is why the middle geometry exists

}  // namespace

SpuFwd3Plan spu_fwd3_plan(int B, int N, int D, int sigma) {
    SpuFwd3Plan pl = {};
    if (N % kP != 0) return pl;
    pl.Q = N / kP;
    if (pl.Q < 8 || pl.Q > 128) return pl;           // the stage-2 matrices of a whole sequence stay in shared memory
    const int nk2 = sigma / kP + 1;                  // values of k2 that reach into the band
    // geometry: 0 narrow, 1 middle, 2 wide; one value of k2 more than the geometry holds is still one pass: the few lanes
    // that reach it (k1 <= sigma - 128 k2max) keep that bin in registers
    pl.geo = nk2 <= GeoNarrow::K2MAX ? 0 : (nk2 <= GeoMid::K2MAX + 1 ? 1 : 2);
    pl.wide = pl.geo != 0;
    const int k2max = pl.geo == 0 ? GeoNarrow::K2MAX : (pl.geo == 1 ? GeoMid::K2MAX : GeoWide::K2MAX);
    pl.slices = (nk2 + k2max - 1) / k2max;
    pl.extra_k2 = 0;
    if (pl.geo != 0 && nk2 == k2max + 1) {
        pl.slices = 1;
        pl.extra_k2 = k2max;
    }
    pl.C = pl.geo == 0 ? GeoNarrow::C : (pl.geo == 1 ? GeoMid::C : GeoWide::C);
    pl.n_ctiles = (D + pl.C - 1) / pl.C;
    const long long items = (long long)B * pl.n_ctiles * pl.slices;
    if (items > 0x7fffffffll) return pl;
    pl.n_items = (int)items;
    const size_t smem = pl.geo == 0 ? fwd3_smem<GeoNarrow>(pl.Q) : (pl.geo == 1 ? fwd3_smem<GeoMid>(pl.Q) : fwd3_smem<GeoWide>(pl.Q));
    if (smem > 220 * 1024) return pl;
    pl.ok = 1;
    return pl;
}

int spu_fwd3_run(const void* hidden, void* yop, int ks_out, float* yx, const float* scale, int B, int N, int D, int sigma,
                 int* status, cudaStream_t stream, void* img) {
    const SpuFwd3Plan pl = spu_fwd3_plan(B, N, D, sigma);
    if (!pl.ok) return LUVC_ERR_INTERNAL;
    Fwd3Args a;
    a.x = reinterpret_cast<const __nv_bfloat16*>(hidden);
    const int k2max = pl.geo == 0 ? GeoNarrow::K2MAX : (pl.geo == 1 ? GeoMid::K2MAX : GeoWide::K2MAX);
    // the extra bin of the middle geometry becomes one more K step of the operand form; that of the wide one goes to yx
    a.extra_in_op = (pl.extra_k2 && ks_out * 4 > k2max) ? 1 : 0;
    if (pl.slices != 1 || ks_out * 4 > k2max + (a.extra_in_op ? 4 : 0)) return LUVC_ERR_INTERNAL;
    if (pl.extra_k2 && !a.extra_in_op && sigma != kP * pl.extra_k2) return LUVC_ERR_INTERNAL;   // yx holds the bin of k1 = 0 only
    a.yop = static_cast<unsigned char*>(yop); a.yx = yx; a.ks_out = ks_out; a.scale = scale; a.status = status;
    a.B = B; a.N = N; a.D = D; a.Q = pl.Q; a.sigma = sigma;
    a.n_ctiles = pl.n_ctiles; a.n_slices = pl.slices; a.n_items = pl.n_items;
    a.extra_k2 = pl.extra_k2;
    // only k1 = 0 reaches the extra bin (sigma = 128 extra_k2): the stage-2 issuing warps form it from the lane-0 values
    // the converters leave in shared memory; else the converter warps that reach it accumulate it
    const int xm = !pl.extra_k2 ? 0 : (sigma == kP * pl.extra_k2 ? 2 : 1);
    a.img = static_cast<const unsigned char*>(img);
    cudaError_t err;
    if (pl.geo == 0) err = launch_fwd3<GeoNarrow, 0>(a, stream);
    else if (pl.geo == 1) err = xm == 0 ? launch_fwd3<GeoMid, 0>(a, stream) : (xm == 1 ? launch_fwd3<GeoMid, 1>(a, stream) : launch_fwd3<GeoMid, 2>(a, stream));
    else if (xm == 1) return LUVC_ERR_INTERNAL;      // a 17th bin that several frequency classes reach: not planned (spu_inv3_plan)
    else err = xm == 0 ? launch_fwd3<GeoWide, 0>(a, stream) : launch_fwd3<GeoWide, 2>(a, stream);
    count_launch(2);
    return err == cudaSuccess ? LUVC_OK : LUVC_ERR_CUDA;
}

}  // namespace luvc
