// Two-stage inverse transform and energy of the Spectrum Pruning Unit (Eq. 7 and Eq. 8) for the
// bf16 path, the mirror image of spu_fwd2.cu.
//
// The filtered signal x'(t) = sum_{k=0..sigma} Re(Y_k e^{2 pi i k t / N}) (Y already carries the
// mask of Eq. 5/6, 1/N and the weight of the conjugate half) is evaluated on the L = P * J
// uniform points t = p Q + jj Q / J of the period (J = Q: the tokens themselves; J < Q: the coarse
// grid from which the squared energies are interpolated).  With k = k1 + P k2:
//   stage 2'  C_jj[k1] = e^{2 pi i k1 jj / L} sum_{k2} Y_{k1 + P k2} e^{2 pi i k2 jj / J}     CUDA cores
//   stage 1'  x'[p, jj] = sum_{k1 < P} Re(e^{2 pi i k1 p / P} C_jj[k1])
//                       = sum_r F[r][p] G_jj[r],  the real P x P matrix of the forward kernel with
//             G[0] = Re C[0], G[1] = Re C[P/2], G[2i] = Re C[i] + Re C[P-i], G[2i+1] = Im C[i] - Im C[P-i]
//             one tcgen05 contraction per tile: A = F transposed (bf16 pair, built once per CTA),
//             B = G for a tile of 64 columns (points x channels), written to shared memory as a bf16
//             pair by the threads that computed it (three products: hi*hi, hi*lo, lo*hi); B and the
//             accumulator are double buffered, so the MMAs of a tile run under the arithmetic of the next
//   energy    S[p J + jj] = sum over the tile's channels of x'^2, read back from TMEM.
// As in the forward kernel the even lane of a pair owns the frequency k1 = i and row 2i, the odd lane
// P - i and row 2i + 1 (they swap one value per column to form G), each keeps its band bins
// Y_{k + P k2} of its warp's channels in registers for the whole work item (sequence x channel tile),
// and P <= 64 puts 128 / P channel blocks on the diagonal of the 128-row operand.  Every mbarrier
// wait is bounded.

#include <cuda_bf16.h>

#include "luvc_internal.h"
#include "sm100_ptx.cuh"
#include "spu_images.cuh"

namespace luvc {
namespace {

using namespace ptx;

constexpr int kWarps = 16;
constexpr int kThreads = kWarps * 32;
// Columns of a tile (TJ points x C channels) are a template parameter NC: 64, or 128 for the few-bin variants, whose
// tiles are short on arithmetic and long on hand-overs (two accumulator buffers of NC columns in tensor memory).
constexpr int kSpin = 1 << 22;

struct InvArgs {
    const float* Y;      // [B][R][D]
    float* part;         // [B][n_parts][L]
    int* status;
    int B, N, D, P, Q, sigma, R, nblk, J, L;
    int n_ctiles, n_items;
    const unsigned char* img;   // stage-1 matrix (both parts) and the table of e^{2 pi i k2 jj / J}, in their
                                // shared-memory layouts, built once per call
};

enum { kBarReady = 0, kBarAccFull = 2, kBarImg = 4, kBars = 5 };

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
// e^{+2 pi i num / den}, 0 <= num < den
__device__ __forceinline__ float2 root_pos(unsigned num, unsigned den) {
    float s, c;
    sincospif(2.0f * (float)num / (float)den, &s, &c);
    return make_float2(c, s);
}

__device__ __forceinline__ uint32_t pack_bf16(__nv_bfloat16 a, __nv_bfloat16 b) {
    return (uint32_t)__bfloat16_as_ushort(a) | ((uint32_t)__bfloat16_as_ushort(b) << 16);
}

// NV bf16 values (NV / 2 packed words) to shared memory
template <int NV> __device__ __forceinline__ void store_bf16(unsigned char* dst, const uint32_t (&v)[NV / 2]) {
    if constexpr (NV == 8) *reinterpret_cast<uint4*>(dst) = make_uint4(v[0], v[1], v[2], v[3]);
    else if constexpr (NV == 4) *reinterpret_cast<uint2*>(dst) = make_uint2(v[0], v[1]);
    else *reinterpret_cast<uint32_t*>(dst) = v[0];
}

// Row `row` of G for the tile's points and this thread's W channels, as a bf16 pair into the B tile.
// NB bins of this lane's frequency are summed (compile time).  G = ga C.x + gb C.y + gc (partner's value).
template <int KB, int W, int NB, int NC>
__device__ __forceinline__ void stage2_tile(const float2 (&y)[KB][W], const float4* __restrict__ w_tab, int jj0, int J,
                                            float2 rot, float2 step, float ga, float gb, float gc, bool odd,
                                            unsigned char* b_hi, unsigned char* b_lo, int sbo, int row, int col0) {
    constexpr int C = 4 * W, TJ = NC / C;
    constexpr int HV = W >= 8 ? 8 : W;        // bf16 values per store
#pragma unroll 1
    for (int jl = 0; jl < TJ; ++jl) {
        const int jj = jj0 + jl;
        float g[W];
        if (jj < J) {
            const float2 rxx = make_float2(rot.x, rot.x), ryy = make_float2(-rot.y, rot.y);
            // s = sum_t y_t w_t with packed FMAs and no operand swaps: sa += (w.x, w.x) * (y.x, y.y),
            // sb += (w.y, w.y) * (y.x, y.y); then s = (sa.x - sb.y, sa.y + sb.x)
            float2 s[W];
            if constexpr (NB <= 6) {            // few bins: the table row stays in registers across the channels
                float4 tw[NB];
#pragma unroll
                for (int t = 0; t < NB; ++t) tw[t] = w_tab[jj * KB + t];
#pragma unroll
                for (int c = 0; c < W; ++c) {
                    float2 sa = make_float2(0.f, 0.f), sb = make_float2(0.f, 0.f);
#pragma unroll
                    for (int t = 0; t < NB; ++t) {
                        sa = __ffma2_rn(make_float2(tw[t].x, tw[t].y), y[t][c], sa);
                        sb = __ffma2_rn(make_float2(tw[t].z, tw[t].w), y[t][c], sb);
                    }
                    s[c] = make_float2(sa.x - sb.y, sa.y + sb.x);
                }
            } else {                            // many bins, few channels: the table streams
                float2 sa[W], sb[W];
#pragma unroll
                for (int c = 0; c < W; ++c) sa[c] = sb[c] = make_float2(0.f, 0.f);
#pragma unroll
                for (int t = 0; t < NB; ++t) {
                    const float4 tw = w_tab[jj * KB + t];
#pragma unroll
                    for (int c = 0; c < W; ++c) {
                        sa[c] = __ffma2_rn(make_float2(tw.x, tw.y), y[t][c], sa[c]);
                        sb[c] = __ffma2_rn(make_float2(tw.z, tw.w), y[t][c], sb[c]);
                    }
                }
#pragma unroll
                for (int c = 0; c < W; ++c) s[c] = make_float2(sa[c].x - sb[c].y, sa[c].y + sb[c].x);
            }
#pragma unroll
            for (int c = 0; c < W; ++c) {
                const float2 cv = __ffma2_rn(rxx, s[c], __fmul2_rn(ryy, make_float2(s[c].y, s[c].x)));   // C = rot * s
                const float got = __shfl_xor_sync(0xffffffffu, odd ? cv.x : cv.y, 1);
                g[c] = fmaf(ga, cv.x, fmaf(gb, cv.y, gc * got));
            }
            rot = cmul(rot, step);
        } else {
#pragma unroll
            for (int c = 0; c < W; ++c) g[c] = 0.f;
        }
        if (row < 0) continue;                 // a lane past the rows in use only takes part in the exchange
        // element (K row r, column n) of a part sits at (n/8) sbo + (r/8) 128 + (r%8) 16 + (n%8) 2
        const int n = jl * C + col0;
        const int off = (n >> 3) * sbo + (n & 7) * 2 + (row >> 3) * 128 + (row & 7) * 16;
#pragma unroll
        for (int h = 0; h < W / HV; ++h) {     // W = 16: two column groups
            uint32_t hv[HV / 2], lv[HV / 2];
#pragma unroll
            for (int c = 0; c < HV; c += 2) {
                const float x0 = g[h * HV + c], x1 = g[h * HV + c + 1];
                const __nv_bfloat16 a0 = __float2bfloat16_rn(x0), a1 = __float2bfloat16_rn(x1);
                hv[c / 2] = pack_bf16(a0, a1);
                lv[c / 2] = pack_bf16(__float2bfloat16_rn(x0 - __bfloat162float(a0)),
                                      __float2bfloat16_rn(x1 - __bfloat162float(a1)));
            }
            store_bf16<HV>(b_hi + off + h * sbo, hv);
            store_bf16<HV>(b_lo + off + h * sbo, lv);
        }
    }
}

// The same for few bins per lane (KB <= 4): the lane carries g[t] = e^{2 pi i jj k_t / L} of each of its bins from
// point to point (k_t = its frequency + P t; times i on the odd lane of a pair, so that its own share of G is the real
// part of C = sum_t Y_t g[t] and the partner's share the imaginary part), which replaces both the table of
// e^{2 pi i k2 jj / J} and the rotation by e^{2 pi i k1 jj / L}.  G = Re C + gc (partner's Im C).
template <int KB, int W, int NB, int NC>
__device__ __forceinline__ void stage2_tile_few(const float2 (&y)[KB][W], float2 (&g)[KB], const float2 (&gstep)[KB], int jj0, int J,
                                                float gc, unsigned char* b_hi, unsigned char* b_lo, int sbo, int row, int col0) {
    constexpr int C = 4 * W, TJ = NC / C;
    constexpr int HV = W >= 8 ? 8 : W;        // bf16 values per store
#pragma unroll 1
    for (int jl = 0; jl < TJ; ++jl) {
        const int jj = jj0 + jl;
        float gv[W];
        if (jj < J) {
            float2 gx[NB], gy[NB];
#pragma unroll
            for (int t = 0; t < NB; ++t) { gx[t] = make_float2(g[t].x, g[t].x); gy[t] = make_float2(g[t].y, g[t].y); }
#pragma unroll
            for (int c = 0; c < W; ++c) {
                float2 sa = make_float2(0.f, 0.f), sb = make_float2(0.f, 0.f);
#pragma unroll
                for (int t = 0; t < NB; ++t) {
                    sa = __ffma2_rn(gx[t], y[t][c], sa);
                    sb = __ffma2_rn(gy[t], y[t][c], sb);
                }
                const float cx = sa.x - sb.y, cy = sa.y + sb.x;
                gv[c] = fmaf(gc, __shfl_xor_sync(0xffffffffu, cy, 1), cx);
            }
        } else {
#pragma unroll
            for (int c = 0; c < W; ++c) gv[c] = 0.f;
        }
#pragma unroll
        for (int t = 0; t < KB; ++t) g[t] = cmul(g[t], gstep[t]);
        if (row < 0) continue;                 // a lane past the rows in use only takes part in the exchange
        const int n = jl * C + col0;
        const int off = (n >> 3) * sbo + (n & 7) * 2 + (row >> 3) * 128 + (row & 7) * 16;
#pragma unroll
        for (int h = 0; h < W / HV; ++h) {
            uint32_t hv[HV / 2], lv[HV / 2];
#pragma unroll
            for (int c = 0; c < HV; c += 2) {
                const float x0 = gv[h * HV + c], x1 = gv[h * HV + c + 1];
                const __nv_bfloat16 a0 = __float2bfloat16_rn(x0), a1 = __float2bfloat16_rn(x1);
                hv[c / 2] = pack_bf16(a0, a1);
                lv[c / 2] = pack_bf16(__float2bfloat16_rn(x0 - __bfloat162float(a0)),
                                      __float2bfloat16_rn(x1 - __bfloat162float(a1)));
            }
            store_bf16<HV>(b_hi + off + h * sbo, hv);
            store_bf16<HV>(b_lo + off + h * sbo, lv);
        }
    }
}

// KB: band bins per lane; W: channels per thread (C = 4 W per channel block, TJ = 64 / C points per tile).
template <int KB, int W, int NC>
__global__ void __launch_bounds__(kThreads, 1) spu_inv2_kernel(const InvArgs a) {
    constexpr int C = 4 * W, TJ = NC / C;
    constexpr int kNcol = NC, kTmemCols = 2 * NC;
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) unsigned long long s_bar[kBars];
    __shared__ uint32_t s_tmem;
    __shared__ int s_fail;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int P = a.P, D = a.D, sigma = a.sigma, J = a.J, L = a.L;
    const int KT = a.nblk * P;                   // rows in use = K extent of the contraction
    const int f_bytes = KT * 256;                // one part of A: KT / 8 K chunks x 128 rows x 16 B
    const int sbo = KT * 16;                     // B: distance between 8-column groups (KT / 8 K groups x 128 B)
    const int b_part = (NC / 8) * sbo, b_buf = 2 * b_part;
    unsigned char* s_fhi = smem;
    unsigned char* s_flo = smem + f_bytes;
    unsigned char* s_b = smem + 2 * f_bytes;     // [2 buffers][hi, lo][8 column groups][KT / 8][128 B]
    float4* s_w = reinterpret_cast<float4*>(s_b + 2 * b_buf);   // [J][KB]: w = e^{2 pi i k2 jj / J} as (w.x, w.x, w.y, w.y)
    const uint32_t bar0 = smem_u32(&s_bar[0]);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    if (tid == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kBarReady + s), kWarps);
            mbar_init(bar(kBarAccFull + s), 1);
        }
        mbar_init(bar(kBarImg), 1);
        s_fail = 0;
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc(smem_u32(&s_tmem), kTmemCols);

    // the operand matrix (both parts) and the table of e^{2 pi i k2 jj / J} were built once per call in global
    // memory in the layouts used here: two bulk copies fetch them (the table sits behind the two B buffers)
    const int w_bytes = J * KB * (int)sizeof(float4);
    if (tid == 0) {
        mbar_arrive_expect_tx(bar(kBarImg), (uint32_t)(2 * f_bytes + w_bytes));
        bulk_load(smem_u32(s_fhi), a.img, (uint32_t)(2 * f_bytes), bar(kBarImg));
        bulk_load(smem_u32(s_w), a.img + 2 * f_bytes, (uint32_t)w_bytes, bar(kBarImg));
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    volatile int* fail = &s_fail;
    if (!__all_sync(0xffffffffu, wait_bar(bar(kBarImg), 0, fail, a.status))) {     // matrix and table have landed
        __syncthreads();
        if (warp == 0) tmem_dealloc(tmem, kTmemCols);
        return;
    }

    const int warp_u = __shfl_sync(0xffffffffu, warp, 0);   // the same in every lane, and the compiler can tell
    const int quarter = warp & 3, grp = warp >> 2;
    const int j = quarter * 32 + lane;               // row (channel block jb, r) of G; row (jb, point p) of the result
    const int jb = j / P, jr = j - jb * P;
    const bool active = j < KT, warp_active = quarter * 32 < KT;
    const int i = jr >> 1;
    const bool odd = jr & 1, special = i == 0;
    const int kf = special ? (odd ? P / 2 : 0) : (odd ? P - i : i);       // this lane's frequency
    const float ga = (odd && !special) ? 0.f : 1.f, gb = (odd && !special) ? -1.f : 0.f, gc = special ? 0.f : 1.f;
    const int tiles_per_item = (J + TJ - 1) / TJ;
    const int item_channels = a.nblk * C;
    const float2 step = root_pos((unsigned)kf % (unsigned)L, L);
    constexpr bool kFew = KB <= 4;               // few bins: the per-bin factors are carried in registers
    float2 gk[KB], gstep[KB];
#pragma unroll
    for (int q = 0; q < KB; ++q) {
        gk[q] = make_float2(1.f, 0.f);
        gstep[q] = kFew ? root_pos((unsigned)((kf + P * q) % L), L) : make_float2(1.f, 0.f);
    }
    const uint32_t idesc = make_idesc_bf16(128, kNcol, false, true);
    const uint64_t a_hi0 = make_desc(smem_u32(s_fhi), 2048, 128), a_lo0 = make_desc(smem_u32(s_flo), 2048, 128);
    const uint64_t b_d0 = make_desc(smem_u32(s_b), 128, sbo);

    // energies of tile `t` (accumulator t & 1) of the item (b, ctile), points jj0 ..: the warp of channel
    // group grp reads the 16 columns [16 grp, 16 grp + 16) of its rows with ONE TMEM load (a load's round
    // trip is long, so the 64 columns are spread over the four warps that share the lanes):
    //   C = 64: the point's channel quarter grp;  C = 32: point grp / 2, channel half grp % 2
    //   C = 16: point grp;                         C = 8: points 2 grp and 2 grp + 1
    constexpr int SPLIT = C == 64 ? 4 : (C == 32 ? 2 : 1);          // partial sums per (channel block, point)
    auto read_tile = [&](int t, int b, int ctile, int jj_first) {
#pragma unroll
        for (int hf = 0; hf < NC / 64; ++hf) {               // each 64 columns of the tile as above
            const int jj0 = jj_first + hf * (64 / C);
            const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)((t & 1) * kNcol + hf * 64 + grp * 16);
            uint32_t v[16];
            tmem_ld16(taddr, v);
            tmem_ld_wait_for(v);
            if (!active) continue;
            const int sub = C == 64 ? grp : (C == 32 ? (grp & 1) : 0);
            float* out = a.part + ((size_t)b * (a.n_ctiles * a.nblk * SPLIT) + (ctile * a.nblk + jb) * SPLIT + sub) * L +
                         (size_t)jr * J;
            constexpr int PTS = C >= 16 ? 1 : 2;          // points among the 16 columns
            constexpr int WP = 16 / PTS;                  // columns per point
#pragma unroll
            for (int pt = 0; pt < PTS; ++pt) {
                float sum = 0.f;
#pragma unroll
                for (int q = 0; q < WP; ++q) { const float x = __uint_as_float(v[pt * WP + q]); sum = fmaf(x, x, sum); }
                const int jl = C == 64 ? 0 : (C == 32 ? (grp >> 1) : (C == 16 ? grp : 2 * grp + pt));
                if (jj0 + jl < J) out[jj0 + jl] = sum;
            }
        }
        tc_fence_before();
    };

    int t = 0;                                       // tiles issued so far by this CTA
    int pb = 0, pct = 0, pj0 = 0;                    // item and first point of tile t - 1
    bool ok = true;
    for (int item = blockIdx.x; item < a.n_items && ok; item += gridDim.x) {
        const int ctile = item % a.n_ctiles, b = item / a.n_ctiles;
        const int ch0 = ctile * item_channels + jb * C + grp * W;
        // band bins of this lane: Y_k = (cos row k) + i (sin row sigma + k), k = kf + P t
        float2 y[KB][W];
        const int nb = (active && kf <= sigma) ? min(KB, (sigma - kf) / P + 1) : 0;
        const float* Yb = a.Y + (size_t)b * a.R * D + ch0;
        constexpr int VEC = W >= 4 ? 4 : 2;
#pragma unroll
        for (int q = 0; q < KB; ++q) {
            const int k = kf + P * q;
            const float* yc = Yb + (size_t)k * D;
            const float* ys = Yb + (size_t)(sigma + k) * D;
#pragma unroll
            for (int c = 0; c < W; c += VEC) {
                float vc[4] = {0.f, 0.f, 0.f, 0.f}, vs[4] = {0.f, 0.f, 0.f, 0.f};
                if (q < nb && ch0 + c < D) {          // D is a multiple of 8, ch0 + c of VEC: the vector is whole or absent
                    if constexpr (VEC == 4) {
                        const float4 t4 = __ldg(reinterpret_cast<const float4*>(yc + c));
                        vc[0] = t4.x; vc[1] = t4.y; vc[2] = t4.z; vc[3] = t4.w;
                        if (k >= 1) {
                            const float4 u4 = __ldg(reinterpret_cast<const float4*>(ys + c));
                            vs[0] = u4.x; vs[1] = u4.y; vs[2] = u4.z; vs[3] = u4.w;
                        }
                    } else {
                        const float2 t2 = __ldg(reinterpret_cast<const float2*>(yc + c));
                        vc[0] = t2.x; vc[1] = t2.y;
                        if (k >= 1) {
                            const float2 u2 = __ldg(reinterpret_cast<const float2*>(ys + c));
                            vs[0] = u2.x; vs[1] = u2.y;
                        }
                    }
                }
#pragma unroll
                for (int e = 0; e < VEC; ++e) y[q][c + e] = make_float2(vc[e], vs[e]);
            }
        }
        const int nb_w = __reduce_max_sync(0xffffffffu, nb);

        for (int tile = 0; tile < tiles_per_item; ++tile, ++t) {
            const int jj0 = tile * TJ;
            // buffer t & 1 of B is free: every warp has seen the MMAs of tile t - 2 finish (below, one tile ago)
            if (kFew && warp_active) {
                if ((tile & 15) == 0) {         // exact restart of the carried factors; in between they are advanced point by point
#pragma unroll
                    for (int q = 0; q < KB; ++q) {
                        const unsigned long long m = (unsigned long long)jj0 * (unsigned)(kf + P * q);
                        gk[q] = root_pos((unsigned)(m % (unsigned)L), L);
                        if (odd && !special) gk[q] = make_float2(-gk[q].y, gk[q].x);      // times i
                    }
                }
                unsigned char* bh = s_b + (t & 1) * b_buf;
                unsigned char* bl = bh + b_part;
                const int col0 = grp * W;
                if (nb_w == KB)
                    stage2_tile_few<KB, W, KB, NC>(y, gk, gstep, jj0, J, gc, bh, bl, sbo, active ? j : -1, col0);
                else if (nb_w == KB - 1 || KB == 2)
                    stage2_tile_few<KB, W, (KB > 1 ? KB - 1 : 1), NC>(y, gk, gstep, jj0, J, gc, bh, bl, sbo, active ? j : -1, col0);
                else
                    stage2_tile_few<KB, W, (KB >= 4 ? KB / 2 : KB), NC>(y, gk, gstep, jj0, J, gc, bh, bl, sbo, active ? j : -1, col0);
            } else if (warp_active) {
                const float2 rot = root_pos(((unsigned)kf * (unsigned)jj0) % (unsigned)L, L);   // kf jj0 < P J = L
                unsigned char* bh = s_b + (t & 1) * b_buf;
                unsigned char* bl = bh + b_part;
                const int col0 = grp * W;
                // lanes past the rows in use take part in the exchange with zeros and store nothing
                if (nb_w == KB)
                    stage2_tile<KB, W, KB, NC>(y, s_w, jj0, J, rot, step, ga, gb, gc, odd, bh, bl, sbo, active ? j : -1, col0);
                else if (nb_w == KB - 1 || KB == 2)
                    stage2_tile<KB, W, (KB > 1 ? KB - 1 : 1), NC>(y, s_w, jj0, J, rot, step, ga, gb, gc, odd, bh, bl, sbo, active ? j : -1, col0);
                else if (KB >= 4 && nb_w <= KB / 2)
                    stage2_tile<KB, W, (KB >= 4 ? KB / 2 : KB), NC>(y, s_w, jj0, J, rot, step, ga, gb, gc, odd, bh, bl, sbo, active ? j : -1, col0);
                else
                    stage2_tile<KB, W, KB, NC>(y, s_w, jj0, J, rot, step, ga, gb, gc, odd, bh, bl, sbo, active ? j : -1, col0);
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarReady + (t & 1)));
            if (warp_u == 0) {
                // every warp has written its share of B (and, before that, read the last of accumulator
                // t & 1, which held tile t - 2): run the three products.  The whole warp waits and one
                // elected lane issues, in warp-uniform code, so that the descriptors stay in uniform
                // registers (a tcgen05.mma issued from divergent code costs its thread twice as long).
                ok = __all_sync(0xffffffffu, wait_bar(bar(kBarReady + (t & 1)), (t >> 1) & 1, fail, a.status));
                if (ok && elect_one()) {
                    tc_fence_after();
                    const uint32_t acc = tmem + (uint32_t)((t & 1) * kNcol);
                    uint64_t ah = a_hi0, al = a_lo0;             // advance by adding to the address field
                    uint64_t bh_d = b_d0 + (uint64_t)(((t & 1) * b_buf) >> 4), bl_d = bh_d + (uint64_t)(b_part >> 4);
                    for (int ks = 0; ks < KT / 16; ++ks) {
                        umma_bf16(acc, ah, bh_d, idesc, ks ? 1u : 0u);
                        umma_bf16(acc, ah, bl_d, idesc, 1u);
                        umma_bf16(acc, al, bh_d, idesc, 1u);
                        ah += 4096 >> 4; al += 4096 >> 4; bh_d += 256 >> 4; bl_d += 256 >> 4;
                    }
                    umma_commit(bar(kBarAccFull + (t & 1)));
                }
                __syncwarp();
            }
            // meanwhile: the energies of the previous tile, whose MMAs ran under the arithmetic above
            if (t >= 1) ok = wait_bar(bar(kBarAccFull + ((t - 1) & 1)), ((t - 1) >> 1) & 1, fail, a.status) && ok;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (t >= 1) {
                tc_fence_after();
                read_tile(t - 1, pb, pct, pj0);
            }
            pb = b; pct = ctile; pj0 = jj0;
        }
    }
    if (ok && t >= 1) {
        ok = wait_bar(bar(kBarAccFull + ((t - 1) & 1)), ((t - 1) >> 1) & 1, fail, a.status);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            tc_fence_after();
            read_tile(t - 1, pb, pct, pj0);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// The operand image and the table of e^{2 pi i k2 jj / J} (spu_images.cuh), built once per call.
__global__ void __launch_bounds__(256) spu_inv2_img_kernel(unsigned char* __restrict__ img, int P, int KT, int J, int KB) {
    spu_inv2_img_element(img, P, KT, J, KB, blockIdx.x * 256 + threadIdx.x);
}

template <int KB, int W, int NC = 64>
cudaError_t launch_inv2(const InvArgs& a, cudaStream_t stream) {
    const int KT = a.nblk * a.P;
    const size_t smem = (size_t)2 * KT * 256 + (size_t)(NC / 32) * KT * 256 + (size_t)a.J * KB * sizeof(float4);
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    cudaFuncSetAttribute(spu_inv2_kernel<KB, W, NC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    const int grid = a.n_items < sms ? a.n_items : sms;
    spu_inv2_kernel<KB, W, NC><<<grid, kThreads, smem, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace

SpuInv2Plan spu_inv2_plan(int B, int N, int D, int sigma) {
    SpuInv2Plan pl = {};
    const SpuFwd2Plan f = spu_fwd2_plan(B, N, D, sigma);
    if (!f.ok) return pl;
    pl.P = f.P; pl.Q = f.Q; pl.nblk = f.nblk;
    // points of the period: J per block of Q tokens, L = P J > 4 sigma (see spu_tc_plan), if that saves a quarter
    const long long need = 4ll * sigma + 2;
    const long long jc = (need + pl.P - 1) / pl.P;
    pl.coarse = (jc * pl.P * 4 <= 3ll * N) ? 1 : 0;
    pl.J = pl.coarse ? (int)jc : pl.Q;
    pl.L = pl.P * pl.J;
    const int nk2 = sigma / pl.P + 1;
    // (up to two bins per class: the four-bin variant when the wide channel tiles of the two-bin variant would leave
    // most SMs without a work item)
    if (nk2 <= 2 && (long long)B * ((D + 64 * pl.nblk - 1) / (64 * pl.nblk)) > 74) { pl.KB = 2; pl.CHT = 16; }
    else if (nk2 <= 4) { pl.KB = 4; pl.CHT = 8; }
    else if (nk2 <= 9) { pl.KB = 9; pl.CHT = 4; }
    else if (nk2 <= 17) { pl.KB = 17; pl.CHT = 2; }
    else return pl;
    if ((size_t)pl.J * pl.KB * sizeof(float4) > 24 * 1024) return pl;
    const int C = 4 * pl.CHT;                          // channels of one block
    pl.n_ctiles = (D + C * pl.nblk - 1) / (C * pl.nblk);
    const long long items = (long long)B * pl.n_ctiles;
    if (items > 0x7fffffffll) return pl;
    pl.n_items = (int)items;
    pl.n_parts = pl.n_ctiles * pl.nblk * (C == 64 ? 4 : (C == 32 ? 2 : 1));
    pl.ok = 1;
    return pl;
}

int spu_inv2_run(const float* Y, float* part, int B, int N, int D, int sigma, int* status, cudaStream_t stream, void* img,
                 bool img_ready) {
    const SpuInv2Plan pl = spu_inv2_plan(B, N, D, sigma);
    if (!pl.ok) return LUVC_ERR_INTERNAL;
    if (!img_ready) {
        const int KT = pl.nblk * pl.P, n = 128 * KT > pl.J * pl.KB ? 128 * KT : pl.J * pl.KB;
        spu_inv2_img_kernel<<<(n + 255) / 256, 256, 0, stream>>>(static_cast<unsigned char*>(img), pl.P, KT, pl.J, pl.KB);
        count_launch();
    }
    InvArgs a;
    a.img = static_cast<const unsigned char*>(img);
    a.Y = Y; a.part = part; a.status = status;
    a.B = B; a.N = N; a.D = D; a.P = pl.P; a.Q = pl.Q; a.sigma = sigma; a.R = 2 * sigma + 1;
    a.nblk = pl.nblk; a.J = pl.J; a.L = pl.L; a.n_ctiles = pl.n_ctiles; a.n_items = pl.n_items;
    cudaError_t err;
    if (pl.KB == 2) err = launch_inv2<2, 16, 128>(a, stream);
    else if (pl.KB == 4) err = launch_inv2<4, 8, 128>(a, stream);
    else if (pl.KB == 9) err = launch_inv2<9, 4>(a, stream);
    else err = launch_inv2<17, 2>(a, stream);
    count_launch();
    return err == cudaSuccess ? LUVC_OK : LUVC_ERR_CUDA;
}

}  // namespace luvc
