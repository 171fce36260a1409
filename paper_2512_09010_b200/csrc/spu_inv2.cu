// Two-stage inverse transform and energy of the Spectrum Pruning Unit (Eq. 7 and Eq. 8) for the
// bf16 path, the mirror image of spu_fwd2.cu.
//
// The filtered signal x'(t) = sum_{k=0..sigma} Re(Y_k e^{2 pi i k t / N}) (Y already carries the
// mask of Eq. 5/6, 1/N and the weight of the conjugate half) is evaluated on the L = P * J
// uniform points t = p Q + jj Q / J of the period (J = Q: the tokens themselves; J < Q: the coarse
// grid from which the squared energies are interpolated).  With k = k1 + P k2:
//   stage 2'  C_jj[k1] = e^{2 pi i k1 jj / L} sum_{k2} Y_{k1 + P k2} e^{2 pi i k2 jj / J}     CUDA cores
//   stage 1'  x'[p, jj] = sum_{k1} cos(2 pi k1 p / P) Re C_jj[k1] - sin(2 pi k1 p / P) Im C_jj[k1]
//             one tcgen05 contraction per tile: A = [cos | -sin] (128 x 2P, bf16 pair, built once per
//             CTA), B = [Re C ; Im C] for a tile of 64 columns (points x channels), written to shared
//             memory as a bf16 pair by the threads that computed it (three products: hi*hi, hi*lo, lo*hi)
//   energy    S[p J + jj] += sum over the tile's channels of x'^2, read back from TMEM.
// The thread that owns row k1 keeps the band bins Y_{k1 + P k2} of its channels in registers for
// the whole work item (sequence x channel tile).  As in the forward kernel, P <= 64 puts 128 / P
// channel blocks on the diagonal of the 128-row operand.  Every mbarrier wait is bounded.

#include <cuda_bf16.h>

#include "luvc_internal.h"
#include "sm100_ptx.cuh"

namespace luvc {
namespace {

using namespace ptx;

constexpr int kWarps = 16;
constexpr int kThreads = kWarps * 32;
constexpr int kNcol = 64;                     // columns of a tile: TJ points x C channels
constexpr int kTmemCols = 128;                // two accumulator buffers
constexpr int kBSbo = 4096;                   // distance between 8-column groups of the B tile (32 K groups x 128 B)
constexpr int kBPart = 8 * kBSbo;             // one part (hi or lo) of the B tile
constexpr int kSpin = 1 << 22;

struct InvArgs {
    const float* Y;      // [B][R][D]
    float* part;         // [B][n_ctiles * nblk * (2 if C = 32)][L]
    int* status;
    int B, N, D, P, Q, sigma, R, nblk, J, L;
    int n_ctiles, n_items;
};

enum { kBarReady = 0, kBarAccFull = 2, kBars = 4 };

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

// C_jj[k1] of the tile's points for one thread's channels, as bf16 pairs into the B tile.
// NA: number of band bins of this row that are summed (compile time).
template <int KB, int CHT, int NA>
__device__ __forceinline__ void stage2_tile(const float (&yv)[KB][CHT][2], const float2* __restrict__ w_tab, int jj0, int J,
                                            float2 rot, float2 step, unsigned char* b_hi, unsigned char* b_lo,
                                            int row_re, int row_im, int col0) {
    constexpr int C = 4 * CHT, TJ = kNcol / C;
#pragma unroll 1
    for (int jl = 0; jl < TJ; ++jl) {
        const int jj = jj0 + jl;
        float re[CHT], im[CHT];
        if (jj < J) {
            float2 g[NA];
#pragma unroll
            for (int t = 0; t < NA; ++t) g[t] = w_tab[jj * KB + t];
#pragma unroll
            for (int c = 0; c < CHT; ++c) {
                float sr = 0.f, si = 0.f;
#pragma unroll
                for (int t = 0; t < NA; ++t) {
                    sr = fmaf(g[t].x, yv[t][c][0], fmaf(-g[t].y, yv[t][c][1], sr));
                    si = fmaf(g[t].x, yv[t][c][1], fmaf(g[t].y, yv[t][c][0], si));
                }
                re[c] = rot.x * sr - rot.y * si;
                im[c] = fmaf(rot.x, si, rot.y * sr);
            }
            rot = cmul(rot, step);
        } else {
#pragma unroll
            for (int c = 0; c < CHT; ++c) re[c] = im[c] = 0.f;
        }
        // element (K row r, column n) of a part sits at (n/8) kBSbo + (r/8) 128 + (r%8) 16 + (n%8) 2
        const int n = jl * C + col0;
        const int off_n = (n >> 3) * kBSbo + (n & 7) * 2;
        const int off_re = off_n + (row_re >> 3) * 128 + (row_re & 7) * 16;
        const int off_im = off_n + (row_im >> 3) * 128 + (row_im & 7) * 16;
        uint32_t hr[CHT / 2], lr[CHT / 2], hi_[CHT / 2], li[CHT / 2];
#pragma unroll
        for (int c = 0; c < CHT; c += 2) {
            const __nv_bfloat16 a0 = __float2bfloat16_rn(re[c]), a1 = __float2bfloat16_rn(re[c + 1]);
            const __nv_bfloat16 b0 = __float2bfloat16_rn(im[c]), b1 = __float2bfloat16_rn(im[c + 1]);
            hr[c / 2] = pack_bf16(a0, a1);
            hi_[c / 2] = pack_bf16(b0, b1);
            lr[c / 2] = pack_bf16(__float2bfloat16_rn(re[c] - __bfloat162float(a0)),
                                  __float2bfloat16_rn(re[c + 1] - __bfloat162float(a1)));
            li[c / 2] = pack_bf16(__float2bfloat16_rn(im[c] - __bfloat162float(b0)),
                                  __float2bfloat16_rn(im[c + 1] - __bfloat162float(b1)));
        }
        if constexpr (CHT == 8) {
            *reinterpret_cast<uint4*>(b_hi + off_re) = make_uint4(hr[0], hr[1], hr[2], hr[3]);
            *reinterpret_cast<uint4*>(b_lo + off_re) = make_uint4(lr[0], lr[1], lr[2], lr[3]);
            *reinterpret_cast<uint4*>(b_hi + off_im) = make_uint4(hi_[0], hi_[1], hi_[2], hi_[3]);
            *reinterpret_cast<uint4*>(b_lo + off_im) = make_uint4(li[0], li[1], li[2], li[3]);
        } else if constexpr (CHT == 4) {
            *reinterpret_cast<uint2*>(b_hi + off_re) = make_uint2(hr[0], hr[1]);
            *reinterpret_cast<uint2*>(b_lo + off_re) = make_uint2(lr[0], lr[1]);
            *reinterpret_cast<uint2*>(b_hi + off_im) = make_uint2(hi_[0], hi_[1]);
            *reinterpret_cast<uint2*>(b_lo + off_im) = make_uint2(li[0], li[1]);
        } else {
            *reinterpret_cast<uint32_t*>(b_hi + off_re) = hr[0];
            *reinterpret_cast<uint32_t*>(b_lo + off_re) = lr[0];
            *reinterpret_cast<uint32_t*>(b_hi + off_im) = hi_[0];
            *reinterpret_cast<uint32_t*>(b_lo + off_im) = li[0];
        }
    }
}

// KB: band bins per row held by a thread; CHT: channels per thread (C = 4 CHT per channel block).
template <int KB, int CHT>
__global__ void __launch_bounds__(kThreads, 1) spu_inv2_kernel(const InvArgs a) {
    constexpr int C = 4 * CHT, TJ = kNcol / C;
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) unsigned long long s_bar[kBars];
    __shared__ uint32_t s_tmem;
    __shared__ int s_fail;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int P = a.P, D = a.D, sigma = a.sigma, J = a.J, L = a.L;
    const int KT = a.nblk * P;                   // rows in use; the contraction runs over 2 KT (real, imaginary)
    const int f_bytes = 2 * KT * 256;            // one part of A: 2 KT / 8 K chunks x 128 rows x 16 B
    unsigned char* s_fhi = smem;
    unsigned char* s_flo = smem + f_bytes;
    unsigned char* s_bhi = smem + 2 * f_bytes;
    unsigned char* s_blo = s_bhi + kBPart;
    float2* s_w = reinterpret_cast<float2*>(s_blo + kBPart);   // [J][KB]: e^{2 pi i k2 jj / J}
    const uint32_t bar0 = smem_u32(&s_bar[0]);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    if (tid == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kBarReady + s), kWarps);
            mbar_init(bar(kBarAccFull + s), 1);
        }
        s_fail = 0;
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc(smem_u32(&s_tmem), kTmemCols);

    // A = [cos | -sin], K-major: element (row m, column kk) at (m/8)*128 + (kk/8)*2048 + (m%8)*16 + (kk%8)*2;
    // row m = jb P + p meets column (part, jb', k1) only for jb == jb'
    for (int idx = tid; idx < 128 * 2 * KT; idx += kThreads) {
        const int m = idx / (2 * KT), kk = idx - m * (2 * KT);
        const int part = kk / KT, kr = kk - part * KT;
        const int jb = m / P, p = m - jb * P, kb = kr / P, k1 = kr - kb * P;
        float v = 0.f;
        if (m < KT && jb == kb) {
            float s, c;
            sincospif(2.0f * (float)((k1 * p) % P) / (float)P, &s, &c);
            v = part ? -s : c;
        }
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        const int off = (m >> 3) * 128 + (kk >> 3) * 2048 + (m & 7) * 16 + (kk & 7) * 2;
        *reinterpret_cast<__nv_bfloat16*>(s_fhi + off) = h;
        *reinterpret_cast<__nv_bfloat16*>(s_flo + off) = __float2bfloat16_rn(v - __bfloat162float(h));
    }
    for (int e = tid; e < J * KB; e += kThreads) {
        const int jj = e / KB, k2 = e - jj * KB;
        s_w[e] = root_pos(((unsigned)jj * (unsigned)k2) % (unsigned)J, J);
    }
    // rows of B that no thread writes (KT < 128 never happens for the K extent 2 KT, which is all
    // the MMAs read), columns of points past J are written as zeros by their owners
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    volatile int* fail = &s_fail;

    const int quarter = warp & 3, grp = warp >> 2;
    const int j = quarter * 32 + lane;               // row: (channel block jb, frequency k1) when producing B,
    const int jb = j / P, k1 = j - jb * P;            //      (channel block jb, point p) when reading the result
    const bool active = j < KT;
    const int tiles_per_item = (J + TJ - 1) / TJ;
    const int item_channels = a.nblk * C;
    const float2 step = root_pos((unsigned)k1 % (unsigned)L, L);
    const uint32_t idesc = make_idesc_bf16(128, kNcol, false, true);
    const uint64_t a_hi0 = make_desc(smem_u32(s_fhi), 2048, 128), a_lo0 = make_desc(smem_u32(s_flo), 2048, 128);
    const uint64_t b_hi0 = make_desc(smem_u32(s_bhi), 128, kBSbo), b_lo0 = make_desc(smem_u32(s_blo), 128, kBSbo);

    // energies of tile `t` (accumulator t & 1) of the item (b, ctile), points jj0 ..: the warp of channel
    // group grp reads the 16 columns [16 grp, 16 grp + 16) of its rows with ONE TMEM load (a load's round
    // trip is long, so the 64 columns are spread over the four warps that share the lanes):
    //   C = 32: point jl = grp / 2, channel half grp % 2 (two partial sums per point)
    //   C = 16: point jl = grp;   C = 8: points 2 grp and 2 grp + 1
    constexpr int SPLIT = C == 32 ? 2 : 1;           // partial sums per (channel block, point)
    auto read_tile = [&](int t, int b, int ctile, int jj0) {
        const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)((t & 1) * kNcol + grp * 16);
        uint32_t v[16];
        tmem_ld16(taddr, v);
        tmem_ld_wait_for(v);
        tc_fence_before();
        if (!active) return;
        const int half = C == 32 ? (grp & 1) : 0;
        float* out = a.part + ((size_t)b * (a.n_ctiles * a.nblk * SPLIT) + (ctile * a.nblk + jb) * SPLIT + half) * L +
                     (size_t)k1 * J;
        constexpr int PTS = C >= 16 ? 1 : 2;          // points among the 16 columns
        constexpr int W = 16 / PTS;                   // columns per point
#pragma unroll
        for (int pt = 0; pt < PTS; ++pt) {
            float sum = 0.f;
#pragma unroll
            for (int q = 0; q < W; ++q) { const float x = __uint_as_float(v[pt * W + q]); sum = fmaf(x, x, sum); }
            const int jl = C == 32 ? (grp >> 1) : (C == 16 ? grp : 2 * grp + pt);
            if (jj0 + jl < J) out[jj0 + jl] = sum;
        }
    };

    int t = 0;                                       // tiles issued so far by this CTA
    int pb = 0, pct = 0, pj0 = 0;                    // item and first point of tile t - 1
    bool ok = true;
    for (int item = blockIdx.x; item < a.n_items && ok; item += gridDim.x) {
        const int ctile = item % a.n_ctiles, b = item / a.n_ctiles;
        const int ch0 = ctile * item_channels + jb * C + grp * CHT;
        // band bins of this row: Y_k = (cos row k) + i (sin row sigma + k), k = k1 + P t
        float yv[KB][CHT][2];
        int nA = (active && k1 <= sigma) ? min(KB, (sigma - k1) / P + 1) : 0;
        const float* Yb = a.Y + (size_t)b * a.R * D + ch0;
#pragma unroll
        for (int q = 0; q < KB; ++q) {
            const int k = k1 + P * q;
            const bool have = q < nA && ch0 < D;          // ch0 is a multiple of CHT and D of 8: all CHT channels exist
            const float* yc = Yb + (size_t)k * D;
            const float* ys = Yb + (size_t)(sigma + k) * D;
            constexpr int VEC = CHT >= 4 ? 4 : 2;
#pragma unroll
            for (int c = 0; c < CHT; c += VEC) {
                float vc[4] = {0.f, 0.f, 0.f, 0.f}, vs[4] = {0.f, 0.f, 0.f, 0.f};
                if (have) {
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
                for (int e = 0; e < VEC; ++e) { yv[q][c + e][0] = vc[e]; yv[q][c + e][1] = vs[e]; }
            }
        }
        const int nA_w = __reduce_max_sync(0xffffffffu, nA);

        for (int tile = 0; tile < tiles_per_item; ++tile, ++t) {
            const int jj0 = tile * TJ;
            // the B tile is single: the MMAs of the previous tile must be done with it
            if (t >= 1) ok = wait_bar(bar(kBarAccFull + ((t - 1) & 1)), ((t - 1) >> 1) & 1, fail, a.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            if (quarter * 32 < KT) {
                const float2 rot = root_pos(((unsigned)k1 * (unsigned)jj0) % (unsigned)L, L);   // k1 jj0 < P J = L
                unsigned char* bh = s_bhi;
                unsigned char* bl = s_blo;
                const int col0 = grp * CHT, rre = j, rim = KT + j;
                if (!active) {
                    // rows past KT of this warp: nothing to write (the MMAs read K rows below 2 KT only,
                    // and row j >= KT as a real-part row is an imaginary-part row of another thread)
                } else if (KB <= 4) {
                    switch (nA_w) {
                        case 1: stage2_tile<KB, CHT, 1>(yv, s_w, jj0, J, rot, step, bh, bl, rre, rim, col0); break;
                        case 2: stage2_tile<KB, CHT, (KB >= 2 ? 2 : KB)>(yv, s_w, jj0, J, rot, step, bh, bl, rre, rim, col0); break;
                        case 3: stage2_tile<KB, CHT, (KB >= 3 ? 3 : KB)>(yv, s_w, jj0, J, rot, step, bh, bl, rre, rim, col0); break;
                        default: stage2_tile<KB, CHT, KB>(yv, s_w, jj0, J, rot, step, bh, bl, rre, rim, col0); break;
                    }
                } else {
                    if (nA_w == KB - 1) stage2_tile<KB, CHT, KB - 1>(yv, s_w, jj0, J, rot, step, bh, bl, rre, rim, col0);
                    else stage2_tile<KB, CHT, KB>(yv, s_w, jj0, J, rot, step, bh, bl, rre, rim, col0);
                }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarReady + (t & 1)));
            if (tid == 0) {
                // every warp has written its share (and has finished reading accumulator t & 1, which it
                // last did for tile t - 2, before it came here): run the three products
                ok = wait_bar(bar(kBarReady + (t & 1)), (t >> 1) & 1, fail, a.status);
                if (ok) {
                    tc_fence_after();
                    const uint32_t acc = tmem + (uint32_t)((t & 1) * kNcol);
                    const int ksteps = 2 * KT / 16;
                    uint64_t ah = a_hi0, al = a_lo0, bh_d = b_hi0, bl_d = b_lo0;   // advance by adding to the address field
                    for (int ks = 0; ks < ksteps; ++ks) {
                        umma_bf16(acc, ah, bh_d, idesc, ks ? 1u : 0u);
                        umma_bf16(acc, ah, bl_d, idesc, 1u);
                        umma_bf16(acc, al, bh_d, idesc, 1u);
                        ah += 4096 >> 4; al += 4096 >> 4; bh_d += 256 >> 4; bl_d += 256 >> 4;
                    }
                    umma_commit(bar(kBarAccFull + (t & 1)));
                }
            }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            // meanwhile: the energies of the previous tile (its accumulator was awaited above)
            if (t >= 1) read_tile(t - 1, pb, pct, pj0);
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

template <int KB, int CHT>
cudaError_t launch_inv2(const InvArgs& a, cudaStream_t stream) {
    const int KT = a.nblk * a.P;
    const size_t smem = (size_t)2 * 2 * KT * 256 + 2 * kBPart + (size_t)a.J * KB * sizeof(float2);
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    cudaFuncSetAttribute(spu_inv2_kernel<KB, CHT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    const int grid = a.n_items < sms ? a.n_items : sms;
    spu_inv2_kernel<KB, CHT><<<grid, kThreads, smem, stream>>>(a);
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
    if (nk2 <= 4) { pl.KB = 4; pl.CHT = 8; }
    else if (nk2 <= 9) { pl.KB = 9; pl.CHT = 4; }
    else if (nk2 <= 17) { pl.KB = 17; pl.CHT = 2; }
    else return pl;
    if ((size_t)pl.J * pl.KB * sizeof(float2) > 24 * 1024) return pl;
    const int C = 4 * pl.CHT * pl.nblk;
    pl.n_ctiles = (D + C - 1) / C;
    const long long items = (long long)B * pl.n_ctiles;
    if (items > 0x7fffffffll) return pl;
    pl.n_items = (int)items;
    pl.n_parts = pl.n_ctiles * pl.nblk * (pl.CHT == 8 ? 2 : 1);
    pl.ok = 1;
    return pl;
}

int spu_inv2_run(const float* Y, float* part, int B, int N, int D, int sigma, int* status, cudaStream_t stream) {
    const SpuInv2Plan pl = spu_inv2_plan(B, N, D, sigma);
    if (!pl.ok) return LUVC_ERR_INTERNAL;
    InvArgs a;
    a.Y = Y; a.part = part; a.status = status;
    a.B = B; a.N = N; a.D = D; a.P = pl.P; a.Q = pl.Q; a.sigma = sigma; a.R = 2 * sigma + 1;
    a.nblk = pl.nblk; a.J = pl.J; a.L = pl.L; a.n_ctiles = pl.n_ctiles; a.n_items = pl.n_items;
    cudaError_t err;
    if (pl.KB == 4) err = launch_inv2<4, 8>(a, stream);
    else if (pl.KB == 9) err = launch_inv2<9, 4>(a, stream);
    else err = launch_inv2<17, 2>(a, stream);
    count_launch();
    return err == cudaSuccess ? LUVC_OK : LUVC_ERR_CUDA;
}

}  // namespace luvc
