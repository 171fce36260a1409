// Inverse transform and energy of the Spectrum Pruning Unit (Eq. 7 and Eq. 8) for bf16 tokens with
// BOTH stages on the tensor cores, for sequence lengths N = 128 Q: the mirror image of spu_fwd3.cu.
//
// The filtered signal x'(t) = sum_{k=0..sigma} Re(Y_k e^{2 pi i k t / N}) (Y already carries the mask
// of Eq. 5/6, 1/N and the weight of the conjugate half) is evaluated on the L = 128 J uniform points
// t = (p J + jj) N / L of the period (J = Q: the tokens themselves; J < Q: the coarse grid from which
// the squared energies are interpolated).  With k = k1 + 128 k2:
//   stage 2'  S_jj[k1] = sum_{k2} Y_{k1 + 128 k2} e^{2 pi i k2 jj / J}      a contraction over k2 with the same small
//                                                                           matrix for every k1 and every channel
//   twiddle   C_jj[k1] = e^{2 pi i k1 jj / L} S_jj[k1]                      CUDA cores, fp32
//   stage 1'  x'[p, jj] = sum_{k1 < 128} Re(e^{2 pi i k1 p / 128} C_jj[k1]) = sum_r F[r][p] G_jj[r]   (as spu_inv2.cu)
//   energy    S[p J + jj] = sum over the channels of x'^2, read back from tensor memory.
// The band spectrum arrives as the A operand of stage 2' ready made ("operand form"): per sequence and
// channel, for every TMEM lane (= frequency k1 of the lane: 0, 64, then i on the even and 128 - i on the
// odd lane of pair i) its bins k2 = 0, 1, .. as four bf16 each (Re hi, Im hi, Re lo, Im lo), K-major, so
// that one bulk copy per tile brings it into shared memory and D2 = A [W; W] + A [W lo; 0] needs two MMAs
// per four bins.  Sixteen converter warps read D2 (lane = k1, columns = (point, re/im)), apply the
// twiddle, exchange one value with the partner lane to form the real row G[r], split it into a bf16 pair
// and store it as the B operand of stage 1' (the contraction of spu_inv2.cu, issued by a warp of its
// own); the same warps then square and sum the result over the channels of a work item in registers.
// One more warp issues the bulk copies and stage 2'.  When one value of k2 too many reaches into the band
// (k = 128 * 16, which only k1 = 0 has), its term is the same for every p (F[0][p] = 1): it is added to
// the result before squaring, from a table the stage-1' warp builds per tile.
// Every mbarrier wait is bounded (on expiry: status word, free TMEM, return).

#include <cuda_bf16.h>

#include "luvc_internal.h"
#include "sm100_ptx.cuh"

namespace luvc {
namespace {

using namespace ptx;

constexpr int kConvWarps = 16;
constexpr int kThreads = (kConvWarps + 2) * 32;   // + the warp of the copies and stage 2', + the warp of stage 1'
constexpr int kP = 128;
constexpr int kSpin = 1 << 22;
constexpr int kA2Bufs = 3;
constexpr int kChanBytes = 4096;              // operand form: bytes per channel and K step (four bins x 128 lanes x 8 B)
constexpr int kItemChannels = 32;             // channels of a work item

struct Inv3Args {
    const unsigned char* yop;   // [B][D][KS][2 K chunks][128 lanes][16 B]
    const float* yx_re;         // the bin k = 128 * 16 (cos row and sin row), element (b, d) at [b * yx_stride + d]
    const float* yx_im;
    long long yx_stride;
    float* part;                // [B][n_parts][L]
    int* status;
    int B, D, J, L, KS, n_ctiles, n_items, n_parts;
    const unsigned char* img;   // stage-1' matrix, stage-2' matrices and the table of the extra bin (built once per call)
};

// barriers
enum {
    kBarImg = 0,
    kBarA2Full = 1,                       // [3] the bulk copy of a tile's operand has landed
    kBarA2Empty = kBarA2Full + kA2Bufs,   // [3] the stage-2' MMAs that read it are done
    kBarD2Full = kBarA2Empty + kA2Bufs,   // [2] stage-2' result of a tile complete
    kBarD2Empty = kBarD2Full + 2,         // [2] every converter warp has read it
    kBarReady = kBarD2Empty + 2,          // [2] every converter warp has written its share of the stage-1' operand
    kBarAccFull = kBarReady + 2,          // [2] stage-1' result of a tile complete
    kBarExtra = kBarAccFull + 2,          // [2] the table of the extra bin's term is written
    kBars = kBarExtra + 2
};

__device__ __forceinline__ bool wait_bar(uint32_t bar, int parity, volatile int* s_fail, int* status) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer();
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
__device__ __forceinline__ bool wait_bar_warp(uint32_t bar, int parity, volatile int* s_fail, int* status) {
    return __all_sync(0xffffffffu, wait_bar(bar, parity, s_fail, status));
}

// e^{+2 pi i num / den}, 0 <= num < den
__device__ __forceinline__ float2 root_pos(unsigned num, unsigned den) {
    float s, c;
    sincospif(2.0f * (float)num / (float)den, &s, &c);
    return make_float2(c, s);
}
__device__ __forceinline__ uint32_t bf16x2_bits(float lo_half, float hi_half) {
    const __nv_bfloat162 p = __floats2bfloat162_rn(lo_half, hi_half);
    return *reinterpret_cast<const uint32_t*>(&p);
}

// Geometry of a variant.
//   JP   points jj per channel held by the stage-2' result (J rounded up to a multiple of 8)
//   CT   channels per tile of stage 1'
template <int JP_, int CT_, int NBUF_>
struct IGeo {
    static constexpr int JP = JP_, CT = CT_, NBUF = NBUF_;    // NBUF: shared-memory buffers of the stage-2' operand (2 or 3)
    static constexpr int N2 = 2 * JP;                         // columns of the stage-2' result per channel: (point, re/im)
    static constexpr int BCOLS = CT * JP;                     // columns of the stage-1' operand that are written: (channel, point)
    static constexpr int TCOL = (BCOLS + 15) / 16 * 16;       // N of the stage-1' MMAs
    static constexpr int NCH = JP / 4;                        // chunks of four points per channel
    static constexpr int TOTCH = CT * NCH;                    // chunks of a tile, dealt out to the four warps of a lane quadrant
    static constexpr int UNITS = (TOTCH + 3) / 4;             // chunks per converter thread and tile
    static constexpr int ECOLS = TCOL / 4;                    // result columns per converter thread
    static constexpr int ACC0 = 0, D20 = 2 * TCOL;
    static constexpr int TMEM_COLS = 512;
    static constexpr int B_PART = BCOLS * 256;                // one part (hi or lo) of the stage-1' operand: BCOLS / 8 groups x 2 KB
    static constexpr int B_BUF = 2 * B_PART;
    static constexpr int W_BYTES = 32 * N2;                   // one part of one K step's stage-2' matrix: 16 x N2 bf16
    static_assert(JP % 8 == 0 && D20 + 2 * CT * N2 <= TMEM_COLS, "tensor memory budget");
    static_assert(CT == 1 || JP % ECOLS == 0, "a converter thread's result columns belong to one channel");
    static_assert(NBUF == 2 || NBUF == 3, "operand buffers");
};

template <typename G, bool EXTRA>
__global__ void __launch_bounds__(kThreads, 1) spu_inv3_kernel(const Inv3Args a) {
    constexpr int JP = G::JP, CT = G::CT, N2 = G::N2;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long s_bar[kBars];
    __shared__ uint32_t s_tmem;
    __shared__ int s_fail;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int D = a.D, J = a.J, L = a.L, KS = a.KS;
    const int a2_bytes = CT * KS * kChanBytes;
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* s_f = smem;                                          // stage-1' matrix, 32 KB per part
    unsigned char* s_w2 = smem + 65536;                                 // [KS][hi, lo][16 x N2]
    float2* s_wx = reinterpret_cast<float2*>(s_w2 + (size_t)KS * 2 * G::W_BYTES);   // e^{2 pi i 16 jj / J}, jj < JP
    float* s_e = reinterpret_cast<float*>(s_wx + JP);                   // [2][JP] the extra bin's term of a tile
    unsigned char* s_b = reinterpret_cast<unsigned char*>(s_e + 2 * JP);   // [2][hi, lo] stage-1' operand
    unsigned char* s_a2 = s_b + 2 * G::B_BUF;                           // [3] stage-2' operand (operand form)
    const uint32_t bar0 = smem_u32(&s_bar[0]);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    if (tid == 0) {
        mbar_init(bar(kBarImg), 1);
        for (int s = 0; s < kA2Bufs; ++s) {
            mbar_init(bar(kBarA2Full + s), 1);
            mbar_init(bar(kBarA2Empty + s), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kBarD2Full + s), 1);
            mbar_init(bar(kBarD2Empty + s), kConvWarps);
            mbar_init(bar(kBarReady + s), kConvWarps);
            mbar_init(bar(kBarAccFull + s), 1);
            mbar_init(bar(kBarExtra + s), 1);
        }
        s_fail = 0;
        mbar_fence_init();
    }
    if (warp == kConvWarps) tmem_alloc(smem_u32(&s_tmem), G::TMEM_COLS);

    const int tab_bytes = KS * 2 * G::W_BYTES + JP * (int)sizeof(float2);
    if (tid == 0) {
        mbar_arrive_expect_tx(bar(kBarImg), (uint32_t)(65536 + tab_bytes));
        bulk_load(smem_u32(s_f), a.img, 65536u, bar(kBarImg));
        bulk_load(smem_u32(s_w2), a.img + 65536, (uint32_t)tab_bytes, bar(kBarImg));
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

    // tiles of work item `item`: its channels in groups of CT (D is a multiple of 8, so groups are whole)
    auto item_tiles = [&](int item) {
        const int c0 = (item % a.n_ctiles) * kItemChannels;
        return (min(kItemChannels, D - c0) + CT - 1) / CT;
    };

    const int warp_u = __shfl_sync(0xffffffffu, warp, 0);   // the same in every lane, and the compiler can tell
    if (warp_u == kConvWarps) {
        // ------------------------------------------------------------------ bulk copies and stage 2'
        const uint32_t idesc2 = make_idesc_bf16(128, N2, false, false);
        const uint64_t w0 = make_desc(smem_u32(s_w2), N2 * 16, 128);
        const uint64_t a0 = make_desc(smem_u32(s_a2), 2048, 128);
        // the copy of the tile that is `ahead` tiles after the one being multiplied: a cursor over (item, tile)
        int c_item = blockIdx.x, c_tile = 0, c_v = 0;
        auto issue_copy = [&]() {                            // tile c_v -> buffer c_v % 3, then advance the cursor
            if (c_item >= a.n_items) return;
            const int ctile = c_item % a.n_ctiles, b = c_item / a.n_ctiles;
            const int c = ctile * kItemChannels + c_tile * CT;
            const int nch = min(CT, D - c);
            const int buf = c_v % G::NBUF;
            if (elect_one()) {
                const uint32_t bytes = (uint32_t)(nch * KS * kChanBytes);
                mbar_arrive_expect_tx(bar(kBarA2Full + buf), bytes);
                bulk_load(smem_u32(s_a2) + (uint32_t)(buf * a2_bytes), a.yop + ((size_t)b * D + c) * (size_t)(KS * kChanBytes), bytes,
                          bar(kBarA2Full + buf));
            }
            __syncwarp();
            ++c_v;
            if (++c_tile == item_tiles(c_item)) { c_tile = 0; c_item += gridDim.x; }
        };
        for (int q = 0; q < G::NBUF - 1; ++q) issue_copy();
        int v = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < a.n_items && ok; item += gridDim.x) {
            const int nt = item_tiles(item);
            const int c_first = (item % a.n_ctiles) * kItemChannels;
            for (int tile = 0; tile < nt && ok; ++tile, ++v) {
                // the copy NBUF - 1 tiles ahead reuses the buffer of tile v - 1, whose MMAs were issued a tile ago
                if (c_v == v + G::NBUF - 1) {
                    if (v >= 1) ok = wait_bar_warp(bar(kBarA2Empty + (v + G::NBUF - 1) % G::NBUF), ((v - 1) / G::NBUF) & 1, fail, a.status);
                    if (!ok) break;
                    issue_copy();
                }
                ok = wait_bar_warp(bar(kBarA2Full + v % G::NBUF), (v / G::NBUF) & 1, fail, a.status);
                if (ok && v >= 2) ok = wait_bar_warp(bar(kBarD2Empty + (v & 1)), ((v - 2) >> 1) & 1, fail, a.status);
                if (!ok) break;
                tc_fence_after();
                const int nch = min(CT, D - (c_first + tile * CT));
                if (elect_one()) {
                    for (int ct = 0; ct < nch; ++ct) {
                        const uint32_t d2 = tmem + (uint32_t)(G::D20 + (v & 1) * CT * N2 + ct * N2);
                        for (int s = 0; s < KS; ++s) {
                            const uint64_t ad = a0 + (uint64_t)(((v % G::NBUF) * a2_bytes + (ct * KS + s) * kChanBytes) >> 4);
                            const uint64_t whi = w0 + (uint64_t)((s * 2 * G::W_BYTES) >> 4), wlo = whi + (uint64_t)(G::W_BYTES >> 4);
                            umma_bf16(d2, ad, whi, idesc2, s ? 1u : 0u);
                            umma_bf16(d2, ad, wlo, idesc2, 1u);
                        }
                    }
                    umma_commit(bar(kBarD2Full + (v & 1)));
                    umma_commit(bar(kBarA2Empty + v % G::NBUF));
                }
                __syncwarp();
            }
        }
    } else if (warp_u == kConvWarps + 1) {
        // ------------------------------------------------------------------ stage 1'
        const uint32_t idesc1 = make_idesc_bf16(128, G::TCOL, false, true);
        const uint64_t a_hi0 = make_desc(smem_u32(s_f), 2048, 128), a_lo0 = make_desc(smem_u32(s_f) + 32768, 2048, 128);
        const uint64_t b_d0 = make_desc(smem_u32(s_b), 128, 2048);
        int t = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < a.n_items && ok; item += gridDim.x) {
            const int nt = item_tiles(item);
            const int ctile = item % a.n_ctiles, b = item / a.n_ctiles;
            for (int tile = 0; tile < nt && ok; ++tile, ++t) {
                float xr = 0.f, xi = 0.f;
                if constexpr (EXTRA) {                       // one channel per tile in this variant
                    const size_t o = (size_t)b * a.yx_stride + ctile * kItemChannels + tile;
                    xr = __ldg(a.yx_re + o);
                    xi = __ldg(a.yx_im + o);
                }
                ok = wait_bar_warp(bar(kBarReady + (t & 1)), (t >> 1) & 1, fail, a.status);
                if (!ok) break;
                if constexpr (EXTRA) {
                    // every converter warp has read the table of tile t - 2 (it arrived on the barrier above after that)
                    for (int jj = lane; jj < JP; jj += 32) {
                        const float2 w = s_wx[jj];
                        s_e[(t & 1) * JP + jj] = xr * w.x - xi * w.y;
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(kBarExtra + (t & 1)));
                }
                tc_fence_after();
                if (elect_one()) {
                    const uint32_t acc = tmem + (uint32_t)(G::ACC0 + (t & 1) * G::TCOL);
                    uint64_t ah = a_hi0, al = a_lo0;
                    uint64_t bh_d = b_d0 + (uint64_t)(((t & 1) * G::B_BUF) >> 4), bl_d = bh_d + (uint64_t)(G::B_PART >> 4);
#pragma unroll
                    for (int ks = 0; ks < kP / 16; ++ks) {
                        umma_bf16(acc, ah, bh_d, idesc1, ks ? 1u : 0u);
                        umma_bf16(acc, ah, bl_d, idesc1, 1u);
                        umma_bf16(acc, al, bh_d, idesc1, 1u);
                        ah += 4096 >> 4; al += 4096 >> 4; bh_d += 256 >> 4; bl_d += 256 >> 4;
                    }
                    umma_commit(bar(kBarAccFull + (t & 1)));
                }
                __syncwarp();
            }
        }
    } else {
        // ------------------------------------------------------------------ converters
        const int quarter = warp & 3, grp = warp >> 2;
        const int j = quarter * 32 + lane;               // TMEM lane = row r of G = point block p of the result
        const int i = j >> 1;
        const bool odd = j & 1, special = i == 0;
        const int kf = special ? (odd ? kP / 2 : 0) : (odd ? kP - i : i);       // this lane's frequency
        const float gc = special ? 0.f : 1.f;
        const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
        // twiddles e^{2 pi i kf jj / L} of this thread's points: unit u is chunk c = grp + 4 u of the tile's chunks
        // (channel c / NCH, points 4 (c % NCH) + e), times i on the odd lane of a pair: then the own contribution
        // to G is the real part and the partner's is the imaginary part
        float2 rot[G::UNITS][4];
#pragma unroll
        for (int u = 0; u < G::UNITS; ++u)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int jj = 4 * ((grp + 4 * u) % G::NCH) + e;
                float2 r = root_pos((unsigned)(((long long)kf * jj) % L), (unsigned)L);
                if (odd && !special) r = make_float2(-r.y, r.x);
                rot[u][e] = r;
            }
        // this thread's ECOLS result columns grp ECOLS + q are points e_jj0 + q of channel e_ct of the tile
        const int e_ct = (grp * G::ECOLS) / JP, e_jj0 = (grp * G::ECOLS) % JP;
        float en[G::ECOLS];                              // energies of this thread's result columns, summed over the item
#pragma unroll
        for (int q = 0; q < G::ECOLS; ++q) en[q] = 0.f;

        // energies of tile tt (accumulator tt & 1): this thread's ECOLS columns of its row
        auto read_tile = [&](int tt) {
            const uint32_t taddr = lane_addr + (uint32_t)(G::ACC0 + (tt & 1) * G::TCOL + grp * G::ECOLS);
            uint32_t x0[G::ECOLS >= 16 ? 16 : 8], x1[4];
            if constexpr (G::ECOLS == 16) {
                tmem_ld16(taddr, x0);
                tmem_ld_wait_for(x0);
            } else if constexpr (G::ECOLS == 12) {
                tmem_ld8(taddr, x0);
                tmem_ld4(taddr + 8, x1);
                tmem_ld_wait_for(x0);
                tmem_ld_wait_for(x1);
            } else {
                tmem_ld16(taddr, x0);
                tmem_ld4(taddr + 16, x1);
                tmem_ld_wait_for(x0);
                tmem_ld_wait_for(x1);
            }
            tc_fence_before();
#pragma unroll
            for (int q = 0; q < G::ECOLS; ++q) {
                constexpr int kFirst = G::ECOLS >= 16 ? 16 : 8;
                float x = __uint_as_float(q < kFirst ? x0[q < kFirst ? q : 0] : x1[q >= kFirst ? q - kFirst : 0]);
                if constexpr (EXTRA) x += s_e[(tt & 1) * JP + min(e_jj0 + q, JP - 1)];
                en[q] = fmaf(x, x, en[q]);
            }
        };
        // the item's energies: part[b][ctile (x channel of the tile)][p J + jj]
        auto flush = [&](int b, int ctile) {
            float* out = a.part + ((size_t)b * a.n_parts + (size_t)ctile * CT + e_ct) * L + (size_t)j * J;
#pragma unroll
            for (int q = 0; q < G::ECOLS; ++q) {
                const int jj = e_jj0 + q;
                if (jj < J) out[jj] = en[q];
                en[q] = 0.f;
            }
        };

        int t = 0;
        int pb = 0, pct = 0;                             // item of tile t - 1
        bool plast = false;                              // tile t - 1 was the last of its item
        bool ok = true;
        for (int item = blockIdx.x; item < a.n_items && ok; item += gridDim.x) {
            const int nt = item_tiles(item);
            const int ctile = item % a.n_ctiles, b = item / a.n_ctiles;
            for (int tile = 0; tile < nt && ok; ++tile, ++t) {
                const int dbuf = t & 1;
                ok = wait_bar(bar(kBarD2Full + dbuf), (t >> 1) & 1, fail, a.status);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                unsigned char* bh = s_b + dbuf * G::B_BUF;
                unsigned char* bl = bh + G::B_PART;
                const uint32_t d2 = lane_addr + (uint32_t)(G::D20 + dbuf * CT * N2);
                // unit u = chunk grp + 4 u of the tile: 8 columns of the stage-2' result of its channel
                uint32_t vb[2][8];                       // units alternate between the two: one in use, one in flight
                tmem_ld8(d2 + (uint32_t)(grp * 8), vb[0]);
#pragma unroll
                for (int u = 0; u < G::UNITS; ++u) {
                    const int c = grp + 4 * u;
                    const int ct = c / G::NCH, ch = c % G::NCH;
                    const bool live = c < G::TOTCH;      // the same for the whole warp
                    uint32_t (&v)[8] = vb[u & 1];
                    if (live) tmem_ld_wait_for(v);
                    if (u + 1 < G::UNITS) {
                        const int c1 = c + 4;
                        if (c1 < G::TOTCH) tmem_ld8(d2 + (uint32_t)((c1 / G::NCH) * N2 + (c1 % G::NCH) * 8), vb[(u + 1) & 1]);
                    }
                    if (!live) continue;
                    float g[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float sx = __uint_as_float(v[2 * e]), sy = __uint_as_float(v[2 * e + 1]);
                        const float2 r = rot[u][e];
                        const float cx = fmaf(r.x, sx, -r.y * sy), cy = fmaf(r.x, sy, r.y * sx);
                        const float got = __shfl_xor_sync(0xffffffffu, cy, 1);
                        g[e] = fmaf(gc, got, cx);
                    }
                    const uint32_t h0 = bf16x2_bits(g[0], g[1]), h1 = bf16x2_bits(g[2], g[3]);
                    const uint32_t l0 = bf16x2_bits(g[0] - __uint_as_float(h0 << 16), g[1] - __uint_as_float(h0 & 0xffff0000u));
                    const uint32_t l1 = bf16x2_bits(g[2] - __uint_as_float(h1 << 16), g[3] - __uint_as_float(h1 & 0xffff0000u));
                    // element (K row r, column n) of a part sits at (n/8) 2048 + (r/8) 128 + (r%8) 16 + (n%8) 2
                    const int n = ct * JP + 4 * ch;
                    const int off = (n >> 3) * 2048 + (n & 7) * 2 + (j >> 3) * 128 + (j & 7) * 16;
                    *reinterpret_cast<uint2*>(bh + off) = make_uint2(h0, h1);
                    *reinterpret_cast<uint2*>(bl + off) = make_uint2(l0, l1);
                }
                // every load of this tile's stage-2' result has completed (the last wait above covered them all)
                tc_fence_before();
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(bar(kBarD2Empty + dbuf));
                    mbar_arrive(bar(kBarReady + dbuf));
                }
                // meanwhile: the energies of the previous tile, whose MMAs ran under the arithmetic above
                if (t >= 1) {
                    ok = wait_bar(bar(kBarAccFull + ((t - 1) & 1)), ((t - 1) >> 1) & 1, fail, a.status);
                    if constexpr (EXTRA) ok = wait_bar(bar(kBarExtra + ((t - 1) & 1)), ((t - 1) >> 1) & 1, fail, a.status) && ok;
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    read_tile(t - 1);
                    if (plast) flush(pb, pct);
                }
                pb = b; pct = ctile; plast = tile == nt - 1;
            }
        }
        if (ok && t >= 1) {
            ok = wait_bar(bar(kBarAccFull + ((t - 1) & 1)), ((t - 1) >> 1) & 1, fail, a.status);
            if constexpr (EXTRA) ok = wait_bar(bar(kBarExtra + ((t - 1) & 1)), ((t - 1) >> 1) & 1, fail, a.status) && ok;
            ok = __all_sync(0xffffffffu, ok);
            if (ok) {
                tc_fence_after();
                read_tile(t - 1);
                flush(pb, pct);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kConvWarps) tmem_dealloc(tmem, G::TMEM_COLS);
}

// The operand images of one call, as the kernel's shared memory holds them:
//   [0, 64 KB)   stage-1' matrix A[m][kk] = F[kk][m] (F: the real 128 x 128 matrix of the forward kernels), K-major:
//                element at (m/8)*128 + (kk/8)*2048 + (m%8)*16 + (kk%8)*2, hi part then lo part
//   then         the stage-2' matrices [KS][hi, lo][16 x N2], K-major [n][k]: element at
//                (n/8)*128 + (k/8)*(N2*16) + (n%8)*16 + (k%8)*2;  k = z*4 + t: bin 4 s + z of the K step, t = Re hi, Im hi,
//                Re lo, Im lo (the lo rows of the hi-part matrix repeat the hi rows; the lo-part matrix has zeros
//                there);  n = (point jj, re/im)
//   then         e^{2 pi i 16 jj / J}, jj < JP (zero past J)
template <typename G>
__global__ void __launch_bounds__(256) spu_inv3_img_kernel(unsigned char* __restrict__ img, int J, int KS, int nk2) {
    constexpr int N2 = G::N2, JP = G::JP;
    const int idx = blockIdx.x * 256 + threadIdx.x;
    if (idx < kP * kP) {
        const int m = idx >> 7, r = idx & 127;
        float v;
        if (r == 0) v = 1.f;
        else if (r == 1) v = (m & 1) ? -1.f : 1.f;
        else {
            float s, c;
            sincospif((float)(((r >> 1) * m) & 127) * (1.0f / 64.0f), &s, &c);
            v = (r & 1) ? -s : c;
        }
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        const int off = (m >> 3) * 128 + (r >> 3) * 2048 + (m & 7) * 16 + (r & 7) * 2;
        *reinterpret_cast<__nv_bfloat16*>(img + off) = h;
        *reinterpret_cast<__nv_bfloat16*>(img + 32768 + off) = __float2bfloat16_rn(v - __bfloat162float(h));
    }
    unsigned char* tabs = img + 65536;
    if (idx < KS * 16 * N2) {
        const int s = idx / (16 * N2), rem = idx - s * 16 * N2;
        const int n = rem >> 4, k = rem & 15;
        const int z = k >> 2, t = k & 3;
        const int jj = n >> 1, ri = n & 1, k2 = 4 * s + z;
        float v = 0.f;
        if (jj < J && k2 < nk2) {
            const float2 w = root_pos((unsigned)(((long long)jj * k2) % J), (unsigned)J);    // e^{2 pi i k2 jj / J}
            // (Re, Im) of Y times w: Re out = Re Y w.x - Im Y w.y, Im out = Re Y w.y + Im Y w.x
            v = (t & 1) == 0 ? (ri == 0 ? w.x : w.y) : (ri == 0 ? -w.y : w.x);
        }
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        const __nv_bfloat16 l = __float2bfloat16_rn(v - __bfloat162float(h));
        const int off = (n >> 3) * 128 + (k >> 3) * (N2 * 16) + (n & 7) * 16 + (k & 7) * 2;
        unsigned char* base = tabs + (size_t)s * 2 * G::W_BYTES;
        *reinterpret_cast<__nv_bfloat16*>(base + off) = h;
        *reinterpret_cast<__nv_bfloat16*>(base + G::W_BYTES + off) = t < 2 ? l : __float2bfloat16_rn(0.f);
    }
    float2* wx = reinterpret_cast<float2*>(tabs + (size_t)KS * 2 * G::W_BYTES);
    if (idx < JP) wx[idx] = idx < J ? root_pos((unsigned)((16ll * idx) % J), (unsigned)J) : make_float2(0.f, 0.f);
}

template <typename G>
size_t inv3_smem(int KS) {
    return 1024 + 65536 + (size_t)KS * 2 * G::W_BYTES + (size_t)G::JP * sizeof(float2) + (size_t)2 * G::JP * sizeof(float) +
           (size_t)2 * G::B_BUF + (size_t)G::NBUF * G::CT * KS * kChanBytes;
}

template <typename G, bool EXTRA>
cudaError_t launch_inv3(const Inv3Args& a, int nk2, cudaStream_t stream) {
    {
        const int n = kP * kP > a.KS * 16 * G::N2 ? kP * kP : a.KS * 16 * G::N2;
        spu_inv3_img_kernel<G><<<(n + 255) / 256, 256, 0, stream>>>(const_cast<unsigned char*>(a.img), a.J, a.KS, nk2);
    }
    const size_t smem = inv3_smem<G>(a.KS);
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    cudaFuncSetAttribute(spu_inv3_kernel<G, EXTRA>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    const int grid = a.n_items < sms ? a.n_items : sms;
    spu_inv3_kernel<G, EXTRA><<<grid, kThreads, smem, stream>>>(a);
    return cudaGetLastError();
}

using GeoSmall = IGeo<16, 4, 3>;
using GeoMid2 = IGeo<40, 2, 2>;      // two channels per tile: 20 chunks split evenly over four warps, one 80-column contraction
using GeoMid = IGeo<40, 1, 3>;       // where the operands of two channels do not fit
using GeoBig = IGeo<72, 1, 3>;

}  // namespace

SpuInv3Plan spu_inv3_plan(int B, int N, int D, int sigma) {
    SpuInv3Plan pl = {};
    const SpuFwd3Plan f = spu_fwd3_plan(B, N, D, sigma);
    if (!f.ok || f.slices != 1) return pl;
    const int Q = N / kP;
    // points of the period: J per block of Q tokens, L = 128 J > 4 sigma, if that saves a quarter (as spu_inv2_plan)
    const long long need = 4ll * sigma + 2;
    const long long jc = (need + kP - 1) / kP;
    pl.coarse = (jc * kP * 4 <= 3ll * N) ? 1 : 0;
    pl.J = pl.coarse ? (int)jc : Q;
    pl.L = kP * pl.J;
    const int nk2 = sigma / kP + 1;
    if (nk2 > 17) return pl;
    pl.extra = nk2 == 17 ? 1 : 0;
    if (pl.extra && sigma != 16 * kP) return pl;     // the 17th bin is passed apart only as the single bin of k1 = 0
    pl.KS = ((pl.extra ? 16 : nk2) + 3) / 4;
    pl.JP = pl.J <= 16 ? 16 : (pl.J <= 40 ? 40 : (pl.J <= 72 ? 72 : 0));
    if (!pl.JP || (pl.extra && pl.JP != 72)) return pl;
    pl.CT = pl.JP == 16 ? 4 : 1;
    if (pl.JP == 40 && inv3_smem<GeoMid2>(pl.KS) <= (size_t)226 * 1024) pl.CT = 2;
    const size_t smem = pl.JP == 16 ? inv3_smem<GeoSmall>(pl.KS)
                        : pl.JP == 40 ? (pl.CT == 2 ? inv3_smem<GeoMid2>(pl.KS) : inv3_smem<GeoMid>(pl.KS)) : inv3_smem<GeoBig>(pl.KS);
    if (smem > 226 * 1024) return pl;
    if (65536 + (size_t)pl.KS * 2 * 64 * pl.JP + (size_t)pl.JP * 8 > kSpuImgBytes) return pl;
    pl.n_ctiles = (D + kItemChannels - 1) / kItemChannels;
    const long long items = (long long)B * pl.n_ctiles;
    if (items > 0x7fffffffll) return pl;
    pl.n_items = (int)items;
    pl.n_parts = pl.n_ctiles * pl.CT;
    pl.yop_bytes = (size_t)B * D * pl.KS * kChanBytes;
    pl.ok = 1;
    return pl;
}

int spu_inv3_run(const void* yop, const float* yx_re, const float* yx_im, long long yx_stride, float* part, int B, int N,
                 int D, int sigma, int* status, cudaStream_t stream, void* img) {
    const SpuInv3Plan pl = spu_inv3_plan(B, N, D, sigma);
    if (!pl.ok) return LUVC_ERR_INTERNAL;
    Inv3Args a;
    a.yop = static_cast<const unsigned char*>(yop);
    a.yx_re = yx_re; a.yx_im = yx_im; a.yx_stride = yx_stride;
    a.part = part; a.status = status;
    a.B = B; a.D = D; a.J = pl.J; a.L = pl.L; a.KS = pl.KS;
    a.n_ctiles = pl.n_ctiles; a.n_items = pl.n_items; a.n_parts = pl.n_parts;
    a.img = static_cast<const unsigned char*>(img);
    const int nk2 = pl.extra ? 16 : sigma / kP + 1;
    const cudaError_t err = pl.JP == 16 ? launch_inv3<GeoSmall, false>(a, nk2, stream)
                            : pl.JP == 40 ? (pl.CT == 2 ? launch_inv3<GeoMid2, false>(a, nk2, stream) : launch_inv3<GeoMid, false>(a, nk2, stream))
                            : pl.extra ? launch_inv3<GeoBig, true>(a, nk2, stream) : launch_inv3<GeoBig, false>(a, nk2, stream);
    count_launch(2);
    return err == cudaSuccess ? LUVC_OK : LUVC_ERR_CUDA;
}

}  // namespace luvc
