// Tensor-core (tcgen05) contraction used by the bf16 path of the Spectrum Pruning Unit.
//
// Both transforms of Eq. 4 and Eq. 7, restricted to the pass band of Eq. 5, are dense
// contractions with the real band matrix PhiT[r][n] (rows: cos / -sin of the passed
// frequencies, see spu.cu).  PhiT is fp32-accurate but the tensor cores take bf16, so it is
// held as a bf16 pair (hi + lo, together about 16 mantissa bits) and every product is issued once
// per part; the token values are bf16 already and need no split.
//
//   pass 1  YT[d][r]   = c[r] * sum_n X[n][d]    * PhiT[r][n]       A = X (1 part),  B = PhiT (hi, lo)
//   pass 2  X'[n][d]   =        sum_r PhiT[r][n] * YT[d][r]         A = PhiT (hi, lo), B = YT (hi, lo)
//           part[n]    = sum_d X'[n][d]^2  over the tile's channels
//
// One kernel serves both: C[m][nn] = sum_k A[k][m] * B[nn][k], with A read from a row-major
// matrix whose M index is contiguous (an MN-major UMMA operand) and B from a row-major matrix
// whose K index is contiguous (a K-major operand).  Tiles are 128 (M) x up to 256 (N) x 64 (K),
// staged in shared memory by 16-byte cp.async copies straight into the no-swizzle core-matrix
// layout (a 16-byte global chunk is a 16-byte shared chunk, so nothing is transposed), double
// buffered; one thread issues tcgen05.mma into a TMEM accumulator of 256 fp32 columns and
// tcgen05.commit reports a finished stage on an mbarrier; all eight warps read the accumulator
// back with tcgen05.ld for the epilogue.  Every mbarrier wait is bounded: on expiry the CTA
// records LUVC_ERR_TIMEOUT in the status word, drains its copies, frees its TMEM and returns.

#include <cuda_bf16.h>

#include "luvc_internal.h"

namespace luvc {
namespace {

constexpr int TM = 128;            // tile rows (TMEM lanes)
constexpr int TK = 64;             // K per stage
constexpr int kStages = 2;
constexpr int kThreads = 256;
constexpr int kTmemCols = 256;
constexpr int kWaitLimit = 1 << 22;

// shared-memory operand layouts (bytes)
//   A part: 16 MN-groups x 8 K-groups of 128-byte core matrices; MN-group stride 1024, K-group stride 128
//   B part: (tn/8) row-groups x 8 K-chunks; row-group stride 128, K-chunk stride tn * 16
constexpr int kABytes = TM * TK * 2;                       // 16 KB per A part
constexpr int kASbo = (TK / 8) * 128, kALbo = 128;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    // no-swizzle UMMA shared-memory descriptor: address, leading and stride offsets in 16-byte units,
    // descriptor version 1 (Blackwell)
    return (uint64_t)((addr >> 4) & 0x3fffu) | ((uint64_t)((lbo >> 4) & 0x3fffu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3fffu) << 32) | (1ull << 46);
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    const int bytes = valid ? 16 : 0;          // 0 source bytes: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, int parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait; false (and the status word set) if the phase never completes.
__device__ bool mbar_wait(uint32_t bar, int parity, int* status) {
    unsigned long long t0 = 0;
    for (int it = 0; it < kWaitLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 1023) == 1023) {               // also bounded in time: one second
            unsigned long long now;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
            if (t0 == 0) t0 = now;
            else if (now - t0 > 1000000000ull) break;
        }
    }
    atomicCAS(status, 0, (int)LUVC_ERR_TIMEOUT);
    return false;
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t addr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(addr) : "memory");
}

struct TcArgs {
    const __nv_bfloat16* a[2];   // A parts: element (k, m) at a[p][batch * a_batch + k * lda + m]
    const __nv_bfloat16* b[2];   // B parts: element (nn, k) at b[p][batch * b_batch + nn * ldb + k]
    long long a_batch, b_batch;
    const int32_t* a_rows;       // optional: row k of A is row a_rows[batch * a_rows_stride + k] of a[0] (gather on load)
    int a_rows_stride;
    int lda, ldb;
    int m_total;                 // valid extent of the M index (multiple of 8)
    int n_total;                 // valid extent of the N index (rows of B)
    int k_a;                     // rows of A that exist (K index); beyond: zero
    int k_blocks;                // ceil(K / 64); B is padded with zeros to k_blocks * 64 columns
    int tn;                      // N tile (64, 128, 192 or 256)
    // epilogues
    const float* scale;          // pass 1: c[nn]
    __nv_bfloat16 *yt_hi, *yt_lo;   // pass 1 out: [batch][m_total][ld_yt]
    int ld_yt;
    float* part;                 // pass 2 out: [batch][2 * gridDim.y][part_n]
    int part_n;
    int* status;
};

// NA, NB: number of bf16 parts of A and B.  PASS2 selects the epilogue.
template <int NA, int NB, bool PASS2>
__global__ void __launch_bounds__(kThreads, 1) spu_tc_kernel(const TcArgs g) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) unsigned long long s_bar[kStages];
    __shared__ uint32_t s_tmem;
    __shared__ int s_fail;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.x * TM, n0 = blockIdx.y * g.tn, batch = blockIdx.z;
    const int tn = g.tn;
    const int b_bytes = tn * TK * 2;
    const int stage_bytes = NA * kABytes + NB * b_bytes;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar0 = smem_u32(&s_bar[0]);

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(bar0 + 8 * s, 1);
        s_fail = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)),
                     "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem;

    // instruction descriptor: fp32 accumulate, bf16 x bf16, A MN-major, B K-major, M = 128, N = tn
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (0u << 16) |
                           ((uint32_t)(tn >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);

    auto load_stage = [&](int kb, int slot) {
        const uint32_t sbase = smem_base + slot * stage_bytes;
        const int k0 = kb * TK;
        // A parts: 16 MN-groups x 64 k rows of 16-byte chunks
#pragma unroll
        for (int p = 0; p < NA; ++p) {
            const __nv_bfloat16* src = g.a[p] + (size_t)batch * g.a_batch;
            for (int c = tid; c < 16 * TK; c += kThreads) {
                const int grp = c & 15, k = c >> 4;
                const int m = m0 + grp * 8, kk = k0 + k;
                const bool ok = m < g.m_total && kk < g.k_a;
                const uint32_t dst = sbase + p * kABytes + grp * kASbo + (k >> 3) * kALbo + (k & 7) * 16;
                const size_t row = (ok && g.a_rows != nullptr) ? (size_t)__ldg(g.a_rows + (size_t)batch * g.a_rows_stride + kk)
                                                               : (size_t)kk;
                cp_async16(dst, ok ? (const void*)(src + row * g.lda + m) : (const void*)src, ok);
            }
        }
        // B parts: tn rows x 8 K-chunks of 16 bytes
#pragma unroll
        for (int p = 0; p < NB; ++p) {
            const __nv_bfloat16* src = g.b[p] + (size_t)batch * g.b_batch;
            for (int c = tid; c < tn * 8; c += kThreads) {
                const int kc = c & 7, row = c >> 3;
                const int nn = n0 + row;
                const bool ok = nn < g.n_total;
                const uint32_t dst = sbase + NA * kABytes + p * b_bytes + (row >> 3) * 128 + (row & 7) * 16 +
                                     kc * (tn * 16);
                cp_async16(dst, ok ? (const void*)(src + (size_t)nn * g.ldb + k0 + kc * 8) : (const void*)src, ok);
            }
        }
    };

    const int KB = g.k_blocks;
    bool alive = true;
    load_stage(0, 0);
    cp_async_commit();
    for (int kb = 0; kb < KB; ++kb) {
        const int slot = kb & 1;
        if (kb + 1 < KB) {
            if (kb >= 1) {
                // the MMAs of block kb-1 read slot (kb+1)&1: wait for their commit before refilling it
                const int j = (kb - 1) >> 1;
                if (!mbar_wait(bar0 + 8 * ((kb + 1) & 1), j & 1, g.status)) s_fail = 1;
            }
            load_stage(kb + 1, (kb + 1) & 1);
        }
        cp_async_commit();
        cp_async_wait<1>();
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
        if (s_fail) { alive = false; break; }
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t sbase = smem_base + slot * stage_bytes;
            const uint32_t b_lbo = tn * 16;
#pragma unroll
            for (int ks = 0; ks < TK / 16; ++ks) {
                uint64_t ad[NA], bd[NB];
#pragma unroll
                for (int p = 0; p < NA; ++p) ad[p] = make_desc(sbase + p * kABytes + ks * 2 * kALbo, kALbo, kASbo);
#pragma unroll
                for (int p = 0; p < NB; ++p)
                    bd[p] = make_desc(sbase + NA * kABytes + p * b_bytes + ks * 2 * b_lbo, b_lbo, 128);
                // hi*hi first (sets or accumulates), then the cross terms
                umma_bf16(tmem, ad[0], bd[0], idesc, (kb | ks) ? 1u : 0u);
                if (NB > 1) umma_bf16(tmem, ad[0], bd[1], idesc, 1u);
                if (NA > 1) umma_bf16(tmem, ad[1], bd[0], idesc, 1u);
            }
            umma_commit(bar0 + 8 * slot);
        }
    }
    cp_async_wait<0>();
    if (alive) {
        const int last = KB - 1;
        if (!mbar_wait(bar0 + 8 * (last & 1), (last >> 1) & 1, g.status)) alive = false;
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

    if (alive) {
        // warps w and w+4 share TMEM lanes 32*(w%4) .. +31 and split the columns
        const int quarter = warp & 3, half = warp >> 2;
        const int row = quarter * 32 + lane;              // accumulator row = M index within the tile
        const int m = m0 + row;
        const int chunks = tn / 32;                        // 32-column chunks in the tile
        float sumsq = 0.f;
        for (int ch = half; ch < chunks; ch += 2) {
            if (n0 + ch * 32 >= g.n_total) break;          // columns past the padded extent (warp-uniform)
            uint32_t v[32];
            tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + ch * 32, v);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (PASS2) {
#pragma unroll
                for (int i = 0; i < 32; ++i) { const float x = __uint_as_float(v[i]); sumsq = fmaf(x, x, sumsq); }
            } else if (m < g.m_total) {
                const int c0 = n0 + ch * 32;
                uint32_t hi[16], lo[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const float x0 = __uint_as_float(v[i]) * __ldg(g.scale + c0 + i);
                    const float x1 = __uint_as_float(v[i + 1]) * __ldg(g.scale + c0 + i + 1);
                    const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
                    const __nv_bfloat16 l0 = __float2bfloat16_rn(x0 - __bfloat162float(h0));
                    const __nv_bfloat16 l1 = __float2bfloat16_rn(x1 - __bfloat162float(h1));
                    hi[i >> 1] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
                    lo[i >> 1] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
                }
                const size_t off = ((size_t)batch * g.m_total + m) * g.ld_yt + c0;
                uint4* ph = reinterpret_cast<uint4*>(g.yt_hi + off);
                uint4* pl = reinterpret_cast<uint4*>(g.yt_lo + off);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    ph[q] = make_uint4(hi[4 * q], hi[4 * q + 1], hi[4 * q + 2], hi[4 * q + 3]);
                    pl[q] = make_uint4(lo[4 * q], lo[4 * q + 1], lo[4 * q + 2], lo[4 * q + 3]);
                }
            }
        }
        if (PASS2 && m < g.part_n)
            g.part[((size_t)batch * (2 * gridDim.y) + 2 * blockIdx.y + half) * g.part_n + m] = sumsq;
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

// PhiT as a bf16 pair, [rows_pad][cols_pad], zero outside [0, R) x [0, N).
__global__ void spu_phi_kernel(const float2* __restrict__ tw, __nv_bfloat16* __restrict__ hi,
                               __nv_bfloat16* __restrict__ lo, int N, int sigma, int rows_pad, int cols_pad) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)rows_pad * cols_pad) return;
    const int r = (int)(i / cols_pad), n = (int)(i % cols_pad);
    float v = 0.f;
    if (r <= 2 * sigma && n < N) {
        const bool is_cos = r <= sigma;
        const int k = is_cos ? r : r - sigma;
        const int j = (int)(((unsigned long long)k * (unsigned long long)n) % (unsigned long long)N);
        const float2 t = __ldg(tw + j);
        v = is_cos ? t.x : -t.y;
    }
    const __nv_bfloat16 h = __float2bfloat16_rn(v);
    hi[i] = h;
    lo[i] = __float2bfloat16_rn(v - __bfloat162float(h));
}

}  // namespace

SpuTcPlan spu_tc_plan(int B, int N, int D, int sigma) {
    SpuTcPlan p;
    const int R = 2 * sigma + 1;
    p.r_pad = (R + 63) / 64 * 64;
    p.n_pad = (N + 127) / 128 * 128;
    p.tiles2 = (D + 255) / 256;
    // The filtered signal has no frequency above sigma, so its squared row norm has none above
    // 2 sigma: L > 4 sigma uniform samples of the period determine it on every token (Eq. 7 and 8
    // evaluated off the token grid, then interpolated).  Used when it saves at least a quarter.
    const long long need = 4ll * sigma + 2;
    const long long lp = (need + 127) / 128 * 128;
    p.coarse = (lp * 4 <= 3ll * p.n_pad) ? 1 : 0;
    p.L = p.coarse ? (int)lp : N;
    p.l_pad = p.coarse ? (int)lp : p.n_pad;
    p.phi_elems = (size_t)p.r_pad * p.n_pad;
    p.phi2_elems = p.coarse ? (size_t)p.r_pad * p.l_pad : 0;
    p.yt_elems = (size_t)B * D * p.r_pad;
    p.part_elems = (size_t)B * 2 * p.tiles2 * p.L;
    return p;
}

int spu_tc_run(const SpuTcBuffers& w, const void* hidden, const float2* tw, const float2* tw2, const float* scale,
               int B, int N, int D, int sigma, int* status, cudaStream_t stream, bool have_yt,
               const int32_t* row_index, int src_rows) {
    const SpuTcPlan pl = spu_tc_plan(B, N, D, sigma);
    if (!have_yt || !pl.coarse) {
        const long long phi_n = (long long)pl.phi_elems;
        spu_phi_kernel<<<(unsigned)((phi_n + 255) / 256), 256, 0, stream>>>(
            tw, reinterpret_cast<__nv_bfloat16*>(w.phi_hi), reinterpret_cast<__nv_bfloat16*>(w.phi_lo), N, sigma,
            pl.r_pad, pl.n_pad);
        count_launch();
    }
    if (pl.coarse) {   // the same rows sampled at t_j = j N / L: angle 2 pi k t_j / N = 2 pi k j / L
        const long long phi2_n = (long long)pl.phi2_elems;
        spu_phi_kernel<<<(unsigned)((phi2_n + 255) / 256), 256, 0, stream>>>(
            tw2, reinterpret_cast<__nv_bfloat16*>(w.phi2_hi), reinterpret_cast<__nv_bfloat16*>(w.phi2_lo), pl.L, sigma,
            pl.r_pad, pl.l_pad);
        count_launch();
    }

    // pass 1: YT[d][r] = c[r] * sum_n X[n][d] PhiT[r][n]
    if (!have_yt) {
        TcArgs g = {};
        g.a[0] = reinterpret_cast<const __nv_bfloat16*>(hidden); g.a[1] = nullptr;
        g.b[0] = reinterpret_cast<const __nv_bfloat16*>(w.phi_hi);
        g.b[1] = reinterpret_cast<const __nv_bfloat16*>(w.phi_lo);
        g.a_batch = (long long)(row_index ? src_rows : N) * D; g.b_batch = 0;
        g.a_rows = row_index; g.a_rows_stride = N;
        g.lda = D; g.ldb = pl.n_pad;
        g.m_total = D; g.n_total = pl.r_pad; g.k_a = N; g.k_blocks = (N + TK - 1) / TK;
        const int tiles = (pl.r_pad + 255) / 256;
        g.tn = pl.r_pad <= 256 ? pl.r_pad : 256;
        g.scale = scale;
        g.yt_hi = reinterpret_cast<__nv_bfloat16*>(w.yt_hi); g.yt_lo = reinterpret_cast<__nv_bfloat16*>(w.yt_lo);
        g.ld_yt = pl.r_pad;
        g.status = status;
        const size_t smem = (size_t)kStages * (kABytes + 2 * g.tn * TK * 2);
        cudaFuncSetAttribute(spu_tc_kernel<1, 2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        spu_tc_kernel<1, 2, false><<<dim3((D + TM - 1) / TM, tiles, B), kThreads, smem, stream>>>(g);
        count_launch();
    }
    // pass 2: part[n] = sum_d (sum_r PhiT[r][n] YT[d][r])^2
    {
        TcArgs g = {};
        g.a[0] = reinterpret_cast<const __nv_bfloat16*>(pl.coarse ? w.phi2_hi : w.phi_hi);
        g.a[1] = reinterpret_cast<const __nv_bfloat16*>(pl.coarse ? w.phi2_lo : w.phi_lo);
        g.b[0] = reinterpret_cast<const __nv_bfloat16*>(w.yt_hi);
        g.b[1] = reinterpret_cast<const __nv_bfloat16*>(w.yt_lo);
        g.a_batch = 0; g.b_batch = (long long)D * pl.r_pad;
        g.lda = pl.l_pad; g.ldb = pl.r_pad;
        g.m_total = pl.l_pad; g.n_total = D; g.k_a = pl.r_pad; g.k_blocks = pl.r_pad / TK;
        g.tn = 256;
        g.part = w.part; g.part_n = pl.L;
        g.status = status;
        const size_t smem = (size_t)kStages * (2 * kABytes + 2 * g.tn * TK * 2);
        cudaFuncSetAttribute(spu_tc_kernel<2, 2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        spu_tc_kernel<2, 2, true><<<dim3(pl.l_pad / TM, pl.tiles2, B), kThreads, smem, stream>>>(g);
        count_launch();
    }
    return cudaGetLastError() == cudaSuccess ? LUVC_OK : LUVC_ERR_CUDA;
}

}  // namespace luvc
