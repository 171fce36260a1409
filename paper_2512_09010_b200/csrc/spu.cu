// Spectrum Pruning Unit (Section 3.3, Eq. 4-8, Algorithm 2) for sm_100a.
//
// The mask of Eq. 5 is zero outside |f| <= sigma, so only the 2*sigma+1 real
// spectral rows of the pass band are ever formed:
//   Phi[n][r] = cos(2 pi r n / N)            r = 0 .. sigma
//   Phi[n][r] = -sin(2 pi (r-sigma) n / N)   r = sigma+1 .. 2 sigma
//   Y  = diag(c) Phi^T X      (Eq. 4 restricted to the band, Eq. 6 and the 1/N and the
//                              factor 2 of the conjugate half folded into c)
//   X' = Phi Y                (Eq. 7; real because the mask is even in f)
//   E[n] = || X'[n, :] ||_2   (Eq. 8)
// followed by an order-preserving top-`keep` selection and a row gather
// (Algorithm 2's last two lines).  fp32 tokens run both contractions on the CUDA
// cores in this file; bf16 tokens run them on the tensor cores (spu_tc.cu) with the
// band matrix and the spectrum held as bf16 pairs and fp32 accumulation.  Reductions
// have a fixed order, so results are reproducible run to run.

#include <cuda_bf16.h>

#include "luvc_internal.h"
#include "spu_images.cuh"

namespace luvc {
namespace {

constexpr int BM = 64, BN = 64, BK = 16;     // tile of the generic contraction
constexpr int kGemmThreads = 256;

// cos / sin of 2 pi j / N for j = 0..N-1, and the per-row constants c[r].
// scale has `scale_len` >= 2 sigma + 1 entries; the extra ones are zero.
// tw2 (may be null) is the same table for a period of L points.
// Blocks past the first `tab_blocks` build the operand images of the two-stage transform kernels (when given):
// `f_blocks` blocks the forward kernel's, the rest the inverse kernel's, so that a call has one set-up launch.
struct SpuImages {
    unsigned char* fwd;     // null: no images in this launch
    unsigned char* inv;
    int P, KT, J, KB_inv, tab_blocks, f_blocks;
};
__global__ void __launch_bounds__(256) spu_tables_kernel(float2* tw, float2* tw2, float* scale, int N, int L, int sigma,
                                                         int scale_len, int no_window, const SpuImages im) {
    if (im.fwd != nullptr && (int)blockIdx.x >= im.tab_blocks) {
        const int rel = (int)blockIdx.x - im.tab_blocks;
        if (rel < im.f_blocks) {
            const int idx = rel * 256 + threadIdx.x;
            if (idx < 128 * im.KT) spu_fwd2_img_element(im.fwd, im.P, im.KT, idx);
        } else {
            spu_inv2_img_element(im.inv, im.P, im.KT, im.J, im.KB_inv, (rel - im.f_blocks) * 256 + threadIdx.x);
        }
        return;
    }
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < N) {
        double s, c;
        sincospi(2.0 * (double)i / (double)N, &s, &c);
        tw[i] = make_float2((float)c, (float)s);
    }
    if (tw2 != nullptr && i < L) {
        double s, c;
        sincospi(2.0 * (double)i / (double)L, &s, &c);
        tw2[i] = make_float2((float)c, (float)s);
    }
    if (i >= 2 * sigma + 1 && i < scale_len) scale[i] = 0.f;
    if (i < 2 * sigma + 1) {
        const int k = i <= sigma ? i : i - sigma;
        double m = 1.0;
        if (!no_window && N > 1) m = 0.54 + 0.46 * cospi(2.0 * (double)k / (double)(N - 1));
        const double mult = (k == 0 || 2 * k == N) ? 1.0 : 2.0;   // bins without a distinct conjugate count once
        scale[i] = (float)(m * mult / (double)N);
    }
}

__device__ __forceinline__ float phi(const float2* __restrict__ tw, int n, int r, int N, int sigma) {
    const bool is_cos = r <= sigma;
    const int k = is_cos ? r : r - sigma;
    // k <= N/2 and n < N: the product fits 32 bits for every N below 65536
    const int j = N < 65536 ? (int)(((unsigned)k * (unsigned)n) % (unsigned)N)
                            : (int)(((unsigned long long)k * (unsigned long long)n) % (unsigned long long)N);
    const float2 t = __ldg(tw + j);
    return is_cos ? t.x : -t.y;
}

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// C[M x D] = A[M x K] * Bm[K x D] with A generated from the twiddle table.
//   FWD:  M = 2 sigma + 1 rows r, K = N tokens;  A[r][n] = Phi[n][r];  Bm = the input (type T);
//         the result, times c[r], is stored to Y[b][r][d].
//   !FWD: M = N tokens, K = 2 sigma + 1;         A[n][r] = Phi[n][r];  Bm = Y (fp32);
//         the squared result is summed over the tile's 64 channels into part[b][d-tile][n].
template <typename T, bool FWD>
__global__ void __launch_bounds__(kGemmThreads) spu_contract_kernel(const void* __restrict__ bm_v,
                                                                    float* __restrict__ out,
                                                                    const float2* __restrict__ tw,
                                                                    const float* __restrict__ scale,
                                                                    int N, int D, int sigma,
                                                                    const int32_t* __restrict__ rows, int src_rows) {
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int R = 2 * sigma + 1;
    const int M = FWD ? R : N, K = FWD ? N : R;
    const int b = blockIdx.z, m0 = blockIdx.y * BM, d0 = blockIdx.x * BN;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const T* xin = reinterpret_cast<const T*>(bm_v) + (size_t)b * (rows ? src_rows : N) * D;   // FWD operand
    const int32_t* rowb = rows ? rows + (size_t)b * N : nullptr;                  // gather on load: token -> row
    const float* yin = reinterpret_cast<const float*>(bm_v) + (size_t)b * R * D;  // !FWD operand

    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int k0 = 0; k0 < K; k0 += BK) {
#pragma unroll
        for (int q = 0; q < BM * BK / kGemmThreads; ++q) {
            const int idx = tid + q * kGemmThreads;
            const int mi = idx % BM, ki = idx / BM;
            const int row = m0 + mi, red = k0 + ki;
            float v = 0.f;
            if (row < M && red < K) v = FWD ? phi(tw, red, row, N, sigma) : phi(tw, row, red, N, sigma);
            As[ki][mi] = v;
        }
#pragma unroll
        for (int q = 0; q < BN * BK / kGemmThreads; ++q) {
            const int idx = tid + q * kGemmThreads;
            const int ni = idx % BN, ki = idx / BN;
            const int red = k0 + ki, d = d0 + ni;
            float v = 0.f;
            if (red < K && d < D)
                v = FWD ? to_f32<T>(xin[(size_t)(rowb ? __ldg(rowb + red) : red) * D + d]) : yin[(size_t)red * D + d];
            Bs[ki][ni] = v;
        }
        __syncthreads();
#pragma unroll
        for (int ki = 0; ki < BK; ++ki) {
            const float4 av = *reinterpret_cast<const float4*>(&As[ki][ty * 4]);
            const float4 bv = *reinterpret_cast<const float4*>(&Bs[ki][tx * 4]);
            const float a[4] = {av.x, av.y, av.z, av.w}, bb[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], bb[j], acc[i][j]);
        }
        __syncthreads();
    }

    if (FWD) {
        float* Y = out + (size_t)b * R * D;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = m0 + ty * 4 + i;
            if (r >= M) continue;
            const float c = scale[r];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int d = d0 + tx * 4 + j;
                if (d < D) Y[(size_t)r * D + d] = c * acc[i][j];
            }
        }
    } else {
        float* part = out + ((size_t)b * gridDim.x + blockIdx.x) * N;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float s = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) s = fmaf(acc[i][j], acc[i][j], s);   // columns beyond D hold zeros
            // the 16 threads that share this row sit in one half-warp
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            const int n = m0 + ty * 4 + i;
            if (tx == 0 && n < M) part[n] = s;
        }
    }
}

// E[b][n] = sqrt(sum over the channel tiles); with `squared` the sum itself.  The order of the sum is
// fixed: thread group g adds tiles g, g + 8, ... in turn, then the eight group sums are added in order.
__global__ void __launch_bounds__(256) spu_energy_kernel(const float* part, float* E, int N, int tiles, long long total,
                                                         int squared) {
    __shared__ float s_sum[8][33];
    const int lane = threadIdx.x & 31, g = threadIdx.x >> 5;
    const long long i = (long long)blockIdx.x * 32 + lane;
    float s = 0.f;
    if (i < total) {
        const int b = (int)(i / N), n = (int)(i % N);
        for (int t = g; t < tiles; t += 8) s += part[((size_t)b * tiles + t) * N + n];
    }
    s_sum[g][lane] = s;
    __syncthreads();
    if (g == 0 && i < total) {
        float r = 0.f;
#pragma unroll
        for (int q = 0; q < 8; ++q) r += s_sum[q][lane];
        E[i] = squared ? r : sqrtf(r);
    }
}

// ---- squared energies from L uniform samples of the period to the N tokens --------------------
//
// S(t) = sum_d x'_d(t)^2 is a real trigonometric polynomial of degree F = 2 sigma, so its L > 2 F
// samples S(j N / L) fix its coefficients g_f = (1/L) sum_j S_j e^{-2 pi i f j / L} exactly, and
// S(n) = g_0 + 2 sum_{f=1..F} Re(g_f e^{2 pi i f n / N}) on the tokens.

constexpr int kSpecChunk = 256;    // samples per partial sum of a coefficient
constexpr int kReseed = 32;        // steps of the rotation recurrence between exact restarts

__device__ __forceinline__ float2 unit_root(long long num, int den) {   // e^{2 pi i num / den}
    const int m = (int)(num % den);
    float s, c;
    sincospif(2.0f * (float)m / (float)den, &s, &c);
    return make_float2(c, s);
}

// gpart[b][chunk][f] = sum over the chunk's samples of S_j e^{-2 pi i f j / L}
__global__ void __launch_bounds__(128) spu_coarse_spectrum_kernel(const float* __restrict__ S, float2* __restrict__ gpart,
                                                                  int L, int F) {
    __shared__ float s_val[kSpecChunk];
    const int b = blockIdx.z, chunk = blockIdx.y, f = blockIdx.x * 128 + threadIdx.x;
    const int j0 = chunk * kSpecChunk, cnt = min(kSpecChunk, L - j0);
    for (int j = threadIdx.x; j < cnt; j += 128) s_val[j] = S[(size_t)b * L + j0 + j];
    __syncthreads();
    if (f > F) return;
    const float2 step = unit_root(f, L);
    float gr = 0.f, gi = 0.f;
    float2 w = make_float2(1.f, 0.f);
    for (int j = 0; j < cnt; ++j) {
        if ((j % kReseed) == 0) w = unit_root((long long)f * (j0 + j), L);
        const float v = s_val[j];
        gr = fmaf(v, w.x, gr);
        gi = fmaf(-v, w.y, gi);                       // conjugate: e^{-i theta}
        const float nx = w.x * step.x - w.y * step.y;
        w.y = fmaf(w.x, step.y, w.y * step.x);
        w.x = nx;
    }
    gpart[((size_t)b * gridDim.y + chunk) * (F + 1) + f] = make_float2(gr, gi);
}

// E[b][n] = sqrt(max(0, S(n))), the coefficient partials summed in chunk order.  A thread forms
// A = sum g.x cos and B = sum g.y sin once and writes two tokens: S(n) = A - B, S(N - n) = A + B.
constexpr int kSynthTile = 2048;   // coefficients staged in shared memory at a time
__global__ void __launch_bounds__(256) spu_coarse_synthesis_kernel(const float2* __restrict__ gpart, float* __restrict__ E,
                                                                   int N, int L, int F, int chunks) {
    __shared__ float2 s_g[kSynthTile];
    const int b = blockIdx.y, n = blockIdx.x * 256 + threadIdx.x;
    const bool live = n <= N / 2;
    const float inv_l = 1.0f / (float)L;
    const float2 step = unit_root(live ? n : 0, N);
    float sa = 0.f, sb = 0.f;
    for (int f0 = 0; f0 <= F; f0 += kSynthTile) {
        const int cnt = min(kSynthTile, F + 1 - f0);
        __syncthreads();
        for (int i = threadIdx.x; i < cnt; i += 256) {
            float gr = 0.f, gi = 0.f;
            for (int c = 0; c < chunks; ++c) {
                const float2 v = gpart[((size_t)b * chunks + c) * (F + 1) + f0 + i];
                gr += v.x; gi += v.y;
            }
            const float m = (f0 + i == 0) ? inv_l : 2.0f * inv_l;
            s_g[i] = make_float2(gr * m, gi * m);
        }
        __syncthreads();
        if (live) {
            float2 w = make_float2(1.f, 0.f);
            for (int i = 0; i < cnt; ++i) {
                if ((i % kReseed) == 0) w = unit_root((long long)(f0 + i) * n, N);
                const float2 g = s_g[i];
                sa = fmaf(g.x, w.x, sa);
                sb = fmaf(g.y, w.y, sb);
                const float nx = w.x * step.x - w.y * step.y;
                w.y = fmaf(w.x, step.y, w.y * step.x);
                w.x = nx;
            }
        }
    }
    if (live) {
        E[(size_t)b * N + n] = sqrtf(fmaxf(sa - sb, 0.f));
        if (n > 0 && n < N - n) E[(size_t)b * N + (N - n)] = sqrtf(fmaxf(sa + sb, 0.f));
    }
}

// ---- the same interpolation in two stages, for L = P J samples and N = P Q tokens ---------------
//
// Analysis, sample j = J j1 + j2, coefficient f = f1 + P f2:
//   g_f = (1/L) sum_{j2} e^{-2 pi i f2 j2 / J} [ e^{-2 pi i f1 j2 / L} sum_{j1} S_{J j1 + j2} e^{-2 pi i f1 j1 / P} ]
// Synthesis, token n = Q n1 + n2:
//   S(n) = Re sum_{f1} e^{2 pi i f1 n1 / P} [ e^{2 pi i f1 n2 / N} sum_{f2} g'_{f1 + P f2} e^{2 pi i f2 n2 / Q} ]
// with g'_0 = g_0, g'_f = 2 g_f.  P (F / P + 1) (J + Q) + P^2 (J + Q) products per sequence instead of (F + 1)(L + N / 2),
// every root taken from an exact table.  A CTA takes eight values of f1 (analysis) or of n2 (synthesis).

constexpr int kInterpSlice = 8;

__device__ __forceinline__ float2 cmul_f(float2 a, float2 b) {
    return make_float2(a.x * b.x - a.y * b.y, fmaf(a.x, b.y, a.y * b.x));
}

// G[b][f] = g'_f, f <= F, from S[b][L]
__global__ void __launch_bounds__(256) spu_interp_analysis_kernel(const float* __restrict__ S, float2* __restrict__ G,
                                                                  int P, int J, int F) {
    extern __shared__ __align__(16) unsigned char interp_smem[];
    const int L = P * J, b = blockIdx.y, f1_0 = blockIdx.x * kInterpSlice;
    float* s_val = reinterpret_cast<float*>(interp_smem);                        // [L]
    float2* s_rp = reinterpret_cast<float2*>(s_val + ((L + 3) & ~3));             // e^{-2 pi i m / P}
    float2* s_rj = s_rp + P;                                                      // e^{-2 pi i m / J}
    float2* s_t = s_rj + J;                                                       // [kInterpSlice][J]
    for (int i = threadIdx.x; i < L; i += 256) s_val[i] = S[(size_t)b * L + i];
    for (int i = threadIdx.x; i < P; i += 256) { const float2 r = unit_root(i, P); s_rp[i] = make_float2(r.x, -r.y); }
    for (int i = threadIdx.x; i < J; i += 256) { const float2 r = unit_root(i, J); s_rj[i] = make_float2(r.x, -r.y); }
    __syncthreads();
    for (int o = threadIdx.x; o < kInterpSlice * J; o += 256) {
        const int fl = o / J, j2 = o - fl * J, f1 = f1_0 + fl;
        float re = 0.f, im = 0.f;
        if (f1 < P) {
            int m = 0;                                   // f1 j1 mod P
            for (int j1 = 0; j1 < P; ++j1) {
                const float v = s_val[J * j1 + j2];
                const float2 w = s_rp[m];
                re = fmaf(v, w.x, re);
                im = fmaf(v, w.y, im);
                m += f1;
                if (m >= P) m -= P;
            }
            const float2 tw = unit_root((long long)f1 * j2, L);       // f1 j2 < P J = L
            const float2 t = cmul_f(make_float2(re, im), make_float2(tw.x, -tw.y));
            re = t.x; im = t.y;
        }
        s_t[o] = make_float2(re, im);
    }
    __syncthreads();
    const int nf2 = F / P + 1;
    const float inv_l = 1.0f / (float)L;
    for (int o = threadIdx.x; o < kInterpSlice * nf2; o += 256) {
        const int fl = o / nf2, f2 = o - fl * nf2, f1 = f1_0 + fl, f = f1 + P * f2;
        if (f1 >= P || f > F) continue;
        float re = 0.f, im = 0.f;
        int m = 0;                                       // f2 j2 mod J
        const int step = f2 % J;
        for (int j2 = 0; j2 < J; ++j2) {
            const float2 t = s_t[fl * J + j2], w = s_rj[m];
            re = fmaf(t.x, w.x, fmaf(-t.y, w.y, re));
            im = fmaf(t.x, w.y, fmaf(t.y, w.x, im));
            m += step;
            if (m >= J) m -= J;
        }
        const float sc = f == 0 ? inv_l : 2.0f * inv_l;
        G[(size_t)b * (F + 1) + f] = make_float2(re * sc, im * sc);
    }
}

// E[b][n] = sqrt(max(0, S(n))) from G[b][f]
__global__ void __launch_bounds__(256) spu_interp_synthesis_kernel(const float2* __restrict__ G, float* __restrict__ E,
                                                                   int P, int Q, int F) {
    extern __shared__ __align__(16) unsigned char interp_smem[];
    const int N = P * Q, b = blockIdx.y, n2_0 = blockIdx.x * kInterpSlice;
    float2* s_g = reinterpret_cast<float2*>(interp_smem);      // [F + 1]
    float2* s_rp = s_g + F + 1;                                 // e^{2 pi i m / P}
    float2* s_rq = s_rp + P;                                    // e^{2 pi i m / Q}
    float2* s_u = s_rq + Q;                                     // [P][kInterpSlice]
    for (int i = threadIdx.x; i <= F; i += 256) s_g[i] = G[(size_t)b * (F + 1) + i];
    for (int i = threadIdx.x; i < P; i += 256) s_rp[i] = unit_root(i, P);
    for (int i = threadIdx.x; i < Q; i += 256) s_rq[i] = unit_root(i, Q);
    __syncthreads();
    for (int o = threadIdx.x; o < P * kInterpSlice; o += 256) {
        const int f1 = o / kInterpSlice, n2 = n2_0 + (o % kInterpSlice);
        float re = 0.f, im = 0.f;
        if (n2 < Q) {
            int m = 0;                                   // f2 n2 mod Q
            for (int f = f1; f <= F; f += P) {
                const float2 g = s_g[f], w = s_rq[m];
                re = fmaf(g.x, w.x, fmaf(-g.y, w.y, re));
                im = fmaf(g.x, w.y, fmaf(g.y, w.x, im));
                m += n2;
                if (m >= Q) m -= Q;
            }
            const float2 t = cmul_f(make_float2(re, im), unit_root((long long)f1 * n2, N));   // f1 n2 < P Q = N
            re = t.x; im = t.y;
        }
        s_u[o] = make_float2(re, im);
    }
    __syncthreads();
    for (int o = threadIdx.x; o < P * kInterpSlice; o += 256) {
        const int n1 = o / kInterpSlice, nl = o % kInterpSlice, n2 = n2_0 + nl;
        if (n2 >= Q) continue;
        float acc = 0.f;
        int m = 0;                                       // f1 n1 mod P
        for (int f1 = 0; f1 < P; ++f1) {
            const float2 u = s_u[f1 * kInterpSlice + nl], w = s_rp[m];
            acc = fmaf(u.x, w.x, fmaf(-u.y, w.y, acc));
            m += n1;
            if (m >= P) m -= P;
        }
        E[(size_t)b * N + (size_t)Q * n1 + n2] = sqrtf(fmaxf(acc, 0.f));
    }
}

size_t interp_analysis_smem(int P, int J) { return ((size_t)((P * J + 3) & ~3)) * 4 + (size_t)(P + J + kInterpSlice * J) * 8; }
size_t interp_synthesis_smem(int P, int Q, int F) { return (size_t)(F + 1 + P + Q + P * kInterpSlice) * 8; }
constexpr size_t kInterpSmemMax = 200 * 1024;

// ---- order-preserving top-k ---------------------------------------------------

constexpr int kSelThreads = 1024;

__device__ __forceinline__ unsigned score_key(float e) {
    // scores are >= 0, so their bit patterns order like the values; anything else
    // (a NaN from non-finite input) ranks lowest
    return (e >= 0.f) ? __float_as_uint(e) : 0u;
}

// Exclusive prefix sum of one int per thread over the block; returns the block total in `total`.
__device__ int block_exclusive_scan(int v, int* s_warp, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();                 // s_warp may still be read from the previous call
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int w = lane < (kSelThreads >> 5) ? s_warp[lane] : 0;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, w, o);
            if (lane >= o) w += t;
        }
        s_warp[lane] = w;            // inclusive totals per warp
    }
    __syncthreads();
    total = s_warp[31];
    return inc - v + (warp ? s_warp[warp - 1] : 0);
}

// One CTA per sequence: radix-select the keep-th largest key (4 passes of 8 bits),
// then one ordered sweep that keeps everything above it plus the first equal ones.
__global__ void __launch_bounds__(kSelThreads) spu_select_kernel(const float* __restrict__ E, int32_t* __restrict__ out_idx,
                                                                 int N, int keep) {
    __shared__ int s_hist[256];
    __shared__ int s_warp[32];
    __shared__ unsigned s_prefix;
    __shared__ int s_remaining;
    const int b = blockIdx.x, tid = threadIdx.x;
    const float* e = E + (size_t)b * N;
    if (tid == 0) { s_prefix = 0u; s_remaining = keep; }
    for (int pass = 3; pass >= 0; --pass) {
        for (int i = tid; i < 256; i += kSelThreads) s_hist[i] = 0;
        __syncthreads();
        const unsigned prefix = s_prefix;
        const unsigned himask = pass == 3 ? 0u : (0xffffffffu << (8 * (pass + 1)));
        for (int n = tid; n < N; n += kSelThreads) {
            const unsigned key = score_key(e[n]);
            if ((key & himask) == prefix) atomicAdd(&s_hist[(key >> (8 * pass)) & 255u], 1);
        }
        __syncthreads();
        if (tid < 32) {
            // the bucket in which the count from the top reaches `rem`: lane l owns buckets 8l .. 8l+7
            const int rem = s_remaining;
            int h[8], mine = 0;
#pragma unroll
            for (int q = 0; q < 8; ++q) { h[q] = s_hist[tid * 8 + q]; mine += h[q]; }
            int above = mine;                                  // inclusive sum over lanes >= tid
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_down_sync(0xffffffffu, above, o);
                if (tid + o < 32) above += v;
            }
            above -= mine;                                     // keys in the buckets of the lanes above this one
            const bool here = above < rem && above + mine >= rem;
            const unsigned who = __ballot_sync(0xffffffffu, here);
            if (who == 0u) {                                   // fewer keys than asked for (cannot happen): bucket 0
                if (tid == 0) { s_prefix = prefix; s_remaining = rem; }
            } else if (tid == 31 - __clz(who)) {
                int r = rem - above, bucket = 7;
                for (; bucket > 0; --bucket) {
                    if (h[bucket] >= r) break;
                    r -= h[bucket];
                }
                s_prefix = prefix | ((unsigned)(tid * 8 + bucket) << (8 * pass));
                s_remaining = r;
            }
        }
        __syncthreads();
    }
    const unsigned thr = s_prefix;      // the keep-th largest key
    const int take_equal = s_remaining; // how many keys equal to it are kept (lowest indices first)
    int32_t* out = out_idx + (size_t)b * keep;
    int eq_seen = 0, written = 0;
    for (int n0 = 0; n0 < N; n0 += kSelThreads) {
        const int n = n0 + tid;
        const unsigned key = n < N ? score_key(e[n]) : 0u;
        const int is_eq = (n < N && key == thr) ? 1 : 0;
        int eq_total;
        const int eq_rank = eq_seen + block_exclusive_scan(is_eq, s_warp, eq_total);
        const int kept = (n < N && (key > thr || (is_eq && eq_rank < take_equal))) ? 1 : 0;
        int kept_total;
        const int pos = written + block_exclusive_scan(kept, s_warp, kept_total);
        if (kept) out[pos] = n;
        eq_seen += eq_total;
        written += kept_total;
    }
}

// out_hidden[b][j][:] = hidden[b][idx[b][j]][:], 16 bytes per thread per trip.
__global__ void __launch_bounds__(128) spu_gather_kernel(const uint4* __restrict__ hidden, const int32_t* __restrict__ idx,
                                                         uint4* __restrict__ out, int N, int keep, int row_vec) {
    const int b = blockIdx.y, j = blockIdx.x;
    const int src = idx[(size_t)b * keep + j];
    const uint4* in = hidden + ((size_t)b * N + src) * row_vec;
    uint4* o = out + ((size_t)b * keep + j) * row_vec;
    for (int v = threadIdx.x; v < row_vec; v += 128) o[v] = __ldg(in + v);
}

struct Workspace {
    float2* tw;
    float2* tw2;     // table for the coarse period (dense inverse)
    float* S;        // squared energies at the coarse points [B][L]
    float2* gpart;   // their spectrum, partial sums [B][chunks][2 sigma * 2 + 1]
    float* scale;
    float* E;
    // fp32 path (CUDA cores)
    float* Y;
    float* part;
    // bf16 path (tensor cores)
    SpuTcBuffers tc;
    float* Y2;       // band spectrum of the two-stage forward transform [B][2 sigma + 1][D]
    void *img_fwd, *img_inv;   // operand images of the forward / inverse transform kernel, built once per call
    void* yop;       // band spectrum in the operand form of the tensor-core inverse
    float* yx;       // [2][B][D] its one bin past sixteen per frequency class
};

// How the bf16 path runs a problem, and the points its inverse is evaluated on.
struct Bf16Mode {
    bool fwd2, inv2;    // two-stage forward / inverse kernels (else the dense contractions of spu_tc.cu)
    bool tc2;           // both of them with their second stage on the tensor cores too (spu_fwd3.cu, spu_inv3.cu)
    int coarse, L;      // the inverse is evaluated on L uniform points of the period (L = N: the tokens)
    int n_parts;        // partial energy sums per point
    int P, Q, J;        // two-stage kernels: N = P Q tokens, L = P J points
};
Bf16Mode bf16_mode(int B, int N, int D, int sigma, bool dense) {
    const SpuTcPlan tc = spu_tc_plan(B, N, D, sigma);
    const SpuInv2Plan iv = spu_inv2_plan(B, N, D, sigma);
    Bf16Mode m;
    m.fwd2 = !dense && spu_fwd2_plan(B, N, D, sigma).ok != 0;   // `dense`: rows come through an index, which only
                                                                // the dense contractions can follow
    m.inv2 = m.fwd2 && iv.ok != 0;
    const SpuInv3Plan iv3 = spu_inv3_plan(B, N, D, sigma);       // (needs the plan of spu_fwd3.cu)
    m.tc2 = m.inv2 && iv3.ok != 0;
    m.coarse = m.inv2 ? iv.coarse : tc.coarse;
    m.L = m.inv2 ? iv.L : tc.L;
    m.n_parts = m.tc2 ? iv3.n_parts : (m.inv2 ? iv.n_parts : 2 * tc.tiles2);
    m.P = m.inv2 ? iv.P : 0; m.Q = m.inv2 ? iv.Q : 0; m.J = m.inv2 ? iv.J : 0;
    return m;
}

size_t coarse_gpart_elems(int B, int L, int sigma) {
    return (size_t)B * ((L + kSpecChunk - 1) / kSpecChunk) * (4 * (size_t)sigma + 1);
}

// Both paths share the twiddle table, the row constants and the scores; the rest differs.
// With ws == nullptr only the size is computed.
Workspace carve(void* ws, int B, int N, int D, int sigma, bool tensor_path, bool dense, size_t* total) {
    unsigned char* p = static_cast<unsigned char*>(ws);
    unsigned char* const p0 = p;
    const int R = 2 * sigma + 1, tiles = (D + BN - 1) / BN;
    const SpuTcPlan pl = spu_tc_plan(B, N, D, sigma);
    Workspace w = {};
    auto take = [&](size_t bytes) { unsigned char* q = p; p += align_up(bytes); return q; };
    w.tw = reinterpret_cast<float2*>(take((size_t)N * sizeof(float2)));
    w.scale = reinterpret_cast<float*>(take((size_t)pl.r_pad * 4));
    w.E = reinterpret_cast<float*>(take((size_t)B * N * 4));
    if (!tensor_path) {
        w.Y = reinterpret_cast<float*>(take((size_t)B * R * D * 4));
        w.part = reinterpret_cast<float*>(take((size_t)B * tiles * N * 4));
    } else {
        const Bf16Mode m = bf16_mode(B, N, D, sigma, dense);
        if (m.coarse) {
            w.S = reinterpret_cast<float*>(take((size_t)B * m.L * 4));
            w.gpart = reinterpret_cast<float2*>(take(coarse_gpart_elems(B, m.L, sigma) * sizeof(float2)));
        }
        if (m.fwd2) {
            if (m.tc2) {
                w.yop = take(spu_inv3_plan(B, N, D, sigma).yop_bytes);
                w.yx = reinterpret_cast<float*>(take((size_t)2 * B * D * sizeof(float)));
            } else {
                w.Y2 = reinterpret_cast<float*>(take((size_t)B * R * D * sizeof(float)));
            }
            w.img_fwd = take(kSpuImgBytes);
            w.img_inv = take(kSpuImgBytes);
        }
        w.tc.part = reinterpret_cast<float*>(take((size_t)B * m.n_parts * m.L * 4));
        if (!m.inv2) {      // the dense inverse (and, without the two-stage forward, the dense forward)
            if (!m.fwd2 || !pl.coarse) {
                w.tc.phi_hi = take(pl.phi_elems * 2);
                w.tc.phi_lo = take(pl.phi_elems * 2);
            }
            if (pl.coarse) {
                w.tc.phi2_hi = take(pl.phi2_elems * 2);
                w.tc.phi2_lo = take(pl.phi2_elems * 2);
                w.tw2 = reinterpret_cast<float2*>(take((size_t)pl.L * sizeof(float2)));
            }
            w.tc.yt_hi = take(pl.yt_elems * 2);
            w.tc.yt_lo = take(pl.yt_elems * 2);
        }
    }
    if (total) *total = (size_t)(p - p0);
    return w;
}

}  // namespace

size_t spu_workspace_bytes(int B, int N, int D, int sigma, int dtype, bool indexed) {
    size_t total = 0;
    carve(nullptr, B, N, D, sigma, dtype != LUVC_F32, indexed, &total);
    return total;
}

bool spu_dense_is_natural(int B, int N, int D, int sigma, int dtype) {
    return dtype == LUVC_F32 || !spu_fwd2_plan(B, N, D, sigma).ok;
}

template <typename T>
static int spu_run_typed(const SpuProblem& p) {
    constexpr bool kTensor = sizeof(T) == 2;     // bf16 tokens go through the tensor cores
    const int N = p.N, D = p.D, B = p.B, sigma = p.sigma, R = 2 * sigma + 1;
    const SpuTcPlan pl = spu_tc_plan(B, N, D, sigma);
    const bool indexed = p.row_index != nullptr;
    Workspace ws = carve(p.workspace, B, N, D, sigma, kTensor, indexed, nullptr);
    float* E = p.out_scores ? p.out_scores : ws.E;
    const Bf16Mode mode = kTensor ? bf16_mode(B, N, D, sigma, indexed) : Bf16Mode{};
    const int tab = max(max(N, pl.r_pad), pl.L);
    const long long bn = (long long)B * N;
    phase_begin(LUVC_PHASE_SPU_TRANSFORM, p.stream);
    SpuImages im = {};
    im.tab_blocks = (tab + 255) / 256;
    int img_blocks = 0;
    if constexpr (kTensor) {
        if (mode.fwd2 && mode.inv2 && !mode.tc2) {      // both two-stage kernels run: their images ride along
            const SpuFwd2Plan fp = spu_fwd2_plan(B, N, D, sigma);
            const SpuInv2Plan ip = spu_inv2_plan(B, N, D, sigma);
            im.fwd = static_cast<unsigned char*>(ws.img_fwd);
            im.inv = static_cast<unsigned char*>(ws.img_inv);
            im.P = fp.P; im.KT = fp.nblk * fp.P; im.J = ip.J; im.KB_inv = ip.KB;
            im.f_blocks = (128 * im.KT + 255) / 256;
            img_blocks = im.f_blocks + (max(128 * im.KT, ip.J * ip.KB) + 255) / 256;
        }
    }
    spu_tables_kernel<<<im.tab_blocks + img_blocks, 256, 0, p.stream>>>(ws.tw, ws.tw2, ws.scale, N, pl.L, sigma, pl.r_pad,
                                                                        p.no_window, im);
    count_launch();
    if constexpr (kTensor) {
        int rc;
        if (mode.tc2) {
            const SpuInv3Plan iv3 = spu_inv3_plan(B, N, D, sigma);
            rc = spu_fwd3_run(p.hidden, ws.yop, iv3.KS, ws.yx, ws.scale, B, N, D, sigma, p.status, p.stream, ws.img_fwd);
            if (rc != LUVC_OK) return rc;
            rc = spu_inv3_run(ws.yop, ws.yx, ws.yx + (size_t)B * D, D, ws.tc.part, B, N, D, sigma, p.status, p.stream,
                              ws.img_inv);
        } else {
            if (mode.fwd2) {
                const int rc1 = spu_fwd2_run(p.hidden, ws.Y2, ws.scale, mode.inv2 ? nullptr : ws.tc.yt_hi,
                                             mode.inv2 ? nullptr : ws.tc.yt_lo, pl.r_pad, B, N, D, sigma, p.status, p.stream, ws.img_fwd,
                                             im.fwd != nullptr);
                if (rc1 != LUVC_OK) return rc1;
            }
            rc = mode.inv2 ? spu_inv2_run(ws.Y2, ws.tc.part, B, N, D, sigma, p.status, p.stream, ws.img_inv, im.fwd != nullptr)
                           : spu_tc_run(ws.tc, p.hidden, ws.tw, ws.tw2, ws.scale, B, N, D, sigma, p.status,
                                        p.stream, mode.fwd2, p.row_index, p.src_rows);
        }
        if (rc != LUVC_OK) return rc;
        if (!mode.coarse) {
            spu_energy_kernel<<<(unsigned)((bn + 31) / 32), 256, 0, p.stream>>>(ws.tc.part, E, N, mode.n_parts, bn, 0);
            count_launch();
        } else {
            const int L = mode.L, F = 2 * sigma, chunks = (L + kSpecChunk - 1) / kSpecChunk;
            const long long bl = (long long)B * L;
            spu_energy_kernel<<<(unsigned)((bl + 31) / 32), 256, 0, p.stream>>>(ws.tc.part, ws.S, L, mode.n_parts, bl, 1);
            const size_t sm_a = mode.inv2 ? interp_analysis_smem(mode.P, mode.J) : 0;
            const size_t sm_s = mode.inv2 ? interp_synthesis_smem(mode.P, mode.Q, F) : 0;
            if (mode.inv2 && sm_a <= kInterpSmemMax && sm_s <= kInterpSmemMax) {
                // L = P J and N = P Q: the interpolation factors into two short stages
                cudaFuncSetAttribute(spu_interp_analysis_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_a);
                cudaFuncSetAttribute(spu_interp_synthesis_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_s);
                spu_interp_analysis_kernel<<<dim3((mode.P + kInterpSlice - 1) / kInterpSlice, B), 256, sm_a, p.stream>>>(
                    ws.S, ws.gpart, mode.P, mode.J, F);
                spu_interp_synthesis_kernel<<<dim3((mode.Q + kInterpSlice - 1) / kInterpSlice, B), 256, sm_s, p.stream>>>(
                    ws.gpart, E, mode.P, mode.Q, F);
            } else {
                spu_coarse_spectrum_kernel<<<dim3((F + 128) / 128, chunks, B), 128, 0, p.stream>>>(ws.S, ws.gpart, L, F);
                spu_coarse_synthesis_kernel<<<dim3((N / 2 + 256) / 256, B), 256, 0, p.stream>>>(ws.gpart, E, N, L, F, chunks);
            }
            count_launch(3);
        }
    } else {
        const int tiles = (D + BN - 1) / BN;
        spu_contract_kernel<T, true><<<dim3(tiles, (R + BM - 1) / BM, B), kGemmThreads, 0, p.stream>>>(
            p.hidden, ws.Y, ws.tw, ws.scale, N, D, sigma, p.row_index, p.src_rows);
        spu_contract_kernel<T, false><<<dim3(tiles, (N + BM - 1) / BM, B), kGemmThreads, 0, p.stream>>>(
            ws.Y, ws.part, ws.tw, ws.scale, N, D, sigma, nullptr, 0);
        spu_energy_kernel<<<(unsigned)((bn + 31) / 32), 256, 0, p.stream>>>(ws.part, E, N, tiles, bn, 0);
        count_launch(3);
    }
    phase_end(LUVC_PHASE_SPU_TRANSFORM, p.stream);
    phase_begin(LUVC_PHASE_SPU_SELECT, p.stream);
    spu_select_kernel<<<B, kSelThreads, 0, p.stream>>>(E, p.out_idx, N, p.keep);
    phase_end(LUVC_PHASE_SPU_SELECT, p.stream);
    count_launch();
    if (p.out_hidden != nullptr && !indexed) {
        phase_begin(LUVC_PHASE_SPU_GATHER, p.stream);
        const int row_vec = (int)((size_t)D * sizeof(T) / 16);
        spu_gather_kernel<<<dim3(p.keep, B), 128, 0, p.stream>>>(reinterpret_cast<const uint4*>(p.hidden), p.out_idx,
                                                                reinterpret_cast<uint4*>(p.out_hidden), N, p.keep, row_vec);
        phase_end(LUVC_PHASE_SPU_GATHER, p.stream);
        count_launch();
    }
    return cudaGetLastError() == cudaSuccess ? LUVC_OK : LUVC_ERR_CUDA;
}

int spu_gather_rows(const void* hidden, const int32_t* idx, void* out, int B, int n_src, int keep, int D, int dtype,
                    cudaStream_t stream) {
    const int row_vec = (int)((size_t)D * (dtype == LUVC_F32 ? 4 : 2) / 16);
    spu_gather_kernel<<<dim3(keep, B), 128, 0, stream>>>(reinterpret_cast<const uint4*>(hidden), idx,
                                                         reinterpret_cast<uint4*>(out), n_src, keep, row_vec);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LUVC_OK : LUVC_ERR_CUDA;
}

__global__ void spu_compose_kernel(const int32_t* __restrict__ prev, const int32_t* __restrict__ cur,
                                   int32_t* __restrict__ out, int n_prev, int keep, long long total) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const int b = (int)(i / keep);
    const int c = cur[i];
    out[i] = prev ? prev[(size_t)b * n_prev + c] : c;
}

int spu_compose_indices(const int32_t* prev, const int32_t* cur, int32_t* out, int B, int n_prev, int keep,
                        cudaStream_t stream) {
    const long long total = (long long)B * keep;
    spu_compose_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(prev, cur, out, n_prev, keep, total);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LUVC_OK : LUVC_ERR_CUDA;
}

int spu_run(const SpuProblem& p) {
    return p.dtype == LUVC_F32 ? spu_run_typed<float>(p) : spu_run_typed<__nv_bfloat16>(p);
}

}  // namespace luvc
