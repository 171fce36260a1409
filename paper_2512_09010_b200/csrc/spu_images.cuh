// Operand images of the two-stage transform kernels (spu_fwd2.cu, spu_inv2.cu), element by element: device
// functions, so that the set-up kernel of a call can build both images and its tables in one launch.
#pragma once

#include <cuda_bf16.h>

namespace luvc {

// Both parts of the forward stage-1 matrix in the layout the kernel's shared memory uses (K-major: element (row j,
// column kk) at (j/8)*128 + (kk/8)*2048 + (j%8)*16 + (kk%8)*2; hi part first, lo part KT*256 bytes later),
// block-diagonal: row j = jb P + jr meets column kk = kb P + p only for jb == kb.  Rows of a block: A[0],
// A[P/2], then Re / Im of A[1 .. P/2-1].  idx < 128 * KT.
__device__ __forceinline__ void spu_fwd2_img_element(unsigned char* __restrict__ img, int P, int KT, int idx) {
    const int j = idx / KT, kk = idx - j * KT;
    const int jb = j / P, jr = j - jb * P, kb = kk / P, p = kk - kb * P;
    float v = 0.f;
    if (j < KT && jb == kb) {
        if (jr == 0) v = 1.f;
        else if (jr == 1) v = (p & 1) ? -1.f : 1.f;
        else {
            const int m = ((jr >> 1) * p) % P;
            float s, c;
            sincospif(2.0f * (float)m / (float)P, &s, &c);
            v = (jr & 1) ? -s : c;
        }
    }
    const __nv_bfloat16 h = __float2bfloat16_rn(v);
    const int off = (j >> 3) * 128 + (kk >> 3) * 2048 + (j & 7) * 16 + (kk & 7) * 2;
    *reinterpret_cast<__nv_bfloat16*>(img + off) = h;
    *reinterpret_cast<__nv_bfloat16*>(img + KT * 256 + off) = __float2bfloat16_rn(v - __bfloat162float(h));
}

// The inverse kernel's image: A[m][kk] = F[kk mod P][m mod P] where row m = jb P + p and column kk = kb P + r share
// the block (jb == kb), K-major as above, hi part then lo part (KT*256 bytes each); behind them
// w[jj][k2] = e^{2 pi i k2 jj / J} as (w.x, w.x, w.y, w.y).  idx < max(128 * KT, J * KB).
__device__ __forceinline__ void spu_inv2_img_element(unsigned char* __restrict__ img, int P, int KT, int J, int KB, int idx) {
    if (idx < 128 * KT) {
        const int m = idx / KT, kk = idx - m * KT;
        const int jb = m / P, p = m - jb * P, kb = kk / P, r = kk - kb * P;
        float v = 0.f;
        if (m < KT && jb == kb) {
            if (r == 0) v = 1.f;
            else if (r == 1) v = (p & 1) ? -1.f : 1.f;
            else {
                float s, c;
                sincospif(2.0f * (float)(((r >> 1) * p) % P) / (float)P, &s, &c);
                v = (r & 1) ? -s : c;
            }
        }
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        const int off = (m >> 3) * 128 + (kk >> 3) * 2048 + (m & 7) * 16 + (kk & 7) * 2;
        *reinterpret_cast<__nv_bfloat16*>(img + off) = h;
        *reinterpret_cast<__nv_bfloat16*>(img + KT * 256 + off) = __float2bfloat16_rn(v - __bfloat162float(h));
    }
    if (idx < J * KB) {
        const int jj = idx / KB, k2 = idx - jj * KB;
        float s, c;
        sincospif(2.0f * (float)(((unsigned)jj * (unsigned)k2) % (unsigned)J) / (float)J, &s, &c);
        reinterpret_cast<float4*>(img + 2 * KT * 256)[idx] = make_float4(c, c, s, s);
    }
}

}  // namespace luvc
