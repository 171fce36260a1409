// Internal declarations shared by the translation units of the library
// (host side only; no device code is shared across files).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/luvc.h"

namespace luvc {

// Counts every kernel launch of the library (reported by luvc_kernel_launches).
void count_launch(int n = 1);

// Phase timing (luvc_profile_*): no-ops unless enabled.
void phase_begin(int phase, cudaStream_t stream);
void phase_end(int phase, cudaStream_t stream);

inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

// ---- OIM -------------------------------------------------------------------

struct OimStep {
    int axis;  // 0: lines are rows, the width shrinks; 1: lines are columns, the height shrinks
    int m;     // cells removed per line
    int h, w;  // grid before the step
};

// Final grid for a target count; false if none fits.
bool oim_final_dims(int H, int W, int target, int* Hf, int* Wf);
// Step list from H x W to Hf x Wf; returns false if unreachable.  `steps` may be null (count only).
// r_w cells leave every row in a width step, r_h cells every column in a height step.
bool oim_schedule(int H, int W, int Hf, int Wf, int r_w, int r_h, int height_first, OimStep* steps, int cap, int* n_steps);

struct OimProblem {
    const void* tokens;
    int B, H, W, D, Hf, Wf, r_w, r_h, height_first, dtype;
    int matching;   // luvc_oim_matching
    void* out_tokens;
    int32_t* out_sizes;
    int32_t* out_map;
    int32_t* trace;
    float* out_log_sizes;
    void* workspace;
    int* status;   // device status block: [0] 0 = ok, else a luvc_status; [1], [2] test knobs (see kStatusWords)
    cudaStream_t stream;
};
// Words of a status block.  [1] and [2] are zero in normal use; the wait-expiry test sets them:
// [1] > 0 replaces the probe limit of the chain's waits, [2] is subtracted from the first image's
// count of finished lines of the first step, so that the waits on it can never be satisfied.
enum { kStatusWord = 0, kStatusProbeLimit = 1, kStatusHoldBack = 2, kStatusWords = 4 };
size_t oim_workspace_bytes(int B, int H, int W, int D, int dtype, int matching = 0);
int oim_run(const OimProblem& p);
int oim_value_enhance(const void* values, const int32_t* sizes, long long rows, int D, int dtype, void* out,
                      cudaStream_t stream);

// ---- SPU -------------------------------------------------------------------

struct SpuProblem {
    const void* hidden;
    int B, N, D, sigma, keep, dtype, no_window;
    // Gather on load (the cascade): when row_index is given, token n of sequence b is row
    // row_index[b][n] of sequence b of `hidden`, which then holds src_rows rows per sequence.
    const int32_t* row_index = nullptr;
    int src_rows = 0;
    int32_t* out_idx;
    void* out_hidden;   // may be null: no rows are gathered (the caller does it later)
    float* out_scores;
    void* workspace;
    int* status;   // device status word (see OimProblem)
    cudaStream_t stream;
};
// `indexed`: the problem reads its rows through a row index (only the dense contractions can).
size_t spu_workspace_bytes(int B, int N, int D, int sigma, int dtype, bool indexed = false);
int spu_run(const SpuProblem& p);
// True when a sequence of N tokens would run the dense band contractions anyway (no two-stage plan),
// i.e. when reading it through a row index costs nothing extra.
bool spu_dense_is_natural(int B, int N, int D, int sigma, int dtype);
// out[b][j][:] = hidden[b][idx[b][j]][:] (hidden holds n_src rows per sequence)
int spu_gather_rows(const void* hidden, const int32_t* idx, void* out, int B, int n_src, int keep, int D, int dtype,
                    cudaStream_t stream);
// out[b][j] = prev[b][cur[b][j]] (prev == nullptr: out = cur)
int spu_compose_indices(const int32_t* prev, const int32_t* cur, int32_t* out, int B, int n_prev, int keep,
                        cudaStream_t stream);

// Tensor-core contraction of the bf16 path (spu_tc.cu).
struct SpuTcPlan {
    int r_pad;          // band rows 2 sigma + 1, padded to a multiple of 64
    int n_pad;          // tokens padded to a multiple of 128
    int tiles2;         // 256-channel tiles of the second pass
    int coarse;         // 1: the inverse is evaluated on L < N uniform points t_j = j N / L of the period
    int L;              // points of the inverse (N when not coarse; a multiple of 128 >= 4 sigma + 2 otherwise)
    int l_pad;          // L padded to a multiple of 128
    size_t phi_elems;   // bf16 elements of each half of the band matrix
    size_t phi2_elems;  // bf16 elements of each half of the coarse band matrix (0 when not coarse)
    size_t yt_elems;    // bf16 elements of each half of the spectrum
    size_t part_elems;  // floats of the per-tile energy partials
};
struct SpuTcBuffers {
    void *phi_hi, *phi_lo, *phi2_hi, *phi2_lo, *yt_hi, *yt_lo;
    float* part;
};
SpuTcPlan spu_tc_plan(int B, int N, int D, int sigma);
// Fills part[b][2 * tiles2][L] with per-tile sums of squares of the filtered signal at the L points
// of the plan.  `scale` must hold r_pad entries (zero beyond 2 sigma + 1); `tw2` is the table of
// cos / sin of 2 pi j / L (used when the plan is coarse).
// With `have_yt` the spectrum (yt_hi / yt_lo) is already in place and only the inverse pass runs.
// row_index / src_rows: see SpuProblem (null: the rows are those of `hidden` in order).
int spu_tc_run(const SpuTcBuffers& w, const void* hidden, const float2* tw, const float2* tw2, const float* scale,
               int B, int N, int D, int sigma, int* status, cudaStream_t stream, bool have_yt,
               const int32_t* row_index = nullptr, int src_rows = 0);

// Scratch for the operand images (stage-1 matrices, stage-2 tables) of one transform kernel.
constexpr size_t kSpuImgBytes = 160 * 1024;

// Two-stage forward transform of the bf16 path (spu_fwd2.cu): N = P * Q, P a multiple of 16.
struct SpuFwd2Plan {
    int ok;             // 0: N has no usable factor, use the dense contraction
    int P, Q;
    int nblk;           // 128 / P channel blocks share one tile (block-diagonal stage-1 operand)
    int KB, CH;         // kernel variant: band bins per frequency class and channels per thread
    int slices;         // passes over the input, each covering KB values of k2
    int n_ctiles, n_items;
};
SpuFwd2Plan spu_fwd2_plan(int B, int N, int D, int sigma);
// Y[b][r][d] = c[r] * (band spectrum); also its transposed bf16 pair [b][d][r_pad] when yt_hi is given.
// `img`: kSpuImgBytes of 16-byte aligned device scratch for the operand images a call builds once for all its CTAs.
int spu_fwd2_run(const void* hidden, float* Y, const float* scale, void* yt_hi, void* yt_lo, int r_pad, int B, int N,
                 int D, int sigma, int* status, cudaStream_t stream, void* img, bool img_ready = false);

// Forward transform with both stages on the tensor cores (spu_fwd3.cu): N = 128 Q, 8 <= Q <= 128.
struct SpuFwd3Plan {
    int ok;             // 0: use the two-stage kernel of spu_fwd2.cu (or the dense contraction)
    int Q;
    int geo;            // bins per frequency class and channels per item: 0: up to 4 x 32; 1: up to 8 x 16; 2: up to 16 x 8
    int wide;           // geo != 0
    int slices;         // passes over the input, each covering 4 / 8 / 16 values of k2
    int extra_k2;       // > 0: this one further value of k2 is kept on the CUDA cores (no second pass for it)
    int C, n_ctiles, n_items;
};
SpuFwd3Plan spu_fwd3_plan(int B, int N, int D, int sigma);
// Writes the band spectrum (times c[r]) in the operand form of spu_inv3.cu, ks_out K steps per channel, and, if one more
// bin per frequency class reaches into the band than a pass holds, that bin's cos and sin values to yx[2][B][D].
int spu_fwd3_run(const void* hidden, void* yop, int ks_out, float* yx, const float* scale, int B, int N, int D, int sigma,
                 int* status, cudaStream_t stream, void* img);

// Inverse transform and energies with both stages on the tensor cores (spu_inv3.cu): N = 128 Q, the band spectrum in
// "operand form" (per sequence and channel: [K step][K chunk][128 lanes][16 B], four bf16 per bin).
struct SpuInv3Plan {
    int ok;             // 0: use the two-stage kernel of spu_inv2.cu
    int coarse, J, L;   // as SpuInv2Plan
    int KS;             // K steps of four bins each
    int JP;             // points per channel held in tensor memory: 16, 40 or 72
    int CT;             // channels per tile of the second contraction: 4, 2 or 1
    int extra;          // 1: the bin k = 128 * 16 reaches into the band and is passed apart
    int n_ctiles, n_items, n_parts;
    size_t yop_bytes;   // size of the band spectrum in operand form
};
SpuInv3Plan spu_inv3_plan(int B, int N, int D, int sigma);
// yx_re / yx_im: the cos and sin value of the bin k = 128 * 16 for (b, d) at [b * yx_stride + d] (read only if plan.extra).
int spu_inv3_run(const void* yop, const float* yx_re, const float* yx_im, long long yx_stride, float* part, int B, int N,
                 int D, int sigma, int* status, cudaStream_t stream, void* img);

// Two-stage inverse transform and energies of the bf16 path (spu_inv2.cu); needs the forward plan.
struct SpuInv2Plan {
    int ok;             // 0: use the dense inverse contraction
    int P, Q, nblk;
    int coarse, J, L;   // L = P J points of the period (J = Q, L = N when not coarse)
    int KB, CHT;        // kernel variant
    int n_ctiles, n_items;
    int n_parts;        // partial sums per point and sequence: part[b][n_parts][L]
};
SpuInv2Plan spu_inv2_plan(int B, int N, int D, int sigma);
// img_ready: the caller has built the image already (spu_images.cuh).
int spu_inv2_run(const float* Y, float* part, int B, int N, int D, int sigma, int* status, cudaStream_t stream, void* img,
                 bool img_ready = false);

}  // namespace luvc
