/*
 * luvc.h - C ABI of the LUVC token-compression library for NVIDIA B200 (sm_100a).
 *
 * Two training-free operators of "Towards Lossless Ultimate Vision Token
 * Compression for VLMs" (arXiv 2512.09010):
 *
 *   OIM  Orthogonal Iterative Merger (Section 3.2; Eq. 3; appendix "Iterative
 *        Strategy and Pseudocode of OIM", Algorithm 1): merges similar
 *        neighbouring vision tokens on the 2D patch grid, alternately along the
 *        width and the height, so that the grid stays rectangular.
 *   SPU  Spectrum Pruning Unit (Section 3.3, Eq. 4-8; Algorithm 2): scores every
 *        visual token by the energy of the low-pass-filtered token sequence and
 *        keeps the highest-scoring tokens in their original order.
 *
 * General rules
 *   - Every function returns a luvc_status (int); 0 is success.  Nothing aborts
 *     or throws.  Argument errors are reported before any work is queued and
 *     leave the outputs untouched.
 *   - Unless a function says "host", every data pointer is a DEVICE pointer
 *     owned by the caller (for PyTorch: tensor.data_ptr()).  The library never
 *     frees or keeps caller memory.  Inputs are not modified.  Outputs must not
 *     overlap inputs.
 *   - Tensors are dense, row-major, innermost dimension D contiguous.  Base
 *     pointers must be 16-byte aligned and D * sizeof(element) a multiple of 16
 *     (D % 8 == 0 for bf16, D % 4 == 0 for fp32), else LUVC_ERR_ALIGN.
 *   - Device calls are asynchronous on the calling thread's luvc stream (see
 *     luvc_set_stream) and do not synchronise the host.
 *   - The plain entry points use library-owned scratch buffers, one set per
 *     device (keyed by the ordinal of the device that is current at the call),
 *     grown with cudaMalloc on demand (a host-synchronous call the first time a
 *     larger problem is seen) and released by luvc_shutdown().  All calls on a
 *     device share that one set: two calls whose GPU work overlaps (two streams,
 *     or two host threads) race on it and give undefined results - keep them on
 *     one stream, order them with events, or give each its own workspace through
 *     the _ex forms.  An _ex call that is given a workspace uses only that
 *     workspace; given a device_status word as well it touches no library-owned
 *     memory at all.
 */
#ifndef LUVC_H_
#define LUVC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LUVC_OK = 0,
    LUVC_ERR_NULL = 1,       /* a required pointer is NULL */
    LUVC_ERR_SHAPE = 2,      /* a dimension is < 1 or too large for 32-bit indexing */
    LUVC_ERR_TARGET = 3,     /* target_count / output grid not reachable from H x W */
    LUVC_ERR_KEEP = 4,       /* keep outside [1, N] */
    LUVC_ERR_CUTOFF = 5,     /* cutoff is NaN or > 1 */
    LUVC_ERR_ALIGN = 6,      /* pointer or row size not 16-byte aligned */
    LUVC_ERR_DTYPE = 7,      /* unknown element type */
    LUVC_ERR_WORKSPACE = 8,  /* caller workspace too small or misaligned */
    LUVC_ERR_CUDA = 9,       /* a CUDA call failed (allocation, copy, launch) */
    LUVC_ERR_TIMEOUT = 10,   /* a bounded device-side wait gave up */
    LUVC_ERR_INTERNAL = 11
} luvc_status;

typedef enum { LUVC_BF16 = 0, LUVC_F32 = 1 } luvc_dtype;

/* Cutoff used when the caller passes cutoff <= 0.  The paper never states the
 * value of its sigma_t; 1/8 of the band is this library's choice. */
#define LUVC_SPU_DEFAULT_CUTOFF 0.125f

/* ---- housekeeping ------------------------------------------------------- */

/* Library version, major * 1000 + minor. */
int luvc_version(void);

/* Static, NUL-terminated description of a status code. */
const char* luvc_status_string(int status);

/* Sets the CUDA stream (a cudaStream_t passed as void*) used by the plain entry
 * points of the calling host thread.  NULL selects the legacy default stream. */
int luvc_set_stream(void* cuda_stream);

/* Device-side conditions (a bounded wait inside a kernel that gave up) are written
 * to a status word in device memory instead of trapping.  This call synchronises
 * the given stream, returns the current device's library-owned word as a
 * luvc_status (LUVC_OK if nothing was reported) and clears it.  While a word is
 * set, operator calls that use it stop early and leave their outputs untouched or
 * partly written (undefined, but every access stays inside the caller's buffers).
 * Calls that were given their own word (device_status of the option structs) report
 * there instead; luvc_read_status reads and clears such a word. */
int luvc_check_status(void* cuda_stream);
int luvc_read_status(int32_t* device_status, void* cuda_stream);

/* Bytes a caller-owned status block must have (device memory, 16-byte aligned, zeroed
 * by the caller before its first use; the library only ever writes its first word). */
#define LUVC_STATUS_BYTES 16

/* Test hook for the give-up path of the bounded device-side waits (no counterpart in the paper).
 * Writes two knobs into a status block (device_status, or the current device's library-owned
 * block when NULL): `probes` > 0 replaces the probe limit of the OIM chain's waits, and
 * `hold_back` > 0 starts the first image's count of finished lines of the first merge step that
 * far below zero, so that no wait on it can ever be satisfied and each gives up after `probes`
 * probes (microseconds).  The call that follows then ends with LUVC_ERR_TIMEOUT in the block.
 * 0, 0 restores normal operation.  Synchronises the stream. */
int luvc_debug_wait_probes(int probes, int hold_back, int32_t* device_status, void* cuda_stream);

/* Frees the library-owned scratch buffers of the current device (and its status
 * word).  Synchronises the device first.  Safe to call more than once. */
int luvc_shutdown(void);

/* Number of kernels this library has launched since it was loaded (all threads). */
long long luvc_kernel_launches(void);

/* Phase timing for benchmarks.  While enabled, every operator call records CUDA
 * events on its stream around its phases (two event records per phase, nothing
 * else changes).  luvc_profile_read synchronises those events and returns the
 * elapsed milliseconds of the most recent call's phases, indexed by luvc_phase;
 * phases that did not run since the last read are reported as 0. */
typedef enum {
    LUVC_PHASE_OIM_STEPS = 0,      /* all merge-step launches of one luvc_oim_merge* call */
    LUVC_PHASE_OIM_TOTAL = 1,      /* the whole call: init, steps, emit, map */
    LUVC_PHASE_SPU_TRANSFORM = 2,  /* tables, forward band DFT, inverse, energies */
    LUVC_PHASE_SPU_SELECT = 3,
    LUVC_PHASE_SPU_GATHER = 4,
    LUVC_PHASE_COUNT = 5
} luvc_phase;
int luvc_profile_enable(int on);
int luvc_profile_read(float* ms, int count);

/* ---- OIM ---------------------------------------------------------------- */

/* Host-only planning.  Maps target_count to the final grid out_h x out_w: the
 * factor pair of target_count with out_h <= H, out_w <= W whose aspect ratio is
 * closest, in log scale, to H / W (tie: larger out_h), and counts the merge
 * steps needed with `merge_per_step` cells removed per line per step
 * (0 = the paper's merge number 2).  LUVC_ERR_TARGET if no such pair exists. */
int luvc_oim_plan(int H, int W, int target_count, int merge_per_step,
                  int* out_h, int* out_w, int* n_steps);

/* Host-only planning for grids whose sides differ (appendix "Iterative Strategy and Pseudocode of
 * OIM": for an encoder that keeps the image's aspect ratio the merges along the two spatial axes
 * follow that ratio; the paper gives no formula, this is the library's reading).  n_ops operations
 * of one width step and one height step each; the shorter side loses merge_per_step (0 = 2) cells
 * per step, the longer side round(merge_per_step * long / short), so the grid keeps its shape.
 * Returns the per-axis numbers (for luvc_oim_opts.merge_per_step_h / _w), the final grid
 * (for out_h / out_w; target_count = out_h * out_w) and the number of steps.
 * LUVC_ERR_TARGET if a side would shrink below one cell. */
int luvc_oim_plan_anyres(int H, int W, int n_ops, int merge_per_step, int* merge_h, int* merge_w,
                         int* out_h, int* out_w, int* n_steps);

/* Bytes of workspace luvc_oim_merge_ex needs for this problem with the adjacent matching;
 * the _ex form takes the luvc_oim_matching (the bipartite matching also keeps a bf16
 * hi + lo copy of every fp32 row).  0 for invalid arguments. */
size_t luvc_oim_workspace_bytes(int B, int H, int W, int D, int dtype);
size_t luvc_oim_workspace_bytes_ex(int B, int H, int W, int D, int dtype, int matching);

/*
 * The two readings of "similarity calculations and binary matching" (Section 3.2).
 * ADJACENT: a cell at an even position of a line is compared with its one or two
 * neighbours in the line.  BIPARTITE: the line is split into its even-position cells
 * (set A) and odd-position cells (set B), every A cell is compared with EVERY B cell
 * of the line (one ceil(len/2) x floor(len/2) similarity matrix per line, the
 * O(n_v^1.5 k) cost the section states), proposes the most similar one (ties: lowest
 * position), and the m best proposals (ties: lowest A position) are merged; several A
 * cells may merge into one B cell.  BIPARTITE needs H <= 256 and W <= 256
 * (LUVC_ERR_SHAPE otherwise) and D a multiple of 8 (LUVC_ERR_ALIGN), a larger workspace
 * (luvc_oim_workspace_bytes_ex), and its trace entries are
 * (position of the merged A cell << 16) | position of the B cell it merged into.
 */
typedef enum {
    LUVC_OIM_MATCH_ADJACENT = 0,
    LUVC_OIM_MATCH_BIPARTITE = 1
} luvc_oim_matching;

typedef struct {
    int dtype;               /* luvc_dtype of tokens and out_tokens */
    void* stream;            /* cudaStream_t; NULL = legacy default stream */
    void* workspace;         /* device, 256-byte aligned; NULL = library-owned scratch */
    size_t workspace_bytes;
    int out_h, out_w;        /* explicit final grid; 0,0 = derive from target_count */
    int merge_per_step;      /* cells removed per line per step; 0 = 2 (appendix of the paper) */
    int height_first;        /* 0: width step first (Section 3.2); 1: Algorithm 1's order */
    int32_t* trace;          /* optional device [B, H*W - out_h*out_w]: one entry per merge,
                                (position of the merged cell in its line) * 2 + direction
                                (0 = into the previous cell of the line, 1 = into the next),
                                ordered by step, line, rank of the candidate */
    size_t trace_bytes;      /* size of the trace buffer; with trace != NULL it must be at least
                                B * (H*W - out_h*out_w) * 4, else LUVC_ERR_WORKSPACE (nothing is queued) */
    float* out_log_sizes;    /* optional device [B, target_count] fp32: log(s), the bias that the
                                value enhancement of Eq. 2 adds to the values (V + log s) */
    int matching;            /* LUVC_OIM_MATCH_ADJACENT (0) or LUVC_OIM_MATCH_BIPARTITE: which cells
                                of a line are compared (see luvc_oim_matching) */
    int32_t* device_status;  /* optional device block of LUVC_STATUS_BYTES (see luvc_read_status);
                                NULL = the library-owned word of the current device */
    int merge_per_step_h;    /* cells removed per COLUMN per height step (0 = merge_per_step) */
    int merge_per_step_w;    /* cells removed per ROW per width step (0 = merge_per_step) */
} luvc_oim_opts;

/*
 * Orthogonal Iterative Merger (Section 3.2).
 *
 * tokens      [B, H, W, D]  patch tokens of B images on their 2D grid
 * out_tokens  [B, target_count, D]  merged tokens, row-major over the final grid;
 *             each is the mean of its source tokens (the size-weighted merge
 *             composed over the steps), rounded once to the element type
 * out_sizes   [B, target_count] int32  number of source tokens per merged token
 *             (the vector s of Eq. 3)
 * out_map     [B, H*W] int32  final cell (row-major index) each source token ended in
 *
 * The iteration alternates one width step and one height step until the grid is
 * out_h x out_w.  A step treats every line (row or column) independently: cells
 * at even positions compare themselves (cosine, fp32 accumulation) with their
 * one or two neighbours in the line, the m cells with the highest similarity
 * (ties: lowest position; direction ties: the previous cell) are merged into
 * that neighbour, and the line closes up keeping its order.
 *
 * luvc_oim_merge takes bf16, luvc_oim_merge_f32 fp32; both run on the thread's
 * luvc stream with library-owned scratch.
 */
int luvc_oim_merge(const void* tokens, int B, int H, int W, int D, int target_count,
                   void* out_tokens, int32_t* out_sizes, int32_t* out_map);
int luvc_oim_merge_f32(const float* tokens, int B, int H, int W, int D, int target_count,
                       float* out_tokens, int32_t* out_sizes, int32_t* out_map);
int luvc_oim_merge_ex(const void* tokens, int B, int H, int W, int D, int target_count,
                      void* out_tokens, int32_t* out_sizes, int32_t* out_map,
                      const luvc_oim_opts* opts);

/* Same operator on HOST buffers (pinned memory recommended): copies the tokens to
 * the device, runs, copies the three outputs back and synchronises the stream
 * before returning.  dtype is a luvc_dtype.  The staging buffers belong to the
 * library and are separate for luvc_oim_merge_host and luvc_spu_prune_host: one
 * call of each may run at the same time from two host threads, each on its own
 * luvc stream (the copies of one then overlap the other's work); two calls of the
 * same entry point must not overlap. */
int luvc_oim_merge_host(const void* tokens, int B, int H, int W, int D, int target_count, int dtype,
                        void* out_tokens, int32_t* out_sizes, int32_t* out_map);

/*
 * Value enhancement of Eq. 2, O = A (V + log s): out[b, t, :] = values[b, t, :] + log(sizes[b, t]),
 * the row-wise bias that lets attention weigh a merged token by the number of tokens it stands for
 * (the attention itself is the caller's).  values / out [B, T, D] of element type `dtype` (DEVICE,
 * out may be the same buffer as values), sizes [B, T] int32 (the out_sizes of luvc_oim_merge*).
 * The sum is formed in fp32 and rounded once.  cuda_stream: a cudaStream_t, NULL = legacy default.
 */
int luvc_oim_value_enhance(const void* values, const int32_t* sizes, int B, int T, int D, int dtype,
                           void* out, void* cuda_stream);

/* ---- SPU ---------------------------------------------------------------- */

/* Last passed frequency bin for a sequence of N tokens:
 * floor(cutoff * floor(N / 2)); cutoff <= 0 selects LUVC_SPU_DEFAULT_CUTOFF.
 * Returns -1 if cutoff is NaN or > 1. */
int luvc_spu_sigma(int N, float cutoff);

/* Bytes of workspace luvc_spu_prune_ex needs for this problem. */
size_t luvc_spu_workspace_bytes(int B, int N, int D, float cutoff, int dtype);

typedef struct {
    int dtype;               /* luvc_dtype of hidden and out_hidden */
    void* stream;
    void* workspace;         /* device, 256-byte aligned; NULL = library-owned scratch */
    size_t workspace_bytes;
    int no_window;           /* 0: Hamming-windowed pass band (Eq. 5); 1: flat pass band
                                (the paper's "without HW" ablation) */
    float* out_scores;       /* optional device [B, N] fp32: the energies E of Eq. 8 */
    int32_t* device_status;  /* optional device block of LUVC_STATUS_BYTES (see luvc_read_status);
                                NULL = the library-owned word of the current device */
} luvc_spu_opts;

/*
 * Spectrum Pruning Unit (Algorithm 2).
 *
 * hidden      [B, N, D]  hidden states of the N visual tokens of B sequences
 * cutoff      fraction of the band [0, floor(N/2)] that is passed, in (0, 1];
 *             <= 0 selects the default
 * keep        number of tokens kept per sequence, 1 <= keep <= N
 * out_idx     [B, keep] int32  kept token indices, strictly ascending
 * out_hidden  [B, keep, D]  the kept rows of `hidden`, bit-exact copies
 *
 * Per sequence and channel the token axis is transformed (Eq. 4), multiplied by
 * the mask of Eq. 5/6 - a Hamming window centred on the zero frequency,
 * 0.54 + 0.46 cos(2 pi f / (N - 1)) for signed frequencies |f| <= sigma and 0
 * elsewhere - and transformed back (Eq. 7); a token's score is the L2 norm over
 * the channels of the filtered signal (Eq. 8).  The `keep` highest scores win,
 * ties go to the lower index.  Arithmetic is fp32.
 */
int luvc_spu_prune(const void* hidden, int B, int N, int D, float cutoff, int keep,
                   int32_t* out_idx, void* out_hidden);
int luvc_spu_prune_f32(const float* hidden, int B, int N, int D, float cutoff, int keep,
                       int32_t* out_idx, float* out_hidden);
int luvc_spu_prune_ex(const void* hidden, int B, int N, int D, float cutoff, int keep,
                      int32_t* out_idx, void* out_hidden, const luvc_spu_opts* opts);

/* Same operator on HOST buffers (see luvc_oim_merge_host). */
int luvc_spu_prune_host(const void* hidden, int B, int N, int D, float cutoff, int keep, int dtype,
                        int32_t* out_idx, void* out_hidden);

/*
 * Cascade of prunes (Section 3.3: the unit is applied again every few layers, each time to the
 * visual tokens that are left; appendix "Hyper-parameters of SPU": start layer and interval).
 * Runs n_stages prunes back to back: stage t keeps keeps[t] of the keeps[t-1] survivors (N for
 * t = 0) with cutoffs[t] (cutoffs == NULL or an entry <= 0: the default).  What the LLM does to the
 * hidden states between two stages is the caller's business and not modelled: every stage sees
 * the rows of `hidden`.
 *
 * keeps, cutoffs  HOST arrays of n_stages entries; 1 <= keeps[t] <= keeps[t-1] <= N
 * out_idx     [B, keeps[n_stages-1]] int32  surviving tokens as indices into the ORIGINAL sequence, ascending
 * out_hidden  [B, keeps[n_stages-1], D]     their rows, bit-exact copies
 * A later stage reads its rows straight out of `hidden`, through the list of survivors composed so far
 * (gather on load): the survivors' rows are written once, by the last stage.  Only a stage whose
 * sequence is long enough for the two-stage transform kernels (which walk dense memory) has its rows
 * copied into library-owned scratch first.  Index lists and the transform workspace live in
 * library-owned scratch (grown with cudaMalloc on demand; see the note on overlapping calls above).
 * Dropping the last survivors altogether, as the paper does at the final layer, needs no kernel.
 */
int luvc_spu_cascade(const void* hidden, int B, int N, int D, int n_stages, const int* keeps, const float* cutoffs,
                     int dtype, void* cuda_stream, int32_t* out_idx, void* out_hidden);

/* ---- SPU without any allocation ------------------------------------------- */

/* Largest workspace (luvc_spu_workspace_bytes) luvc_spu_prune_static accepts: 32 MiB. */
#define LUVC_SPU_STATIC_MAX_BYTES (32u * 1024u * 1024u)

/*
 * luvc_spu_prune with a fixed, built-in workspace.  (The paper has no counterpart:
 * this is a deployment variant of the same operator, not another method.)
 *
 * For callers that cannot allocate device memory when they prune: a server whose
 * own allocator already owns the device's memory, a loop that cannot afford the
 * device-wide synchronisation an allocation may cause, a process under a fixed
 * memory budget.  This call never calls cudaMalloc, cudaFree or any routine that
 * allocates, and needs no caller workspace.  Its workspace is an array of
 * LUVC_SPU_STATIC_MAX_BYTES (+256) bytes that is part of the library's device
 * image: every GPU that loads that image holds it until the process exits.
 * With CUDA's lazy module loading (the default of current toolkits) the image, and
 * with it the array, is loaded by the first call on a device, and each kernel's
 * code by its first launch: those first uses can reserve device memory and can
 * synchronise.  So make ONE warm-up call per device (and per kind of problem: element
 * type, and a sequence length of the same factor class) at start-up, before the
 * device's memory is handed to another allocator - or run with
 * CUDA_MODULE_LOADING=EAGER; from then on no call reserves anything.
 *
 * Arguments and results are those of luvc_spu_prune_ex with default options
 * (Hamming-windowed pass band, no score export): hidden [B,N,D], out_idx [B,keep],
 * out_hidden [B,keep,D] are DEVICE pointers owned by the caller, dtype is a
 * luvc_dtype, cuda_stream a cudaStream_t (NULL = legacy default stream); the work
 * is queued on that stream and the host is not synchronised.
 *
 * Errors: those of luvc_spu_prune_ex, and LUVC_ERR_WORKSPACE when
 * luvc_spu_workspace_bytes(B, N, D, cutoff, dtype) exceeds LUVC_SPU_STATIC_MAX_BYTES
 * (nothing is queued; use the other entry points for such sizes).
 *
 * The first call on each device looks up the array's device address (with that
 * device current); make that first call outside any stream capture.  All calls on
 * a device share the one array and it keeps the previous call's contents: the
 * call clears the part that must start at zero, but two calls whose GPU work
 * overlaps (different streams, or several host threads) race on it - run them on
 * one stream or order them with events.  A bounded device-side wait that gives up
 * is recorded inside the array, not in the word luvc_check_status reads:
 * luvc_spu_static_status reads it; the outputs of such a call are undefined.
 * With luvc_profile_enable(1) the first
 * call creates CUDA events; leave profiling off where that matters.
 */
int luvc_spu_prune_static(const void* hidden, int B, int N, int D, float cutoff, int keep, int dtype,
                          void* cuda_stream, int32_t* out_idx, void* out_hidden);

/* Synchronises the stream and returns, as a luvc_status, what the most recent
 * luvc_spu_prune_static call on the current device recorded inside the array (LUVC_OK, or
 * LUVC_ERR_TIMEOUT when a bounded wait gave up); the next call clears it.  Allocates nothing.
 * (No counterpart in the paper.) */
int luvc_spu_static_status(void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* LUVC_H_ */
