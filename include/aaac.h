/*
 * aaac.h -- C ABI of the B200 (sm_100a) AAAC per-layer quantisation library.
 *
 * AAAC replaces the fixed 4-bit table of a group-quantised linear layer by two learned
 * 16-entry scalar codebooks T0, T1; every group of g weights picks the codebook with the
 * lower activation-weighted error and stores that choice in the sign bit of its (always
 * positive) scale.  This library is the per-layer fitting path of Algorithm 1.
 *
 * Conventions for every entry point
 *   - Pointers are DEVICE pointers unless the name ends in _host.  The caller owns every
 *     buffer; the library allocates no device memory and keeps no per-call state, except for
 *     four process-wide diagnostics / conveniences that are documented where they are declared:
 *     the event table of aaac_timing_begin / aaac_timing_end, the launch counter of
 *     aaac_launch_count, the built-in scratch array of aaac_act_stats_noalloc, and the seven
 *     streams and eight events per device that aaac_fit_layers / aaac_quantize_layers create at
 *     their first call with more than one layer.
 *   - W is [N x K] row-major BF16 (N = output rows, K = input channels, y = x W^T, Sec. 3.1),
 *     leading dimension ldw (elements).  Groups are g contiguous elements of a row.
 *     X is [T x K] row-major BF16 calibration activations, leading dimension ldx.
 *   - mode AAAC_INT4 : g = 128, scales BF16 [N][K/g], no tensor scale (tensor_scale[0] = 1).
 *     mode AAAC_NVFP4: g = 16, scales E4M3 bytes [N][K/g] plus one FP32 tensor scale.
 *   - Tables are [2][16]: T0[0..15] then T1[0..15].
 *   - `stream` is a cudaStream_t passed as void*.  Work is enqueued and never synchronised:
 *     results are valid once the stream has been synchronised by the caller.
 *   - Return value: AAAC_OK or an aaac_status for argument / launch errors (checked before any
 *     work is enqueued).  Conditions that only the device sees are OR-ed into the optional
 *     device word `dev_status` instead (AAAC_DEV_* bits); nothing traps.  AAAC_DEV_NONFINITE:
 *     W, X or a multiplier holds Inf / NaN.  AAAC_DEV_TIMEOUT: a bounded wait between the
 *     blocks of the fit-rounds kernel ran out (the kernel then returns early and the tables,
 *     and whatever is packed from them, are NOT valid).  Without a dev_status word neither can
 *     be seen by the caller; the host-buffer calls always keep one.
 *   - Alignment: W, X, codes, What 16-byte aligned; K % 8 == 0; K % g == 0; ldw, ldx, ldo
 *     multiples of 8.
 *   - ws is scratch of at least aaac_workspace_bytes(...) bytes, 256-byte aligned.  Calls
 *     that share a workspace must be ordered on one stream.
 */
#ifndef AAAC_H
#define AAAC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    AAAC_OK = 0,
    AAAC_ERR_NULL = 1,          /* a required pointer is NULL */
    AAAC_ERR_MODE = 2,          /* unknown mode / init, or group does not match the mode */
    AAAC_ERR_SHAPE = 3,         /* N < 1, K % g, K % 8, ld < K, ld % 8, T < 1, n_outer < 0 */
    AAAC_ERR_ALIGN = 4,         /* a pointer is not 16-byte aligned (ws: 256) */
    AAAC_ERR_WORKSPACE = 5,     /* ws_bytes too small (host-buffer calls: also AAAC_DEV_SCRATCH was set) */
    AAAC_ERR_CUDA = 6,          /* a CUDA runtime call or launch failed */
    AAAC_ERR_NONFINITE = 7,     /* (dev_status bit) W or X holds Inf / NaN */
    AAAC_ERR_UNIMPLEMENTED = 8, /* reserved */
    AAAC_ERR_TOO_LARGE = 9,     /* size beyond a fixed capacity: K of a no-allocation entry point, N * ldw of a fit */
    AAAC_ERR_TIMEOUT = 10       /* (dev_status bit AAAC_DEV_TIMEOUT) a bounded device-side wait ran out */
} aaac_status;

typedef enum { AAAC_INT4 = 0, AAAC_NVFP4 = 1 } aaac_mode;

typedef enum {
    AAAC_INIT_QUANTILE = 0,     /* Eq. 9 / Eq. 10 */
    AAAC_INIT_GRID = 1,         /* T0 = the format's table, T1 = T0 moved up half a step */
    AAAC_INIT_USER = 2          /* T01 holds the start tables */
} aaac_init;

/* bits OR-ed into *dev_status by the kernels */
#define AAAC_DEV_NONFINITE 1u
#define AAAC_DEV_TIMEOUT 2u      /* a bounded wait inside a kernel ran out; results are not valid */
#define AAAC_DEV_SCRATCH 4u      /* the quantile start needed more scratch than ws holds (see aaac_workspace_bytes); the
                                    start tables, and everything fitted from them, are not valid */

const char* aaac_status_string(int status);

/* Bytes of scratch that any call below needs for a layer of this shape (T = calibration
 * tokens, 0 if activations are never passed): a few megabytes of fixed regions plus the candidate
 * list of the quantile start (Eq. 9-10), 4 bytes for a sixteenth of the layer's weights -- about
 * an eighth of the layer's own size.  The list holds the normalised weights that fall into the
 * (at most 64) histogram bins of width 2^-10 around the requested quantiles, usually 1-3 % of
 * the weights.  A bin whose weights do not fit the list is still resolved when they all have one
 * value (a constant or pruned layer); otherwise AAAC_DEV_SCRATCH is set in dev_status.  A caller
 * who wants to rule that out passes a larger workspace: whatever ws_bytes holds beyond the fixed
 * regions is used for the list, and aaac_workspace_bytes_full is the size that can never fall
 * short (one list entry per weight: twice the layer's size). */
size_t aaac_workspace_bytes(int mode, int64_t N, int64_t K, int64_t T);
size_t aaac_workspace_bytes_full(int mode, int64_t N, int64_t K, int64_t T);

/*
 * Activation importance, Eq. 7:  I[k] = sum_t X[t,k]^2.
 * The squares are exact in FP32 and are added without rounding error (an FP32 value pair per
 * column, strips combined in a fixed order in double); the sum is rounded once to FP32.
 * accumulate = 0 overwrites I; 1 adds to the existing I (FP32 add), so that the tokens can
 * be streamed in chunks.  Sets AAAC_DEV_NONFINITE if a sum is not finite.
 */
int aaac_act_stats(const void* X, int64_t T, int64_t K, int64_t ldx, float* I, int accumulate,
                   uint32_t* dev_status /* may be NULL */, void* ws, size_t ws_bytes, void* stream);

/*
 * aaac_act_stats for callers that have no scratch buffer to give and must not allocate one.
 * (The paper has no counterpart: this entry point exists for the integration, not the method.)
 *
 * Who needs it: code that runs where device allocation is off limits -- inside a serving
 * engine whose memory pool was sized and handed out at start-up, in a plugin or callback that
 * is only given its input and output tensors, or on a path that must not stall on cudaMalloc's
 * implicit synchronisation.  Such a caller cannot create the workspace aaac_act_stats asks for.
 *
 * Same inputs, outputs, accumulate flag and result as aaac_act_stats.  The strip partials go
 * to an 8 MiB array that is part of the library's device image (one copy on every GPU that
 * loads the library, held until the process exits).  Limits and rules:
 *   - K <= 32768, otherwise AAAC_ERR_TOO_LARGE is returned and nothing is enqueued;
 *   - no cudaMalloc / cudaFree or other allocating call is made, on any call;
 *   - the first call on each device looks up the array's device address (a host-side step
 *     done once per device, with that device current); make that first call before starting
 *     any stream capture;
 *   - all calls on a GPU share the array: calls that may overlap on the GPU (different
 *     streams without ordering) race on it and give wrong sums.  The array keeps the previous
 *     call's partials; every value a call reads it has first written itself, so nothing needs
 *     clearing between calls;
 *   - the looked-up address is kept for the life of the device's primary context; after a
 *     cudaDeviceReset the library must be reloaded before this entry point is used again.
 */
int aaac_act_stats_noalloc(const void* X, int64_t T, int64_t K, int64_t ldx, float* I, int accumulate,
                           uint32_t* dev_status /* may be NULL */, void* stream);

/*
 * Algorithm 1 lines 1-16 for one layer: scales (line 1), normalisation w~ = w / s (Eq. 2,
 * line 2; w~ = fl32(w * fl32(1/s)) is recomputed on the fly, never stored), importance
 * (line 3; taken from I, or computed from X when I == NULL), initial tables (lines 4-5),
 * then n_outer rounds of { assignment step Eq. 8; n_inner iterations of the weighted-centroid
 * update Eq. 11 with the selection frozen, each from the Voronoi cells of the table as it stood
 * before the iteration, an entry whose cell has no weight keeping its value; sort }.  With
 * n_inner = 1 a round is a single pass over W (the cells of the update are the nearest-entry
 * indices of the assignment step); every further inner iteration is one more, cheaper pass.
 * n_inner >= 1 and n_outer * n_inner <= 2^20, else AAAC_ERR_SHAPE.  A layer must span fewer than
 * 2^32 elements (N * ldw < 2^32; the fit kernels index it with 32 bits), else AAAC_ERR_TOO_LARGE.
 *
 *   scales        out  positive scales (sign bit clear).  INT4: s = bf16(absmax/7) (1 for an
 *                      all-zero group).  NVFP4: E4M3(absmax / (6 s_t)) in 0x01..0x7E with
 *                      s_t = layer absmax / 2688.
 *   tensor_scale  out  [1] FP32 (1.0 for INT4)
 *   T01           in (AAAC_INIT_USER) / out  [2][16] FP32 tables after the last round, sorted
 *   err_trace     out  [n_outer] double or NULL: Eq. 8 objective (sum over groups of the
 *                      smaller weighted error, normalised units) of each round's assignment
 *   dev_status    out  device word or NULL
 */
int aaac_fit_layer(const void* W, int64_t N, int64_t K, int64_t ldw, int mode, int group,
                   const float* I, const void* X, int64_t T, int64_t ldx,
                   int n_outer, int n_inner, int init,
                   float* T01, void* scales, float* tensor_scale, double* err_trace,
                   uint32_t* dev_status, void* ws, size_t ws_bytes, void* stream);

/*
 * Algorithm 1 lines 17-20: round the tables to BF16 (RNE of the FP32 values), recompute
 * sigma for every group with Eq. 8, store the nearest-entry index under the chosen table
 * (Eq. 6) as a 4-bit code, and put sigma into the sign bit of the scale.  As for the fit, a layer
 * must span fewer than 2^32 elements (N * ldw < 2^32), else AAAC_ERR_TOO_LARGE.
 *
 *   T01_f32   in   [2][16]
 *   T01_bf16  out  [2][16] BF16 bit patterns (64 bytes)
 *   scales    in: positive scales from aaac_fit_layer; out: sign bit (bit 15 of the BF16 /
 *             bit 7 of the E4M3 byte) = sigma
 *   codes     out  [N][K/2]; element 2i in the low nibble of byte i, 2i+1 in the high nibble
 *   err_out   out  [2] double or NULL: {Eq. 8 objective under the BF16 tables,
 *             sum_k I_k (w - w^)^2 in weight units}
 *   stats     out  [4] uint64 or NULL: {groups with E0 == E1 exactly, weights exactly half-way
 *             between two different entries of their table, groups re-evaluated in double,
 *             reserved}
 * Decisions are those of a double-precision evaluation: the codes are exact, and a group whose
 * FP32 errors lie within the proven rounding bound of each other is re-evaluated in double
 * (each lane adds its eight terms in index order, the lanes of a group are then combined
 * pairwise; against a strictly index-ordered double sum this can differ by a few 2^-53
 * relative, far inside what "E0 == E1 exactly" can resolve on non-degenerate data).
 */
int aaac_pack(const void* W, int64_t N, int64_t K, int64_t ldw, int mode, int group,
              const float* I, const float* T01_f32, uint16_t* T01_bf16,
              void* scales, const float* tensor_scale, uint8_t* codes,
              double* err_out, uint64_t* stats, void* ws, size_t ws_bytes, void* stream);

/*
 * Eq. 5:  w^ = T_sigma[c] * s, sigma = sign bit of the stored scale, s = its magnitude (times
 * tensor_scale[0] for NVFP4, the product rounded to FP32), one FP32 multiply, BF16 (RNE) out.
 */
int aaac_dequant(const uint8_t* codes, const void* scales, const float* tensor_scale,
                 const uint16_t* T01_bf16, int64_t N, int64_t K, int mode, int group,
                 void* What, int64_t ldo, void* stream);

/*
 * Selection group S smaller than the scale group g (Sec. 3.1, "granularity"; Algorithm 1
 * line 20, "separately if S < g"): the same three calls with the selection group size given
 * apart from the scale group.  Built for sel_group == group (then identical to the calls
 * above; sigma_bits is ignored) and for the paper's INT4 variant group = 128, sel_group = 16;
 * anything else returns AAAC_ERR_MODE.  With sel_group < group the selection costs 1/S bit per
 * weight and lives in
 *   sigma_bits  [N][K / (8 S)] bytes, row-major: selection group j of a row (columns
 *               j S .. j S + S - 1) in bit j % 8 of the row's byte j / 8
 * which aaac_pack_sel writes and aaac_dequant_sel reads, while the scales keep a clear sign
 * bit.  aaac_fit_layer_sel's assignment step (Eq. 8) sums over selection groups of S weights.
 */
int aaac_fit_layer_sel(const void* W, int64_t N, int64_t K, int64_t ldw, int mode, int group, int sel_group,
                       const float* I, const void* X, int64_t T, int64_t ldx,
                       int n_outer, int n_inner, int init,
                       float* T01, void* scales, float* tensor_scale, double* err_trace,
                       uint32_t* dev_status, void* ws, size_t ws_bytes, void* stream);
int aaac_pack_sel(const void* W, int64_t N, int64_t K, int64_t ldw, int mode, int group, int sel_group,
                  const float* I, const float* T01_f32, uint16_t* T01_bf16,
                  void* scales, const float* tensor_scale, uint8_t* codes, uint8_t* sigma_bits,
                  double* err_out, uint64_t* stats, void* ws, size_t ws_bytes, void* stream);
int aaac_dequant_sel(const uint8_t* codes, const void* scales, const uint8_t* sigma_bits, const float* tensor_scale,
                     const uint16_t* T01_bf16, int64_t N, int64_t K, int mode, int group, int sel_group,
                     void* What, int64_t ldo, void* stream);

/*
 * Algorithm 1 lines 1-16 for several layers of one format at once.  The paper processes layers
 * independently (Sec. 3.3, "Computational cost"), so a batch is only a way of running them: the
 * result for every layer is what aaac_fit_layer_sel gives for it, up to the rounding of the FP32
 * partial sums (a layer's rows are dealt to a share of the GPU's blocks instead of all of them;
 * the fitted tables agree to about 1e-7 relative and are bitwise reproducible from call to call).
 * With n_inner = 1 the rounds of up to eight layers run in one launch, each layer on its own
 * share of the blocks, so that the cost of a round that does not depend on the layer's size is
 * paid once per batch and small layers do not leave most of the GPU idle; more layers, and
 * n_inner > 1, are run in turn.  Scales, importances (from X where I is NULL) and start tables
 * are computed per layer exactly as by aaac_fit_layer_sel, except that layers given the same
 * activations (the same X, T, K and ldx, with I == NULL) share their importances, which are
 * computed once (into the workspace of the first of them).  With more than one layer these
 * per-layer passes are queued on up to seven streams the library keeps per device (created at the
 * first such call), forked from `stream` and joined back to it before the fit launch: seen from
 * `stream`, the call is ordered like any other.
 *
 *   layers   HOST array of n_layers descriptors (read before the call returns); every pointer
 *            inside is a DEVICE pointer with the meaning, layout and alignment of the
 *            argument of the same name of aaac_fit_layer_sel; every layer has its own ws
 *   mode, group, sel_group, n_outer, n_inner, init   shared by all layers of the batch
 * Returns the first error found (nothing is enqueued for an invalid batch).
 */
typedef struct {
    const void* W;
    int64_t N, K, ldw;
    const float* I;          /* [K], or NULL with X given */
    const void* X;
    int64_t T, ldx;
    float* T01;              /* [2][16] in (AAAC_INIT_USER) / out */
    void* scales;            /* out */
    float* tensor_scale;     /* out [1] */
    double* err_trace;       /* out [n_outer] or NULL */
    void* ws;
    size_t ws_bytes;
} aaac_layer;

int aaac_fit_layers(const aaac_layer* layers, int n_layers, int mode, int group, int sel_group,
                    int n_outer, int n_inner, int init, uint32_t* dev_status /* may be NULL */, void* stream);

/*
 * The whole path of Algorithm 1 for several layers in one call: aaac_fit_layers on the batch,
 * then for every layer the pack pass (Eq. 6, Eq. 8) and, where `What` is given, the
 * dequantisation (Eq. 5).  The results are those of the separate calls on each layer; the
 * per-layer passes before and after the fit launch are queued on the library's side streams
 * (see aaac_fit_layers), forked from `stream` and joined back to it.
 *
 *   layers   as for aaac_fit_layers (the pack pass uses the importance the fit used: I, or
 *            the one computed from X, which stays in the layer's ws)
 *   outs     HOST array of n_layers descriptors, DEVICE pointers inside:
 *              T01_bf16   [2][16] BF16 bit patterns, written (the tables as stored, Sec. 3.2)
 *              codes      [N][K/2] packed 4-bit codes, written; 16-byte aligned
 *              sigma_bits [N][K/128] selection bytes, written; only where sel_group != group, else ignored
 *              err_out    [2] doubles: Eq. 2 objective with the stored tables, sum of w^2 I; or NULL
 *              stats      [4] counters of aaac_pack; or NULL
 *              What       [N][ldo] BF16 reconstruction, written; or NULL: no dequantisation
 *              ldo        elements between rows of What (>= K, multiple of 8)
 * Returns the first error found (nothing is enqueued for an invalid batch).
 */
typedef struct {
    uint16_t* T01_bf16;
    uint8_t* codes;
    uint8_t* sigma_bits;
    double* err_out;
    uint64_t* stats;
    void* What;
    int64_t ldo;
} aaac_layer_out;

int aaac_quantize_layers(const aaac_layer* layers, const aaac_layer_out* outs, int n_layers, int mode, int group,
                         int sel_group, int n_outer, int n_inner, int init, uint32_t* dev_status /* may be NULL */,
                         void* stream);

/*
 * Per-input-channel scaling before the fit (Section 4, "Combining AAAC with AWQ": AWQ scales
 * the weights, AAAC then learns its tables on the scaled distribution).  The multipliers a_k
 * themselves come from the caller (AWQ's search is not part of the method).
 *
 *   a       in   [K] FP32, positive and finite (else AAAC_DEV_NONFINITE is OR-ed into dev_status)
 *   W_out   out  [N][ldo] BF16: bf16_rne(fl32(w * a_k)); may be W itself (in place)
 *   I, I_out     both NULL, or [K] FP32 in / out: I_out[k] = I[k] / a_k^2 (double, rounded once) --
 *                the importance of the layer's input once it is divided by a_k; may alias
 * Feed W_out and I_out to aaac_fit_layer / aaac_pack; the dequantised weights are then those of
 * the scaled layer.  K % 8 == 0, ldw and ldo multiples of 8, 16-byte aligned W, W_out, a.
 */
int aaac_prescale_columns(const void* W, int64_t N, int64_t K, int64_t ldw, const float* a,
                          void* W_out, int64_t ldo, const float* I, float* I_out,
                          uint32_t* dev_status /* may be NULL */, void* stream);

/*
 * Whole path for one layer with HOST buffers: copies W and X to the device (into ws), runs
 * aaac_act_stats, aaac_fit_layer and aaac_pack, and copies tables, scales, tensor scale,
 * codes and errors back.  Host buffers should be page-locked for the copies to be
 * asynchronous.  ws must hold aaac_host_workspace_bytes(...) bytes of DEVICE memory.
 * Synchronises the stream before returning; returns AAAC_ERR_TIMEOUT or AAAC_ERR_NONFINITE
 * if the corresponding bit of the device status word was set (the outputs are then not valid).
 */
size_t aaac_host_workspace_bytes(int mode, int64_t N, int64_t K, int64_t T);
int aaac_quantize_layer_host(const void* W_host, int64_t N, int64_t K, int mode, int group,
                             const void* X_host, int64_t T, int n_outer, int init,
                             float* T01_host, uint16_t* T01_bf16_host, void* scales_host,
                             float* tensor_scale_host, uint8_t* codes_host, double* err_out_host,
                             void* ws, size_t ws_bytes, void* stream);

/*
 * The same without the final synchronisation: everything, the copies back included, is only
 * enqueued on the stream, so layers issued on different streams (each with its own ws)
 * overlap their copies and kernels.  status_host receives the device status word
 * (AAAC_DEV_* bits) once the stream has been synchronised by the caller; it and the other host
 * buffers must stay valid until then and should be page-locked.
 */
int aaac_quantize_layer_host_async(const void* W_host, int64_t N, int64_t K, int mode, int group,
                                   const void* X_host, int64_t T, int n_outer, int init,
                                   float* T01_host, uint16_t* T01_bf16_host, void* scales_host,
                                   float* tensor_scale_host, uint8_t* codes_host, double* err_out_host,
                                   uint32_t* status_host, void* ws, size_t ws_bytes, void* stream);

/*
 * Optional timing of the fit-rounds kernel: after aaac_timing_begin(n) the next n launches of
 * it (one per aaac_fit_layer call with n_outer > 0, covering all rounds of that call) on the
 * calling thread's device are bracketed by CUDA events on their stream;
 * aaac_timing_end synchronises those events and returns how many were recorded, writing each
 * launch's device time (milliseconds) to ms_host[0..].  Not re-entrant; diagnostics only.
 */
int aaac_timing_begin(int max_launches);
int aaac_timing_end(float* ms_host, int capacity);

/*
 * Diagnostics for the bounded wait of the fit-rounds kernel (Algorithm 1's rounds run in one
 * persistent kernel whose blocks wait for each other's sums once per pass; a wait that runs out
 * sets AAAC_DEV_TIMEOUT and ends the kernel).  extra_arrivals > 0 makes every later
 * aaac_fit_layer call of the process wait for that many more blocks than exist, so the wait must
 * run out after spin_limit polls (0 = the default of several seconds); extra_arrivals = 0 and
 * spin_limit = 0 restore normal operation.  For tests of the error path; process-wide, not
 * thread-safe against concurrent aaac_fit_layer calls.
 */
int aaac_debug_fit_wait(int extra_arrivals, unsigned spin_limit);

/*
 * Diagnostics for the quantile start's candidate list: entries > 0 caps the list of every later
 * call of the process at that many entries (never below what the fit's selection words need), so
 * that the paths taken when a bin's weights do not fit -- one shared value: resolved; several:
 * AAAC_DEV_SCRATCH -- can be tested on small layers; 0 restores the normal capacity.  Process-wide.
 */
int aaac_debug_quantile_cap(size_t entries);

/*
 * Number of kernels this library has launched in the calling process so far (all entry points,
 * all devices and streams; a process-wide counter, diagnostics only).  The benchmark reports
 * the difference across its timed region.
 */
unsigned long long aaac_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* AAAC_H */
