/*
 * moqe.h -- C ABI of the routed, weight-only-quantized linear layer of MoQE
 * (Mixture of Quantization Experts) for NVIDIA B200 (sm_100a).
 *
 * The method (paper, Section 3.1 "Mixture of Quantization Experts"): one
 * full-precision model is quantized into several frozen variants, the
 * "quantization experts"; a router scores the experts and every sample (one
 * sequence or one image) is run by exactly ONE expert (Section 3.2 "Router
 * Model"; Appendix "Convergence Observations", r(x) in [M]).  This library is
 * the linear layer of such a model when a batch mixes samples routed to
 * different experts that are all resident in device memory:
 *
 *     Y[m][:] = X[m][:] . dequant(W_e(m))^T ,   e(m) = expert of row m
 *
 * computed as  sort rows by expert -> grouped dequant-GEMM -> unsort.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its name starts with h_.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     All work is enqueued on it; no call synchronises except where stated.
 *   - Matrices are dense row-major: W[N][K] (N output features, K input
 *     features, K contiguous), X[M][K], Y[M][N]; bf16 = bfloat16 bit patterns.
 *   - Every call returns a moqe_status.  Argument errors are detected on the
 *     host before anything is launched and leave outputs untouched.  Errors
 *     only a kernel can see (an expert id outside [0,E)) never trap: the
 *     offending rows are written as zeros, a status word is set on the device
 *     and moqe_async_status() reports it.
 *   - The caller owns X, Y, ids, perm, offsets and workspaces.  The library
 *     owns only what a moqe_expert* points at.
 *   - Row pointers and row pitches must be 16-byte aligned (K % 8 == 0 for
 *     bf16 rows), else MOQE_ERR_UNSUPPORTED.
 */
#ifndef MOQE_H_
#define MOQE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define MOQE_API __attribute__((visibility("default")))
#else
#define MOQE_API
#endif

typedef enum {
    MOQE_OK = 0,
    MOQE_ERR_NULL = 1,         /* a required pointer is NULL */
    MOQE_ERR_SHAPE = 2,        /* a size is negative, zero where it may not be, or inconsistent */
    MOQE_ERR_UNSUPPORTED = 3,  /* bits not in {2,3,4,8}; group not 0, 32, 64 or a multiple of 128;
                                  K % 8 != 0; E > MOQE_MAX_EXPERTS; misaligned pointer */
    MOQE_ERR_ALLOC = 4,        /* device allocation failed */
    MOQE_ERR_WORKSPACE = 5,    /* workspace NULL or smaller than the *_workspace() figure */
    MOQE_ERR_MISMATCH = 6,     /* experts of one call disagree on N or K */
    MOQE_ERR_CUDA = 7,         /* a CUDA runtime / driver call failed */
    MOQE_ERR_EXPERT_ID = 8,    /* asynchronous: an id outside [0,E) was seen by a kernel */
    MOQE_ERR_TIMEOUT = 9,      /* asynchronous: a bounded in-kernel wait ran out */
    MOQE_ERR_IO = 10           /* a file could not be opened, read or written, or is not a whole expert image */
} moqe_status;

#define MOQE_MAX_EXPERTS 32

/* One quantization expert of one linear layer: b-bit codes in the library's
 * private packed layout plus fp16 scales and integer zero-points, on device. */
typedef struct moqe_expert moqe_expert;

/* ---------------------------------------------------------------------------
 * Expert construction (Section 3.1: the experts are quantized variants of the
 * same full-precision model, frozen afterwards).  The paper names no quantizer
 * for this library's purpose; the one implemented is affine round-to-nearest:
 * for every output channel n and every group of `group` consecutive k
 * (group == 0: the whole row), in IEEE fp32 with round-half-to-even,
 *   symmetric : a = max|w|, qmax = 2^(b-1)-1, s = fp16(a/qmax),
 *               c = clamp(rint(w/s), -qmax, qmax) + 2^(b-1),  z = 2^(b-1)
 *   asymmetric: lo = min(0,min w), hi = max(0,max w), s = fp16((hi-lo)/(2^b-1)),
 *               z = clamp(rint(-lo/s), 0, 2^b-1), c = clamp(rint(w/s)+z, 0, 2^b-1)
 *   s == 0 or non-finite after the fp16 rounding -> s = 1;   dequant = s*(c-z).
 * W: device fp32 [N][K], finite.  bits in {2,3,4,8}; group 0, 32, 64 or a multiple
 * of 128, dividing K.  On success *out owns new device buffers (cudaMalloc'ed by
 * this call; it is therefore not capturable in a CUDA graph) and must be
 * released with moqe_expert_destroy.  The kernels run on `stream`.
 * ------------------------------------------------------------------------- */
MOQE_API moqe_status moqe_quantize_rtn(const float* W, int N, int K, int bits, int group, int sym,
                              void* stream, moqe_expert** out);

/* Canonical, layout-independent view of an expert, for checking and storage:
 * codes [N][K] one code per byte, scales_f16 [N][K/g] and zeros_f16 [N][K/g]
 * as IEEE binary16 bit patterns (zeros hold the integer zero-point; symmetric
 * experts export 2^(b-1)).  g = K when group == 0.  Any output may be NULL. */
MOQE_API moqe_status moqe_expert_export(const moqe_expert* e, uint8_t* codes, uint16_t* scales_f16,
                               uint16_t* zeros_f16, void* stream);

/* Inverse of export: build an expert from canonical device arrays.  For a
 * symmetric expert zeros_f16 may be NULL. */
MOQE_API moqe_status moqe_expert_import(int N, int K, int bits, int group, int sym, const uint8_t* codes,
                               const uint16_t* scales_f16, const uint16_t* zeros_f16, void* stream,
                               moqe_expert** out);

/* Host-side description.  code_bytes = N*K*bits/8 exactly (the paper's storage
 * ratios FP16 : Int8 : Int4 = 1 : 1/2 : 1/4, Appendix "Peak VRAM and CPU RAM
 * usage analysis"); meta_bytes = scales (+ zeros when asymmetric), 2 bytes each;
 * alloc_bytes = what the packed buffers really occupy (padding included).
 * Any output may be NULL. */
MOQE_API moqe_status moqe_expert_info(const moqe_expert* e, int* N, int* K, int* bits, int* group, int* sym,
                             size_t* code_bytes, size_t* meta_bytes, size_t* alloc_bytes);

/* Frees the expert's device buffers (cudaFree: synchronises the device). */
MOQE_API moqe_status moqe_expert_destroy(moqe_expert* e);

/* ---------------------------------------------------------------------------
 * Expert residency (Section 4.4 and the appendix table "Router model and expert loading overhead": one expert
 * stays on the GPU, the others wait in CPU RAM and are loaded when the routing changes).  A packed expert is a
 * plain byte image, so parking and reloading it is copy-engine work only:
 *   moqe_expert_offload   : device expert -> a copy in PINNED host memory (synchronises `stream`; the device expert
 *                           is left as it is and may be destroyed afterwards).
 *   moqe_expert_prefetch  : pinned host copy -> a NEW device expert; allocates (synchronously), then enqueues the
 *                           host-to-device copies on `stream` and returns at once.  Give it a side stream to
 *                           overlap the copy with the layer that is running; the expert may be used by work
 *                           ordered after those copies (same stream, or an event recorded on it).  The host copy
 *                           must stay alive until the copies have completed.
 *   moqe_expert_host_save / _load : the host copy to / from a file.  The file holds a header (magic, packed-layout
 *                           version, N, K, bits, group, sym, byte counts) and the packed image; it is tied to
 *                           the packed layout of the library that wrote it.  A file that is not exactly one
 *                           image of a supported format is refused (MOQE_ERR_IO / _UNSUPPORTED / _SHAPE).
 * The library owns what *out points at; destroy with moqe_expert_host_destroy / moqe_expert_destroy.
 * ------------------------------------------------------------------------- */
typedef struct moqe_expert_host moqe_expert_host;
MOQE_API moqe_status moqe_expert_offload(const moqe_expert* e, void* stream, moqe_expert_host** out);
MOQE_API moqe_status moqe_expert_prefetch(const moqe_expert_host* h, void* stream, moqe_expert** out);
MOQE_API moqe_status moqe_expert_host_info(const moqe_expert_host* h, int* N, int* K, int* bits, int* group, int* sym,
                                           size_t* image_bytes);
MOQE_API moqe_status moqe_expert_host_save(const moqe_expert_host* h, const char* path);
MOQE_API moqe_status moqe_expert_host_load(const char* path, moqe_expert_host** out);
MOQE_API moqe_status moqe_expert_host_destroy(moqe_expert_host* h);

/* ---------------------------------------------------------------------------
 * Hard routing (Section 3.2; Appendix: the router's decision r(x) is one expert
 * index per sample, and the expert's output is not weighted by the score).
 * ids[s] = smallest index attaining the maximum of logits[s][0..E); NaN never
 * wins; an all-NaN row gives 0.  logits fp32 [S][E]; ids int32 [S].
 * ------------------------------------------------------------------------- */
MOQE_API moqe_status moqe_route(const float* logits, int S, int E, int32_t* ids, void* stream);

/* Per-sample ids -> per-row ids: rows [row_offsets[s], row_offsets[s+1]) take
 * ids[s].  row_offsets int32 [S+1], non-decreasing, row_offsets[0] == 0,
 * row_offsets[S] == M.  row_ids int32 [M]. */
MOQE_API moqe_status moqe_expand_ids(const int32_t* ids, const int32_t* row_offsets, int S, int M,
                            int32_t* row_ids, void* stream);

/* moqe_route, moqe_expand_ids and the index part of moqe_permute (below) in ONE launch, for small batches (a decode
 * step): S <= 1024 samples, M <= 1024 rows (else MOQE_ERR_UNSUPPORTED, nothing launched).  logits fp32 [S][E],
 * row_offsets int32 [S+1] as for moqe_expand_ids, or NULL for one row per sample (then M == S); written: ids int32 [S],
 * row_ids int32 [M], perm int32 [M], offsets int32 [E+1], with exactly the values the three calls give.  All device
 * pointers; no workspace; E <= MOQE_MAX_EXPERTS. */
MOQE_API moqe_status moqe_route_permute(const float* logits, int S, int E, const int32_t* row_offsets, int M, int32_t* ids,
                                        int32_t* row_ids, int32_t* perm, int32_t* offsets, void* stream);

/* ---------------------------------------------------------------------------
 * Stable counting sort of rows by expert id, and the row gather / scatter.
 * (The batching glue between "one expert per sample" and a grouped GEMM; the
 * per-expert counts are the n_i of the load statistic F_i = n_i / B of
 * Section 3.3 "Router Fine-Tuning".)
 *   offsets[e] = number of rows with id < e            (int32 [E+1])
 *   perm[offsets[e] + r] = the r-th row, in increasing row index, with id e
 *   Xp[j][:] = X[perm[j]][:]                            (rows of C bf16, C % 8 == 0)
 * moqe_permute: X and Xp may both be NULL (indices only).  Rows whose id is
 * outside [0,E) are sorted behind all valid rows (offsets[E] then counts only
 * the valid ones), their Xp rows are zero, and MOQE_ERR_EXPERT_ID is latched.
 * workspace: moqe_permute_workspace(M, E) bytes, contents irrelevant on entry.
 * moqe_unpermute: Y[perm[j]][:] = Yp[j][:].
 * ------------------------------------------------------------------------- */
MOQE_API size_t moqe_permute_workspace(int M, int E);
MOQE_API moqe_status moqe_permute(const void* X_bf16, const int32_t* row_ids, int M, int C, int E, void* Xp_bf16,
                         int32_t* perm, int32_t* offsets, void* workspace, size_t workspace_bytes,
                         void* stream);
MOQE_API moqe_status moqe_unpermute(const void* Yp_bf16, const int32_t* perm, int M, int C, void* Y_bf16,
                           void* stream);

/* moqe_permute for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a deployment convenience of the library.)
 * Who needs it: code that runs where cudaMalloc is off limits -- a plug-in inside
 * a serving process whose memory pool is owned and fully handed out by the host
 * framework, a real-time loop that may not take the allocator's lock or trigger
 * its implicit device synchronisation, or a process kept under a fixed memory
 * budget.  moqe_permute needs a caller-provided workspace for batches above 1024
 * rows; this variant keeps that scratch (per-block bucket totals, 132 KiB) in a
 * fixed array inside the library image, which every GPU that loads the library
 * holds until the process exits.  It performs no allocation at all: no cudaMalloc
 * or cudaFree, no allocating library call.
 *   - Same arguments, results and row limit semantics as moqe_permute, minus the
 *     workspace.  M above MOQE_PERMUTE_STATIC_MAX_ROWS returns MOQE_ERR_WORKSPACE
 *     (nothing is launched): use moqe_permute for such batches.
 *   - Ids outside [0,E) are sorted behind the valid rows and their Xp rows are
 *     zero, exactly as in moqe_permute, but NO error is latched for
 *     moqe_async_status (the status word lives in allocated memory); compare
 *     offsets[E] with M to detect them.
 *   - The first call on each device looks up the device address of the built-in
 *     array (a host-side query, not an allocation).  Make that first call outside
 *     any stream capture.
 *   - All calls on a device share the one array.  Nothing in it needs clearing
 *     between calls (each call writes every entry before reading it), but two
 *     calls that overlap on the GPU -- different streams, or concurrent host
 *     threads on different streams -- race on it: serialise them. */
#define MOQE_PERMUTE_STATIC_MAX_ROWS (1 << 20)
MOQE_API moqe_status moqe_permute_static(const void* X_bf16, const int32_t* row_ids, int M, int C, int E,
                                         void* Xp_bf16, int32_t* perm, int32_t* offsets, void* stream);

/* ---------------------------------------------------------------------------
 * Router front end on the device (Section 3.2 "Router Model": the router ends in an MLP that maps the sample's
 * feature vector to one score per expert, and one expert index leaves it).  The paper's trained encoders are not
 * part of this library; the feature vector is the mean of the sample's rows:
 *   pooled[s][h] = mean over rows r in [row_offsets[s], row_offsets[s+1]) of X[r][h]   (0 for a sample without rows)
 *   hidden[s][d] = max(0, sum_h pooled[s][h] * W1[d][h]),   logits[s][e] = sum_d hidden[s][d] * W2[e][d]
 *   ids[s]       = first maximum of logits[s] (as moqe_route)
 * X bf16 [rows][H] (H a multiple of 8, 16-byte aligned), row_offsets int32 [S+1], W1 fp32 [D][H] (16-byte aligned),
 * W2 fp32 [E][D], logits fp32 [S][E] and ids int32 [S] are written.  All device pointers; fp32 arithmetic in a fixed
 * summation order (the same call gives the same bits).  workspace: moqe_router_mlp_workspace(S, H, D) bytes,
 * 256-byte aligned, contents irrelevant.  E <= MOQE_MAX_EXPERTS.
 *
 * moqe_router_load_report (Section 3.3 "Router Fine-Tuning", the balance term, evaluated on a routed batch):
 *   report[i] = P_i = mean over the S samples of softmax(logits[s])_i,   report[E + i] = F_i = n_i / S,
 *   report[2E] = L_bal = E * sum_i P_i * F_i,   counts[i] = n_i = samples with ids[s] == i   (counts may be NULL).
 * ------------------------------------------------------------------------- */
MOQE_API size_t moqe_router_mlp_workspace(int S, int H, int D);
MOQE_API moqe_status moqe_router_mlp(const void* X_bf16, const int32_t* row_offsets, int S, int H, const float* W1, int D,
                                     const float* W2, int E, float* logits, int32_t* ids, void* workspace,
                                     size_t workspace_bytes, void* stream);
MOQE_API moqe_status moqe_router_load_report(const float* logits, const int32_t* ids, int S, int E, float* report,
                                             int32_t* counts, void* stream);

/* ---------------------------------------------------------------------------
 * The routed dequant-GEMM (Section 3.1: "the activated quantization expert
 * performs the inference on this sample" -- here for a whole mixed batch):
 *   Y[m][n] = bf16( sum_k X[m][k] * s_e[n][k/g] * (c_e[n][k] - z_e[n][k/g]) ),
 *   e = row_ids[m], accumulated in fp32.
 * X bf16 [M][K]; row_ids int32 [M]; h_experts: HOST array of E expert handles
 * that agree on N and K; Y bf16 [M][N] (every row is written; rows with an
 * invalid id are written as zeros).  M == 0 is valid.  workspace:
 * moqe_routed_qgemm_workspace(M, N, K, E) bytes, contents irrelevant on entry;
 * calls that share a workspace must not overlap on the device.
 * Decode batches (at most 32 rows, experts per-channel or with groups of 128 k or more) stream each touched
 * expert's packed weights once through the decode kernel (bulk-copy ring, warp-level MMAs on fp16 operands,
 * stream-K split that follows the routing: experts without rows cost nothing).  That kernel converts the bf16
 * activations to fp16: values with |x| > 65504 are outside its domain (they become infinities); every other
 * kernel takes the whole bf16 range.  Other small batches take the split-K mma.sync streaming kernel; large
 * batches run the persistent tcgen05 grouped GEMM.
 * ------------------------------------------------------------------------- */
MOQE_API size_t moqe_routed_qgemm_workspace(int M, int N, int K, int E);
MOQE_API moqe_status moqe_routed_qgemm(const void* X_bf16, const int32_t* row_ids, int M,
                              const moqe_expert* const* h_experts, int E, void* Y_bf16,
                              void* workspace, size_t workspace_bytes, void* stream);

/* Same, with the kernel chosen by the caller (testing / measurement):
 * path 0 = automatic, 1 = split-K dequant-MMA streaming kernel, 2 = tcgen05 grouped GEMM (automatic
 * token tile), 3 / 4 = tcgen05 grouped GEMM with 128- / 256-token tiles, 5 = decode kernel
 * (MOQE_ERR_UNSUPPORTED if the batch has more than 32 rows or an expert has groups narrower than 128 k),
 * 6 = dense-weights tcgen05 GEMM for large batches on small layers (more than 128 rows, K <= 1024, at most 1024
 * output channels; the automatic choice there: the layer is bound by its activations, so each expert's weights
 * are expanded to bf16 once per call and X / Y are streamed; MOQE_ERR_UNSUPPORTED otherwise). */
MOQE_API moqe_status moqe_routed_qgemm_path(const void* X_bf16, const int32_t* row_ids, int M,
                                   const moqe_expert* const* h_experts, int E, void* Y_bf16,
                                   void* workspace, size_t workspace_bytes, void* stream, int path);

/* The same product for a batch that is already sorted: `perm` [M] and `offsets`
 * [E+1] as moqe_permute wrote them (device pointers; rows perm[offsets[E]..M) are
 * left untouched in Y).  One sort then serves every linear layer of a block,
 * since a sample keeps its expert through the whole model (Section 3.1).
 * The split-K arrival counters at the head of the workspace body must be zero on
 * entry -- clear them once with moqe_routed_qgemm_workspace_clear after
 * allocating the workspace (same M, N, K, E) -- and every call leaves them zero,
 * except a call that ended in MOQE_ERR_TIMEOUT (moqe_async_status): clear the
 * workspace again before it is reused after that.
 * `path` as for moqe_routed_qgemm_path. */
MOQE_API moqe_status moqe_routed_qgemm_sorted(const void* X_bf16, const int32_t* perm, const int32_t* offsets, int M,
                                              const moqe_expert* const* h_experts, int E, void* Y_bf16,
                                              void* workspace, size_t workspace_bytes, void* stream, int path);
/* Several linear layers of one decode batch in ONE launch: layers that share the routing (`perm`, `offsets`
 * and M as above) and do not depend on one another -- the q/k/v projections of a block, or its gate and up
 * projections (Section 3.1: a sample keeps its expert through the whole model).  h_X_bf16[l] / h_Y_bf16[l] are
 * host arrays of device pointers to layer l's input [M][K_l] and output [M][N_l]; h_experts[l * E + e] is expert
 * e of layer l (the E experts of a layer agree on N and K; layers may differ).  Same workspace rules as
 * moqe_routed_qgemm_sorted, sized for layer 0 (moqe_routed_qgemm_workspace(M, N_0, K_0, E)).
 * Only what the decode kernel takes: M <= 32, experts per-channel or with groups of 128 k or more,
 * n_layers * E <= MOQE_MAX_EXPERTS; otherwise MOQE_ERR_UNSUPPORTED and nothing is launched (call
 * moqe_routed_qgemm_sorted per layer instead). */
MOQE_API moqe_status moqe_routed_qgemm_sorted_multi(const void* const* h_X_bf16, const int32_t* perm, const int32_t* offsets,
                                                    int M, int n_layers, const moqe_expert* const* h_experts, int E,
                                                    void* const* h_Y_bf16, void* workspace, size_t workspace_bytes,
                                                    void* stream);
/* Two steps of an expert's forward pass fused into the routed product of a DECODE batch (Section 4.4 times whole
 * expert forwards, so what sits between two linear layers counts).  Same `perm` / `offsets` / workspace rules as
 * moqe_routed_qgemm_sorted; only batches of at most 16 rows of what the decode kernel takes (experts per-channel or with groups of
 * 128 k or more), otherwise MOQE_ERR_UNSUPPORTED and nothing is launched.
 *   _gated    : Y[m][n] = bf16( silu(a) * b ),  a = (X . Wgate_e^T)[m][n],  b = (X . Wup_e^T)[m][n],  e = the row's
 *               expert, silu(a) = a / (1 + exp(-a)); a and b are the fp32 sums, rounded once at the end.  h_gate[e] and
 *               h_up[e] must agree on N, K, bits, group and sym (MOQE_ERR_MISMATCH).  One launch streams both experts'
 *               weights; the [M][N] intermediate of each projection is never written.
 *   _residual : Y[m][n] = bf16( (X . W_e^T)[m][n] + R[m][n] ),  R bf16 [M][N] in original row order (may be Y itself). */
MOQE_API moqe_status moqe_routed_qgemm_sorted_gated(const void* X_bf16, const int32_t* perm, const int32_t* offsets, int M,
                                                    const moqe_expert* const* h_gate, const moqe_expert* const* h_up, int E,
                                                    void* Y_bf16, void* workspace, size_t workspace_bytes, void* stream);
MOQE_API moqe_status moqe_routed_qgemm_sorted_residual(const void* X_bf16, const int32_t* perm, const int32_t* offsets, int M,
                                                       const moqe_expert* const* h_experts, int E, const void* R_bf16,
                                                       void* Y_bf16, void* workspace, size_t workspace_bytes, void* stream);
MOQE_API moqe_status moqe_routed_qgemm_workspace_clear(void* workspace, size_t workspace_bytes, int M, int N, int K,
                                                       int E, void* stream);

/* Synchronises `stream`, then returns and clears the first error latched by a
 * kernel on the current device (MOQE_OK if none). */
MOQE_API moqe_status moqe_async_status(void* stream);

MOQE_API const char* moqe_status_str(moqe_status s);

/* Measurement knobs (process-wide, not thread-safe; defaults are the tuned values):
 *   "stream_tile_cost_w8" / "_w4" / "_w3" : relative cost of one packed 128x128 tile of
 *                            that bit-width in the streaming kernel's work split
 *                            (defaults 8 / 8 / 8).
 *   "decode_tile_cost_w8" / "_w4" / "_w3" : the same for the decode kernel (defaults 10 / 10 / 10).
 *   "auto_decode"          : whether path 0 takes the decode kernel where it applies (default 1).
 *   "auto_dense"           : whether path 0 takes the dense-weights GEMM where it applies (default 1).
 * Unknown key: MOQE_ERR_UNSUPPORTED. */
MOQE_API moqe_status moqe_tune(const char* key, int value);

/* Self-test of the bounded waits every kernel of this library uses (no counterpart in the paper): launches one
 * small kernel whose only thread waits, with a limit of `limit_us` microseconds (1 .. 1 000 000), on an mbarrier
 * nobody ever arrives on.  The wait must give up by itself: the kernel then writes 2 to *d_returned (device int;
 * 1 would mean the barrier completed), latches MOQE_ERR_TIMEOUT in the device status word -- read and cleared by
 * the next moqe_async_status -- and returns; the context stays usable and later calls work as usual. */
MOQE_API moqe_status moqe_selftest_timeout(unsigned limit_us, int* d_returned, void* stream);

/* Number of kernels this library has launched so far in this process. */
MOQE_API unsigned long long moqe_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* MOQE_H_ */
