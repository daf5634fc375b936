/*
 * scap.h - C ABI of the SCAP sparse fully-connected library for NVIDIA B200 (sm_100a).
 *
 * SCAP (Statistical Calibrated Activation Pruning) sparsifies the INPUT activation of a
 * fully-connected layer at decode time: the input is mode-centred (x' = x - m), every entry
 * with |x'| < tau is dropped, and the matrix-vector product only fetches the weight rows of
 * the surviving input channels; m W is folded into the bias offline so the layer's function is
 * unchanged before pruning.
 *
 * Notation (paper's in brackets):  K input channels [IC], N output channels [OC], B batch rows.
 *   x[B,K]      row-major activations, fp16 or bf16
 *   W[K,N]      row-major weights, fp16 or bf16; row k holds every output of input channel k
 *               [W in R^{IC x OC} of Eq. 1], so a kept channel is one contiguous row
 *   m[K]        per-channel mode, fp32 (the paper's scalar eta is the constant vector)
 *   tau[1]      pruning threshold, fp32, in DEVICE memory (no host round trip)
 *   b_fused[N]  b + m W, fp32 (Eq. 6)
 *   y[B,N]      fp32
 *
 * General rules for every entry point
 *   - All data pointers are DEVICE pointers unless the parameter name ends in _host.
 *   - The caller owns every buffer; the library allocates no device memory and keeps no state
 *     between calls except the process-wide tuning set by scap_tune().
 *   - Calls enqueue work on `stream` and return without synchronising; they perform no host
 *     synchronisation, so they may be recorded into a CUDA graph.  Two calls that share a
 *     workspace must be ordered on one stream.
 *   - Data pointers must be 16-byte aligned and N (and F, D for the FFN calls) a multiple of 8,
 *     else SCAP_ERR_ALIGN.  B outside 1..16, K < 1, K > 1048576 or N < 1 give SCAP_ERR_SHAPE.  A
 *     NULL required pointer gives SCAP_ERR_INVALID_ARG, a workspace smaller than the matching
 *     *_workspace() query SCAP_ERR_WORKSPACE, an unknown dtype SCAP_ERR_DTYPE, a failed launch
 *     SCAP_ERR_CUDA, a device that is not compute capability 10.x SCAP_ERR_UNSUPPORTED_ARCH.
 *     Nothing throws, aborts, traps or prints.  On error nothing has been enqueued.
 *   - Workspace contents are scratch: undefined on entry, undefined on exit.
 *   - Every kernel of a call waits for the work placed before it on the stream before it reads the activations,
 *     m, tau, the scales, the biases or a row map, and reads whatever a kernel may have rewritten through L2.  So
 *     these may be produced on the same stream directly before the call that uses them (scap_calibrate,
 *     scap_fold_bias, or any kernel or copy of the caller's), with no further synchronisation.  The weight matrix W
 *     is the exception: it is a constant of the layer and must be complete in device memory when the call is
 *     ISSUED (not written by work still pending on the stream), because kernels that know their first weight rows
 *     without looking at the activations (the batch 5..16 kernel, the dense calls, a sparse call with "head_rows"
 *     set) request them before that wait, so that the memory system does not idle between consecutive calls.  Consecutive calls overlap where they can: a kernel may
 *     become resident and set up its shared memory while its predecessor drains (programmatic dependent launch,
 *     "pdl" below).
 */
#ifndef SCAP_H_
#define SCAP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SCAP_OK = 0,
    SCAP_ERR_INVALID_ARG = 1,
    SCAP_ERR_SHAPE = 2,
    SCAP_ERR_DTYPE = 3,
    SCAP_ERR_ALIGN = 4,
    SCAP_ERR_WORKSPACE = 5,
    SCAP_ERR_CUDA = 6,
    SCAP_ERR_TIMEOUT = 7,
    SCAP_ERR_UNSUPPORTED_ARCH = 8
} scap_status;

typedef enum { SCAP_F16 = 0, SCAP_BF16 = 1 } scap_dtype;

/* A CUDA stream handle (cudaStream_t); NULL is the legacy default stream. */
typedef struct CUstream_st *scap_stream_t;

#define SCAP_MAX_BATCH 16
#define SCAP_MAX_EXPERTS 32
#define SCAP_MAX_TOP_K 4

/* Static string naming a status code. */
const char *scap_status_string(scap_status st);

/* Library version, major * 1000 + minor. */
int scap_version(void);

/* Process-wide tuning knobs (plain ints, not thread-safe against concurrent calls):
 *   "split_k"  cap the split-K factor (thread-block cluster size) of the FC kernel: 0 = automatic, else 1..8
 *   "tile"     columns of the output a CTA of the FC kernel owns: 0 = automatic (default), else 128 or 256
 *   "pdl"      1 = launch dependent kernels with programmatic dependent launch (default), 0 = off
 *   "fma_rows" largest batch that runs on the fp32-FMA form of the FC kernel: 4 (default) or 2; larger
 *              batches (up to 16) run on a tensor-core form
 *   "tcgen05"  tensor-core batches of the FC and SwiGLU entry points: 0 = always the mma.sync variants,
 *              1 = the tcgen05 (TMEM accumulator) kernel where its shared-memory operand region holds
 *              the call's kept channels in one pass, else mma.sync (default), 2 = always tcgen05
 *   "dense_stream"  batches above "fma_rows": 1 (default) = the dense-stream tensor-core kernel, which reads every row of
 *              its weight tile with TMA box loads and prunes on the activation operand (with that many rows the union
 *              mask of unrelated rows keeps nearly every channel anyway); 0 = the gather kernels, which fetch kept rows
 *              only (better when the rows of a batch share their pattern and the union keeps less than about half);
 *              2 = the dense-stream kernel from batch 3 on
 *   "tc_spin"  tcgen05 kernels: how often a wait on one of its shared-memory barriers polls before it gives up
 *              (0 = the built-in limit of about a million polls, the default).  A limit of 1 makes the waits of
 *              the next call run out at once, which is how the error path of scap_device_status() is exercised
 *              without a fault; y of such a call is incomplete.
 *   "host_direct"  scap_sparse_fc_host: 1 = when x_host and y_host are page-locked and addressable by the
 *              device, a kernel pulls x and the FC kernel writes y to host memory (default), 0 = always copies
 *   "cal_strip"  scap_calibrate: channels per CTA of the per-channel histogram kernel, 16 (default: 256 threads,
 *              two CTAs per SM) or 32 (512 threads, one CTA per SM)
 *   "head_rows" batch 1..4 FC kernel, sparse calls: number of 32-channel chunks per CTA (0..64, default 0) whose weight
 *              rows are asked into L2 at kernel start, before the kept set is known.  It fills the idle time between
 *              calls with reads of which the pruned share is wasted: measured at K = 11008, N = 4096 with 6 chunks,
 *              -0.4 us per call at 50 % sparsity, -0.25 us at 60 %, +0.3 us at 90 %, for 12.6 MB of requests per
 *              call.  Dense calls, which need every row, always ask for their first 4 chunks.
 *   "l2_hints"  batch 1..4 FC kernel: 1 = loads carry L2 eviction hints (default): activations and modes, which every
 *              column tile of a call reads again, are kept (evict_last); weight rows, read once, go first
 *              (evict_first); 0 = no hints
 * Unknown keys return SCAP_ERR_INVALID_ARG.  Tuning never changes what is computed; split_k
 * changes the (fixed) summation order and therefore the last bits of y.  Query workspace sizes
 * after tuning.                                                                               */
scap_status scap_tune(const char *key, int value);

/* The tcgen05 kernel bounds every wait on a shared-memory barrier; a wait that runs out (which a
 * correct run never does) makes the CTA stop issuing work, so y is then incomplete.  This call
 * synchronises the device, returns SCAP_ERR_TIMEOUT if that happened since the last call (and
 * clears the record), SCAP_OK otherwise.  Not for use during stream capture.                   */
scap_status scap_device_status(void);

/* ------------------------------------------------------------------------------------------
 * Offline calibration (Section 3, "Mode-Centering Calibration"; Eq. 2 for tau)
 *
 * scap_calibrate reads calibration activations x_calib[T,K] (row-major, dtype dt) and writes
 *   m_out[K]   per-channel mode: arg-max bin centre of an nbins-bin histogram over the channel's
 *              [min, max] range (lowest bin wins ties; a constant channel returns that constant).
 *              nbins = 0 disables centring and writes zeros.  1 <= nbins <= 2048 otherwise.
 *   tau_out[1] the `sparsity` quantile (linear interpolation between order statistics) of the
 *              importance |x - m| pooled over all T*K values; sparsity <= 0 gives tau = 0.
 * Binary32 arithmetic with every operation rounded separately, so results are bit-reproducible.
 * Inputs must be finite.  sparsity must lie in [0, 1); T*K < 2^31; T <= 65535; K a multiple of 8
 * (else SCAP_ERR_ALIGN).
 * ------------------------------------------------------------------------------------------ */
size_t scap_calibrate_workspace(int T, int K, int nbins);
scap_status scap_calibrate(const void *x_calib, int T, int K, scap_dtype dt, double sparsity, int nbins,
                           float *m_out, float *tau_out, void *ws, size_t ws_bytes, scap_stream_t stream);

/* Section 3, "Determination of mode value": the paper names the empirical mean and the median as fast
 * estimates of the mode, and its eta is one scalar per FC.  scap_calibrate_ex is scap_calibrate with the
 * estimator and the scope chosen by the caller (same workspace query, same tau computation on |x - m|):
 *   SCAP_MODE_HISTOGRAM  arg-max bin centre as in scap_calibrate
 *   SCAP_MODE_MEAN       per channel: the column added in row order in binary64, divided by T, rounded once
 *   SCAP_MODE_MEDIAN     per channel: the middle value, or the mean of the two middle values (binary64,
 *                        rounded once) for even T
 *   SCAP_MODE_KDE        per channel only: peak of a Gaussian kernel density estimate, bandwidth sigma * T^(-1/5)
 *                        (Scott's rule, sample standard deviation), evaluated in binary64 on nbins >= 2 grid points
 *                        from the channel's minimum to its maximum; the first point of largest density.  T <= 4096
 *                        (else SCAP_ERR_SHAPE); with SCAP_ETA_SCALAR or nbins < 2: SCAP_ERR_INVALID_ARG.  Where two
 *                        grid points have densities equal to within rounding, either may be returned.
 *   SCAP_ETA_PER_CHANNEL one value per input channel in m_out[K]
 *   SCAP_ETA_SCALAR      one value for the whole tensor, written to all K entries of m_out: the estimator
 *                        applied to all T*K values as one sample (mean: the column sums of the per-channel
 *                        form added in channel order, divided by T*K)
 * A result of -0 is returned as +0.  Inputs must be finite.                                            */
typedef enum { SCAP_MODE_HISTOGRAM = 0, SCAP_MODE_MEAN = 1, SCAP_MODE_MEDIAN = 2, SCAP_MODE_KDE = 3 } scap_mode_estimator;
typedef enum { SCAP_ETA_PER_CHANNEL = 0, SCAP_ETA_SCALAR = 1 } scap_eta_scope;
scap_status scap_calibrate_ex(const void *x_calib, int T, int K, scap_dtype dt, double sparsity,
                              scap_mode_estimator estimator, scap_eta_scope scope, int nbins, float *m_out,
                              float *tau_out, void *ws, size_t ws_bytes, scap_stream_t stream);

/* Eq. 5-6: b_fused[n] = b[n] + sum_k m[k] W[k,n].  b is in the weight dtype and may be NULL
 * (zero bias).  Run once per layer after calibration.                                          */
size_t scap_fold_bias_workspace(int K, int N);
scap_status scap_fold_bias(const void *W, const float *m, const void *b, int K, int N, scap_dtype dt,
                           float *b_fused, void *ws, size_t ws_bytes, scap_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * Decode-time sparse FC (Eq. 2-3, Eq. 6; Alg. 3 "SCAP FC with Mode Centering")
 *
 *   d[b,k]   = float(x[b,k]) - m[k]            one binary32 subtraction (m == NULL: d = x)
 *   keep     = |d| >= tau                      (a NaN is dropped)
 *   y[b,n]   = b_fused[n] + sum_k keep[b,k] d[b,k] W[k,n]      fp32 accumulation, fixed order
 * Only rows of W whose channel is kept by at least one batch row are read.  Pruning is per
 * element, so row b of a batched call equals the batch-1 call on row b up to summation order.
 * Optional outputs for inspection: idx_out[K] receives the ascending list of fetched channels
 * (first *nnz_out entries valid), nnz_out[1] their number.  m, b_fused, idx_out, nnz_out may
 * be NULL.  Results are bitwise reproducible for fixed shapes and tuning.
 * Arithmetic: batches up to the tuning value "fma_rows" (default 4) multiply-accumulate in fp32 FMAs.
 * Larger batches (up to 16) run on the tensor cores with d split exactly into parts of the weight dtype
 * (bf16: three parts, fp16: two) and fp32 accumulation, so the result carries the same information as
 * the FMA path; with fp16 weights the parts overflow for |d| > 65504 (such an activation yields inf/NaN
 * in its row only).  In the tensor-core forms a non-finite weight makes its column non-finite whether
 * or not its channel is kept (0 * inf): weights must be finite.
 * ------------------------------------------------------------------------------------------ */
size_t scap_fc_workspace(int B, int K, int N);
scap_status scap_sparse_fc(const void *x, const void *W, const float *m, const float *tau, const float *b_fused,
                           float *y, int B, int K, int N, scap_dtype dt, uint32_t *idx_out, int *nnz_out,
                           void *ws, size_t ws_bytes, scap_stream_t stream);

/* Eq. 1: y = x W + b over the same layout, no pruning; the library's own dense baseline.
 * b is fp32 [N] or NULL.  Uses scap_fc_workspace(B, K, N).                                     */
scap_status scap_dense_fc(const void *x, const void *W, const float *b, float *y, int B, int K, int N,
                          scap_dtype dt, void *ws, size_t ws_bytes, scap_stream_t stream);

/* 8-bit weights (Table 4 applies SCAP to 8-bit models).  Storage: Wq[K,N] signed 8-bit, row-major like W, and
 * wscale[K] fp32, one scale per input channel: W[k,n] = wscale[k] * Wq[k,n] (symmetric, no zero point).  x has
 * dtype xdt (fp16 or bf16); everything else as in scap_sparse_fc / scap_dense_fc / scap_fold_bias, with these
 * differences: N must be a multiple of 16; the bias b of the dense call and of the folding is fp32 [N] or
 * NULL; batches of more than two rows are processed two rows at a time (results per row as in scap_sparse_fc;
 * idx_out / nnz_out are only available for B <= 2, else SCAP_ERR_SHAPE).  Workspace: scap_fc_workspace(B, K, N). */
scap_status scap_sparse_fc_q8(const void *x, scap_dtype xdt, const signed char *Wq, const float *wscale, const float *m,
                              const float *tau, const float *b_fused, float *y, int B, int K, int N, uint32_t *idx_out,
                              int *nnz_out, void *ws, size_t ws_bytes, scap_stream_t stream);
scap_status scap_dense_fc_q8(const void *x, scap_dtype xdt, const signed char *Wq, const float *wscale, const float *b,
                             float *y, int B, int K, int N, void *ws, size_t ws_bytes, scap_stream_t stream);
scap_status scap_fold_bias_q8(const signed char *Wq, const float *wscale, const float *m, const float *b, int K, int N,
                              float *b_fused, void *ws, size_t ws_bytes, scap_stream_t stream);

/* Group-wise 4-bit weights (Table 4 applies SCAP to AWQ 4-bit models; the paper names the models, not a layout - this one is
 * the library's).  Storage: Wq[K, N/2] bytes, two unsigned codes q in 0..15 per byte (column 2j in the low nibble of byte
 * j, column 2j+1 in the high nibble), row-major like W, so a kept input channel is still one contiguous row; groups of
 * `group` consecutive INPUT channels share, per output column, scale[K/group rounded up, N] (fp32) and a zero point
 * zero[same shape] (one byte, 0..15):  W[k,n] = scale[k / group, n] * (q[k,n] - zero[k / group, n]).
 * group: a multiple of 32, 32..2048 (else SCAP_ERR_SHAPE); N a multiple of 16.  Everything else - x of dtype xdt, m, tau,
 * b_fused, y, the optional kept list, the batch rule (more than two rows run two at a time; idx_out / nnz_out only for
 * B <= 2), the workspace query - as for the 8-bit calls above.  The sum over the kept channels of one group is formed
 * on the integer codes in fp32 as sum d * q - zero * sum d, and scaled once.                                          */
scap_status scap_sparse_fc_q4(const void *x, scap_dtype xdt, const unsigned char *Wq, const float *scale,
                              const unsigned char *zero, int group, const float *m, const float *tau, const float *b_fused,
                              float *y, int B, int K, int N, uint32_t *idx_out, int *nnz_out, void *ws, size_t ws_bytes,
                              scap_stream_t stream);
scap_status scap_dense_fc_q4(const void *x, scap_dtype xdt, const unsigned char *Wq, const float *scale,
                             const unsigned char *zero, int group, const float *b, float *y, int B, int K, int N, void *ws,
                             size_t ws_bytes, scap_stream_t stream);
scap_status scap_fold_bias_q4(const unsigned char *Wq, const float *scale, const unsigned char *zero, int group, const float *m,
                              const float *b, int K, int N, float *b_fused, void *ws, size_t ws_bytes, scap_stream_t stream);

/* Appendix C ("overlapping sparsity"): the union mask of a batch keeps its sparsity only as far as the rows' patterns
 * overlap.  scap_sparse_fc_grouped is scap_sparse_fc for up to 64 rows whose groups the caller names - rows that are
 * expected to share their pattern, e.g. the beams of one prompt or the tokens of one request: group_of_row_host[b]
 * (a HOST array, read during the call only) is the group 0..15 of row b; at most 16 rows per group (else
 * SCAP_ERR_SHAPE).  Each group is pruned with the union mask of its own rows only and fetches only the weight rows
 * that mask keeps, all groups in one launch; y[b] is the same function of x[b] as in scap_sparse_fc (pruning is per
 * element), whatever the grouping.  No idx / nnz outputs.  Workspace: scap_grouped_workspace() bytes.              */
size_t scap_grouped_workspace(void);
scap_status scap_sparse_fc_grouped(const void *x, const void *W, const float *m, const float *tau, const float *b_fused,
                                   float *y, int B, int K, int N, scap_dtype dt, const int *group_of_row_host, void *ws,
                                   size_t ws_bytes, scap_stream_t stream);

/* scap_sparse_fc for a caller whose activations live in HOST memory: copies x_host[B,K]
 * (dtype dt; pinned memory recommended) to the device, runs the sparse FC, and copies y back to
 * y_host[B,N] (fp32), all enqueued on `stream`; y_host is valid once the stream has drained.
 * If both buffers are page-locked and addressable by the device (cudaHostAlloc, cudaHostRegister), the
 * transfers are done by the library's kernels instead of copy operations (a small kernel pulls x into
 * the workspace, the FC kernel stores y to host memory); x_host must stay unchanged until then.
 * W, m, tau, b_fused stay device-resident.  Needs scap_fc_host_workspace(B, K, N) bytes.        */
size_t scap_fc_host_workspace(int B, int K, int N);
scap_status scap_sparse_fc_host(const void *x_host, const void *W, const float *m, const float *tau,
                                const float *b_fused, float *y_host, int B, int K, int N, scap_dtype dt,
                                void *ws, size_t ws_bytes, scap_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * SwiGLU FFN block (Alg. 2 "SCAP's SwiGLU")
 *
 *   [g | u] = sparse_fc(h; Wgu, m1, tau1, bgu_fused)     one mask shared by gate and up
 *   z       = u * silu(g),  silu(g) = g / (1 + exp(-g))  kept in fp32
 *   y       = sparse_fc(z; Wd, m2, tau2, bd_fused)
 * h[B,D]; Wgu[D,2F] with gate in columns 0..F-1 and up in columns F..2F-1 of each row; Wd[F,D];
 * bgu_fused[2F]; bd_fused[D]; y[B,D].  m1, m2 and the two fused biases may be NULL.  Optional
 * outputs: z_out[B,F] (the fp32 z the second mask was taken on), idx1_out[D]/nnz1_out[1],
 * idx2_out[F]/nnz2_out[1].  D and F must be multiples of 8.
 * ------------------------------------------------------------------------------------------ */
size_t scap_glu_workspace(int B, int D, int F);
scap_status scap_glu_ffn(const void *h, const void *Wgu, const void *Wd, const float *m1, const float *tau1,
                         const float *bgu_fused, const float *m2, const float *tau2, const float *bd_fused,
                         float *y, int B, int D, int F, scap_dtype dt, float *z_out, uint32_t *idx1_out,
                         int *nnz1_out, uint32_t *idx2_out, int *nnz2_out, void *ws, size_t ws_bytes,
                         scap_stream_t stream);

/* Non-GLU FFN block (Section 4.3, the Falcon / MPT ablation of mode centring): up projection, exact GELU,
 * mode-centred sparse down projection.
 *   u = scap_sparse_fc(h; Wu[D,F], m1, tau1, bu_fused)      (tau1 = 0 runs the up projection on every channel)
 *   z = gelu(u) = u/2 (1 + erf(u / sqrt 2))                 fp32, formed in the epilogue of the first kernel
 *   y = scap_sparse_fc(z; Wd[F,D], m2, tau2, bd_fused)      z in fp32, never leaves L2
 * Arguments, optional outputs (z_out[B,F], idx1_out .. nnz2_out), workspace rules and errors as scap_glu_ffn; the workspace
 * query returns the same size as scap_glu_workspace.                                                           */
size_t scap_gelu_ffn_workspace(int B, int D, int F);
scap_status scap_gelu_ffn(const void *h, const void *Wu, const void *Wd, const float *m1, const float *tau1,
                          const float *bu_fused, const float *m2, const float *tau2, const float *bd_fused, float *y,
                          int B, int D, int F, scap_dtype dt, float *z_out, uint32_t *idx1_out, int *nnz1_out,
                          uint32_t *idx2_out, int *nnz2_out, void *ws, size_t ws_bytes, scap_stream_t stream);

/* scap_glu_ffn without a workspace argument (the paper has no counterpart; this is a deployment aid).
 *
 * Some callers must not allocate device memory on the decode path: a serving process that handed all
 * free HBM to its KV-cache pool at start-up, a plug-in that runs inside a host framework's memory
 * budget, or code on a latency-critical path where cudaMalloc's implicit device synchronisation is not
 * acceptable.  For them the scratch of the SwiGLU block (the fp32 intermediate z[B,F] plus a few mask
 * words) lives in a fixed array inside the library image instead of a caller workspace.  The call
 * performs no cudaMalloc / cudaFree and uses no allocating library routine.
 *
 *   - Capacity: scap_glu_static_capacity() bytes (2 MiB), held by every GPU that loads the library
 *     until the process exits.  A shape needing more (scap_glu_workspace(B, D, F) > capacity, i.e.
 *     roughly B * F > 520000) is rejected with SCAP_ERR_WORKSPACE and nothing is enqueued.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress) and
 *     caches it; make that first call outside any stream capture.  The cached address belongs to the
 *     device's current context: it is not valid after a cudaDeviceReset.
 *   - All calls on a device share the one array.  It keeps whatever the last call left there; nothing
 *     needs clearing because each call writes every word before reading it.  Two calls that overlap
 *     on the GPU (different streams, or graphs replayed concurrently) race on it: keep them on one
 *     stream or order them with events.
 *   - Arguments, results and error codes are otherwise those of scap_glu_ffn (no idx/nnz outputs).   */
size_t scap_glu_static_capacity(void);
scap_status scap_glu_ffn_static(const void *h, const void *Wgu, const void *Wd, const float *m1, const float *tau1,
                                const float *bgu_fused, const float *m2, const float *tau2, const float *bd_fused,
                                float *y, int B, int D, int F, scap_dtype dt, float *z_out, scap_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * Mixture-of-experts FFN layer (the paper applies SCAP to Mixtral-8x7B, Table 4; it does not
 * describe the router, so the convention is this library's): p = softmax(logits[b, 0..E-1]),
 * the top_k largest are selected (ties to the lower index), their weights renormalised to sum
 * to one, and y[b] = sum_j w[b,j] * glu_ffn_{e(b,j)}(h[b]), summed in selection order.  Each
 * expert has its own calibration (m1, tau1, m2, tau2) and fused biases; the rows routed to one
 * expert share that expert's union mask.
 * experts_host: HOST array of E structs holding DEVICE pointers (read during the call only).
 * logits[B,E] fp32.  Optional outputs expert_out[B,top_k] (int32), weight_out[B,top_k] (fp32).
 * 1 <= E <= SCAP_MAX_EXPERTS, 1 <= top_k <= min(E, SCAP_MAX_TOP_K).
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    const void *Wgu;        /* [D,2F] */
    const void *Wd;         /* [F,D]  */
    const float *m1;        /* [D]  nullable */
    const float *tau1;      /* [1]  */
    const float *bgu_fused; /* [2F] nullable */
    const float *m2;        /* [F]  nullable */
    const float *tau2;      /* [1]  */
    const float *bd_fused;  /* [D]  nullable */
} scap_expert;

size_t scap_moe_workspace(int B, int D, int F, int E, int top_k);
scap_status scap_moe_ffn(const void *h, const float *logits, const scap_expert *experts_host, int E, int top_k,
                         float *y, int B, int D, int F, scap_dtype dt, int *expert_out, float *weight_out,
                         void *ws, size_t ws_bytes, scap_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* SCAP_H_ */
