/*
 * codistill.h -- C ABI of the fused codistillation objective (loss forward + gradient
 * with respect to the logits) for NVIDIA B200 (sm_100a).
 *
 * The operation is the per-model objective inside the update of Algorithm 1
 * ("Codistillation") of "A Closer Look at Codistillation for Distributed Training"
 * (arXiv 2010.02838): for model i with logits z and peers z^(j), j != i,
 *
 *     loss_row = L(y, z) + alpha * 1/(n-1) * sum_{j != i} D(z, z^(j))
 *
 * where L is the supervised loss of Section 2, here the cross-entropy of softmax(z) against the
 * label y (the paper's experiments are all classification), and D is, as in the paper's
 * experiments (Appendix, "Implementation Details"), the mean squared error between the raw,
 * un-centred logits of the two models.  The KL divergence between temperature softmaxes
 * that Section 2 attributes to earlier work is available as a second form of D.  The
 * gradient is taken with respect to model i's logits only; the peers are constants
 * (Algorithm 1 differentiates with respect to theta_i alone; Section 3).
 *
 * Conventions common to every entry point
 *   - Unless a parameter says HOST, a pointer is a DEVICE pointer owned by the caller; the
 *     library never frees or keeps it.  Inputs are never written.  grad_logits must not
 *     alias an input.
 *   - Work is enqueued on the caller's stream and the call returns immediately; outputs are
 *     valid once that stream has been synchronised.
 *   - Return value: CODISTILL_OK, or a CODISTILL_ERR_* code for anything the host can
 *     check, in which case nothing was launched.  Conditions only the device can see set
 *     bits in *dev_status (CODISTILL_DEV_*).  Nothing traps, aborts or prints.
 *   - Tensors are row-major [rows, classes] with a common row pitch `row_stride` (in
 *     elements, >= classes) for logits, every peer and grad_logits.
 *   - rows == 0 is valid: reduced loss 0, counters 0.
 *   - NaN / Inf inputs propagate by IEEE rules and are outside the tested domain.
 */
#ifndef CODISTILL_H_
#define CODISTILL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* host-side return codes */
enum {
  CODISTILL_OK = 0,
  CODISTILL_ERR_NULL = 1,        /* a required pointer is NULL */
  CODISTILL_ERR_SHAPE = 2,       /* n < 1, rows < 0, classes < 1, row_stride < classes, sizes too large */
  CODISTILL_ERR_DTYPE = 3,       /* dtype is not CODISTILL_F32 / CODISTILL_BF16 */
  CODISTILL_ERR_PARAM = 4,       /* temperature <= 0, non-finite alpha, label_smoothing outside [0,1), bad enum */
  CODISTILL_ERR_UNSUPPORTED = 5, /* valid request this build cannot serve (e.g. n - 1 > CODISTILL_MAX_PEERS) */
  CODISTILL_ERR_CUDA = 6,        /* a CUDA runtime call failed; the CUDA error is left for cudaGetLastError */
  CODISTILL_ERR_WORKSPACE = 7,   /* workspace NULL, misaligned (256 B) or smaller than codistill_workspace_bytes */
  CODISTILL_ERR_TOO_LARGE = 8    /* codistill_loss_fwd_bwd_static only: rows > CODISTILL_STATIC_MAX_ROWS */
};

/* element type of logits, peers and grad_logits */
enum { CODISTILL_F32 = 0, CODISTILL_BF16 = 1 };

/* form of the distillation distance D */
enum {
  CODISTILL_DIST_MSE_LOGITS = 0, /* D(z, z') = 1/C * sum_c (z_c - z'_c)^2 (Appendix "Implementation Details") */
  CODISTILL_DIST_KL_SOFTMAX = 1, /* D(z, z') = T^2 * KL(softmax(z'/T) || softmax(z/T)) (Section 2, earlier work) */
  CODISTILL_DIST_MSE_CENTRED = 2, /* MSE between logits centred on their class means (Appendix "Implementation Details":
                                    centring gave similar results): D(z, z') = 1/C * sum_c ((z_c - mean z) - (z'_c - mean z'))^2 */
  CODISTILL_DIST_KL_REVERSE = 3, /* the other direction of Section 2's KL divergence (the paper does not fix it):
                                    D(z, z') = T^2 * KL(softmax(z/T) || softmax(z'/T)) */
  CODISTILL_DIST_KL_SYMMETRIC = 4 /* half the sum of the two directions */
};

/* how the n-1 peers enter D */
enum {
  CODISTILL_PEERS_PAIRWISE_MEAN = 0, /* 1/(n-1) * sum_j D(z, z^(j))      -- Algorithm 1 as printed          */
  CODISTILL_PEERS_MEAN_TARGET = 1    /* D(z, zbar), zbar = 1/(n-1) * sum_j z^(j) -- distance to the averaged peer */
};

/* reduction over rows; the gradient is the gradient of the reduced loss */
enum { CODISTILL_REDUCE_MEAN_VALID = 0, CODISTILL_REDUCE_SUM = 1 };

/* bits OR-ed into *dev_status by the kernels */
enum {
  CODISTILL_DEV_BAD_LABEL = 1, /* a valid row had a label outside [0, classes); that row was treated as masked */
  CODISTILL_DEV_TIMEOUT = 2    /* a bounded wait on an asynchronous copy expired; outputs are not to be trusted */
};

#define CODISTILL_MAX_PEERS 31 /* n <= 32 */

/* layout of counters[]: [0] n_valid, [1] n_masked, [2] n_correct, [3 + j] n_agree with peer j */
#define CODISTILL_COUNTERS_FIXED 3

/*
 * Full parameter block (Algorithm 1's objective with every knob this library exposes).
 *
 *   struct_bytes     sizeof(codistill_params_t) as seen by the caller (ABI check).
 *   logits           [rows, row_stride] own logits z of model i.
 *   peer_logits      HOST array of n-1 device pointers, each [rows, row_stride]; may be NULL when n == 1.
 *   labels           [rows] int32 class ids y.
 *   mask             [rows] uint8, non-zero = valid row; NULL = all rows valid.  The paper does not
 *                    mention padding; masked rows get zero loss and an all-zero gradient row.
 *   n                number of codistilled models (n == 1: plain training, no distillation term).
 *   alpha            penalty coefficient alpha^k of Algorithm 1.  alpha == 0 skips the term.
 *   temperature      T > 0; used by the KL form only (the paper's MSE form has no temperature).
 *   label_smoothing  eps in [0,1): target q = (1-eps)*onehot(y) + eps/C for the task loss.
 *   row_loss         [rows] float output, per-row loss (0 for masked rows); may be NULL.
 *   reduced_loss     [1] float output: sum over valid rows (SUM) or that / max(n_valid,1) (MEAN_VALID).
 *   grad_logits      [rows, row_stride] output in `dtype` (bf16: round-to-nearest-even); NULL = forward only.
 *                    Only the first `classes` elements of each row are written.
 *   counters         [3 + (n-1)] int64 output (bit-exact integers), may be NULL:
 *                    n_valid, n_masked, n_correct = #{valid r: argmax z = y},
 *                    n_agree[j] = #{valid r: argmax z = argmax z^(j)}; lowest index wins ties.
 *   dev_status       [1] int32 output, CODISTILL_DEV_* bits; may be NULL.
 *   workspace        scratch of at least codistill_workspace_bytes(...) bytes, 256-byte aligned.
 *                    Contents on entry are irrelevant; calls sharing a workspace must not overlap.
 */
typedef struct codistill_params {
  uint64_t struct_bytes;
  const void* logits;
  const void* const* peer_logits;
  const int32_t* labels;
  const uint8_t* mask;
  int32_t n;
  int32_t dtype;
  int64_t rows;
  int64_t classes;
  int64_t row_stride;
  float alpha;
  float temperature;
  float label_smoothing;
  int32_t dist_kind;
  int32_t peer_reduce;
  int32_t reduction;
  float* row_loss;
  float* reduced_loss;
  void* grad_logits;
  int64_t* counters;
  int32_t* dev_status;
  void* workspace;
  uint64_t workspace_bytes;
} codistill_params_t;

/*
 * The objective of Algorithm 1 in the form the paper's experiments use: cross-entropy task
 * loss, D = MSE on raw logits averaged over the n-1 peers (PAIRWISE_MEAN), no label
 * smoothing, mean over valid rows, dense rows (row_stride == classes).  `temperature` is
 * validated (> 0) and otherwise unused because the MSE form has none.
 * The call draws its scratch from the CUDA stream-ordered allocator (cudaMallocAsync /
 * cudaFreeAsync on `stream`); use codistill_loss_fwd_bwd_ex to supply the scratch yourself.
 * `stream` is a cudaStream_t (NULL = default stream).
 */
int codistill_loss_fwd_bwd(const void* logits, const void* const* peer_logits /* HOST array */,
                           const int32_t* labels, const uint8_t* mask, int n, int64_t rows,
                           int64_t classes, float alpha, float temperature, int dtype,
                           float* row_loss, float* reduced_loss, void* grad_logits, void* stream);

/*
 * Allocation-free form of codistill_loss_fwd_bwd.  (The paper has no counterpart for this entry
 * point; it exists for deployment reasons only.)
 *
 * Who needs it: programs that must not touch a CUDA allocator when they call the loss.  Typical
 * cases are a serving or training process whose framework claimed all device memory at start-up,
 * so that a later cudaMalloc / cudaMallocAsync fails or stalls, and latency-critical loops that ban
 * allocator calls because those may synchronise the device.  The basic entry point above takes its
 * scratch from the stream-ordered allocator and the _ex form expects the caller to have allocated
 * a workspace; this one needs neither.
 *
 * How: the scratch (row-validity counts, per-row flag words, the completion ticket) lives in a
 * fixed array inside the library's device image.  Every GPU that loads the library holds that
 * array (about 0.5 MiB) until the process exits.  The array is sized for at most
 * CODISTILL_STATIC_MAX_ROWS rows; a larger `rows` returns CODISTILL_ERR_TOO_LARGE and launches
 * nothing.  The call performs no cudaMalloc, cudaFree or other allocating routine.
 *
 * Arguments, defaults and outputs are exactly those of codistill_loss_fwd_bwd (row_loss may be NULL:
 * the per-row losses then stay inside the built-in scratch).
 *
 * Set-up: the first call on each device looks up the device address of the array (the device
 * must be current, as for every call).  Make that first call outside any stream capture, and while
 * the device still has room for this library's code and the array itself: the CUDA runtime may
 * load both only when the library is first used on a device, so a process that fills the device
 * memory before its first call into the library can see that call fail with CODISTILL_ERR_CUDA.
 * Host threads may make their first calls concurrently.
 *
 * Sharing: all calls on a device use the same array, which keeps whatever the previous call left
 * in it; each call clears the words that must start at zero before using them.  Two calls that
 * overlap on the GPU (different streams, no ordering between them) race on the array and give
 * wrong results: order them, or use codistill_loss_fwd_bwd_ex with separate workspaces.
 */
#define CODISTILL_STATIC_MAX_ROWS 65536
int codistill_loss_fwd_bwd_static(const void* logits, const void* const* peer_logits /* HOST array */,
                                  const int32_t* labels, const uint8_t* mask, int n, int64_t rows,
                                  int64_t classes, float alpha, float temperature, int dtype,
                                  float* row_loss, float* reduced_loss, void* grad_logits, void* stream);

/* Same operation with every option of codistill_params_t; allocates nothing. */
int codistill_loss_fwd_bwd_ex(const codistill_params_t* params, void* stream);

/*
 * Host-buffer variant used for end-to-end use from pageable or pinned HOST memory: every data
 * pointer in `params` (logits, each peer, labels, mask, row_loss, reduced_loss, grad_logits,
 * counters, dev_status) is a HOST pointer; params->workspace is a DEVICE buffer of at least
 * codistill_host_workspace_bytes(...) bytes.  Rows are processed in slices of `chunk_rows`
 * (0 = library default): host->device copy of a slice, the same kernels as above, device->host
 * copy of that slice's gradient and losses, software-pipelined over internal streams.  The
 * call is synchronous: on return every host output is valid.  No arithmetic of the objective
 * runs on the host.
 */
int codistill_loss_fwd_bwd_host(const codistill_params_t* params, int64_t chunk_rows, void* stream);

/* Scratch size for codistill_loss_fwd_bwd_ex (bytes; multiple of 256). */
size_t codistill_workspace_bytes(int n, int64_t rows, int64_t classes, int dtype);

/* Device scratch size for codistill_loss_fwd_bwd_host with the given slice height (0 = default).
 * Pass the row pitch as `classes` when row_stride > classes. */
size_t codistill_host_workspace_bytes(int n, int64_t rows, int64_t classes, int dtype, int64_t chunk_rows);

/*
 * All models in one call: Algorithm 1 updates every model i = 1..n on the same minibatch (its inner
 * loop over the models), and each update needs the objective with model i as "own" and the other n-1 as
 * peers.  Done with n calls above, every logit tensor is read n times and n gradients are written:
 * n (n + 1) tensor passes.  This entry point computes the n objectives together: the per-column sums
 * over the models are shared, so that 3 n passes suffice (each tensor read twice, each gradient
 * written once).  Distances: MSE on logits, plain or centred (dist_kind = CODISTILL_DIST_MSE_LOGITS or
 * CODISTILL_DIST_MSE_CENTRED), and the KL form (CODISTILL_DIST_KL_SOFTMAX, `temperature` > 0) reduced
 * pairwise over the peers (peer_reduce = CODISTILL_PEERS_PAIRWISE_MEAN; with n = 2 the mean target is
 * the same thing and is accepted; otherwise CODISTILL_ERR_UNSUPPORTED): the per-column sums
 * sum_j t_j and sum_j t_j log t_j of the tempered softmaxes serve all n models.
 *
 *   logits        HOST array of n device pointers, each [rows, row_stride] in `dtype`, 16-byte aligned.
 *   grad_logits   HOST array of n device pointers (same layout), or NULL = forward only.
 *   row_loss      [n, rows] float device output (model-major), may be NULL.
 *   reduced_loss  [n] float device output.
 *   counters      [n, 3 + (n-1)] int64 device output, may be NULL: row i as for a single call with
 *                 model i as own and the other models, in increasing index, as its peers.
 *   n             2 .. CODISTILL_ALL_MAX_MODELS.
 * Everything else as in codistill_params_t.  Results equal those of the n single calls within the
 * stated tolerances; integer outputs are identical.
 */
#define CODISTILL_ALL_MAX_MODELS 8
typedef struct codistill_all_params {
  uint64_t struct_bytes;
  const void* const* logits;
  const int32_t* labels;
  const uint8_t* mask;
  int32_t n;
  int32_t dtype;
  int64_t rows;
  int64_t classes;
  int64_t row_stride;
  float alpha;
  float label_smoothing;
  int32_t peer_reduce;
  int32_t reduction;
  int32_t dist_kind;
  float temperature;  /* T of the KL form; ignored by the MSE forms */
  float* row_loss;
  float* reduced_loss;
  void* const* grad_logits;
  int64_t* counters;
  int32_t* dev_status;
  void* workspace;
  uint64_t workspace_bytes;
} codistill_all_params_t;
int codistill_loss_fwd_bwd_all(const codistill_all_params_t* params, void* stream);

/* Scratch size for codistill_loss_fwd_bwd_all (bytes; multiple of 256). */
size_t codistill_all_workspace_bytes(int n, int64_t rows);

/* Human-readable name of a CODISTILL_ERR_* code (static storage). */
const char* codistill_status_string(int status);

/*
 * Compression of the predictions exchanged between the model groups (Section 3: every device sends the
 * predictions of its minibatch, b_pred bits per sample, to the devices that train the other models).
 * Packing 32-bit logits to bfloat16 (round to nearest, ties to even; NaN stays NaN) halves b_pred; the
 * receiver either runs the loss on the bfloat16 tensors or widens them again (exact) with the second call.
 *   src / dst      DEVICE pointers, row-major [rows, stride] with stride >= classes (elements); only the first
 *                  `classes` elements of a row are read and written.  16-byte aligned bases with pitches that
 *                  are multiples of 8 (bf16) / 4 (fp32) elements take the 16-byte path, anything else works too.
 * Asynchronous on `stream`; CODISTILL_ERR_SHAPE / CODISTILL_ERR_NULL on bad arguments, nothing launched.
 */
int codistill_pack_predictions(const float* src, void* dst_bf16, int64_t rows, int64_t classes, int64_t src_stride,
                               int64_t dst_stride, void* stream);
int codistill_unpack_predictions(const void* src_bf16, float* dst, int64_t rows, int64_t classes, int64_t src_stride,
                                 int64_t dst_stride, void* stream);

/*
 * Diagnostic, not part of the objective.  Every wait of the kernels on an asynchronous copy is bounded:
 * when its time limit runs out the kernel raises CODISTILL_DEV_TIMEOUT in the status word, stops waiting
 * and leaves normally; the context stays usable.  This call shows that path without a copy that never
 * lands: it launches one small CTA that waits `limit_ns` nanoseconds (1 .. 100 000 000) on a barrier
 * that nothing completes, then writes the status bits to *dev_status (DEVICE pointer; expected value
 * CODISTILL_DEV_TIMEOUT).  Asynchronous on `stream` like every call.
 */
int codistill_selftest_bounded_wait(int32_t* dev_status, uint64_t limit_ns, void* stream);

/*
 * Text of the CUDA runtime error behind the most recent CODISTILL_ERR_CUDA on this host thread
 * ("no error" when there was none).  The library carries its own copy of the CUDA runtime, so the
 * error is not visible through the caller's cudaGetLastError.  Reading it clears it.  Static storage.
 */
const char* codistill_last_cuda_error(void);

/* Library version: major * 10000 + minor * 100 + patch. */
int codistill_version(void);

/*
 * Name of the kernel regime the dispatcher picks for a problem, so that tests and benchmarks can
 * state which kernel they exercised: "short" (up to 1024 classes, up to 7 peers, MSE distance, at most 16384
 * rows: one launch, one warp per row, the row held in registers), "warp" (rows up to 8 KiB, one warp per row), "tma" (long rows,
 * MSE distance, own row staged in shared memory by bulk copies), "stream" (long rows, direct loads,
 * own row read twice: MSE rows beyond 64 KiB, the softmax-KL and centred-MSE distances), "cluster"
 * (long rows, all n row images of a row index kept in the shared memory of a thread-block cluster: by
 * default only the peer counts the two kernels before are not built for, 4 to 6) or "block"
 * (everything else).  The answer assumes
 * 16-byte aligned tensor bases (the long-row kernels need them).  For measurements the environment
 * variable CODISTILL_REGIME = warp | tma | stream | cluster | block overrides the choice where the named
 * kernel can serve the call, and CODISTILL_CLUSTER_SIZE = 1 | 2 | 4 | 8 | 16 fixes the number of
 * CTAs per cluster of the "cluster" kernel.  Static storage; NULL on bad arguments.
 */
const char* codistill_kernel_regime(int n, int64_t rows, int64_t classes, int64_t row_stride, int dtype,
                                    int dist_kind, int peer_reduce);

#ifdef __cplusplus
}
#endif
#endif /* CODISTILL_H_ */
