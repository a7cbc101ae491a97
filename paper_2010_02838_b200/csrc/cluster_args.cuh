// Argument block and host entry points of the cluster-resident row kernel (rows_cluster.cu), shared
// with the dispatchers of the single-model and all-models calls.
#pragma once
#include "common.cuh"

namespace codistill {

constexpr int kClMax = CODISTILL_ALL_MAX_MODELS;   // tensors resident at most

enum ClMode { kClMse = 0, kClKlPairwise = 1, kClKlMeanTarget = 2 };

struct ClArgs {
  const void* model[kClMax];    // model[0]: own logits of a single-model call
  void* grad[kClMax];           // all-models call: n outputs or all null; single-model call: grad[0] or null
  const int32_t* labels;
  const uint8_t* mask;          // nullable
  float* row_loss;              // [n_out][rows_total]
  uint32_t* row_flags;          // [n_out][rows_total]
  WsHeader* hdr;
  const int64_t* partials;
  int64_t rows_total;           // rows of the whole call (labels / mask / row_loss length)
  int64_t row_begin, row_end;   // rows of this launch; the tensor pointers are those of row_begin
  int64_t classes, row_stride;
  int n;                        // resident tensors
  int pairwise;                 // MSE: loss from the pairwise distances (else distance to the averaged peers)
  int reduction;
  int centred;                  // MSE between logits centred on their class means
  float alpha, eps, temperature;
  int spc;                      // segments of a row image per CTA
  uint32_t slice_bytes;         // shared-memory bytes of one tensor's range (16 * spc rounded up to 128)
};

// Launches the kernel for rows [row_begin, row_end) of `a` (spc and slice_bytes are filled in here).
// `mode`: ClMode; `all`: every model's outputs, else model 0's.  cudaErrorNotSupported when the row
// images do not fit the shared memory of the largest cluster.
cudaError_t launch_cluster(ClArgs a, int dtype, int mode, bool all, int smem_optin, cudaStream_t stream);

// Whether n row images of this shape fit (16-byte aligned tensor bases are checked by the callers).
bool cluster_fits(int n, int64_t classes, int64_t row_stride, int dtype, int smem_optin);

}  // namespace codistill
