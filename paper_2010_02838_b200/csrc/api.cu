// Host side of the C ABI declared in include/codistill.h: argument validation, workspace
// layout, regime dispatch, the prep / finalize kernels and the host-buffer pipeline.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>

#include "bulk_copy.cuh"
#include "common.cuh"

static_assert(sizeof(codistill_params_t) == 152, "ABI: size of codistill_params_t");

namespace codistill {

cudaError_t launch_generic(const KArgs& a, int dtype, bool warp_regime, bool vec, int num_sms, cudaStream_t stream);
bool tma_supported(const KArgs& a, int dtype, int smem_optin);
int tma_ctas_per_sm(const KArgs& a, int dtype, int smem_optin);
cudaError_t launch_tma(const KArgs& a, int dtype, int num_sms, int smem_optin, cudaStream_t stream);
bool stream_supported(const KArgs& a, int dtype);
cudaError_t launch_stream(const KArgs& a, int dtype, int num_sms, cudaStream_t stream);
bool short_supported(const KArgs& a, int dtype);
cudaError_t launch_short(const KArgs& a, int dtype, bool vec, int num_sms, cudaStream_t stream);
bool cluster_supported(const KArgs& a, int dtype, int smem_optin);
cudaError_t launch_cluster_single(const KArgs& a, int dtype, int smem_optin, cudaStream_t stream);

static thread_local cudaError_t g_last_cuda_error = cudaSuccess;
static thread_local const char* g_last_cuda_call = "";
static thread_local char g_last_cuda_text[256];
cudaError_t cuda_note(cudaError_t e, const char* what) {
  if (e != cudaSuccess) g_last_cuda_call = what;
  return e;
}
int cuda_status(cudaError_t e) {
  if (e == cudaSuccess) return CODISTILL_OK;
  g_last_cuda_error = e;
  cudaGetLastError();   // a launch failure also sits in the runtime's own slot: clear it
  return CODISTILL_ERR_CUDA;
}

// ------------------------------------------------------------------ prep and finalize kernels
// Zeroes the workspace header and counts valid / masked rows (one partial pair per block, summed
// later in block order).  A valid row with a label that is not a class id counts as masked and
// raises CODISTILL_DEV_BAD_LABEL.
__global__ void __launch_bounds__(1024) prep_kernel(WsHeader* hdr, int64_t* partials, const int32_t* labels,
                                                     const uint8_t* mask, int64_t rows, int64_t classes) {
  __shared__ long long sh[2][32];
  __shared__ int sh_bad;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  release_dependent_grid();  // the main kernel may start its set-up now; it waits for this grid before reading the workspace
  if (tid == 0) sh_bad = 0;
  __syncthreads();
  long long valid = 0, masked = 0;
  int bad = 0;
  for (int64_t r = (int64_t)blockIdx.x * blockDim.x + tid; r < rows; r += (int64_t)gridDim.x * blockDim.x) {
    const bool on = (mask == nullptr) || mask[r] != 0;
    const int32_t y = labels[r];
    const bool ok = y >= 0 && (int64_t)y < classes;
    if (on && ok) ++valid; else ++masked;
    bad |= (on && !ok);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    valid += __shfl_down_sync(0xffffffffu, valid, o);
    masked += __shfl_down_sync(0xffffffffu, masked, o);
  }
  if (bad) sh_bad = 1;
  if (lane == 0) { sh[0][warp] = valid; sh[1][warp] = masked; }
  __syncthreads();
  if (tid == 0) {
    long long v = 0, m = 0;
    for (int k = 0; k < (int)(blockDim.x >> 5); ++k) { v += sh[0][k]; m += sh[1][k]; }
    partials[2 * blockIdx.x] = v;
    partials[2 * blockIdx.x + 1] = m;
  }
  // Header: block 0 clears the words the main kernels accumulate into.  The bad-label flag of each
  // block goes to a word of its own, so that no block races with the clearing.
  if (tid == 0) hdr->pad[blockIdx.x] = sh_bad ? 1u : 0u;
  if (blockIdx.x == 0 && tid == 0) {
    hdr->ticket = 0u;
    hdr->next_row = 0u;
    hdr->sched_done = 0u;
    hdr->status = 0;
    hdr->prep_blocks = (int)gridDim.x;
  }
}
static_assert(kPrepMaxBlocks <= 59, "per-block bad-label words live in the header padding");

// One CTA running the final reduction, for calls whose main kernels do not do it themselves.
__global__ void __launch_bounds__(1024) finalize_kernel(const __grid_constant__ KArgs a) {
  __shared__ double sh[32];
  finalize_cta(a, sh);
}

// Diagnostic: one CTA waits, with the library's bounded wait, on an mbarrier that nothing ever completes
// (no copy is in flight, so the CTA may leave at once afterwards).  Shows that an expired wait ends in a
// status bit and a normal kernel exit.
__global__ void __launch_bounds__(64) bounded_wait_probe_kernel(int32_t* dev_status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    mbar_init_fence();
    abort_flag = 0;
    *dev_status = 0;
  }
  __syncthreads();
  // warp 0 polls back to back like a consumer, warp 1 with back-off like a producer
  mbar_wait_limited(&bar, 0u, &abort_flag, dev_status, CODISTILL_DEV_TIMEOUT, limit_ns, true, threadIdx.x >= 32);
}

// ------------------------------------------------------------------ host helpers
struct DeviceInfo { int device = -1; int num_sms = 0; int smem_optin = 0; };

static cudaError_t device_info(DeviceInfo* out) {
  static thread_local DeviceInfo cache[64];
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64 && cache[dev].device == dev) { *out = cache[dev]; return cudaSuccess; }
  DeviceInfo d;
  d.device = dev;
  if ((e = cudaDeviceGetAttribute(&d.num_sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess) return e;
  if (dev >= 0 && dev < 64) cache[dev] = d;
  *out = d;
  return cudaSuccess;
}

static int validate(const codistill_params_t* p, bool host_pointers) {
  if (p == nullptr) return CODISTILL_ERR_NULL;
  if (p->struct_bytes != sizeof(codistill_params_t)) return CODISTILL_ERR_PARAM;
  if (p->n < 1 || p->rows < 0 || p->classes < 1 || p->row_stride < p->classes) return CODISTILL_ERR_SHAPE;
  if (p->classes > (int64_t)1 << 30 || p->rows > (int64_t)1 << 40) return CODISTILL_ERR_SHAPE;
  if (p->dtype != CODISTILL_F32 && p->dtype != CODISTILL_BF16) return CODISTILL_ERR_DTYPE;
  if (!(p->temperature > 0.f) || !isfinite(p->temperature) || !isfinite(p->alpha)) return CODISTILL_ERR_PARAM;
  if (!(p->label_smoothing >= 0.f && p->label_smoothing < 1.f)) return CODISTILL_ERR_PARAM;
  if (p->dist_kind < CODISTILL_DIST_MSE_LOGITS || p->dist_kind > CODISTILL_DIST_KL_SYMMETRIC) return CODISTILL_ERR_PARAM;
  if (p->peer_reduce != CODISTILL_PEERS_PAIRWISE_MEAN && p->peer_reduce != CODISTILL_PEERS_MEAN_TARGET) return CODISTILL_ERR_PARAM;
  if (p->reduction != CODISTILL_REDUCE_MEAN_VALID && p->reduction != CODISTILL_REDUCE_SUM) return CODISTILL_ERR_PARAM;
  if (p->n - 1 > kMaxPeers) return CODISTILL_ERR_UNSUPPORTED;
  if (p->reduced_loss == nullptr) return CODISTILL_ERR_NULL;
  if (p->rows > 0) {
    if (p->logits == nullptr || p->labels == nullptr) return CODISTILL_ERR_NULL;
    if (p->n > 1) {
      if (p->peer_logits == nullptr) return CODISTILL_ERR_NULL;
      for (int j = 0; j < p->n - 1; ++j)
        if (p->peer_logits[j] == nullptr) return CODISTILL_ERR_NULL;
    }
  }
  if (p->workspace == nullptr || (reinterpret_cast<uintptr_t>(p->workspace) & 255u) != 0) return CODISTILL_ERR_WORKSPACE;
  (void)host_pointers;
  return CODISTILL_OK;
}

enum Regime { kRegimeWarp = 0, kRegimeBlock = 1, kRegimeTma = 2, kRegimeStream = 3, kRegimeCluster = 4 };

// Long rows with the MSE distance have two kernels: "tma" (own row staged in shared memory by bulk
// copies) and "stream" (direct loads, own row re-read through L2).  The staged kernel is the faster
// one while two of its CTAs fit an SM (rows up to 64 KiB); beyond that, and for rows it cannot hold
// at all, the direct-load kernel is.  The environment variable CODISTILL_REGIME = stream | tma |
// block overrides the default choice where the named kernel supports the call (for measurements;
// results are the same within rounding).
static Regime pick_regime(const KArgs& a, int dtype, int smem_optin) {
  const int64_t row_bytes = a.classes * (dtype == CODISTILL_F32 ? 4 : 2);
  const Regime generic = row_bytes <= 8192 ? kRegimeWarp : kRegimeBlock;
  const bool can_tma = tma_supported(a, dtype, smem_optin), can_stream = stream_supported(a, dtype);
  const bool can_cluster = cluster_supported(a, dtype, smem_optin);
  if (const char* want = getenv("CODISTILL_REGIME")) {
    if (strcmp(want, "tma") == 0 && can_tma) return kRegimeTma;
    if (strcmp(want, "stream") == 0 && can_stream) return kRegimeStream;
    if (strcmp(want, "cluster") == 0 && can_cluster) return kRegimeCluster;
    if (strcmp(want, "block") == 0) return generic;
  }
  if (can_tma && (!can_stream || tma_ctas_per_sm(a, dtype, smem_optin) >= 2)) return kRegimeTma;
  if (can_stream) return kRegimeStream;
  if (can_cluster) return kRegimeCluster;   // peer counts the two MSE kernels above are not built for (4, 5, 6)
  return generic;
}

// CODISTILL_REGIME=warp (or block) keeps short rows on the two-launch generic kernels, for measurements
static bool regime_forced_away_from_short() {
  const char* want = getenv("CODISTILL_REGIME");
  return want != nullptr && (strcmp(want, "warp") == 0 || strcmp(want, "block") == 0);
}

static bool rows_vectorizable(const KArgs& a, int dtype) {
  const size_t es = dtype == CODISTILL_F32 ? 4 : 2;
  if ((a.row_stride * es) % 16 != 0) return false;
  uintptr_t bits = reinterpret_cast<uintptr_t>(a.own) | reinterpret_cast<uintptr_t>(a.grad);
  for (int j = 0; j < a.n_peers; ++j) bits |= reinterpret_cast<uintptr_t>(a.peers[j]);
  return (bits & 15u) == 0;
}

// Fills the kernel argument block for rows [row_begin, row_end) whose logits start at the given pointers.
static void fill_args(KArgs* a, const codistill_params_t* p, void* workspace) {
  memset(a, 0, sizeof(*a));
  const WsLayout l = ws_layout(p->rows);
  char* ws = static_cast<char*>(workspace);
  a->own = p->logits;
  for (int j = 0; j < p->n - 1; ++j) a->peers[j] = p->peer_logits[j];
  a->grad = p->grad_logits;
  a->labels = p->labels;
  a->mask = p->mask;
  a->row_loss = p->row_loss ? p->row_loss : reinterpret_cast<float*>(ws + l.row_loss);
  a->row_flags = reinterpret_cast<uint32_t*>(ws + l.row_flags);
  a->hdr = reinterpret_cast<WsHeader*>(ws);
  a->partials = reinterpret_cast<const int64_t*>(ws + l.partials);
  a->reduced_loss = p->reduced_loss;
  a->counters = p->counters;
  a->dev_status = p->dev_status;
  a->rows_total = p->rows;
  a->row_begin = 0;
  a->row_end = p->rows;
  a->classes = p->classes;
  a->row_stride = p->row_stride;
  a->n_peers = p->n - 1;
  a->dist = p->dist_kind;
  a->peer_reduce = p->peer_reduce;
  a->reduction = p->reduction;
  a->want_flags = p->counters != nullptr;
  a->fused_finalize = 1;
  a->alpha = p->alpha;
  a->temperature = p->temperature;
  a->eps = p->label_smoothing;
}

static int prep_grid(int64_t rows) {
  int64_t g = (rows + 8191) / 8192;
  if (g < 1) g = 1;
  return (int)(g > kPrepMaxBlocks ? kPrepMaxBlocks : g);
}

static cudaError_t launch_prep(const KArgs& a, cudaStream_t stream) {
  prep_kernel<<<prep_grid(a.rows_total), 1024, 0, stream>>>(a.hdr, const_cast<int64_t*>(a.partials), a.labels, a.mask,
                                                           a.rows_total, a.classes);
  return cudaGetLastError();
}

// the prep kernel for callers outside this file (the all-models entry point)
cudaError_t launch_prep_rows(WsHeader* hdr, int64_t* partials, const int32_t* labels, const uint8_t* mask, int64_t rows,
                             int64_t classes, cudaStream_t stream) {
  prep_kernel<<<prep_grid(rows), 1024, 0, stream>>>(hdr, partials, labels, mask, rows, classes);
  return cudaGetLastError();
}

static cudaError_t launch_main(const KArgs& a, int dtype, const DeviceInfo& di, cudaStream_t stream) {
  const Regime reg = pick_regime(a, dtype, di.smem_optin);
  if (reg == kRegimeTma) return launch_tma(a, dtype, di.num_sms, di.smem_optin, stream);
  if (reg == kRegimeStream) return launch_stream(a, dtype, di.num_sms, stream);
  if (reg == kRegimeCluster) {
    const cudaError_t e = launch_cluster_single(a, dtype, di.smem_optin, stream);
    if (e != cudaSuccess || !a.fused_finalize) return e;
    finalize_kernel<<<1, 1024, 0, stream>>>(a);   // this kernel leaves the final reduction to a launch of its own
    return cudaGetLastError();
  }
  return launch_generic(a, dtype, reg == kRegimeWarp, rows_vectorizable(a, dtype), di.num_sms, stream);
}

static int run_device(const codistill_params_t* p, cudaStream_t stream) {
  if (p->workspace_bytes < ws_layout(p->rows).total) return CODISTILL_ERR_WORKSPACE;
  DeviceInfo di;
  if (const int rc_cuda = cuda_status(device_info(&di))) return rc_cuda;
  KArgs a;
  fill_args(&a, p, p->workspace);
  // short rows: one cooperative launch does the counting, the rows and the final reduction
  if (short_supported(a, p->dtype) && !regime_forced_away_from_short())
    return cuda_status(launch_short(a, p->dtype, rows_vectorizable(a, p->dtype), di.num_sms, stream));
  if (const int rc_cuda = cuda_status(launch_prep(a, stream))) return rc_cuda;
  if (p->rows == 0) {
    a.fused_finalize = 0;
    finalize_kernel<<<1, 1024, 0, stream>>>(a);
    return cuda_status(cudaGetLastError());
  }
  if (const int rc_cuda = cuda_status(launch_main(a, p->dtype, di, stream))) return rc_cuda;
  return CODISTILL_OK;
}

// ------------------------------------------------------------------ host-buffer pipeline
// Device workspace of the host-buffer entry point: the ordinary workspace, device copies of the
// per-row vectors and scalars, and two slots of (n inputs + 1 gradient) slices.
struct HostLayout {
  size_t ws, labels, mask, row_loss, scalars, slots, slot_bytes, tensor_bytes, total;
  int64_t chunk_rows;
};
constexpr size_t kHostScalarBytes = 1024;  // reduced loss, status, counters

static int64_t default_chunk_rows(int64_t rows, int64_t row_stride, size_t es) {
  const size_t target = size_t(32) << 20;  // about 32 MiB per tensor slice
  int64_t c = (int64_t)(target / ((size_t)row_stride * es));
  if (c < 1) c = 1;
  return c > rows ? (rows > 0 ? rows : 1) : c;
}

static HostLayout host_layout(int n, int64_t rows, int64_t row_stride, int dtype, int64_t chunk_rows) {
  const size_t es = dtype == CODISTILL_F32 ? 4 : 2;
  HostLayout h;
  h.chunk_rows = chunk_rows > 0 ? (chunk_rows > rows && rows > 0 ? rows : chunk_rows) : default_chunk_rows(rows, row_stride, es);
  const size_t R = (size_t)(rows > 0 ? rows : 1);
  h.ws = 0;
  h.labels = round256(ws_layout(rows).total);
  h.mask = h.labels + round256(4 * R);
  h.row_loss = h.mask + round256(R);
  h.scalars = h.row_loss + round256(4 * R);
  h.slots = h.scalars + kHostScalarBytes;
  h.tensor_bytes = round256((size_t)h.chunk_rows * (size_t)row_stride * es);
  h.slot_bytes = h.tensor_bytes * (size_t)(n + 1);
  h.total = h.slots + 2 * h.slot_bytes;
  return h;
}

#define CODISTILL_CK(expr) do { if ((rc = cuda_status(expr)) != CODISTILL_OK) goto done; } while (0)

static int run_host(const codistill_params_t* p, int64_t chunk_rows_req, cudaStream_t stream) {
  const size_t es = p->dtype == CODISTILL_F32 ? 4 : 2;
  const HostLayout h = host_layout(p->n, p->rows, p->row_stride, p->dtype, chunk_rows_req);
  if (p->workspace_bytes < h.total) return CODISTILL_ERR_WORKSPACE;
  DeviceInfo di;
  if (const int rc_cuda = cuda_status(device_info(&di))) return rc_cuda;
  char* base = static_cast<char*>(p->workspace);
  const int64_t R = p->rows;
  const int P = p->n - 1;
  int rc = CODISTILL_OK;
  cudaStream_t s_in = nullptr, s_out = nullptr;
  cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_k[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
  cudaEvent_t ev_start = nullptr;

  // device-side view of the call: per-row vectors and scalars live in the workspace
  codistill_params_t d = *p;
  d.labels = reinterpret_cast<const int32_t*>(base + h.labels);
  d.mask = p->mask ? reinterpret_cast<const uint8_t*>(base + h.mask) : nullptr;
  d.row_loss = reinterpret_cast<float*>(base + h.row_loss);
  d.reduced_loss = reinterpret_cast<float*>(base + h.scalars);
  d.dev_status = reinterpret_cast<int32_t*>(base + h.scalars + 16);
  d.counters = p->counters ? reinterpret_cast<int64_t*>(base + h.scalars + 64) : nullptr;
  KArgs a;
  fill_args(&a, &d, base + h.ws);
  a.fused_finalize = 0;

  CODISTILL_CK(cudaStreamCreateWithFlags(&s_in, cudaStreamNonBlocking));
  CODISTILL_CK(cudaStreamCreateWithFlags(&s_out, cudaStreamNonBlocking));
  for (int i = 0; i < 2; ++i) {
    CODISTILL_CK(cudaEventCreateWithFlags(&ev_in[i], cudaEventDisableTiming));
    CODISTILL_CK(cudaEventCreateWithFlags(&ev_k[i], cudaEventDisableTiming));
    CODISTILL_CK(cudaEventCreateWithFlags(&ev_out[i], cudaEventDisableTiming));
  }
  CODISTILL_CK(cudaEventCreateWithFlags(&ev_start, cudaEventDisableTiming));
  CODISTILL_CK(cudaEventRecord(ev_start, stream));       // copies must not run ahead of the caller's stream
  CODISTILL_CK(cudaStreamWaitEvent(s_in, ev_start, 0));
  CODISTILL_CK(cudaStreamWaitEvent(s_out, ev_start, 0));

  if (R > 0) {
    CODISTILL_CK(cudaMemcpyAsync(base + h.labels, p->labels, 4 * (size_t)R, cudaMemcpyHostToDevice, stream));
    if (p->mask) CODISTILL_CK(cudaMemcpyAsync(base + h.mask, p->mask, (size_t)R, cudaMemcpyHostToDevice, stream));
  }
  CODISTILL_CK(launch_prep(a, stream));

  for (int64_t r0 = 0, k = 0; r0 < R; r0 += h.chunk_rows, ++k) {
    const int slot = (int)(k & 1);
    const int64_t r1 = r0 + h.chunk_rows < R ? r0 + h.chunk_rows : R;
    // the last row of the call may be shorter than the pitch in the caller's buffers
    const size_t elems = (size_t)(r1 - r0 - 1) * (size_t)p->row_stride + (size_t)(r1 == R ? p->classes : p->row_stride);
    const size_t bytes = elems * es, off = (size_t)r0 * (size_t)p->row_stride * es;
    char* sb = base + h.slots + (size_t)slot * h.slot_bytes;
    if (k >= 2) CODISTILL_CK(cudaStreamWaitEvent(s_in, ev_k[slot], 0));  // slot inputs free once chunk k-2 has run
    CODISTILL_CK(cudaMemcpyAsync(sb, static_cast<const char*>(p->logits) + off, bytes, cudaMemcpyHostToDevice, s_in));
    for (int j = 0; j < P; ++j)
      CODISTILL_CK(cudaMemcpyAsync(sb + (size_t)(j + 1) * h.tensor_bytes, static_cast<const char*>(p->peer_logits[j]) + off,
                                   bytes, cudaMemcpyHostToDevice, s_in));
    CODISTILL_CK(cudaEventRecord(ev_in[slot], s_in));
    CODISTILL_CK(cudaStreamWaitEvent(stream, ev_in[slot], 0));
    if (k >= 2) CODISTILL_CK(cudaStreamWaitEvent(stream, ev_out[slot], 0));  // gradient slice of chunk k-2 copied out
    a.own = sb;
    for (int j = 0; j < P; ++j) a.peers[j] = sb + (size_t)(j + 1) * h.tensor_bytes;
    a.grad = p->grad_logits ? sb + (size_t)(P + 1) * h.tensor_bytes : nullptr;
    a.row_begin = r0;
    a.row_end = r1;
    CODISTILL_CK(launch_main(a, p->dtype, di, stream));
    CODISTILL_CK(cudaEventRecord(ev_k[slot], stream));
    if (p->grad_logits) {
      CODISTILL_CK(cudaStreamWaitEvent(s_out, ev_k[slot], 0));
      CODISTILL_CK(cudaMemcpyAsync(static_cast<char*>(p->grad_logits) + off, sb + (size_t)(P + 1) * h.tensor_bytes, bytes,
                                   cudaMemcpyDeviceToHost, s_out));
    }
    CODISTILL_CK(cudaEventRecord(ev_out[slot], s_out));
  }
  finalize_kernel<<<1, 1024, 0, stream>>>(a);
  CODISTILL_CK(cudaGetLastError());
  CODISTILL_CK(cudaMemcpyAsync(p->reduced_loss, d.reduced_loss, sizeof(float), cudaMemcpyDeviceToHost, stream));
  if (p->dev_status) CODISTILL_CK(cudaMemcpyAsync(p->dev_status, d.dev_status, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
  if (p->counters) CODISTILL_CK(cudaMemcpyAsync(p->counters, d.counters, sizeof(int64_t) * (size_t)(2 + p->n), cudaMemcpyDeviceToHost, stream));
  if (p->row_loss && R > 0) CODISTILL_CK(cudaMemcpyAsync(p->row_loss, d.row_loss, 4 * (size_t)R, cudaMemcpyDeviceToHost, stream));
  CODISTILL_CK(cudaStreamSynchronize(s_out));
  CODISTILL_CK(cudaStreamSynchronize(stream));
done:
  if (rc != CODISTILL_OK) { cudaStreamSynchronize(stream); if (s_in) cudaStreamSynchronize(s_in); if (s_out) cudaStreamSynchronize(s_out); }
  for (int i = 0; i < 2; ++i) {
    if (ev_in[i]) cudaEventDestroy(ev_in[i]);
    if (ev_k[i]) cudaEventDestroy(ev_k[i]);
    if (ev_out[i]) cudaEventDestroy(ev_out[i]);
  }
  if (ev_start) cudaEventDestroy(ev_start);
  if (s_in) cudaStreamDestroy(s_in);
  if (s_out) cudaStreamDestroy(s_out);
  return rc;
}
#undef CODISTILL_CK

}  // namespace codistill

using namespace codistill;

extern "C" {

int codistill_version(void) { return 200; }

int codistill_selftest_bounded_wait(int32_t* dev_status, uint64_t limit_ns, void* stream) {
  if (dev_status == nullptr) return CODISTILL_ERR_NULL;
  if (limit_ns == 0 || limit_ns > 100000000ull) return CODISTILL_ERR_PARAM;   // at most 100 ms
  bounded_wait_probe_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(dev_status, limit_ns);
  return cuda_status(cudaGetLastError());
}

const char* codistill_last_cuda_error(void) {
  const cudaError_t e = g_last_cuda_error;
  snprintf(g_last_cuda_text, sizeof(g_last_cuda_text), "%s%s%s", cudaGetErrorString(e), g_last_cuda_call[0] ? " in " : "", g_last_cuda_call);
  g_last_cuda_error = cudaSuccess;
  g_last_cuda_call = "";
  return g_last_cuda_text;
}

const char* codistill_status_string(int status) {
  switch (status) {
    case CODISTILL_OK: return "ok";
    case CODISTILL_ERR_NULL: return "a required pointer is NULL";
    case CODISTILL_ERR_SHAPE: return "invalid shape (n, rows, classes or row_stride)";
    case CODISTILL_ERR_DTYPE: return "unknown dtype";
    case CODISTILL_ERR_PARAM: return "invalid parameter (temperature, alpha, label_smoothing, enum or struct size)";
    case CODISTILL_ERR_UNSUPPORTED: return "request not supported by this build";
    case CODISTILL_ERR_CUDA: return "a CUDA runtime call failed";
    case CODISTILL_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case CODISTILL_ERR_TOO_LARGE: return "rows exceed CODISTILL_STATIC_MAX_ROWS, the capacity of the built-in scratch";
    default: return "unknown status";
  }
}

size_t codistill_workspace_bytes(int n, int64_t rows, int64_t classes, int dtype) {
  (void)n; (void)classes; (void)dtype;
  return ws_layout(rows < 0 ? 0 : rows).total;
}

int codistill_loss_fwd_bwd_ex(const codistill_params_t* params, void* stream) {
  const int v = validate(params, false);
  if (v != CODISTILL_OK) return v;
  return run_device(params, static_cast<cudaStream_t>(stream));
}

int codistill_loss_fwd_bwd(const void* logits, const void* const* peer_logits, const int32_t* labels,
                           const uint8_t* mask, int n, int64_t rows, int64_t classes, float alpha,
                           float temperature, int dtype, float* row_loss, float* reduced_loss, void* grad_logits,
                           void* stream) {
  codistill_params_t p;
  memset(&p, 0, sizeof(p));
  p.struct_bytes = sizeof(p);
  p.logits = logits;
  p.peer_logits = peer_logits;
  p.labels = labels;
  p.mask = mask;
  p.n = n;
  p.dtype = dtype;
  p.rows = rows;
  p.classes = classes;
  p.row_stride = classes;
  p.alpha = alpha;
  p.temperature = temperature;
  p.label_smoothing = 0.f;
  p.dist_kind = CODISTILL_DIST_MSE_LOGITS;
  p.peer_reduce = CODISTILL_PEERS_PAIRWISE_MEAN;
  p.reduction = CODISTILL_REDUCE_MEAN_VALID;
  p.row_loss = row_loss;
  p.reduced_loss = reduced_loss;
  p.grad_logits = grad_logits;
  p.workspace = reinterpret_cast<void*>(uintptr_t(256));  // placeholder so that validation sees a non-null, aligned value
  p.workspace_bytes = 0;
  const int v = validate(&p, false);
  if (v != CODISTILL_OK) return v;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t bytes = ws_layout(rows).total;
  void* ws = nullptr;
  if (const int rc_cuda = cuda_status(cudaMallocAsync(&ws, bytes, s))) return rc_cuda;
  p.workspace = ws;
  p.workspace_bytes = bytes;
  const int rc = run_device(&p, s);
  if (const int rc_cuda = cuda_status(cudaFreeAsync(ws, s))) return rc_cuda;
  return rc;
}

size_t codistill_host_workspace_bytes(int n, int64_t rows, int64_t classes, int dtype, int64_t chunk_rows) {
  if (n < 1 || rows < 0 || classes < 1) return 0;
  return host_layout(n, rows, classes, dtype, chunk_rows).total;
}

int codistill_loss_fwd_bwd_host(const codistill_params_t* params, int64_t chunk_rows, void* stream) {
  const int v = validate(params, true);
  if (v != CODISTILL_OK) return v;
  if (chunk_rows < 0) return CODISTILL_ERR_SHAPE;
  return run_host(params, chunk_rows, static_cast<cudaStream_t>(stream));
}

const char* codistill_kernel_regime(int n, int64_t rows, int64_t classes, int64_t row_stride, int dtype,
                                    int dist_kind, int peer_reduce) {
  if (n < 1 || rows < 0 || classes < 1 || row_stride < classes) return nullptr;
  if (dtype != CODISTILL_F32 && dtype != CODISTILL_BF16) return nullptr;
  DeviceInfo di;
  if (device_info(&di) != cudaSuccess) { di.smem_optin = 232448; di.num_sms = 148; }
  KArgs a;
  memset(&a, 0, sizeof(a));
  a.classes = classes;
  a.row_stride = row_stride;
  a.n_peers = n - 1;
  a.dist = dist_kind;
  a.peer_reduce = peer_reduce;
  a.row_end = rows;
  a.rows_total = rows;
  a.fused_finalize = 1;
  if (short_supported(a, dtype) && !regime_forced_away_from_short()) return "short";
  switch (pick_regime(a, dtype, di.smem_optin)) {
    case kRegimeWarp: return "warp";
    case kRegimeBlock: return "block";
    case kRegimeStream: return "stream";
    case kRegimeCluster: return "cluster";
    default: return "tma";
  }
}

}  // extern "C"

// ------------------------------------------------------------------ allocation-free entry point
// Scratch of codistill_loss_fwd_bwd_static: one workspace for up to CODISTILL_STATIC_MAX_ROWS rows,
// part of the device image of this library (each GPU that loads it keeps the array until exit).
// In host code `g_static_scratch` is only a handle for cudaGetSymbolAddress, never a device address.
namespace codistill {
constexpr size_t kStaticScratchBytes = 256 + 1024 + 2 * 4 * (size_t)CODISTILL_STATIC_MAX_ROWS;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of the scratch array on the current device, looked up once per device.  Host threads
// may make their first calls on a device at the same time: the table is filled under a mutex and read
// through acquire loads, so that no thread ever sees a half-published entry.
static int static_scratch_address(void** out) {
  static std::atomic<void*> cache[64];
  static std::mutex fill;
  int dev = 0;
  if (const int rc_cuda = cuda_status(cudaGetDevice(&dev))) return rc_cuda;
  const bool cached = dev >= 0 && dev < 64;
  if (cached) {
    if (void* known = cache[dev].load(std::memory_order_acquire)) { *out = known; return CODISTILL_OK; }
  }
  std::lock_guard<std::mutex> lock(fill);
  void* ptr = nullptr;
  if (const int rc_cuda = cuda_status(cudaGetSymbolAddress(&ptr, g_static_scratch))) return rc_cuda;
  if (ptr == nullptr) return CODISTILL_ERR_CUDA;
  if (cached) cache[dev].store(ptr, std::memory_order_release);
  *out = ptr;
  return CODISTILL_OK;
}
}  // namespace codistill

extern "C" int codistill_loss_fwd_bwd_static(const void* logits, const void* const* peer_logits, const int32_t* labels,
                                             const uint8_t* mask, int n, int64_t rows, int64_t classes, float alpha,
                                             float temperature, int dtype, float* row_loss, float* reduced_loss,
                                             void* grad_logits, void* stream) {
  using namespace codistill;
  codistill_params_t p;
  memset(&p, 0, sizeof(p));
  p.struct_bytes = sizeof(p);
  p.logits = logits;
  p.peer_logits = peer_logits;
  p.labels = labels;
  p.mask = mask;
  p.n = n;
  p.dtype = dtype;
  p.rows = rows;
  p.classes = classes;
  p.row_stride = classes;
  p.alpha = alpha;
  p.temperature = temperature;
  p.dist_kind = CODISTILL_DIST_MSE_LOGITS;
  p.peer_reduce = CODISTILL_PEERS_PAIRWISE_MEAN;
  p.reduction = CODISTILL_REDUCE_MEAN_VALID;
  p.row_loss = row_loss;
  p.reduced_loss = reduced_loss;
  p.grad_logits = grad_logits;
  p.workspace = reinterpret_cast<void*>(uintptr_t(256));  // placeholder for validation; replaced below
  const int v = validate(&p, false);
  if (v != CODISTILL_OK) return v;
  if (rows > (int64_t)CODISTILL_STATIC_MAX_ROWS) return CODISTILL_ERR_TOO_LARGE;
  if (ws_layout(rows).total > kStaticScratchBytes) return CODISTILL_ERR_TOO_LARGE;
  void* scratch = nullptr;
  const int rc = static_scratch_address(&scratch);
  if (rc != CODISTILL_OK) return rc;
  p.workspace = scratch;
  p.workspace_bytes = kStaticScratchBytes;
  return run_device(&p, static_cast<cudaStream_t>(stream));
}
