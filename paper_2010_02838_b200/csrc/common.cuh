// Shared declarations of the codistillation kernels: kernel argument block, workspace layout,
// element conversion and group reductions.  Device code only; the host dispatcher is in api.cu.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

#include "../../include/codistill.h"

namespace codistill {

constexpr int kMaxPeers = CODISTILL_MAX_PEERS;
constexpr int kPrepMaxBlocks = 56;        // partial valid-row counts written by the prep kernel
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// First 256 bytes of the workspace.  Zeroed by the prep kernel at the start of every call.
struct WsHeader {
  unsigned int ticket;        // CTAs that finished their rows (the last one runs the final reduction)
  unsigned int next_row;      // dynamic row scheduler of the persistent kernel
  int status;                 // CODISTILL_DEV_* bits
  int prep_blocks;            // number of valid entries in the partial counts
  unsigned int sched_done;    // CTAs of the persistent kernel that are done with the row counter
  unsigned int pad[59];       // [b] != 0: prep block b saw a valid row with a label outside [0, classes)
};
static_assert(sizeof(WsHeader) == 256, "header is 256 bytes");

// Byte offsets inside the workspace (all multiples of 256).
struct WsLayout {
  size_t partials;   // int64[kPrepMaxBlocks][2]  (valid, masked) per prep block
  size_t row_flags;  // uint32[rows]  bit 0: arg-max == label, bit 1+j: arg-max agrees with peer j
  size_t row_loss;   // float[rows]   used when the caller passes no row_loss
  size_t total;
};
__host__ __device__ inline size_t round256(size_t v) { return (v + 255) & ~size_t(255); }
__host__ __device__ inline WsLayout ws_layout(int64_t rows) {
  WsLayout l;
  l.partials = sizeof(WsHeader);
  l.row_flags = l.partials + round256(sizeof(int64_t) * 2 * kPrepMaxBlocks);
  l.row_loss = l.row_flags + round256(sizeof(uint32_t) * (size_t)(rows > 0 ? rows : 1));
  l.total = l.row_loss + round256(sizeof(float) * (size_t)(rows > 0 ? rows : 1));
  return l;
}

// Arguments of every main kernel.  Data pointers of logits / peers / grad are those of row
// `row_begin`; labels, mask, row_loss and row_flags are indexed by the global row id.
struct KArgs {
  const void* own;
  const void* peers[kMaxPeers];
  void* grad;                  // nullable
  const int32_t* labels;
  const uint8_t* mask;         // nullable
  float* row_loss;             // never null here (caller's or workspace)
  uint32_t* row_flags;
  WsHeader* hdr;
  const int64_t* partials;
  float* reduced_loss;
  int64_t* counters;           // nullable
  int32_t* dev_status;         // nullable
  int64_t rows_total;          // rows of the whole call (labels / mask length)
  int64_t row_begin, row_end;  // rows handled by this launch
  int64_t classes, row_stride;
  int n_peers;
  int dist, peer_reduce, reduction;
  int want_flags;              // compute arg-max agreement bits (counters requested)
  int fused_finalize;          // last CTA reduces losses and counters
  float alpha, temperature, eps;
};

// ------------------------------------------------------------------ CUDA errors
// CODISTILL_OK for cudaSuccess; otherwise the error is kept for codistill_last_cuda_error() (per host
// thread) and CODISTILL_ERR_CUDA is returned.  Defined in api.cu.
int cuda_status(cudaError_t e);
// Same, for code that hands a cudaError_t on: remembers which call failed (a string literal) and returns e.
cudaError_t cuda_note(cudaError_t e, const char* what);

// ------------------------------------------------------------------ programmatic dependent launch
// The main kernels are launched with programmatic stream serialisation: their CTAs may start while
// the prep kernel of the same call still runs, so that launch latency and set-up overlap with it.
// Nothing the prep kernel writes (workspace header, partial counts) may be touched before
// wait_for_prior_grid() returns; it returns once the preceding grid has finished and its writes are visible.
__device__ __forceinline__ void wait_for_prior_grid() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void release_dependent_grid() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Launches `kernel` so that it may overlap the tail of the kernel before it in the stream.
template <typename... KP, typename... Args>
inline cudaError_t launch_overlapped(void (*kernel)(KP...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// ------------------------------------------------------------------ element conversion
template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int kVec = 4;  // elements per 16-byte packet
  __device__ static float to_f32(float v) { return v; }
  __device__ static float from_f32(float v) { return v; }
};
template <> struct Elem<__nv_bfloat16> {
  static constexpr int kVec = 8;
  __device__ static float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
  __device__ static __nv_bfloat16 from_f32(float v) { return __float2bfloat16_rn(v); }
};

// Load V consecutive elements starting at element c of a row (V == 1 or a full 16-byte packet).
template <typename T, int V>
__device__ __forceinline__ void load_packet(const T* __restrict__ row, int64_t c, float (&out)[V]) {
  if constexpr (V == 1) {
    out[0] = Elem<T>::to_f32(row[c]);
  } else {
    const uint4 raw = *reinterpret_cast<const uint4*>(row + c);
    if constexpr (sizeof(T) == 4) {
      out[0] = __uint_as_float(raw.x); out[1] = __uint_as_float(raw.y);
      out[2] = __uint_as_float(raw.z); out[3] = __uint_as_float(raw.w);
    } else {
      const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        out[2 * i] = __uint_as_float(w[i] << 16);
        out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
      }
    }
  }
}

// Store V consecutive elements (rounded to T); only the first `nvalid` are written.
template <typename T, int V>
__device__ __forceinline__ void store_packet(T* __restrict__ row, int64_t c, const float (&v)[V], int nvalid) {
  if constexpr (V == 1) {
    row[c] = Elem<T>::from_f32(v[0]);
  } else {
    if (nvalid >= V) {
      uint4 raw;
      if constexpr (sizeof(T) == 4) {
        raw.x = __float_as_uint(v[0]); raw.y = __float_as_uint(v[1]);
        raw.z = __float_as_uint(v[2]); raw.w = __float_as_uint(v[3]);
      } else {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const __nv_bfloat162 p = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
          w[i] = *reinterpret_cast<const uint32_t*>(&p);
        }
        raw.x = w[0]; raw.y = w[1]; raw.z = w[2]; raw.w = w[3];
      }
      *reinterpret_cast<uint4*>(row + c) = raw;
    } else {
#pragma unroll
      for (int i = 0; i < V; ++i)
        if (i < nvalid) row[c + i] = Elem<T>::from_f32(v[i]);
    }
  }
}

// ------------------------------------------------------------------ reductions
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
// larger value wins; on equal values the lower index wins (first arg-max)
__device__ __forceinline__ void argmax_combine(float& v, int& i, float ov, int oi) {
  if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
}
__device__ __forceinline__ void warp_argmax(float& v, int& i) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, v, o);
    const int oi = __shfl_xor_sync(0xffffffffu, i, o);
    argmax_combine(v, i, ov, oi);
  }
}

// A group of threads working on one row: one warp (kThreads == 32) or the whole CTA.
// Every reduction returns the result to all threads of the group.  `scratch` is shared memory
// of at least 33 * 4 floats private to the group (unused for a warp).
template <int kThreads>
struct Group {
  static constexpr int kWarps = kThreads / 32;
  template <int N>
  __device__ static void sum(float (&v)[N], float* scratch) {
#pragma unroll
    for (int k = 0; k < N; ++k) v[k] = warp_sum(v[k]);
    if constexpr (kThreads > 32) {
      const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
      __syncthreads();
      if (lane == 0) {
#pragma unroll
        for (int k = 0; k < N; ++k) scratch[k * 32 + warp] = v[k];
      }
      __syncthreads();
#pragma unroll
      for (int k = 0; k < N; ++k) {
        float t = (lane < kWarps) ? scratch[k * 32 + lane] : 0.f;
        v[k] = warp_sum(t);
      }
    }
  }
  __device__ static float max(float v, float* scratch) {
    v = warp_max(v);
    if constexpr (kThreads > 32) {
      const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
      __syncthreads();
      if (lane == 0) scratch[warp] = v;
      __syncthreads();
      v = warp_max((lane < kWarps) ? scratch[lane] : -INFINITY);
    }
    return v;
  }
  __device__ static void argmax(float& v, int& i, float* scratch) {
    warp_argmax(v, i);
    if constexpr (kThreads > 32) {
      const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
      __syncthreads();
      if (lane == 0) { scratch[warp] = v; reinterpret_cast<int*>(scratch)[32 + warp] = i; }
      __syncthreads();
      v = (lane < kWarps) ? scratch[lane] : -INFINITY;
      i = (lane < kWarps) ? reinterpret_cast<int*>(scratch)[32 + lane] : 0x7fffffff;
      warp_argmax(v, i);
    }
  }
};

// A row takes part iff its mask byte is non-zero (or there is no mask) and its label is a class id.
__device__ __forceinline__ bool row_valid(const KArgs& a, int64_t r) {
  if (a.mask != nullptr && a.mask[r] == 0) return false;
  const int32_t y = a.labels[r];
  return y >= 0 && (int64_t)y < a.classes;
}

// n_valid of the whole call, from the prep kernel's partial counts (fixed order).
__device__ __forceinline__ int64_t total_valid(const KArgs& a) {
  const int nb = a.hdr->prep_blocks;
  int64_t v = 0;
  for (int b = 0; b < nb; ++b) v += a.partials[2 * b];
  return v;
}

// Final reduction, run by one whole CTA after every row has been written: per-row losses are
// summed in a fixed order in double precision, flag bits are counted, outputs are written.
// `sh` is shared memory of at least 32 doubles.  The result does not depend on which CTA runs it.
__device__ inline void finalize_cta(const KArgs& a, double* sh) {
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = (nt + 31) >> 5;
  const int64_t R = a.rows_total;
  int64_t n_valid = 0, n_masked = 0;
  for (int b = 0; b < a.hdr->prep_blocks; ++b) { n_valid += a.partials[2 * b]; n_masked += a.partials[2 * b + 1]; }

  double s = 0.0;
  for (int64_t r = tid; r < R; r += nt) s += (double)__ldcg(a.row_loss + r);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
  __syncthreads();
  if (lane == 0) sh[warp] = s;
  __syncthreads();
  if (tid == 0) {
    double total = 0.0;
    for (int k = 0; k < nw; ++k) total += sh[k];
    if (a.reduction == CODISTILL_REDUCE_MEAN_VALID) total /= (double)(n_valid > 1 ? n_valid : 1);
    *a.reduced_loss = (float)total;
    if (a.dev_status) {
      int st = a.hdr->status;
      for (int b = 0; b < a.hdr->prep_blocks; ++b)
        if (a.hdr->pad[b]) st |= CODISTILL_DEV_BAD_LABEL;  // per-block words written by the prep kernel
      *a.dev_status = st;
    }
    if (a.counters) { a.counters[0] = n_valid; a.counters[1] = n_masked; }
  }
  if (a.counters) {
    long long* shi = reinterpret_cast<long long*>(sh);
    for (int bit = 0; bit <= a.n_peers; ++bit) {
      long long cnt = 0;
      for (int64_t r = tid; r < R; r += nt) cnt += (__ldcg(a.row_flags + r) >> bit) & 1u;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) cnt += __shfl_down_sync(0xffffffffu, cnt, o);
      __syncthreads();
      if (lane == 0) shi[warp] = cnt;
      __syncthreads();
      if (tid == 0) {
        long long total = 0;
        for (int k = 0; k < nw; ++k) total += shi[k];
        a.counters[2 + bit] = total;
      }
    }
  }
}

// Called by every CTA of a main kernel once its rows are written.  With fused_finalize the last
// CTA to arrive runs the final reduction.  `sh_flag` is one int of shared memory.
__device__ inline void finish_cta(const KArgs& a, double* sh, int* sh_flag) {
  if (!a.fused_finalize) return;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned int prev = atomicAdd(&a.hdr->ticket, 1u);
    *sh_flag = (prev == gridDim.x - 1);
  }
  __syncthreads();
  if (*sh_flag) {
    __threadfence();
    finalize_cta(a, sh);
  }
}

}  // namespace codistill
