// Compression of the predictions that codistilled models exchange (Section 3: every device sends its
// B x C predictions to the other model groups; b_pred bits per sample): 32-bit logits packed to bfloat16
// (round to nearest even) before they are sent, and widened again (exactly) on the receiving side when the
// loss runs on 32-bit logits.  Element-wise, memory-bound: 16-byte loads and stores where rows allow.
#include <cuda_bf16.h>

#include "common.cuh"

namespace codistill {

constexpr int kPackThreads = 256;

// rows x classes elements; pitches in elements.  VEC: both pitches and both bases allow 8-element packets.
template <bool VEC>
__global__ void __launch_bounds__(kPackThreads) pack_predictions_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst,
                                                                         int64_t rows, int64_t classes, int64_t src_stride, int64_t dst_stride) {
  const int64_t per_row = VEC ? (classes + 7) / 8 : classes;
  const int64_t total = rows * per_row;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = idx / per_row, k = idx - r * per_row;
    if constexpr (VEC) {
      const int64_t c = k * 8;
      const float* s = src + r * src_stride + c;
      __nv_bfloat16* d = dst + r * dst_stride + c;
      if (c + 8 <= classes) {
        const float4 a = *reinterpret_cast<const float4*>(s), b = *reinterpret_cast<const float4*>(s + 4);
        const __nv_bfloat162 p0 = __floats2bfloat162_rn(a.x, a.y), p1 = __floats2bfloat162_rn(a.z, a.w);
        const __nv_bfloat162 p2 = __floats2bfloat162_rn(b.x, b.y), p3 = __floats2bfloat162_rn(b.z, b.w);
        uint4 o;
        o.x = *reinterpret_cast<const uint32_t*>(&p0); o.y = *reinterpret_cast<const uint32_t*>(&p1);
        o.z = *reinterpret_cast<const uint32_t*>(&p2); o.w = *reinterpret_cast<const uint32_t*>(&p3);
        *reinterpret_cast<uint4*>(d) = o;
      } else {
        for (int64_t i = 0; c + i < classes; ++i) d[i] = __float2bfloat16_rn(s[i]);
      }
    } else {
      dst[r * dst_stride + k] = __float2bfloat16_rn(src[r * src_stride + k]);
    }
  }
}

template <bool VEC>
__global__ void __launch_bounds__(kPackThreads) unpack_predictions_kernel(const __nv_bfloat16* __restrict__ src, float* __restrict__ dst,
                                                                           int64_t rows, int64_t classes, int64_t src_stride, int64_t dst_stride) {
  const int64_t per_row = VEC ? (classes + 7) / 8 : classes;
  const int64_t total = rows * per_row;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = idx / per_row, k = idx - r * per_row;
    if constexpr (VEC) {
      const int64_t c = k * 8;
      const __nv_bfloat16* s = src + r * src_stride + c;
      float* d = dst + r * dst_stride + c;
      if (c + 8 <= classes) {
        const uint4 raw = *reinterpret_cast<const uint4*>(s);
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
        float4 a, b;
        a.x = __uint_as_float(w[0] << 16); a.y = __uint_as_float(w[0] & 0xFFFF0000u);
        a.z = __uint_as_float(w[1] << 16); a.w = __uint_as_float(w[1] & 0xFFFF0000u);
        b.x = __uint_as_float(w[2] << 16); b.y = __uint_as_float(w[2] & 0xFFFF0000u);
        b.z = __uint_as_float(w[3] << 16); b.w = __uint_as_float(w[3] & 0xFFFF0000u);
        *reinterpret_cast<float4*>(d) = a;
        *reinterpret_cast<float4*>(d + 4) = b;
      } else {
        for (int64_t i = 0; c + i < classes; ++i) d[i] = __bfloat162float(s[i]);
      }
    } else {
      dst[r * dst_stride + k] = __bfloat162float(src[r * src_stride + k]);
    }
  }
}

static int predictions_check(const void* src, void* dst, int64_t rows, int64_t classes, int64_t src_stride, int64_t dst_stride) {
  if (rows < 0 || classes < 1 || src_stride < classes || dst_stride < classes) return CODISTILL_ERR_SHAPE;
  if (rows > 0 && (src == nullptr || dst == nullptr)) return CODISTILL_ERR_NULL;
  return CODISTILL_OK;
}

static int predictions_grid(int64_t work) {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int64_t blocks = (work + kPackThreads - 1) / kPackThreads;
  const int64_t cap = (int64_t)sms * 8;   // eight resident CTAs per SM cover the memory latency
  return (int)(blocks < 1 ? 1 : blocks < cap ? blocks : cap);
}

}  // namespace codistill

using namespace codistill;

extern "C" int codistill_pack_predictions(const float* src, void* dst_bf16, int64_t rows, int64_t classes, int64_t src_stride,
                                          int64_t dst_stride, void* stream) {
  if (const int rc = predictions_check(src, dst_bf16, rows, classes, src_stride, dst_stride)) return rc;
  if (rows == 0) return CODISTILL_OK;
  __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(dst_bf16);
  const bool vec = (reinterpret_cast<uintptr_t>(src) & 15u) == 0 && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0 &&
                   src_stride % 4 == 0 && dst_stride % 8 == 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (vec)
    pack_predictions_kernel<true><<<predictions_grid(rows * ((classes + 7) / 8)), kPackThreads, 0, s>>>(src, dst, rows, classes, src_stride, dst_stride);
  else
    pack_predictions_kernel<false><<<predictions_grid(rows * classes), kPackThreads, 0, s>>>(src, dst, rows, classes, src_stride, dst_stride);
  return cuda_status(cudaGetLastError());
}

extern "C" int codistill_unpack_predictions(const void* src_bf16, float* dst, int64_t rows, int64_t classes, int64_t src_stride,
                                            int64_t dst_stride, void* stream) {
  if (const int rc = predictions_check(src_bf16, dst, rows, classes, src_stride, dst_stride)) return rc;
  if (rows == 0) return CODISTILL_OK;
  const __nv_bfloat16* src = static_cast<const __nv_bfloat16*>(src_bf16);
  const bool vec = (reinterpret_cast<uintptr_t>(src) & 15u) == 0 && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0 &&
                   src_stride % 8 == 0 && dst_stride % 4 == 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (vec)
    unpack_predictions_kernel<true><<<predictions_grid(rows * ((classes + 7) / 8)), kPackThreads, 0, s>>>(src, dst, rows, classes, src_stride, dst_stride);
  else
    unpack_predictions_kernel<false><<<predictions_grid(rows * classes), kPackThreads, 0, s>>>(src, dst, rows, classes, src_stride, dst_stride);
  return cuda_status(cudaGetLastError());
}
