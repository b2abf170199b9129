// Layout conversions between the boundary's NCHW fp32 tensors and the internal
// channels-last tensors (state import/export and debug taps only; not on the hot path).
#include "tt_internal.h"

namespace tt {
namespace {

template <typename SRC, typename DST, bool TO_NCHW>
__global__ void convert_kernel(const SRC* __restrict__ src, DST* __restrict__ dst, int C, int plane) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long long)C * plane) return;
  // i enumerates the destination linearly
  int c, px;
  if (TO_NCHW) { c = (int)(i / plane); px = (int)(i % plane); }
  else { px = (int)(i / C); c = (int)(i % C); }
  const SRC v = TO_NCHW ? src[(size_t)px * C + c] : src[(size_t)c * plane + px];
  dst[i] = (DST)v;
}

template <typename SRC, typename DST, bool TO_NCHW>
cudaError_t run(const SRC* src, DST* dst, int C, int plane, cudaStream_t s) {
  const long long n = (long long)C * plane;
  convert_kernel<SRC, DST, TO_NCHW><<<(unsigned)((n + 255) / 256), 256, 0, s>>>(src, dst, C, plane);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_nhwc_to_nchw_f32(const float* src, float* dst, int C, int plane, cudaStream_t s) {
  return run<float, float, true>(src, dst, C, plane, s);
}
cudaError_t launch_nchw_to_nhwc_f32(const float* src, float* dst, int C, int plane, cudaStream_t s) {
  return run<float, float, false>(src, dst, C, plane, s);
}
cudaError_t launch_nhwc_bf16_to_nchw_f32(const __nv_bfloat16* src, float* dst, int C, int plane, cudaStream_t s) {
  return run<__nv_bfloat16, float, true>(src, dst, C, plane, s);
}
cudaError_t launch_nchw_f32_to_nhwc_bf16(const float* src, __nv_bfloat16* dst, int C, int plane, cudaStream_t s) {
  return run<float, __nv_bfloat16, false>(src, dst, C, plane, s);
}

}  // namespace tt
