// First encoder layer of the bf16 path: 3 input channels (planar fp32 from preprocess) ->
// COUT channels, 3x3, pad 1, stride 1 or 2, bias, ReLU, output bf16 channels-last.
//
// K = 27 is too thin for a tensor-core contraction and the layer is bound by plain fp32 FMA
// throughput and HBM.  One thread produces one output pixel for all COUT channels.  The
// 27*COUT weights travel in the kernel's parameter block, i.e. in the constant bank, and the
// loops are fully unrolled, so every FMA takes its weight as a constant-bank operand: no
// shared memory, no weight loads, one issue slot per FMA.
#include "tt_internal.h"

namespace tt {
namespace {

template <int COUT>
__global__ void __launch_bounds__(256) conv_first_kernel(const __grid_constant__ ConvFirstParams p) {
  const int xo = blockIdx.x * 32 + threadIdx.x;
  const int yo = blockIdx.y * 8 + threadIdx.y;
  const int n = blockIdx.z;
  if (xo >= p.Wo || yo >= p.Ho) return;
  const size_t plane = (size_t)p.H * p.W;
  const float* __restrict__ src = p.in + (size_t)n * 3 * plane;
  const int x0 = xo * p.stride - 1, y0 = yo * p.stride - 1;

  float v[27];
#pragma unroll
  for (int c = 0; c < 3; ++c)
#pragma unroll
    for (int ky = 0; ky < 3; ++ky)
#pragma unroll
      for (int kx = 0; kx < 3; ++kx) {
        const int yi = y0 + ky, xi = x0 + kx;
        const bool ok = yi >= 0 && yi < p.H && xi >= 0 && xi < p.W;
        v[(c * 3 + ky) * 3 + kx] = ok ? __ldg(src + (size_t)c * plane + (size_t)yi * p.W + xi) : 0.0f;
      }

  __nv_bfloat16* dst = p.out + (((size_t)n * p.Ho + yo) * p.Wo + xo) * COUT;
#pragma unroll
  for (int o0 = 0; o0 < COUT; o0 += 8) {
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = p.b[o0 + i];
#pragma unroll
    for (int t = 0; t < 27; ++t)
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] = fmaf(v[t], p.w[t * COUT + o0 + i], acc[i]);
    uint4 u;
    __nv_bfloat162 q0 = __floats2bfloat162_rn(fmaxf(acc[0], 0.f), fmaxf(acc[1], 0.f));
    __nv_bfloat162 q1 = __floats2bfloat162_rn(fmaxf(acc[2], 0.f), fmaxf(acc[3], 0.f));
    __nv_bfloat162 q2 = __floats2bfloat162_rn(fmaxf(acc[4], 0.f), fmaxf(acc[5], 0.f));
    __nv_bfloat162 q3 = __floats2bfloat162_rn(fmaxf(acc[6], 0.f), fmaxf(acc[7], 0.f));
    u.x = *reinterpret_cast<uint32_t*>(&q0);
    u.y = *reinterpret_cast<uint32_t*>(&q1);
    u.z = *reinterpret_cast<uint32_t*>(&q2);
    u.w = *reinterpret_cast<uint32_t*>(&q3);
    *reinterpret_cast<uint4*>(dst + o0) = u;
  }
}

template <int COUT>
cudaError_t launch_t(const ConvFirstParams& q, cudaStream_t s) {
  dim3 grid((q.Wo + 31) / 32, (q.Ho + 7) / 8, q.K), block(32, 8);
  conv_first_kernel<COUT><<<grid, block, 0, s>>>(q);
  return cudaGetLastError();
}

}  // namespace

bool conv_first_supported(int cout) { return cout == 16 || cout == 32 || cout == 64; }

cudaError_t launch_conv_first(const ConvFirstParams& q, cudaStream_t s) {
  switch (q.cout) {
    case 16: return launch_t<16>(q, s);
    case 32: return launch_t<32>(q, s);
    case 64: return launch_t<64>(q, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace tt
