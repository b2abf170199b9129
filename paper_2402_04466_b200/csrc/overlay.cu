// S6: alpha-blend the thresholded tool masks as colours onto an RGBA8 copy of the source
// frame (integer arithmetic, bit-exact).  HBM-bound: 3 bytes in, 4 bytes out per pixel.
// When the frame is dense (pitch == 3*W) and 4-byte aligned the image is processed as a
// flat stream: a thread takes 4 consecutive pixels = three 32-bit loads and one 128-bit
// store, both fully coalesced.
#include "tt_internal.h"

namespace tt {
namespace {

template <bool PACKED>
__device__ __forceinline__ uint32_t mask_bits(const OverlayParams& p, int n, int x, int y) {
  const int mx = (int)(((long long)x * p.Wm) / p.src_w);
  const int my = (int)(((long long)y * p.Hm) / p.src_h);
  const int plane = p.Hm * p.Wm;
  if (PACKED) return __ldg(p.bits + (size_t)n * plane + my * p.Wm + mx);
  uint32_t b = 0;
  for (int t = 0; t < p.T; ++t) b |= (uint32_t)(__ldg(p.masks + ((size_t)n * p.T + t) * plane + my * p.Wm + mx) != 0) << t;
  return b;
}

__device__ __forceinline__ uint32_t blend_px(int r, int g, int b, uint32_t bits, const OverlayParams& p) {
  while (bits) {
    const int t = __ffs(bits) - 1;
    bits &= bits - 1;
    r = (153 * r + 102 * (int)p.palette[t][0] + 127) / 255;
    g = (153 * g + 102 * (int)p.palette[t][1] + 127) / 255;
    b = (153 * b + 102 * (int)p.palette[t][2] + 127) / 255;
  }
  return (uint32_t)r | ((uint32_t)g << 8) | ((uint32_t)b << 16) | 0xFF000000u;
}

template <bool PACKED, bool FLAT>
__global__ void __launch_bounds__(256) overlay_kernel(const __grid_constant__ OverlayParams p) {
  const int n = blockIdx.y;
  const uint8_t* __restrict__ src = p.src_tab ? p.src_tab[n] : p.src.p[n];
  const long long npx = (long long)p.src_w * p.src_h;
  uint8_t* dst = p.dst + (size_t)n * npx * 4;
  const long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x;  // group of 4 pixels
  const long long i0 = q * 4;
  if (i0 >= npx) return;
  uint32_t out[4];
  if (FLAT && i0 + 3 < npx) {
    const uint32_t* s32 = reinterpret_cast<const uint32_t*>(src) + q * 3;
    const uint32_t w0 = __ldg(s32), w1 = __ldg(s32 + 1), w2 = __ldg(s32 + 2);
    const int r[4] = {(int)(w0 & 255), (int)(w0 >> 24), (int)((w1 >> 16) & 255), (int)((w2 >> 8) & 255)};
    const int g[4] = {(int)((w0 >> 8) & 255), (int)(w1 & 255), (int)(w1 >> 24), (int)((w2 >> 16) & 255)};
    const int b[4] = {(int)((w0 >> 16) & 255), (int)((w1 >> 8) & 255), (int)(w2 & 255), (int)(w2 >> 24)};
    int x = (int)(i0 % p.src_w), y = (int)(i0 / p.src_w);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      out[j] = blend_px(r[j], g[j], b[j], mask_bits<PACKED>(p, n, x, y), p);
      if (++x == p.src_w) { x = 0; ++y; }
    }
    *reinterpret_cast<uint4*>(dst + i0 * 4) = make_uint4(out[0], out[1], out[2], out[3]);
  } else {
    for (int j = 0; j < 4 && i0 + j < npx; ++j) {
      const int x = (int)((i0 + j) % p.src_w), y = (int)((i0 + j) / p.src_w);
      const uint8_t* s = src + (size_t)y * p.src_pitch + 3 * x;
      const uint32_t v = blend_px(s[0], s[1], s[2], mask_bits<PACKED>(p, n, x, y), p);
      *reinterpret_cast<uint32_t*>(dst + (i0 + j) * 4) = v;
    }
  }
}

}  // namespace

cudaError_t launch_overlay(const OverlayParams& p, cudaStream_t s) {
  const long long npx = (long long)p.src_w * p.src_h;
  const long long groups = (npx + 3) / 4;
  dim3 grid((unsigned)((groups + 255) / 256), p.K), block(256);
  bool flat = p.src_pitch == 3 * p.src_w;
  for (int n = 0; n < p.K; ++n) flat = flat && (((uintptr_t)p.src.p[n] & 3) == 0);
  flat = flat && (((uintptr_t)p.dst & 15) == 0) && ((npx * 4) % 16 == 0 || p.K == 1);
  const bool packed = p.bits != nullptr;
  if (packed) {
    if (flat) overlay_kernel<true, true><<<grid, block, 0, s>>>(p);
    else overlay_kernel<true, false><<<grid, block, 0, s>>>(p);
  } else {
    if (flat) overlay_kernel<false, true><<<grid, block, 0, s>>>(p);
    else overlay_kernel<false, false><<<grid, block, 0, s>>>(p);
  }
  return cudaGetLastError();
}

}  // namespace tt
