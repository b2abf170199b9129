// Stand-in for the visualisation load, scaled up: a full-resolution, multi-layer blend of the tool
// masks onto the frame (layer l repeats the S6 blend with the palette rotated by l), written as an
// RGBA8 image.  The paper's central finding is that the visualisation work sharing the GPU with
// the inference work is what spreads the latencies (Section VI), and it names single-GPU spatial
// isolation of the two as future work (Section VIII).  This kernel exists to ask that question
// with CUDA only: it can run time-shared (one block per 1024 pixels, spread over every
// multiprocessor, competing with whatever else is running) or carved out (a fixed, small number
// of blocks, each claiming enough shared memory that the large tensor-core blocks of the
// inference path cannot share its multiprocessor, looping over the image).
// The arithmetic per pixel is the same in both modes and does not depend on the mask values
// (every tool's blend is computed and then selected), so the load is the same for any input.
#include "tt_internal.h"

namespace tt {
namespace {

constexpr int RENDER_THREADS = 256;
constexpr int RENDER_PX_PER_THREAD = 4;

__device__ __forceinline__ uint32_t render_px(int r, int g, int b, uint32_t bits, const RenderParams& p) {
  for (int l = 0; l < p.layers; ++l) {
#pragma unroll
    for (int t = 0; t < TT_MAX_TOOLS; ++t) {
      if (t < p.T) {
        int c = t + l;
        c -= (c / p.T) * p.T;                      // palette entry (t + l) mod T
        const int r2 = (153 * r + 102 * (int)p.palette[c][0] + 127) / 255;
        const int g2 = (153 * g + 102 * (int)p.palette[c][1] + 127) / 255;
        const int b2 = (153 * b + 102 * (int)p.palette[c][2] + 127) / 255;
        const bool m = (bits >> t) & 1u;
        r = m ? r2 : r;
        g = m ? g2 : g;
        b = m ? b2 : b;
      }
    }
  }
  return (uint32_t)r | ((uint32_t)g << 8) | ((uint32_t)b << 16) | 0xFF000000u;
}

__global__ void __launch_bounds__(RENDER_THREADS) render_kernel(const __grid_constant__ RenderParams p) {
  const long long npx = (long long)p.src_w * p.src_h;
  const long long groups_per_img = (npx + RENDER_PX_PER_THREAD - 1) / RENDER_PX_PER_THREAD;
  const long long total = groups_per_img * p.K;
  const int plane = p.Hm * p.Wm;
  // grid-stride over groups of 4 pixels: with a full grid every thread takes one group, with a
  // carved-out grid the few blocks walk through the whole batch
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < total; q += (long long)gridDim.x * blockDim.x) {
    const int n = (int)(q / groups_per_img);
    const long long i0 = (q - (long long)n * groups_per_img) * RENDER_PX_PER_THREAD;
    const uint8_t* __restrict__ src = p.src.p[n];
    uint8_t* dst = p.dst + (size_t)n * npx * 4;
    for (int j = 0; j < RENDER_PX_PER_THREAD && i0 + j < npx; ++j) {
      const int x = (int)((i0 + j) % p.src_w), y = (int)((i0 + j) / p.src_w);
      const uint8_t* s = src + (size_t)y * p.src_pitch + 3 * x;
      const int mx = (int)(((long long)x * p.Wm) / p.src_w), my = (int)(((long long)y * p.Hm) / p.src_h);
      uint32_t bits = 0;
      for (int t = 0; t < p.T; ++t) bits |= (uint32_t)(__ldg(p.masks + ((size_t)n * p.T + t) * plane + my * p.Wm + mx) != 0) << t;
      *reinterpret_cast<uint32_t*>(dst + (i0 + j) * 4) = render_px(__ldg(s), __ldg(s + 1), __ldg(s + 2), bits, p);
    }
  }
}

}  // namespace

cudaError_t launch_render(const RenderParams& p, cudaStream_t s) {
  const long long npx = (long long)p.src_w * p.src_h;
  const long long groups = ((npx + RENDER_PX_PER_THREAD - 1) / RENDER_PX_PER_THREAD) * p.K;
  const long long full = (groups + RENDER_THREADS - 1) / RENDER_THREADS;
  if (p.carve_ctas > 0) {
    // a block of the carved-out form claims this much shared memory so that the inference path's
    // large blocks (about 200 KB each) cannot be placed beside it
    constexpr int CLAIM = 64 * 1024;
    cudaError_t e = cudaFuncSetAttribute(render_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, CLAIM);
    if (e != cudaSuccess) return e;
    const int grid = (int)(full < p.carve_ctas ? full : p.carve_ctas);
    render_kernel<<<grid, RENDER_THREADS, CLAIM, s>>>(p);
  } else {
    render_kernel<<<(unsigned)full, RENDER_THREADS, 0, s>>>(p);
  }
  return cudaGetLastError();
}

}  // namespace tt
