// S1: uint8 RGB interleaved frame -> bilinear resize -> normalise -> planar fp32.
//
// HBM-bound stage.  Each thread produces 4 consecutive output samples of one row for all
// three channels (three 128-bit stores).  The source rows a block needs are staged in
// shared memory with 128-bit loads of the aligned byte range that covers them (row pitch
// 3*W is in general not a multiple of 16, so rows are treated as a byte stream and indexed
// from the remainder), then sampled from shared memory.
#include "tt_internal.h"

namespace tt {
namespace {

constexpr int PRE_TX = 32;          // threads along x; each makes 4 outputs -> 128 outputs per block row
constexpr int PRE_TY = 8;           // output rows per block
constexpr int PRE_OUT_W = PRE_TX * 4;
constexpr int PRE_SMEM_BYTES = 40 * 1024;

struct AxisSample {
  int i0, i1;
  float f;
};

// Exact integer evaluation of s = clamp((o + 1/2) * in/out - 1/2, 0, in - 1):
// s = num/den with num = (2o+1)*in - out, den = 2*out.
__device__ __forceinline__ AxisSample axis_sample(int o, int in, int out) {
  int den = 2 * out;
  int num = (2 * o + 1) * in - out;
  int hi = (in - 1) * den;
  num = max(0, min(num, hi));
  AxisSample r;
  r.i0 = num / den;
  r.i1 = min(r.i0 + 1, in - 1);
  r.f = (float)(num - r.i0 * den) / (float)den;  // both integers are exact in fp32
  return r;
}

__device__ __forceinline__ int axis_lo(int o, int in, int out) {
  int den = 2 * out;
  int num = (2 * o + 1) * in - out;
  num = max(0, min(num, (in - 1) * den));
  return num / den;
}

template <bool STAGED>
__global__ void __launch_bounds__(PRE_TX* PRE_TY)
preprocess_kernel(const PreprocessParams p, int row_cap_bytes) {
  extern __shared__ __align__(16) uint8_t s_rows[];
  const int n = blockIdx.z;
  const uint8_t* __restrict__ src = p.src.p[n];
  const int xo_blk = blockIdx.x * PRE_OUT_W;
  const int yo_blk = blockIdx.y * PRE_TY;
  const int tid = threadIdx.y * PRE_TX + threadIdx.x;

  // Source footprint of this block.
  const int xo_last = min(xo_blk + PRE_OUT_W, p.net_w) - 1;
  const int yo_last = min(yo_blk + PRE_TY, p.net_h) - 1;
  const int sx_lo = axis_lo(xo_blk, p.src_w, p.net_w);
  const int sx_hi = min(axis_lo(xo_last, p.src_w, p.net_w) + 1, p.src_w - 1);
  const int sy_lo = axis_lo(yo_blk, p.src_h, p.net_h);
  const int sy_hi = min(axis_lo(yo_last, p.src_h, p.net_h) + 1, p.src_h - 1);
  const int n_rows = sy_hi - sy_lo + 1;

  if (STAGED) {
    // Row r of the footprint occupies s_rows[r*row_cap_bytes ...]; byte b of the staged
    // row corresponds to global byte (row_start_aligned + b).
    for (int r = 0; r < n_rows; ++r) {
      const size_t g_first = (size_t)(sy_lo + r) * p.src_pitch + 3 * sx_lo;
      const size_t g_last = (size_t)(sy_lo + r) * p.src_pitch + 3 * sx_hi + 2;
      const uintptr_t a_first = ((uintptr_t)src + g_first) & ~(uintptr_t)15;
      const uintptr_t a_end = (((uintptr_t)src + g_last) | 15) + 1;
      const int n_vec = (int)((a_end - a_first) >> 4);
      const uint4* gv = reinterpret_cast<const uint4*>(a_first);
      uint4* sv = reinterpret_cast<uint4*>(s_rows + (size_t)r * row_cap_bytes);
      for (int i = tid; i < n_vec; i += PRE_TX * PRE_TY) sv[i] = __ldg(gv + i);
    }
    __syncthreads();
  }

  const int yo = yo_blk + threadIdx.y;
  const int xo0 = xo_blk + threadIdx.x * 4;
  if (yo >= p.net_h || xo0 >= p.net_w) return;

  const AxisSample sy = axis_sample(yo, p.src_h, p.net_h);
  const uint8_t* r0;
  const uint8_t* r1;
  if (STAGED) {
    // offset of source column 0 inside a staged row: (global address of the row's byte
    // 3*sx_lo) minus its aligned start, minus 3*sx_lo
    const size_t g0 = (size_t)sy.i0 * p.src_pitch + 3 * sx_lo;
    const size_t g1 = (size_t)sy.i1 * p.src_pitch + 3 * sx_lo;
    const int off0 = (int)(((uintptr_t)src + g0) & 15) - 3 * sx_lo;
    const int off1 = (int)(((uintptr_t)src + g1) & 15) - 3 * sx_lo;
    r0 = s_rows + (size_t)(sy.i0 - sy_lo) * row_cap_bytes + off0;
    r1 = s_rows + (size_t)(sy.i1 - sy_lo) * row_cap_bytes + off1;
  } else {
    r0 = src + (size_t)sy.i0 * p.src_pitch;
    r1 = src + (size_t)sy.i1 * p.src_pitch;
  }

  float outv[3][4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int xo = min(xo0 + j, p.net_w - 1);
    const AxisSample sx = axis_sample(xo, p.src_w, p.net_w);
#pragma unroll
    for (int c = 0; c < 3; ++c) {
      const float p00 = (float)r0[3 * sx.i0 + c], p01 = (float)r0[3 * sx.i1 + c];
      const float p10 = (float)r1[3 * sx.i0 + c], p11 = (float)r1[3 * sx.i1 + c];
      const float top = p00 + sx.f * (p01 - p00);
      const float bot = p10 + sx.f * (p11 - p10);
      const float v = top + sy.f * (bot - top);
      outv[c][j] = (v * p.inv_div - p.mean) * p.inv_std;
    }
  }

  const size_t plane = (size_t)p.net_h * p.net_w;
  float* dst = p.dst + (size_t)n * 3 * plane + (size_t)yo * p.net_w + xo0;
  const bool vec_ok = ((p.net_w & 3) == 0) && (xo0 + 3 < p.net_w);
#pragma unroll
  for (int c = 0; c < 3; ++c) {
    float* d = dst + c * plane;
    if (vec_ok) {
      *reinterpret_cast<float4*>(d) = make_float4(outv[c][0], outv[c][1], outv[c][2], outv[c][3]);
    } else {
      for (int j = 0; j < 4 && xo0 + j < p.net_w; ++j) d[j] = outv[c][j];
    }
  }
}

}  // namespace

cudaError_t launch_preprocess(const PreprocessParams& p, cudaStream_t s) {
  dim3 block(PRE_TX, PRE_TY);
  dim3 grid((p.net_w + PRE_OUT_W - 1) / PRE_OUT_W, (p.net_h + PRE_TY - 1) / PRE_TY, p.K);
  // Worst-case staged footprint of one block: rows = ceil(TY * sh/nh) + 2, bytes per row =
  // 3 * (ceil(OUT_W * sw/nw) + 2) + 32 (alignment slack on both ends), rounded to 16.
  const long rows = ((long)PRE_TY * p.src_h + p.net_h - 1) / p.net_h + 2;
  const long cols = ((long)PRE_OUT_W * p.src_w + p.net_w - 1) / p.net_w + 2;
  long row_cap = ((3 * cols + 32 + 15) / 16) * 16;
  if (rows * row_cap <= PRE_SMEM_BYTES) {
    preprocess_kernel<true><<<grid, block, (size_t)(rows * row_cap), s>>>(p, (int)row_cap);
  } else {
    preprocess_kernel<false><<<grid, block, 0, s>>>(p, 0);
  }
  return cudaGetLastError();
}

}  // namespace tt
