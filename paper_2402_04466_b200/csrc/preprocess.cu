// S1: uint8 RGB interleaved frame -> bilinear resize -> normalise -> planar fp32.
//
// HBM-bound stage.  A block produces a 128 x 16 tile of the output.  The source rows it needs
// are staged in shared memory with 128-bit loads of the aligned byte range that covers them
// (row pitch 3*W is in general not a multiple of 16, so rows are treated as a byte stream and
// indexed from the remainder).  The horizontal sample positions of the tile's 128 columns are
// computed once per block into shared memory.  A thread produces 4 consecutive outputs of two
// rows for all three channels: each bilinear tap pair (two neighbouring RGB pixels = 6 bytes) is
// fetched as three 32-bit shared loads plus funnel shifts, bytes become floats by a byte
// permute into the mantissa of 2^23, and the results leave as three 128-bit stores.
#include "tt_internal.h"
#include "pre_math.cuh"

namespace tt {
namespace {

using namespace pre;

constexpr int PRE_TX = 32;          // threads along x; each makes 4 outputs -> 128 outputs per block row
constexpr int PRE_TY = 8;           // output rows per block
constexpr int PRE_OUT_W = PRE_TX * 4;
constexpr int PRE_THREADS = PRE_TX * PRE_TY;
constexpr int PRE_SMEM_BYTES = 44 * 1024;

// Six bytes starting at byte offset `b` of a word-aligned shared buffer: the RGB triples of two
// neighbouring pixels.  lo = bytes b..b+3 (R0 G0 B0 R1), hi = bytes b+4..b+7 (G1 B1 . .).
__device__ __forceinline__ void fetch_pair(const uint32_t* s_words, int b, uint32_t& lo, uint32_t& hi) {
  const int w = b >> 2;
  const uint32_t sh = (uint32_t)(b & 3) * 8u;
  const uint32_t w0 = s_words[w], w1 = s_words[w + 1], w2 = s_words[w + 2];
  lo = __funnelshift_r(w0, w1, sh);
  hi = __funnelshift_r(w1, w2, sh);
}

constexpr int PRE_ROWS = 16;          // output rows per block of the staged kernel: 2 per thread

__global__ void __launch_bounds__(PRE_THREADS)
preprocess_staged_kernel(const __grid_constant__ PreprocessParams p, int row_cap_bytes, float scale, float shift) {
  extern __shared__ __align__(16) uint8_t s_mem[];
  __shared__ __align__(16) int s_xoff[PRE_OUT_W];    // 3 * (i0 - sx_lo) per output column of the tile
  __shared__ __align__(16) float s_fx[PRE_OUT_W];
  __shared__ int s_y0[PRE_ROWS], s_y1[PRE_ROWS];     // source rows of every output row of the tile
  __shared__ float s_fy[PRE_ROWS];
  __shared__ int s_xlo, s_xhi;                       // source column range of the tile
  // the next kernel of the stream, if it was launched as a programmatic dependent, may start its set-up now;
  // it waits for this grid to finish before it reads the output
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int n = blockIdx.z;
  const uint8_t* __restrict__ src = p.src_tab ? p.src_tab[n] : p.src.p[n];
  const uint32_t src_lo = (uint32_t)(uintptr_t)src;  // only the low bits matter for 16-byte alignment
  const int xo_blk = blockIdx.x * PRE_OUT_W;
  const int yo_blk = blockIdx.y * PRE_ROWS;
  const int tid = threadIdx.y * PRE_TX + threadIdx.x;

  // Phase 0: one sample position per thread (the only integer divisions of the kernel).
  if (tid < PRE_OUT_W) {
    const AxisSample sx = axis_sample(min(xo_blk + tid, p.net_w - 1), p.src_w, p.net_w);
    s_xoff[tid] = 3 * sx.i0;
    s_fx[tid] = sx.f;
    if (tid == 0) s_xlo = sx.i0;
    if (tid == PRE_OUT_W - 1) s_xhi = min(sx.i0 + 1, p.src_w - 1);
  } else if (tid < PRE_OUT_W + PRE_ROWS) {
    const int r = tid - PRE_OUT_W;
    const AxisSample sy = axis_sample(min(yo_blk + r, p.net_h - 1), p.src_h, p.net_h);
    s_y0[r] = sy.i0;
    s_y1[r] = sy.i1;
    s_fy[r] = sy.f;
  }
  __syncthreads();
  const int sx_lo = s_xlo, sx_hi = s_xhi;
  const int sy_lo = s_y0[0], sy_hi = s_y1[PRE_ROWS - 1];
  const int n_rows = sy_hi - sy_lo + 1;

  // Phase 1: row r of the footprint goes to s_mem[r*row_cap_bytes ...]; byte b of a staged row is
  // the global byte (aligned start of that row's range) + b.  Warp w copies rows w, w+8, ...; its
  // lanes copy 16-byte vectors lane, lane+32, ... of the row.
  for (int r = threadIdx.y; r < n_rows; r += PRE_TY) {
    const size_t g_first = (size_t)(sy_lo + r) * p.src_pitch + 3 * sx_lo;
    const uintptr_t a_first = ((uintptr_t)src + g_first) & ~(uintptr_t)15;
    const uintptr_t a_end = (((uintptr_t)src + g_first + 3 * (sx_hi - sx_lo) + 2) | 15) + 1;
    const int n_vec = (int)((a_end - a_first) >> 4);
    uint4* srow = reinterpret_cast<uint4*>(s_mem + (size_t)r * row_cap_bytes);
    for (int i = threadIdx.x; i < n_vec; i += PRE_TX) srow[i] = __ldg(reinterpret_cast<const uint4*>(a_first) + i);
  }
  __syncthreads();

  // Phase 2: 4 consecutive outputs of rows threadIdx.y and threadIdx.y + 8.
  const int xl = threadIdx.x * 4;
  const int xo0 = xo_blk + xl;
  if (xo0 >= p.net_w) return;
  const uint32_t* s_words = reinterpret_cast<const uint32_t*>(s_mem);
  const int4 xoff4 = *reinterpret_cast<const int4*>(s_xoff + xl);
  const float4 fx4 = *reinterpret_cast<const float4*>(s_fx + xl);
  const int xoffs[4] = {xoff4.x - 3 * sx_lo, xoff4.y - 3 * sx_lo, xoff4.z - 3 * sx_lo, xoff4.w - 3 * sx_lo};
  const float fxs[4] = {fx4.x, fx4.y, fx4.z, fx4.w};
  const size_t plane = (size_t)p.net_h * p.net_w;
  // with a row length that is a multiple of 4 every row start is as aligned as the tensor itself
  const bool vec_ok = ((p.net_w & 3) == 0) && (xo0 + 3 < p.net_w) && (((uintptr_t)p.dst & 15) == 0);

#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    const int r = threadIdx.y + rr * PRE_TY;
    const int yo = yo_blk + r;
    if (yo >= p.net_h) break;
    const int y0 = s_y0[r], y1 = s_y1[r];
    const float fy = s_fy[r];
    // byte position of source column sx_lo inside the two staged rows
    const int base0 = (y0 - sy_lo) * row_cap_bytes + (int)((src_lo + (uint32_t)(y0 * p.src_pitch + 3 * sx_lo)) & 15u);
    const int base1 = (y1 - sy_lo) * row_cap_bytes + (int)((src_lo + (uint32_t)(y1 * p.src_pitch + 3 * sx_lo)) & 15u);
    float o0[4], o1[4], o2[4];  // the three channels of the 4 outputs
    if (fy == 0.0f) {
      // The sample sits exactly on a source row (every row of an axis that is not resized): the
      // lower row has weight zero, so top + 0 * (bot - top) = top and only one row is fetched.
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        uint32_t lo0, hi0;
        fetch_pair(s_words, base0 + xoffs[j], lo0, hi0);
        sample_row(lo0, hi0, fxs[j], scale, shift, o0[j], o1[j], o2[j]);
      }
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        uint32_t lo0, hi0, lo1, hi1;
        fetch_pair(s_words, base0 + xoffs[j], lo0, hi0);
        fetch_pair(s_words, base1 + xoffs[j], lo1, hi1);
        sample_rows(lo0, hi0, lo1, hi1, fxs[j], fy, scale, shift, o0[j], o1[j], o2[j]);
      }
    }
    float* d0 = p.dst + (size_t)n * 3 * plane + (size_t)yo * p.net_w + xo0;
    float* d1 = d0 + plane;
    float* d2 = d1 + plane;
    if (vec_ok) {
      *reinterpret_cast<float4*>(d0) = make_float4(o0[0], o0[1], o0[2], o0[3]);
      *reinterpret_cast<float4*>(d1) = make_float4(o1[0], o1[1], o1[2], o1[3]);
      *reinterpret_cast<float4*>(d2) = make_float4(o2[0], o2[1], o2[2], o2[3]);
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (xo0 + j < p.net_w) {
          d0[j] = o0[j];
          d1[j] = o1[j];
          d2[j] = o2[j];
        }
    }
  }
}

// Fallback for extreme down-scaling factors whose footprint does not fit in shared memory:
// taps are read straight from global memory (L1-cached byte loads).
__global__ void __launch_bounds__(PRE_THREADS) preprocess_direct_kernel(const __grid_constant__ PreprocessParams p, float scale, float shift) {
  const int n = blockIdx.z;
  const uint8_t* __restrict__ src = p.src_tab ? p.src_tab[n] : p.src.p[n];
  const int yo = blockIdx.y * PRE_TY + threadIdx.y;
  const int xo0 = blockIdx.x * PRE_OUT_W + threadIdx.x * 4;
  if (yo >= p.net_h || xo0 >= p.net_w) return;
  const AxisSample sy = axis_sample(yo, p.src_h, p.net_h);
  const uint8_t* r0 = src + (size_t)sy.i0 * p.src_pitch;
  const uint8_t* r1 = src + (size_t)sy.i1 * p.src_pitch;
  const size_t plane = (size_t)p.net_h * p.net_w;
  float* dst = p.dst + (size_t)n * 3 * plane + (size_t)yo * p.net_w + xo0;
  for (int j = 0; j < 4 && xo0 + j < p.net_w; ++j) {
    const AxisSample sx = axis_sample(xo0 + j, p.src_w, p.net_w);
#pragma unroll
    for (int c = 0; c < 3; ++c) {
      const float p00 = (float)__ldg(r0 + 3 * sx.i0 + c), p01 = (float)__ldg(r0 + 3 * sx.i1 + c);
      const float p10 = (float)__ldg(r1 + 3 * sx.i0 + c), p11 = (float)__ldg(r1 + 3 * sx.i1 + c);
      const float top = p00 + sx.f * (p01 - p00);
      const float bot = p10 + sx.f * (p11 - p10);
      dst[c * plane + j] = fmaf(top + sy.f * (bot - top), scale, shift);
    }
  }
}

}  // namespace

cudaError_t launch_preprocess(const PreprocessParams& p, cudaStream_t s) {
  dim3 block(PRE_TX, PRE_TY);
  const float scale = pre::norm_scale(p.inv_div, p.inv_std), shift = pre::norm_shift(p.mean, p.inv_std);
  // Worst-case staged footprint of one block: rows = ceil(TY * sh/nh) + 2; bytes per row =
  // 3 * (ceil(OUT_W * sw/nw) + 2) + 15 (alignment at the front) + 15 (at the end) + 12 (the tap
  // fetch reads three whole words from its first byte), rounded up to 16.
  const long rows = ((long)PRE_ROWS * p.src_h + p.net_h - 1) / p.net_h + 2;
  const long cols = ((long)PRE_OUT_W * p.src_w + p.net_w - 1) / p.net_w + 2;
  const long row_cap = ((3 * cols + 48 + 15) / 16) * 16;
  if (rows * row_cap <= PRE_SMEM_BYTES) {
    dim3 grid((p.net_w + PRE_OUT_W - 1) / PRE_OUT_W, (p.net_h + PRE_ROWS - 1) / PRE_ROWS, p.K);
    preprocess_staged_kernel<<<grid, block, (size_t)(rows * row_cap), s>>>(p, (int)row_cap, scale, shift);
  } else {
    dim3 grid((p.net_w + PRE_OUT_W - 1) / PRE_OUT_W, (p.net_h + PRE_TY - 1) / PRE_TY, p.K);
    preprocess_direct_kernel<<<grid, block, 0, s>>>(p, scale, shift);
  }
  return cudaGetLastError();
}

}  // namespace tt
