// S1: uint8 RGB interleaved frame -> bilinear resize -> normalise -> planar fp32.
//
// HBM-bound stage.  A block produces a 128 x 8 tile of the output.  The source rows it needs
// are staged in shared memory with 128-bit loads of the aligned byte range that covers them
// (row pitch 3*W is in general not a multiple of 16, so rows are treated as a byte stream and
// indexed from the remainder).  The horizontal sample positions of the tile's 128 columns are
// computed once per block into shared memory.  A thread produces 4 consecutive outputs of one
// row for all three channels: each bilinear tap pair (two neighbouring RGB pixels = 6 bytes) is
// fetched as three 32-bit shared loads plus funnel shifts, bytes become floats by a byte
// permute into the mantissa of 2^23 and one subtraction, and the results leave as three
// 128-bit stores.
#include "tt_internal.h"

namespace tt {
namespace {

constexpr int PRE_TX = 32;          // threads along x; each makes 4 outputs -> 128 outputs per block row
constexpr int PRE_TY = 8;           // output rows per block
constexpr int PRE_OUT_W = PRE_TX * 4;
constexpr int PRE_THREADS = PRE_TX * PRE_TY;
constexpr int PRE_SMEM_BYTES = 44 * 1024;

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

// byte k of x -> float (exact): build 0x4B0000bb = 2^23 + b, subtract 2^23
__device__ __forceinline__ float byte_to_float(uint32_t x, uint32_t selector) {
  return __uint_as_float(__byte_perm(x, 0x4B000000u, selector)) - 8388608.0f;
}

// Six bytes starting at byte offset `b` of a word-aligned shared buffer: the RGB triples of two
// neighbouring pixels.  lo = bytes b..b+3 (R0 G0 B0 R1), hi = bytes b+4..b+7 (G1 B1 . .).
__device__ __forceinline__ void fetch_pair(const uint32_t* s_words, int b, uint32_t& lo, uint32_t& hi) {
  const int w = b >> 2;
  const uint32_t sh = (uint32_t)(b & 3) * 8u;
  const uint32_t w0 = s_words[w], w1 = s_words[w + 1], w2 = s_words[w + 2];
  lo = __funnelshift_r(w0, w1, sh);
  hi = __funnelshift_r(w1, w2, sh);
}

// bilinear blend of the four taps (left/right on the upper row, left/right on the lower row)
// followed by the normalisation as one fused multiply-add
__device__ __forceinline__ float blend(float l0, float r0, float l1, float r1, float fx, float fy, float scale,
                                       float shift) {
  const float top = l0 + fx * (r0 - l0);
  const float bot = l1 + fx * (r1 - l1);
  return fmaf(top + fy * (bot - top), scale, shift);
}

__global__ void __launch_bounds__(PRE_THREADS)
preprocess_staged_kernel(const __grid_constant__ PreprocessParams p, int row_cap_bytes, float scale, float shift) {
  extern __shared__ __align__(16) uint8_t s_mem[];
  __shared__ int s_xoff[PRE_OUT_W];    // 3 * (i0 - sx_lo) per output column of the tile
  __shared__ float s_fx[PRE_OUT_W];
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
  const int vec_cap = row_cap_bytes >> 4;

  if (tid < PRE_OUT_W) {
    const AxisSample sx = axis_sample(min(xo_blk + tid, p.net_w - 1), p.src_w, p.net_w);
    s_xoff[tid] = 3 * (sx.i0 - sx_lo);
    s_fx[tid] = sx.f;
  }
  // Row r of the footprint occupies s_mem[r*row_cap_bytes ...]; byte b of a staged row is the
  // global byte (aligned start of that row's range) + b.  All rows' vectors are spread over the
  // whole block so that every thread has independent loads in flight.
  for (int idx = tid; idx < n_rows * vec_cap; idx += PRE_THREADS) {
    const int r = idx / vec_cap, i = idx - r * vec_cap;
    const size_t g_first = (size_t)(sy_lo + r) * p.src_pitch + 3 * sx_lo;
    const size_t g_last = (size_t)(sy_lo + r) * p.src_pitch + 3 * sx_hi + 2;
    const uintptr_t a_first = ((uintptr_t)src + g_first) & ~(uintptr_t)15;
    const uintptr_t a_end = (((uintptr_t)src + g_last) | 15) + 1;
    const uintptr_t a = a_first + (uintptr_t)i * 16;
    if (a < a_end) reinterpret_cast<uint4*>(s_mem + (size_t)r * row_cap_bytes)[i] = __ldg(reinterpret_cast<const uint4*>(a));
  }
  __syncthreads();

  const int yo = yo_blk + threadIdx.y;
  const int xl = threadIdx.x * 4;
  const int xo0 = xo_blk + xl;
  if (yo >= p.net_h || xo0 >= p.net_w) return;

  const AxisSample sy = axis_sample(yo, p.src_h, p.net_h);
  // byte position of source column sx_lo inside staged rows i0 / i1
  const size_t g0 = (size_t)sy.i0 * p.src_pitch + 3 * sx_lo;
  const size_t g1 = (size_t)sy.i1 * p.src_pitch + 3 * sx_lo;
  const int base0 = (sy.i0 - sy_lo) * row_cap_bytes + (int)(((uintptr_t)src + g0) & 15);
  const int base1 = (sy.i1 - sy_lo) * row_cap_bytes + (int)(((uintptr_t)src + g1) & 15);
  const uint32_t* s_words = reinterpret_cast<const uint32_t*>(s_mem);

  float o0[4], o1[4], o2[4];  // the three channels of the thread's 4 outputs
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int xoff = s_xoff[xl + j];
    const float fx = s_fx[xl + j];
    uint32_t lo0, hi0, lo1, hi1;
    fetch_pair(s_words, base0 + xoff, lo0, hi0);
    fetch_pair(s_words, base1 + xoff, lo1, hi1);
    // channel c of the left pixel is byte c of lo; of the right pixel: byte 3 of lo, bytes 0, 1 of hi
    o0[j] = blend(byte_to_float(lo0, 0x7440), byte_to_float(lo0, 0x7443), byte_to_float(lo1, 0x7440),
                  byte_to_float(lo1, 0x7443), fx, sy.f, scale, shift);
    o1[j] = blend(byte_to_float(lo0, 0x7441), byte_to_float(hi0, 0x7440), byte_to_float(lo1, 0x7441),
                  byte_to_float(hi1, 0x7440), fx, sy.f, scale, shift);
    o2[j] = blend(byte_to_float(lo0, 0x7442), byte_to_float(hi0, 0x7441), byte_to_float(lo1, 0x7442),
                  byte_to_float(hi1, 0x7441), fx, sy.f, scale, shift);
  }

  const size_t plane = (size_t)p.net_h * p.net_w;
  float* d0 = p.dst + (size_t)n * 3 * plane + (size_t)yo * p.net_w + xo0;
  float* d1 = d0 + plane;
  float* d2 = d1 + plane;
  if (((p.net_w & 3) == 0) && (xo0 + 3 < p.net_w)) {
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

// Fallback for extreme down-scaling factors whose footprint does not fit in shared memory:
// taps are read straight from global memory (L1-cached byte loads).
__global__ void __launch_bounds__(PRE_THREADS) preprocess_direct_kernel(const __grid_constant__ PreprocessParams p, float scale, float shift) {
  const int n = blockIdx.z;
  const uint8_t* __restrict__ src = p.src.p[n];
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
  dim3 grid((p.net_w + PRE_OUT_W - 1) / PRE_OUT_W, (p.net_h + PRE_TY - 1) / PRE_TY, p.K);
  // ((v / div) - mean) / std as one fused multiply-add: v * scale + shift
  const float scale = p.inv_div * p.inv_std, shift = -p.mean * p.inv_std;
  // Worst-case staged footprint of one block: rows = ceil(TY * sh/nh) + 2; bytes per row =
  // 3 * (ceil(OUT_W * sw/nw) + 2) + 15 (alignment at the front) + 15 (at the end) + 12 (the tap
  // fetch reads three whole words from its first byte), rounded up to 16.
  const long rows = ((long)PRE_TY * p.src_h + p.net_h - 1) / p.net_h + 2;
  const long cols = ((long)PRE_OUT_W * p.src_w + p.net_w - 1) / p.net_w + 2;
  const long row_cap = ((3 * cols + 48 + 15) / 16) * 16;
  if (rows * row_cap <= PRE_SMEM_BYTES) {
    preprocess_staged_kernel<<<grid, block, (size_t)(rows * row_cap), s>>>(p, (int)row_cap, scale, shift);
  } else {
    preprocess_direct_kernel<<<grid, block, 0, s>>>(p, scale, shift);
  }
  return cudaGetLastError();
}

}  // namespace tt
