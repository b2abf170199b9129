// Arithmetic of the preprocessing stage (bilinear resize of a uint8 RGB frame + normalisation), shared by
// the stand-alone preprocess kernel and by the first encoder layer when it samples the frame itself.
// Both must give the same fp32 bits, so both evaluate exactly these expressions.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace tt {
namespace pre {

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

// floor(n / d) for 0 <= n < 2^27 and 0 < d, without the integer division sequence: an estimate from the
// reciprocal (inv_d = 1.0f / d, any rounding), then exact correction steps.  The estimate is off by less than
// two for quotients below 2^16.
__device__ __forceinline__ int div_by(int n, int d, float inv_d) {
  int q = __float2int_rz(__int2float_rn(n) * inv_d);
  int r = n - q * d;
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    if (r < 0) { r += d; --q; }
    if (r >= d) { r -= d; ++q; }
  }
  return q;
}

// axis_sample with the quotient from div_by: the same i0, i1 and f, bit for bit (inv_den = 1.0f / (2 * out)).
__device__ __forceinline__ AxisSample axis_sample_fast(int o, int in, int out, float inv_den) {
  int den = 2 * out;
  int num = (2 * o + 1) * in - out;
  int hi = (in - 1) * den;
  num = max(0, min(num, hi));
  AxisSample r;
  r.i0 = div_by(num, den, inv_den);
  r.i1 = min(r.i0 + 1, in - 1);
  r.f = (float)(num - r.i0 * den) / (float)den;
  return r;
}

// byte k of x as the float 2^23 + b (exact)
__device__ __forceinline__ float byte_to_magic(uint32_t x, uint32_t selector) {
  return __uint_as_float(__byte_perm(x, 0x4B000000u, selector));
}

// Bilinear blend of four taps given as 2^23 + byte, then the normalisation as one fused
// multiply-add.  Differences of two such floats are the exact byte differences, so only the
// left taps need the 2^23 removed.
__device__ __forceinline__ float blend_magic(float l0, float r0, float l1, float r1, float fx, float fy, float scale,
                                             float shift) {
  const float top = fmaf(fx, r0 - l0, l0 - 8388608.0f);
  const float bot = fmaf(fx, r1 - l1, l1 - 8388608.0f);
  return fmaf(fmaf(fy, bot - top, top), scale, shift);
}

// The three channels of one output sample whose vertical weight is zero (the sample sits exactly on a
// source row, as on every row of an axis that is not resized): top + 0 * (bot - top) = top, so only
// one source row is needed.  lo = bytes R0 G0 B0 R1 of the tap pair, hi = bytes G1 B1 . .
__device__ __forceinline__ void sample_row(uint32_t lo0, uint32_t hi0, float fx, float scale, float shift, float& o0,
                                           float& o1, float& o2) {
  o0 = fmaf(fmaf(fx, byte_to_magic(lo0, 0x7443) - byte_to_magic(lo0, 0x7440), byte_to_magic(lo0, 0x7440) - 8388608.0f), scale, shift);
  o1 = fmaf(fmaf(fx, byte_to_magic(hi0, 0x7440) - byte_to_magic(lo0, 0x7441), byte_to_magic(lo0, 0x7441) - 8388608.0f), scale, shift);
  o2 = fmaf(fmaf(fx, byte_to_magic(hi0, 0x7441) - byte_to_magic(lo0, 0x7442), byte_to_magic(lo0, 0x7442) - 8388608.0f), scale, shift);
}

// The three channels of one output sample from the tap pairs of two source rows.
// Channel c of the left pixel is byte c of lo; of the right pixel: byte 3 of lo, bytes 0, 1 of hi.
__device__ __forceinline__ void sample_rows(uint32_t lo0, uint32_t hi0, uint32_t lo1, uint32_t hi1, float fx, float fy,
                                            float scale, float shift, float& o0, float& o1, float& o2) {
  o0 = blend_magic(byte_to_magic(lo0, 0x7440), byte_to_magic(lo0, 0x7443), byte_to_magic(lo1, 0x7440),
                   byte_to_magic(lo1, 0x7443), fx, fy, scale, shift);
  o1 = blend_magic(byte_to_magic(lo0, 0x7441), byte_to_magic(hi0, 0x7440), byte_to_magic(lo1, 0x7441),
                   byte_to_magic(hi1, 0x7440), fx, fy, scale, shift);
  o2 = blend_magic(byte_to_magic(lo0, 0x7442), byte_to_magic(hi0, 0x7441), byte_to_magic(lo1, 0x7442),
                   byte_to_magic(hi1, 0x7441), fx, fy, scale, shift);
}

// ((v / div) - mean) / std as one fused multiply-add: v * scale + shift
__host__ __device__ inline float norm_scale(float inv_div, float inv_std) { return inv_div * inv_std; }
__host__ __device__ inline float norm_shift(float mean, float inv_std) { return -mean * inv_std; }

}  // namespace pre
}  // namespace tt
