// S2/S3 on plain fp32 ALUs: direct 3x3 convolution (pad 1, stride 1 or 2) with fused
// bias + ReLU, or with the fused ConvLSTM gate math.  Used by the fp32 precision path and
// for the first encoder layer of the bf16 path (3 input channels: too thin for a
// tensor-core contraction, HBM/ALU bound).
//
// Block = 32 x 8 output pixels x OCB output channels; 256 threads, one pixel each, OCB
// accumulators per thread.  Input channels are consumed in chunks of CB: the haloed input
// tile and the [CB][9][OCB] weight slice are staged in shared memory.
#include "tt_internal.h"

namespace tt {
namespace {

constexpr int TW = 32, TH = 8, CB = 8;

template <int OCB>
__device__ __forceinline__ void store_bf16_vec(__nv_bfloat16* dst, const float* v, int n_valid) {
  if (n_valid == OCB && ((uintptr_t)dst & 15) == 0) {
#pragma unroll
    for (int i = 0; i < OCB; i += 8) {
      __nv_bfloat162 a = __floats2bfloat162_rn(v[i + 0], v[i + 1]);
      __nv_bfloat162 b = __floats2bfloat162_rn(v[i + 2], v[i + 3]);
      __nv_bfloat162 c = __floats2bfloat162_rn(v[i + 4], v[i + 5]);
      __nv_bfloat162 d = __floats2bfloat162_rn(v[i + 6], v[i + 7]);
      uint4 u;
      u.x = *reinterpret_cast<uint32_t*>(&a);
      u.y = *reinterpret_cast<uint32_t*>(&b);
      u.z = *reinterpret_cast<uint32_t*>(&c);
      u.w = *reinterpret_cast<uint32_t*>(&d);
      *reinterpret_cast<uint4*>(dst + i) = u;
    }
  } else {
    for (int i = 0; i < n_valid; ++i) dst[i] = __float2bfloat16_rn(v[i]);
  }
}

__device__ __forceinline__ float sigmoid_acc(float z) { return 1.0f / (1.0f + expf(-z)); }

template <int STRIDE, int EPI, int OCB>
__global__ void __launch_bounds__(TW* TH) conv3x3_simt_kernel(const __grid_constant__ ConvSimtParams p) {
  constexpr int IN_W = TW * STRIDE + 2;
  constexpr int IN_H = TH * STRIDE + 2;
  constexpr int IN_WP = IN_W + 1;  // pad against bank conflicts
  extern __shared__ __align__(16) float smem[];
  float* s_in = smem;                       // [CB][IN_H][IN_WP]
  float* s_w = smem + CB * IN_H * IN_WP;    // [CB][9][OCB]

  const int tiles_x = (p.Wo + TW - 1) / TW;
  const int tile_x = blockIdx.x % tiles_x, tile_y = blockIdx.x / tiles_x;
  const int grp = blockIdx.y;  // output-channel group
  const int n = blockIdx.z;
  const int tx = threadIdx.x, ty = threadIdx.y;
  const int tid = ty * TW + tx;
  const int xo = tile_x * TW + tx, yo = tile_y * TH + ty;
  const int x_in0 = tile_x * TW * STRIDE - 1, y_in0 = tile_y * TH * STRIDE - 1;
  const int cin = p.C0 + p.C1;
  const size_t in_plane = (size_t)p.H * p.W;
  const float* base0 = p.in0 + (size_t)p.idx0.v[n] * p.img_stride0;
  const float* base1 = p.C1 ? p.in1 + (size_t)p.idx1.v[n] * p.img_stride1 : nullptr;

  float acc[OCB];
#pragma unroll
  for (int i = 0; i < OCB; ++i) acc[i] = 0.0f;

  for (int c0 = 0; c0 < cin; c0 += CB) {
    for (int i = tid; i < CB * IN_H * IN_W; i += TW * TH) {
      const int c = i / (IN_H * IN_W);
      const int r = (i / IN_W) % IN_H;
      const int col = i % IN_W;
      const int ci = c0 + c, yi = y_in0 + r, xi = x_in0 + col;
      float v = 0.0f;
      if (ci < cin && yi >= 0 && yi < p.H && xi >= 0 && xi < p.W) {
        const float* src = ci < p.C0 ? base0 + (size_t)ci * in_plane : base1 + (size_t)(ci - p.C0) * in_plane;
        v = __ldg(src + (size_t)yi * p.W + xi);
        // on the bf16 path every contraction takes bf16 operands, like the tensor-core layers
        if (EPI == EPI_RELU_BF16_NHWC) v = __bfloat162float(__float2bfloat16_rn(v));
      }
      s_in[(c * IN_H + r) * IN_WP + col] = v;
    }
    for (int i = tid; i < CB * 9 * OCB; i += TW * TH) {
      const int c = i / (9 * OCB);
      const int rest = i % (9 * OCB);
      const int ci = c0 + c;
      s_w[i] = ci < cin ? __ldg(p.wgt + ((size_t)ci * 9) * p.cout_packed + (size_t)(rest / OCB) * p.cout_packed +
                                grp * OCB + (rest % OCB))
                        : 0.0f;
    }
    __syncthreads();
#pragma unroll 2
    for (int c = 0; c < CB; ++c) {
      float v[9];
#pragma unroll
      for (int ky = 0; ky < 3; ++ky)
#pragma unroll
        for (int kx = 0; kx < 3; ++kx) v[ky * 3 + kx] = s_in[(c * IN_H + ty * STRIDE + ky) * IN_WP + tx * STRIDE + kx];
      const float4* wv = reinterpret_cast<const float4*>(s_w + c * 9 * OCB);
#pragma unroll
      for (int t = 0; t < 9; ++t) {
#pragma unroll
        for (int o4 = 0; o4 < OCB / 4; ++o4) {
          const float4 w4 = wv[t * (OCB / 4) + o4];
          acc[o4 * 4 + 0] = fmaf(v[t], w4.x, acc[o4 * 4 + 0]);
          acc[o4 * 4 + 1] = fmaf(v[t], w4.y, acc[o4 * 4 + 1]);
          acc[o4 * 4 + 2] = fmaf(v[t], w4.z, acc[o4 * 4 + 2]);
          acc[o4 * 4 + 3] = fmaf(v[t], w4.w, acc[o4 * 4 + 3]);
        }
      }
    }
    __syncthreads();
  }

  if (xo >= p.Wo || yo >= p.Ho) return;
  const size_t out_plane = (size_t)p.Ho * p.Wo;
  const size_t pix = (size_t)yo * p.Wo + xo;
  const float* bias = p.bias + grp * OCB;

  if (EPI == EPI_RELU_F32_NCHW) {
    float* out = reinterpret_cast<float*>(p.out) + (size_t)n * p.out_img_stride;
#pragma unroll
    for (int i = 0; i < OCB; ++i) {
      const int o = grp * OCB + i;
      if (o < p.cout) out[(size_t)o * out_plane + pix] = fmaxf(acc[i] + __ldg(bias + i), 0.0f);
    }
  } else if (EPI == EPI_RELU_BF16_NHWC) {
    __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.out) + (size_t)n * p.out_img_stride;
#pragma unroll
    for (int i = 0; i < OCB; ++i) acc[i] = fmaxf(acc[i] + __ldg(bias + i), 0.0f);
    const int n_valid = min(OCB, p.cout - grp * OCB);
    store_bf16_vec<OCB>(out + pix * p.cout + grp * OCB, acc, n_valid);
  } else {
    // Packed order inside the group: local = gate*(OCB/4) + jj, hidden unit j = grp*(OCB/4) + jj.
    constexpr int HB = OCB / 4;
    float* c_img = p.c_state + (size_t)p.c_idx.v[n] * p.hidden * out_plane;
    float* h_img = p.h_state + (size_t)p.h_out_idx.v[n] * p.hidden * out_plane;
#pragma unroll
    for (int jj = 0; jj < HB; ++jj) {
      const int j = grp * HB + jj;
      if (j >= p.hidden) break;
      const float gi = acc[0 * HB + jj] + __ldg(bias + 0 * HB + jj);
      const float gf = acc[1 * HB + jj] + __ldg(bias + 1 * HB + jj);
      const float gg = acc[2 * HB + jj] + __ldg(bias + 2 * HB + jj);
      const float go = acc[3 * HB + jj] + __ldg(bias + 3 * HB + jj);
      const size_t idx = (size_t)j * out_plane + pix;
      const float c_new = sigmoid_acc(gf) * c_img[idx] + sigmoid_acc(gi) * tanhf(gg);
      c_img[idx] = c_new;
      h_img[idx] = sigmoid_acc(go) * tanhf(c_new);
    }
  }
}

template <int STRIDE, int EPI, int OCB>
cudaError_t launch_one(const ConvSimtParams& p, cudaStream_t s) {
  constexpr int IN_W = TW * STRIDE + 2, IN_H = TH * STRIDE + 2;
  const size_t smem = (size_t)(CB * IN_H * (IN_W + 1) + CB * 9 * OCB) * sizeof(float);
  auto kern = conv3x3_simt_kernel<STRIDE, EPI, OCB>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  const int tiles = ((p.Wo + TW - 1) / TW) * ((p.Ho + TH - 1) / TH);
  dim3 grid(tiles, p.cout_packed / OCB, p.K), block(TW, TH);
  kern<<<grid, block, smem, s>>>(p);
  return cudaGetLastError();
}

template <int STRIDE, int EPI>
cudaError_t launch_ocb(const ConvSimtParams& p, cudaStream_t s) {
  if (p.ocb == 16) return launch_one<STRIDE, EPI, 16>(p, s);
  if (p.ocb == 32) return launch_one<STRIDE, EPI, 32>(p, s);
  return cudaErrorInvalidValue;
}

template <int STRIDE>
cudaError_t launch_epi(const ConvSimtParams& p, cudaStream_t s) {
  switch (p.epilogue) {
    case EPI_RELU_F32_NCHW: return launch_ocb<STRIDE, EPI_RELU_F32_NCHW>(p, s);
    case EPI_RELU_BF16_NHWC: return launch_ocb<STRIDE, EPI_RELU_BF16_NHWC>(p, s);
    case EPI_LSTM_F32_NCHW: return launch_ocb<STRIDE, EPI_LSTM_F32_NCHW>(p, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_conv_simt(const ConvSimtParams& p, cudaStream_t s) {
  if (p.stride == 1) return launch_epi<1>(p, s);
  if (p.stride == 2) return launch_epi<2>(p, s);
  return cudaErrorInvalidValue;
}

}  // namespace tt
