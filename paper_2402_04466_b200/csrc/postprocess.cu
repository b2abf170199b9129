// S4 + S5: mask head (1x1 conv hidden -> tools), sigmoid, threshold, per-tool confidence
// and mask centroid.  HBM-bound: the hidden state is read exactly once.
//
// Pass 1 (post_tile_kernel): a block stages 64 pixels x Ch hidden values in shared memory
// with coalesced 128-bit loads, four threads per pixel form the T dot products, the masks,
// logits and probabilities are written, and the block's partial sums (count, sum x, sum y
// as integers; sum p and per-channel sum h as floats) are written to scratch.
// Pass 2 (post_finalize_kernel): one block per stream adds the partials in a fixed order
// (bitwise reproducible, no float atomics) and forms confidence and centroid.
#include <mutex>

#include "tt_internal.h"

namespace tt {
namespace {

constexpr int PIX = 64;        // pixels per block
constexpr int POST_THREADS = 256;
constexpr int ROW_PAD = 16;    // floats of padding per staged pixel row

__host__ __device__ inline int post_blocks_per_img(int plane) { return (plane + PIX - 1) / PIX; }

struct ScratchLayout {
  size_t off_int, off_p, off_h, total;
};
__host__ __device__ inline ScratchLayout scratch_layout(int K, int plane, int ch, int T) {
  const size_t nb = (size_t)K * post_blocks_per_img(plane);
  ScratchLayout l;
  l.off_int = 0;
  l.off_p = l.off_int + nb * TT_MAX_TOOLS * 4 * sizeof(int32_t);
  l.off_h = l.off_p + nb * TT_MAX_TOOLS * sizeof(float);
  l.total = l.off_h + nb * (size_t)ch * sizeof(float);
  l.total = (l.total + 255) & ~(size_t)255;
  return l;
}

__device__ __forceinline__ float sigmoid_acc(float z) { return 1.0f / (1.0f + expf(-z)); }

__global__ void __launch_bounds__(POST_THREADS) post_tile_kernel(const __grid_constant__ PostParams p) {
  extern __shared__ __align__(16) float s_mem[];
  const int Ch = p.Ch, T = p.T;
  const int row = Ch + ROW_PAD;
  float* s_tile = s_mem;                     // [PIX][row]
  float* s_w = s_tile + PIX * row;           // [T][Ch]
  float* s_red_f = s_w + TT_MAX_TOOLS * Ch;  // [8 warps][T]
  int* s_red_i = reinterpret_cast<int*>(s_red_f + 8 * TT_MAX_TOOLS);  // [8 warps][T][3]

  const int plane = p.Hm * p.Wm;
  const int nb = post_blocks_per_img(plane);
  const int n = blockIdx.x / nb, blk = blockIdx.x % nb;
  const int pix0 = blk * PIX;
  const int npix = min(PIX, plane - pix0);
  const int tid = threadIdx.x;
  const float* h_img = p.h + (size_t)p.idx.v[n] * p.img_stride;

  for (int i = tid; i < T * Ch; i += POST_THREADS) s_w[i] = __ldg(p.head_w + i);

  if (p.channels_last) {
    const int row4 = Ch >> 2;
    const float4* g = reinterpret_cast<const float4*>(h_img + (size_t)pix0 * Ch);
    for (int i = tid; i < npix * row4; i += POST_THREADS) {
      const int pp = i / row4, c4 = i % row4;
      *reinterpret_cast<float4*>(s_tile + pp * row + 4 * c4) = __ldg(g + i);
    }
  } else {
    for (int i = tid; i < Ch * PIX; i += POST_THREADS) {
      const int c = i / PIX, pp = i % PIX;
      if (pp < npix) s_tile[pp * row + c] = __ldg(h_img + (size_t)c * plane + pix0 + pp);
    }
  }
  __syncthreads();

  // --- T dot products per pixel: 4 threads per pixel, 128-bit chunks interleaved by q.
  const int pp = tid >> 2, q = tid & 3;
  float acc[TT_MAX_TOOLS];
#pragma unroll
  for (int t = 0; t < TT_MAX_TOOLS; ++t) acc[t] = 0.0f;
  if (pp < npix) {
    for (int c4 = q; c4 < (Ch >> 2); c4 += 4) {
      const float4 hv = *reinterpret_cast<const float4*>(s_tile + pp * row + 4 * c4);
#pragma unroll
      for (int t = 0; t < TT_MAX_TOOLS; ++t) {
        if (t < T) {
          const float4 wv = *reinterpret_cast<const float4*>(s_w + t * Ch + 4 * c4);
          acc[t] = fmaf(hv.x, wv.x, acc[t]);
          acc[t] = fmaf(hv.y, wv.y, acc[t]);
          acc[t] = fmaf(hv.z, wv.z, acc[t]);
          acc[t] = fmaf(hv.w, wv.w, acc[t]);
        }
      }
    }
  }
#pragma unroll
  for (int t = 0; t < TT_MAX_TOOLS; ++t) {
    acc[t] += __shfl_xor_sync(0xffffffffu, acc[t], 1);
    acc[t] += __shfl_xor_sync(0xffffffffu, acc[t], 2);
  }

  // --- sigmoid, threshold, outputs, per-pixel statistics (lanes with q == 0 own a pixel)
  const bool owner = (q == 0) && (pp < npix);
  const int pix = pix0 + pp;
  const int px = owner ? pix % p.Wm : 0, py = owner ? pix / p.Wm : 0;
  uint32_t bits = 0;
  float prob[TT_MAX_TOOLS];
#pragma unroll
  for (int t = 0; t < TT_MAX_TOOLS; ++t) {
    prob[t] = 0.0f;
    if (t < T && owner) {
      const float z = acc[t] + __ldg(p.head_b + t);
      const float pr = sigmoid_acc(z);
      const bool m = z > p.zthr;
      prob[t] = pr;
      bits |= (m ? 1u : 0u) << t;
      const size_t o = ((size_t)n * T + t) * plane + pix;
      p.logits[o] = z;
      p.probs[o] = pr;
      p.masks[o] = m ? 1 : 0;
    }
  }
  if (owner && p.bits) p.bits[(size_t)n * plane + pix] = (uint8_t)bits;

  // --- block partial sums: shuffle over the 8 pixel owners of a warp, then over 8 warps
  const int warp = tid >> 5, lane = tid & 31;
#pragma unroll
  for (int t = 0; t < TT_MAX_TOOLS; ++t) {
    if (t < T) {
      int cnt = (bits >> t) & 1u;
      int sx = cnt ? px : 0, sy = cnt ? py : 0;
      float sp = prob[t];
#pragma unroll
      for (int d = 4; d < 32; d <<= 1) {
        cnt += __shfl_xor_sync(0xffffffffu, cnt, d);
        sx += __shfl_xor_sync(0xffffffffu, sx, d);
        sy += __shfl_xor_sync(0xffffffffu, sy, d);
        sp += __shfl_xor_sync(0xffffffffu, sp, d);
      }
      if (lane == 0) {
        s_red_i[(warp * TT_MAX_TOOLS + t) * 3 + 0] = cnt;
        s_red_i[(warp * TT_MAX_TOOLS + t) * 3 + 1] = sx;
        s_red_i[(warp * TT_MAX_TOOLS + t) * 3 + 2] = sy;
        s_red_f[warp * TT_MAX_TOOLS + t] = sp;
      }
    }
  }
  __syncthreads();

  const ScratchLayout sl = scratch_layout(p.K, plane, Ch, T);
  uint8_t* scr = reinterpret_cast<uint8_t*>(p.scratch);
  int32_t* part_i = reinterpret_cast<int32_t*>(scr + sl.off_int) + (size_t)blockIdx.x * TT_MAX_TOOLS * 4;
  float* part_p = reinterpret_cast<float*>(scr + sl.off_p) + (size_t)blockIdx.x * TT_MAX_TOOLS;
  float* part_h = reinterpret_cast<float*>(scr + sl.off_h) + (size_t)blockIdx.x * Ch;
  if (tid < T) {
    int cnt = 0, sx = 0, sy = 0;
    float sp = 0.0f;
    for (int w = 0; w < 8; ++w) {
      cnt += s_red_i[(w * TT_MAX_TOOLS + tid) * 3 + 0];
      sx += s_red_i[(w * TT_MAX_TOOLS + tid) * 3 + 1];
      sy += s_red_i[(w * TT_MAX_TOOLS + tid) * 3 + 2];
      sp += s_red_f[w * TT_MAX_TOOLS + tid];
    }
    part_i[tid * 4 + 0] = cnt;
    part_i[tid * 4 + 1] = sx;
    part_i[tid * 4 + 2] = sy;
    part_i[tid * 4 + 3] = 0;
    part_p[tid] = sp;
  }
  if (p.conf_mode == TT_CONF_GAP_LINEAR) {
    for (int c = tid; c < Ch; c += POST_THREADS) {
      float s = 0.0f;
      for (int i = 0; i < npix; ++i) s += s_tile[i * row + c];
      part_h[c] = s;
    }
  }
}

// Channels-last fast path (hidden a multiple of 128): no shared-memory staging of the hidden
// state.  A warp takes 8 of the block's 64 pixels, 4 at a time.  Lane l owns channels
// [128*k + 4*l, +4) of every 128-channel chunk k, so each load instruction of a warp reads 512
// contiguous bytes.  The lane's partial dot products for (4 pixels x 8 tool slots) = 32 values
// are summed across the warp by a transposing butterfly (31 shuffles for all 32 values, fixed
// order), after which lane i holds the logit of pixel i/8, tool i%8.  The pooled hidden state
// accumulates in registers on the way.
template <int NCHUNK>
__global__ void __launch_bounds__(POST_THREADS) post_direct_kernel(const __grid_constant__ PostParams p) {
  constexpr int CH = NCHUNK * 128;
  extern __shared__ __align__(16) float s_dyn[];
  float* s_h = s_dyn;                         // [8 warps][8 pixels][CH]: each warp's pixels, filled by cp.async
  float* s_w = s_h + PIX * CH;                // [TT_MAX_TOOLS][CH]
  float (*s_gapw)[CH] = reinterpret_cast<float (*)[CH]>(s_w + TT_MAX_TOOLS * CH);  // [8][CH]
  __shared__ float s_red_f[8 * TT_MAX_TOOLS];
  __shared__ int s_red_i[8 * TT_MAX_TOOLS * 3];

  const int T = p.T;
  const int plane = p.Hm * p.Wm;
  const int nb = post_blocks_per_img(plane);
  const int n = blockIdx.x / nb, blk = blockIdx.x % nb;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const float* h_img = p.h + (size_t)p.idx.v[n] * p.img_stride;

  // Every lane copies, for each of its warp's 8 pixels, the 16 bytes per 128-channel chunk that it
  // will consume itself: the copies need no registers, are all in flight at once, and a lane only
  // ever reads back what it copied, so waiting for its own copies is the only synchronisation.
  float* my_h = s_h + (size_t)warp * 8 * CH;
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    const int pix = blk * PIX + warp * 8 + q;
#pragma unroll
    for (int k = 0; k < NCHUNK; ++k) {
      float* dst = my_h + q * CH + k * 128 + lane * 4;
      if (pix < plane) {
        const float* src = h_img + (size_t)pix * CH + k * 128 + lane * 4;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
      } else {
        *reinterpret_cast<float4*>(dst) = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
  }
  asm volatile("cp.async.commit_group;" ::: "memory");

  for (int i = tid; i < TT_MAX_TOOLS * CH; i += POST_THREADS) s_w[i] = i < T * CH ? __ldg(p.head_w + i) : 0.0f;
  __syncthreads();
  asm volatile("cp.async.wait_group 0;" ::: "memory");

  const int slot = lane >> 3, t = lane & 7;       // after the butterfly this lane owns (pixel slot, tool)
  const float bias = t < T ? __ldg(p.head_b + t) : 0.0f;
  float gap[NCHUNK * 4];
#pragma unroll
  for (int i = 0; i < NCHUNK * 4; ++i) gap[i] = 0.0f;
  int cnt = 0, sx = 0, sy = 0;
  float sp = 0.0f;

#pragma unroll 1
  for (int it = 0; it < 2; ++it) {
    const int pix0 = blk * PIX + warp * 8 + it * 4;
    float4 hv[4][NCHUNK];
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
      for (int k = 0; k < NCHUNK; ++k)
        hv[q][k] = *reinterpret_cast<const float4*>(my_h + (it * 4 + q) * CH + k * 128 + lane * 4);
    float v[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = 0.0f;
#pragma unroll
    for (int k = 0; k < NCHUNK; ++k) {
#pragma unroll
      for (int tt = 0; tt < TT_MAX_TOOLS; ++tt) {
        const float4 w = *(reinterpret_cast<const float4*>(s_w + tt * CH + k * 128) + lane);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          float a = v[q * 8 + tt];
          a = fmaf(hv[q][k].x, w.x, a);
          a = fmaf(hv[q][k].y, w.y, a);
          a = fmaf(hv[q][k].z, w.z, a);
          a = fmaf(hv[q][k].w, w.w, a);
          v[q * 8 + tt] = a;
        }
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        gap[k * 4 + 0] += hv[q][k].x;
        gap[k * 4 + 1] += hv[q][k].y;
        gap[k * 4 + 2] += hv[q][k].z;
        gap[k * 4 + 3] += hv[q][k].w;
      }
    }
    // transposing butterfly: after the round with offset d a lane keeps the half of its values
    // selected by its own bit d; five rounds leave value index == lane
#pragma unroll
    for (int d = 16, half = 16; d >= 1; d >>= 1, half >>= 1) {
      const bool upper = (lane & d) != 0;
#pragma unroll
      for (int j = 0; j < half; ++j) {
        const float send = upper ? v[j] : v[j + half];
        const float keep = upper ? v[j + half] : v[j];
        v[j] = keep + __shfl_xor_sync(0xffffffffu, send, d);
      }
    }
    const int pix = pix0 + slot;
    const bool live = (pix < plane) && (t < T);
    const float z = v[0] + bias;
    const float pr = sigmoid_acc(z);
    const bool m = live && (z > p.zthr);
    if (live) {
      const size_t o = ((size_t)n * T + t) * plane + pix;
      p.logits[o] = z;
      p.probs[o] = pr;
      p.masks[o] = m ? 1 : 0;
      sp += pr;
    }
    if (m) {
      cnt += 1;
      sx += pix % p.Wm;
      sy += pix / p.Wm;
    }
    const uint32_t ballot = __ballot_sync(0xffffffffu, m);
    if (p.bits && lane < 4 && pix0 + lane < plane) p.bits[(size_t)n * plane + pix0 + lane] = (uint8_t)(ballot >> (8 * lane));
  }

  // pixel slots -> one value per tool (lanes 0..7), then the 8 warps in order
#pragma unroll
  for (int d = 8; d <= 16; d <<= 1) {
    cnt += __shfl_xor_sync(0xffffffffu, cnt, d);
    sx += __shfl_xor_sync(0xffffffffu, sx, d);
    sy += __shfl_xor_sync(0xffffffffu, sy, d);
    sp += __shfl_xor_sync(0xffffffffu, sp, d);
  }
  if (lane < TT_MAX_TOOLS) {
    s_red_i[(warp * TT_MAX_TOOLS + lane) * 3 + 0] = cnt;
    s_red_i[(warp * TT_MAX_TOOLS + lane) * 3 + 1] = sx;
    s_red_i[(warp * TT_MAX_TOOLS + lane) * 3 + 2] = sy;
    s_red_f[warp * TT_MAX_TOOLS + lane] = sp;
  }
  if (p.conf_mode == TT_CONF_GAP_LINEAR) {
#pragma unroll
    for (int k = 0; k < NCHUNK; ++k)
      *(reinterpret_cast<float4*>(&s_gapw[warp][k * 128]) + lane) = make_float4(gap[k * 4], gap[k * 4 + 1], gap[k * 4 + 2], gap[k * 4 + 3]);
  }
  __syncthreads();

  const ScratchLayout sl = scratch_layout(p.K, plane, CH, T);
  uint8_t* scr = reinterpret_cast<uint8_t*>(p.scratch);
  int32_t* part_i = reinterpret_cast<int32_t*>(scr + sl.off_int) + (size_t)blockIdx.x * TT_MAX_TOOLS * 4;
  float* part_p = reinterpret_cast<float*>(scr + sl.off_p) + (size_t)blockIdx.x * TT_MAX_TOOLS;
  float* part_h = reinterpret_cast<float*>(scr + sl.off_h) + (size_t)blockIdx.x * CH;
  if (tid < T) {
    int c = 0, x = 0, y = 0;
    float f = 0.0f;
    for (int w = 0; w < 8; ++w) {
      c += s_red_i[(w * TT_MAX_TOOLS + tid) * 3 + 0];
      x += s_red_i[(w * TT_MAX_TOOLS + tid) * 3 + 1];
      y += s_red_i[(w * TT_MAX_TOOLS + tid) * 3 + 2];
      f += s_red_f[w * TT_MAX_TOOLS + tid];
    }
    part_i[tid * 4 + 0] = c;
    part_i[tid * 4 + 1] = x;
    part_i[tid * 4 + 2] = y;
    part_i[tid * 4 + 3] = 0;
    part_p[tid] = f;
  }
  if (p.conf_mode == TT_CONF_GAP_LINEAR) {
    for (int c = tid; c < CH; c += POST_THREADS) {
      float a = 0.0f;
#pragma unroll
      for (int w = 0; w < 8; ++w) a += s_gapw[w][c];
      part_h[c] = a;
    }
  }
}

// One block of 1024 threads per stream.  Pooled hidden state: the tile blocks are split into
// G = 1024 / Ch interleaved groups, thread (g, c) adds channel c over group g's blocks in
// order, and the G group sums are added in order.  Tool statistics: warp t reduces the partials
// of tool t (lanes stride over the tile blocks, then a fixed shuffle tree).  The order of the
// additions never depends on timing, so results are bitwise reproducible.
constexpr int FIN_THREADS = 1024;

__global__ void __launch_bounds__(FIN_THREADS) post_finalize_kernel(const __grid_constant__ PostParams p) {
  __shared__ float s_part[FIN_THREADS];
  __shared__ float s_gap[512];
  const int n = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int plane = p.Hm * p.Wm, Ch = p.Ch, T = p.T;
  const int nb = post_blocks_per_img(plane);
  const ScratchLayout sl = scratch_layout(p.K, plane, Ch, T);
  const uint8_t* scr = reinterpret_cast<const uint8_t*>(p.scratch);
  const int4* part_i = reinterpret_cast<const int4*>(scr + sl.off_int) + (size_t)n * nb * TT_MAX_TOOLS;
  const float* part_p = reinterpret_cast<const float*>(scr + sl.off_p) + (size_t)n * nb * TT_MAX_TOOLS;
  const float* part_h = reinterpret_cast<const float*>(scr + sl.off_h) + (size_t)n * nb * Ch;
  const float inv_plane = 1.0f / (float)plane;

  if (p.conf_mode == TT_CONF_GAP_LINEAR) {
    const int G = FIN_THREADS / Ch;          // Ch <= 512, so G >= 2
    const int g = tid / Ch, c = tid - g * Ch;
    float s = 0.0f;
    if (g < G) {
#pragma unroll 32
      for (int b = g; b < nb; b += G) s += part_h[(size_t)b * Ch + c];
    }
    s_part[tid] = s;
    __syncthreads();
    if (tid < Ch) {
      float a = 0.0f;
      for (int k = 0; k < G; ++k) a += s_part[k * Ch + tid];
      s_gap[tid] = a * inv_plane;
    }
  }
  __syncthreads();
  if (warp < T) {
    const int t = warp;
    long long cnt = 0, sx = 0, sy = 0;
    float sp = 0.0f;
#pragma unroll 8
    for (int b = lane; b < nb; b += 32) {
      const int4 v = part_i[(size_t)b * TT_MAX_TOOLS + t];
      cnt += v.x; sx += v.y; sy += v.z;
      sp += part_p[(size_t)b * TT_MAX_TOOLS + t];
    }
    float a = 0.0f;
    if (p.conf_mode == TT_CONF_GAP_LINEAR)
      for (int c = lane; c < Ch; c += 32) a = fmaf(__ldg(p.conf_w + t * Ch + c), s_gap[c], a);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      cnt += __shfl_xor_sync(0xffffffffu, cnt, d);
      sx += __shfl_xor_sync(0xffffffffu, sx, d);
      sy += __shfl_xor_sync(0xffffffffu, sy, d);
      sp += __shfl_xor_sync(0xffffffffu, sp, d);
      a += __shfl_xor_sync(0xffffffffu, a, d);
    }
    if (lane == 0) {
      const float conf = p.conf_mode == TT_CONF_GAP_LINEAR ? sigmoid_acc(a + __ldg(p.conf_b + t)) : sp * inv_plane;
      tt_result* r = p.results + n;
      r->conf[t] = conf;
      r->count[t] = (int32_t)cnt;
      r->cx[t] = cnt ? (float)((double)sx / (double)cnt) : -1.0f;
      r->cy[t] = cnt ? (float)((double)sy / (double)cnt) : -1.0f;
    }
  }
}

// Scratch of the entry point that allocates nothing: one fixed array inside the library image.
// Every device that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_post_scratch[TT_POSTPROCESS_STATIC_SCRATCH_BYTES];

size_t post_smem_bytes(int ch) {
  return (size_t)(PIX * (ch + ROW_PAD) + TT_MAX_TOOLS * ch + 8 * TT_MAX_TOOLS) * sizeof(float) +
         (size_t)8 * TT_MAX_TOOLS * 3 * sizeof(int);
}

}  // namespace

size_t post_scratch_bytes(int K, int hm, int wm, int ch, int T) { return scratch_layout(K, hm * wm, ch, T).total; }

// In host code the array's name is only a handle; the device address has to be asked for,
// once per device, with that device current.
cudaError_t post_static_scratch(void** ptr) {
  constexpr int MAX_DEV = 64;
  static void* addr[MAX_DEV] = {};
  static std::mutex mu;
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEV) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lk(mu);
  if (!addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_post_scratch);
    if (e != cudaSuccess) return e;
    addr[dev] = p;
  }
  *ptr = addr[dev];
  return cudaSuccess;
}

cudaError_t post_prepare() {
  cudaError_t e = cudaFuncSetAttribute(post_tile_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)post_smem_bytes(512));
  if (e != cudaSuccess) return e;
  const int per_ch = (PIX + TT_MAX_TOOLS + 8) * (int)sizeof(float);
  e = cudaFuncSetAttribute(post_direct_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, per_ch * 128);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(post_direct_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, per_ch * 256);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(post_direct_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, per_ch * 512);
}

cudaError_t launch_postprocess(const PostParams& p, cudaStream_t s) {
  const int plane = p.Hm * p.Wm;
  const int nb = post_blocks_per_img(plane);
  const bool direct = p.channels_last && (p.Ch == 128 || p.Ch == 256 || p.Ch == 512) &&
                      (((uintptr_t)p.h & 15) == 0) && ((p.img_stride & 3) == 0);
  const size_t dsm = (size_t)(PIX + TT_MAX_TOOLS + 8) * p.Ch * sizeof(float);
  if (direct && p.Ch == 128) post_direct_kernel<1><<<p.K * nb, POST_THREADS, dsm, s>>>(p);
  else if (direct && p.Ch == 256) post_direct_kernel<2><<<p.K * nb, POST_THREADS, dsm, s>>>(p);
  else if (direct) post_direct_kernel<4><<<p.K * nb, POST_THREADS, dsm, s>>>(p);
  else post_tile_kernel<<<p.K * nb, POST_THREADS, post_smem_bytes(p.Ch), s>>>(p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  post_finalize_kernel<<<p.K, FIN_THREADS, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace tt
