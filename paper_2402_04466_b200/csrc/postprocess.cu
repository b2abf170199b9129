// S4 + S5: mask head (1x1 conv hidden -> tools), sigmoid, threshold, per-tool confidence
// and mask centroid.  HBM-bound: the hidden state is read exactly once.
//
// Generic kernel (post_tile_kernel): a block stages 64 pixels x Ch hidden values in shared
// memory with coalesced 128-bit loads, four threads per pixel form the T dot products, and the
// masks, logits and probabilities are written.
// The block's partial sums go into per-stream accumulators with integer atomics (fixed point for
// the float sums: bitwise reproducible whatever the order); the block that finishes a stream last
// forms confidence and centroid and re-zeroes the accumulators.
#include <mutex>

#include "tt_internal.h"

namespace tt {
namespace {

constexpr int PIX = 64;        // pixels per block
constexpr int POST_THREADS = 256;
constexpr int ROW_PAD = 16;    // floats of padding per staged pixel row

__host__ __device__ inline int post_blocks_per_img(int plane) { return (plane + PIX - 1) / PIX; }

// Scratch: per-stream accumulators that the tile blocks add into with integer atomics (the order
// of integer additions does not matter, so results stay bitwise reproducible).  Floating-point
// sums (probabilities, pooled hidden state) are accumulated in fixed point with 30 fractional
// bits.  The block that finishes a stream last turns the accumulators into the result record and
// zeroes them again, so the scratch must be zero before a launch and is zero after it.
constexpr float FIX_SCALE = 1073741824.0f;          // 2^30
constexpr float FIX_INV = 1.0f / 1073741824.0f;

struct ScratchLayout {
  size_t off_counter, off_acc, acc_stride, total;   // acc block per stream: [Ch] pooled sums, then [TT_MAX_TOOLS][4]
};
__host__ __device__ inline ScratchLayout scratch_layout(int K, int plane, int ch, int T) {
  (void)plane; (void)T;
  ScratchLayout l;
  l.off_counter = 0;
  l.off_acc = 256;                                   // TT_MAX_STREAMS counters fit in front
  l.acc_stride = ((size_t)ch + TT_MAX_TOOLS * 4) * sizeof(long long);
  l.total = l.off_acc + (size_t)K * l.acc_stride;
  l.total = (l.total + 255) & ~(size_t)255;
  return l;
}

__device__ __forceinline__ long long to_fixed(float v) { return __float2ll_rn(v * FIX_SCALE); }

__device__ __forceinline__ float sigmoid_acc(float z) { return 1.0f / (1.0f + expf(-z)); }

// Called by every thread of a tile block after the block has added its partial sums into the
// stream's accumulators.  The last block of the stream to arrive finalises: confidence, count,
// centroid -> result record; accumulators and counter back to zero.
__device__ __forceinline__ void finish_stream(const PostParams& p, int n, int nb, int tid) {
  __shared__ float s_gap_fin[512];
  __shared__ int s_last;
  const int plane = p.Hm * p.Wm, Ch = p.Ch, T = p.T;
  const ScratchLayout sl = scratch_layout(p.K, plane, Ch, T);
  uint8_t* scr = reinterpret_cast<uint8_t*>(p.scratch);
  unsigned int* counter = reinterpret_cast<unsigned int*>(scr + sl.off_counter) + n;
  long long* acc = reinterpret_cast<long long*>(scr + sl.off_acc + (size_t)n * sl.acc_stride);
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(counter, 1u) == (unsigned int)(nb - 1));
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const float inv_plane = 1.0f / (float)plane;
  if (p.conf_mode == TT_CONF_GAP_LINEAR) {
    for (int c = tid; c < Ch; c += POST_THREADS) s_gap_fin[c] = (float)((double)__ldcg(acc + c) * (double)FIX_INV) * inv_plane;
  }
  __syncthreads();
  const int warp = tid >> 5, lane = tid & 31;
  if (warp < T) {
    const int t = warp;
    float a = 0.0f;
    if (p.conf_mode == TT_CONF_GAP_LINEAR)
      for (int c = lane; c < Ch; c += 32) a = fmaf(__ldg(p.conf_w + t * Ch + c), s_gap_fin[c], a);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) a += __shfl_xor_sync(0xffffffffu, a, d);
    if (lane == 0) {
      const long long* st = acc + Ch + t * 4;
      const long long cnt = __ldcg(st + 0), sx = __ldcg(st + 1), sy = __ldcg(st + 2), spf = __ldcg(st + 3);
      const float conf = p.conf_mode == TT_CONF_GAP_LINEAR ? sigmoid_acc(a + __ldg(p.conf_b + t))
                                                          : (float)((double)spf * (double)FIX_INV) * inv_plane;
      tt_result* r = p.results + n;
      r->conf[t] = conf;
      r->count[t] = (int32_t)cnt;
      r->cx[t] = cnt ? (float)((double)sx / (double)cnt) : -1.0f;
      r->cy[t] = cnt ? (float)((double)sy / (double)cnt) : -1.0f;
    }
  }
  __syncthreads();
  for (int i = tid; i < Ch + TT_MAX_TOOLS * 4; i += POST_THREADS) acc[i] = 0;
  if (tid == 0) *counter = 0u;
}

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
  long long* sacc = reinterpret_cast<long long*>(reinterpret_cast<uint8_t*>(p.scratch) + sl.off_acc + (size_t)n * sl.acc_stride);
  if (tid < T) {
    int cnt = 0, sx = 0, sy = 0;
    float sp = 0.0f;
    for (int w = 0; w < 8; ++w) {
      cnt += s_red_i[(w * TT_MAX_TOOLS + tid) * 3 + 0];
      sx += s_red_i[(w * TT_MAX_TOOLS + tid) * 3 + 1];
      sy += s_red_i[(w * TT_MAX_TOOLS + tid) * 3 + 2];
      sp += s_red_f[w * TT_MAX_TOOLS + tid];
    }
    unsigned long long* st = reinterpret_cast<unsigned long long*>(sacc + Ch + tid * 4);
    atomicAdd(st + 0, (unsigned long long)(long long)cnt);
    atomicAdd(st + 1, (unsigned long long)(long long)sx);
    atomicAdd(st + 2, (unsigned long long)(long long)sy);
    atomicAdd(st + 3, (unsigned long long)to_fixed(sp));
  }
  if (p.conf_mode == TT_CONF_GAP_LINEAR) {
    for (int c = tid; c < Ch; c += POST_THREADS) {
      float s = 0.0f;
      for (int i = 0; i < npix; ++i) s += s_tile[i * row + c];
      atomicAdd(reinterpret_cast<unsigned long long*>(sacc + c), (unsigned long long)to_fixed(s));
    }
  }
  finish_stream(p, n, nb, tid);
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
  long long* sacc = reinterpret_cast<long long*>(reinterpret_cast<uint8_t*>(p.scratch) + sl.off_acc + (size_t)n * sl.acc_stride);
  if (tid < T) {
    int c = 0, x = 0, y = 0;
    float f = 0.0f;
    for (int w = 0; w < 8; ++w) {
      c += s_red_i[(w * TT_MAX_TOOLS + tid) * 3 + 0];
      x += s_red_i[(w * TT_MAX_TOOLS + tid) * 3 + 1];
      y += s_red_i[(w * TT_MAX_TOOLS + tid) * 3 + 2];
      f += s_red_f[w * TT_MAX_TOOLS + tid];
    }
    unsigned long long* st = reinterpret_cast<unsigned long long*>(sacc + CH + tid * 4);
    atomicAdd(st + 0, (unsigned long long)(long long)c);
    atomicAdd(st + 1, (unsigned long long)(long long)x);
    atomicAdd(st + 2, (unsigned long long)(long long)y);
    atomicAdd(st + 3, (unsigned long long)to_fixed(f));
  }
  if (p.conf_mode == TT_CONF_GAP_LINEAR) {
    for (int c = tid; c < CH; c += POST_THREADS) {
      float a = 0.0f;
#pragma unroll
      for (int w = 0; w < 8; ++w) a += s_gapw[w][c];
      atomicAdd(reinterpret_cast<unsigned long long*>(sacc + c), (unsigned long long)to_fixed(a));
    }
  }
  finish_stream(p, n, nb, tid);
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
  return cudaGetLastError();
}

}  // namespace tt
