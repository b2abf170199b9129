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

// Channels-last fast path (hidden a multiple of 128): a persistent kernel of independent warps.
// Every stream's pixels are cut into units of 32 consecutive pixels (8 rounds of 4).  A block
// takes a contiguous range of the (stream, unit) list and its warps take the units of that range
// in turn (warp w: units w, w + WARPS, ...).  Each warp runs its own ring of bulk-copy stages:
// lane 0 issues one cp.async.bulk per round (the round's 4 x CH floats are contiguous in memory)
// that completes on a warp-private mbarrier, so the ring keeps STAGES rounds per warp in flight
// with no block-wide synchronisation in the streaming phase.  Lane l owns channels
// [128*k + 4*l, +4) of every 128-channel chunk k; its partial dot products for 4 pixels x 8 tool
// slots = 32 values (formed two at a time by packed fp32 FMAs) are summed across the warp by a
// transposing butterfly (31 shuffles, fixed order), after which lane i holds the logit of pixel
// i/8, tool i%8.  Logits are parked in a warp-private shared buffer and written out once per unit,
// lane = pixel, so that every store instruction covers whole 128-byte lines.  Mask statistics and
// the pooled hidden state accumulate in registers and reach the per-stream accumulators through
// block-wide sums in shared memory.  Floating-point sums turn into fixed point at a granularity
// that does not depend on how the work is divided (the pooled state per unit, probabilities per
// pixel), so a stream's results are bit for bit the same whatever else shares the launch.
constexpr int SW_ROUND_PIX = 4;
// Rounds per unit: 8 (32 pixels, whole 128-byte lines per store) on large maps; 2 on small ones,
// where a launch has so few units that the time of one warp's unit sets the kernel's duration.
// A function of the map size alone, so that a stream's sums are grouped the same way whatever
// else shares the launch.
__host__ __device__ inline int sw_unit_rounds(int plane) { return plane >= 8192 ? 8 : 2; }
constexpr int SW_OUT_ROW = 36;              // floats per tool row of the parked logits: (4*t + pixel) % 32 is conflict-free
constexpr int SW_OUT_FLOATS = TT_MAX_TOOLS * SW_OUT_ROW;
constexpr long long SW_WAIT_LIMIT_CYCLES = 4000000000ll;   // about 2 s of SM cycles

template <int NCHUNK>
struct StreamCfg {
  static constexpr int CH = NCHUNK * 128;
  static constexpr int ROUND_BYTES = SW_ROUND_PIX * CH * 4;
  static constexpr int STAGES_RAW = ((NCHUNK <= 2 ? 12 : 16) * 1024) / ROUND_BYTES;   // 12 or 16 KB of copies in flight per warp
  static constexpr int STAGES = STAGES_RAW > 8 ? 8 : STAGES_RAW;
  static constexpr int WARPS = NCHUNK <= 2 ? 16 : 8;       // warps per block (one block per multiprocessor)
  static constexpr int THREADS = WARPS * 32;
  static constexpr int WARP_BYTES = STAGES * ROUND_BYTES + SW_OUT_FLOATS * 4 + 64 /*barriers*/;
  static constexpr int SMEM_BYTES = WARPS * WARP_BYTES + 2 * (CH + TT_MAX_TOOLS * 4) * 8 /*block sums*/ +
                                    TT_MAX_TOOLS * CH * 4 /*head weights*/ + 128 /*alignment slack*/;
  static_assert(SMEM_BYTES + 2560 <= 227 * 1024, "dynamic plus static shared memory must fit one block per multiprocessor");
};

// Two fp32 values in one 64-bit register, and the packed fused multiply-add acc += a * b on both halves.
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void fma2(unsigned long long& acc, unsigned long long a, unsigned long long b) {
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}

__device__ __forceinline__ uint32_t sw_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Bounded wait on a warp-private mbarrier; false when the limit ran out (the caller gives up).
__device__ __forceinline__ bool sw_wait(uint32_t bar, uint32_t parity, long long limit) {
  long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (ok) return true;
    if ((it & 63u) == 63u) {
      const long long now = clock64();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit) return false;
    }
  }
}

// Turns the accumulators of stream n into its result record and zeroes them again; run by one
// whole warp after the stream's last contribution has been added.
__device__ __forceinline__ void finish_stream_warp(const PostParams& p, int n, long long* acc, unsigned int* counter, int lane) {
  const int Ch = p.Ch, T = p.T;
  const float inv_plane = 1.0f / (float)(p.Hm * p.Wm);
  float a[TT_MAX_TOOLS];
#pragma unroll
  for (int tt = 0; tt < TT_MAX_TOOLS; ++tt) a[tt] = 0.0f;
  if (p.conf_mode == TT_CONF_GAP_LINEAR) {
    for (int c = lane; c < Ch; c += 32) {
      const float g = (float)((double)__ldcg(acc + c) * (double)FIX_INV) * inv_plane;
#pragma unroll
      for (int tt = 0; tt < TT_MAX_TOOLS; ++tt)
        if (tt < T) a[tt] = fmaf(__ldg(p.conf_w + tt * Ch + c), g, a[tt]);
    }
#pragma unroll
    for (int tt = 0; tt < TT_MAX_TOOLS; ++tt)
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) a[tt] += __shfl_xor_sync(0xffffffffu, a[tt], d);
  }
#pragma unroll
  for (int tt = 0; tt < TT_MAX_TOOLS; ++tt) {
    if (lane == tt && tt < T) {
      const long long* st = acc + Ch + tt * 4;
      const long long c = __ldcg(st + 0), x = __ldcg(st + 1), y = __ldcg(st + 2), spf = __ldcg(st + 3);
      const float conf = p.conf_mode == TT_CONF_GAP_LINEAR ? sigmoid_acc(a[tt] + __ldg(p.conf_b + tt))
                                                          : (float)((double)spf * (double)FIX_INV) * inv_plane;
      tt_result* r = p.results + n;
      r->conf[tt] = conf;
      r->count[tt] = (int32_t)c;
      r->cx[tt] = c ? (float)((double)x / (double)c) : -1.0f;
      r->cy[tt] = c ? (float)((double)y / (double)c) : -1.0f;
    }
  }
  __syncwarp();
  for (int i = lane; i < Ch + TT_MAX_TOOLS * 4; i += 32) acc[i] = 0;
  if (lane == 0) *counter = 0u;
}

template <int NCHUNK>
__global__ void __launch_bounds__(StreamCfg<NCHUNK>::THREADS, 1) post_stream_kernel(const __grid_constant__ PostParams p) {
  pdl_launch_dependents();
  using Cfg = StreamCfg<NCHUNK>;
  constexpr int CH = Cfg::CH;
  constexpr int STAGES = Cfg::STAGES;
  constexpr int ACC_N = CH + TT_MAX_TOOLS * 4;     // accumulators per stream
  constexpr int SW_WARPS = Cfg::WARPS, SW_THREADS = Cfg::THREADS;
  extern __shared__ uint8_t s_raw[];
  uint8_t* s_base = reinterpret_cast<uint8_t*>(((uintptr_t)s_raw + 127) & ~(uintptr_t)127);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint8_t* my = s_base + (size_t)warp * Cfg::WARP_BYTES;
  float* s_out = reinterpret_cast<float*>(my + STAGES * Cfg::ROUND_BYTES);
  uint64_t* bars = reinterpret_cast<uint64_t*>(my + STAGES * Cfg::ROUND_BYTES + SW_OUT_FLOATS * 4);
  unsigned long long* s_acc = reinterpret_cast<unsigned long long*>(s_base + (size_t)SW_WARPS * Cfg::WARP_BYTES);  // [2][ACC_N]
  // Head weights, four tools per 16-byte entry: entry (k*8 + c*2 + g)*32 + lane holds the weights
  // of tools 4g .. 4g+3 for channel 128*k + 4*lane + c.
  float4* s_w = reinterpret_cast<float4*>(s_acc + 2 * ACC_N);
  __shared__ unsigned int s_rounds[2];             // rounds this block added to its first two streams
  __shared__ int s_last[2];
  __shared__ float s_gap_fin[512];

  const int T = p.T;
  const long long wait_limit = p.wait_limit > 0 ? p.wait_limit : SW_WAIT_LIMIT_CYCLES;
  const int plane = p.Hm * p.Wm;
  const int rpi = (plane + SW_ROUND_PIX - 1) / SW_ROUND_PIX;    // rounds per image
  const int unit_rounds = sw_unit_rounds(plane), unit_pix = unit_rounds * SW_ROUND_PIX;
  const int upi = (plane + unit_pix - 1) / unit_pix;            // units per image
  const int total_units = p.K * upi;
  const int u_begin = (int)((long long)blockIdx.x * total_units / gridDim.x);
  const int u_end = (int)((long long)(blockIdx.x + 1) * total_units / gridDim.x);
  // Sums for the first two streams this block's range touches are combined in shared memory and
  // reach the global accumulators once per block; a range that runs on into further streams
  // (very small grids only) adds to the global accumulators warp by warp.
  const int n_block0 = u_begin / upi;

  for (int i = tid; i < 2 * ACC_N; i += SW_THREADS) s_acc[i] = 0ull;
  if (tid < 2) s_rounds[tid] = 0u;
  for (int u = tid; u < NCHUNK * 8 * 32; u += SW_THREADS) {
    const int l = u & 31, j = (u >> 5) & 7, k = u >> 8;
    const int c = j >> 1, t0 = (j & 1) * 4;
    const int ch = k * 128 + 4 * l + c;
    float w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) w[i] = t0 + i < T ? __ldg(p.head_w + (t0 + i) * CH + ch) : 0.0f;
    s_w[u] = make_float4(w[0], w[1], w[2], w[3]);
  }
  if (lane == 0) {
    for (int s = 0; s < STAGES; ++s)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(sw_smem_u32(bars + s)), "r"(1u) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  pdl_wait();   // head weights and barriers are set up; the hidden state is the previous kernel's output

  const ScratchLayout sl = scratch_layout(p.K, plane, CH, T);
  uint8_t* scr = reinterpret_cast<uint8_t*>(p.scratch);

  if (u_begin + warp < u_end) {
    // lane 0: the next round to copy (unit, stream, first pixel, rounds left in the unit)
    int iss_unit = u_begin + warp, iss_n = iss_unit / upi, iss_pix = (iss_unit % upi) * unit_pix, iss_stage = 0;
    auto issue = [&]() {
      const int npix = min(SW_ROUND_PIX, plane - iss_pix);
      const uint32_t bytes = (uint32_t)npix * CH * 4u;
      const float* src = p.h + (size_t)p.idx.v[iss_n] * p.img_stride + (size_t)iss_pix * CH;
      const uint32_t dst = sw_smem_u32(my + iss_stage * Cfg::ROUND_BYTES);
      const uint32_t bar = sw_smem_u32(bars + iss_stage);
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
      if (++iss_stage == STAGES) iss_stage = 0;
      iss_pix += SW_ROUND_PIX;
      if ((iss_pix & (unit_pix - 1)) == 0 || iss_pix >= plane) {   // unit exhausted: on to this warp's next one
        iss_unit += SW_WARPS;
        iss_n = iss_unit / upi;
        iss_pix = (iss_unit % upi) * unit_pix;
      }
    };
    if (lane == 0)
      for (int i = 0; i < STAGES && iss_unit < u_end; ++i) issue();

    static_assert(SW_ROUND_PIX == 4, "the butterfly below reduces exactly four pixels x eight tools");
    const int slot = lane >> 3, t = lane & 7;       // after the butterfly this lane owns (pixel slot, tool)
    const float bias = t < T ? __ldg(p.head_b + t) : 0.0f;

    long long gap[NCHUNK * 4];                       // pooled hidden state of this lane's channels, fixed point
#pragma unroll
    for (int i = 0; i < NCHUNK * 4; ++i) gap[i] = 0;
    int cnt = 0, sx = 0, sy = 0;                     // lane t < T: statistics of tool t
    long long spf = 0;                               // lane t < T: sum of tool t's probabilities, fixed point
    int stream_rounds = 0;                           // rounds of the current stream done by this warp

    // write out the parked logits of one unit of stream n (pixels pix0 .. pix0 + 4*rounds - 1); lane = pixel
    auto write_unit = [&](int n, int pix0, int rounds) {
      __syncwarp();
      const int pix = pix0 + lane;
      const bool live = lane < rounds * SW_ROUND_PIX && pix < plane;
      const int px = live ? pix % p.Wm : 0, py = live ? pix / p.Wm : 0;
      uint32_t bits = 0;
#pragma unroll
      for (int tt = 0; tt < TT_MAX_TOOLS; ++tt) {
        if (tt < T) {
          const float z = s_out[tt * SW_OUT_ROW + lane];
          const float pr = sigmoid_acc(z);
          const bool m = live && (z > p.zthr);
          if (live) {
            const size_t o = ((size_t)n * T + tt) * plane + pix;
            p.logits[o] = z;
            p.probs[o] = pr;
            p.masks[o] = m ? 1 : 0;
          }
          bits |= (m ? 1u : 0u) << tt;
          const int c1 = __popc(__ballot_sync(0xffffffffu, m));
          const int x1 = __reduce_add_sync(0xffffffffu, m ? px : 0);
          const int y1 = __reduce_add_sync(0xffffffffu, m ? py : 0);
          if (lane == tt) { cnt += c1; sx += x1; sy += y1; }
          if (p.conf_mode == TT_CONF_MEAN_SIGMOID) {
            // probabilities in units of 2^-26: 32 of them fit an unsigned 32-bit sum
            const unsigned q1 = __reduce_add_sync(0xffffffffu, live ? __float2uint_rn(pr * 67108864.0f) : 0u);
            if (lane == tt) spf += (long long)q1 << 4;
          }
        }
      }
      if (p.bits && live) p.bits[(size_t)n * plane + pix] = (uint8_t)bits;
      __syncwarp();
    };

    // hand this warp's sums for stream n on: to the block's shared accumulators, or, beyond the
    // block's first two streams, straight to the global ones (then the warp that completes the
    // stream also forms its result record)
    auto flush_stream = [&](int n) {
      const int bslot = n - n_block0;
      if (bslot < 2) {
        unsigned long long* acc = s_acc + bslot * ACC_N;
        if (lane < T) {
          atomicAdd(acc + CH + lane * 4 + 0, (unsigned long long)(long long)cnt);
          atomicAdd(acc + CH + lane * 4 + 1, (unsigned long long)(long long)sx);
          atomicAdd(acc + CH + lane * 4 + 2, (unsigned long long)(long long)sy);
          atomicAdd(acc + CH + lane * 4 + 3, (unsigned long long)spf);
        }
        if (p.conf_mode == TT_CONF_GAP_LINEAR) {
#pragma unroll
          for (int k = 0; k < NCHUNK; ++k)
#pragma unroll
            for (int j = 0; j < 4; ++j) atomicAdd(acc + k * 128 + lane * 4 + j, (unsigned long long)gap[k * 4 + j]);
        }
        if (lane == 0) atomicAdd(&s_rounds[bslot], (unsigned int)stream_rounds);
      } else {
        long long* acc = reinterpret_cast<long long*>(scr + sl.off_acc + (size_t)n * sl.acc_stride);
        unsigned int* counter = reinterpret_cast<unsigned int*>(scr + sl.off_counter) + n;
        if (lane < T) {
          unsigned long long* st = reinterpret_cast<unsigned long long*>(acc + CH + lane * 4);
          atomicAdd(st + 0, (unsigned long long)(long long)cnt);
          atomicAdd(st + 1, (unsigned long long)(long long)sx);
          atomicAdd(st + 2, (unsigned long long)(long long)sy);
          atomicAdd(st + 3, (unsigned long long)spf);
        }
        if (p.conf_mode == TT_CONF_GAP_LINEAR) {
#pragma unroll
          for (int k = 0; k < NCHUNK; ++k)
#pragma unroll
            for (int j = 0; j < 4; ++j)
              atomicAdd(reinterpret_cast<unsigned long long*>(acc + k * 128 + lane * 4 + j), (unsigned long long)gap[k * 4 + j]);
        }
        __threadfence();
        __syncwarp();
        int last = 0;
        if (lane == 0) last = (atomicAdd(counter, (unsigned int)stream_rounds) + (unsigned int)stream_rounds == (unsigned int)rpi);
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
          __threadfence();
          finish_stream_warp(p, n, acc, counter, lane);
        }
      }
      cnt = 0; sx = 0; sy = 0; spf = 0;
#pragma unroll
      for (int i = 0; i < NCHUNK * 4; ++i) gap[i] = 0;
      stream_rounds = 0;
    };

    int cur_n = (u_begin + warp) / upi;
    int stage = 0;
    uint32_t parity = 0;
    bool ok = true;
#pragma unroll 1
    for (int unit = u_begin + warp; unit < u_end && ok; unit += SW_WARPS) {
      const int n = unit / upi;
      const int unit_pix0 = (unit % upi) * unit_pix;
      const int rounds = min(unit_rounds, (plane - unit_pix0 + SW_ROUND_PIX - 1) / SW_ROUND_PIX);
      if (n != cur_n) {                              // this warp's units run on into the next stream
        flush_stream(cur_n);
        cur_n = n;
      }
      float gsum[NCHUNK * 4];                        // pooled hidden state over this unit
#pragma unroll
      for (int i = 0; i < NCHUNK * 4; ++i) gsum[i] = 0.0f;
#pragma unroll 1
      for (int r = 0; r < rounds; ++r) {
        const int pix0 = unit_pix0 + r * SW_ROUND_PIX;
        const int npix = min(SW_ROUND_PIX, plane - pix0);
        ok = sw_wait(sw_smem_u32(bars + stage), parity, wait_limit);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) {
          // a copy never arrived: record it, give copies still in flight time to land, stop
          if (lane == 0 && p.status) atomicCAS(p.status, 0, 0x700 + stage);
          for (int w = 0; w < 64; ++w) __nanosleep(16000);
          break;
        }
        const float* sh = reinterpret_cast<const float*>(my + stage * Cfg::ROUND_BYTES);
        float4 hv[SW_ROUND_PIX][NCHUNK];
#pragma unroll
        for (int qq = 0; qq < SW_ROUND_PIX; ++qq)
#pragma unroll
          for (int k = 0; k < NCHUNK; ++k)
            hv[qq][k] = qq < npix ? *(reinterpret_cast<const float4*>(sh + qq * CH + k * 128) + lane) : make_float4(0.f, 0.f, 0.f, 0.f);
        __syncwarp();
        if (lane == 0 && iss_unit < u_end) {
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the lanes' reads are done before the refill lands
          issue();
        }
        if (++stage == STAGES) { stage = 0; parity ^= 1u; }

        // partial dot products as packed pairs (tools 2tp, 2tp+1) of one pixel: two fp32 FMAs per instruction
        unsigned long long v2[SW_ROUND_PIX][4];
#pragma unroll
        for (int qq = 0; qq < SW_ROUND_PIX; ++qq)
#pragma unroll
          for (int tp = 0; tp < 4; ++tp) v2[qq][tp] = 0ull;
#pragma unroll
        for (int k = 0; k < NCHUNK; ++k) {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const float4 wa = s_w[(k * 8 + c * 2 + 0) * 32 + lane];    // tools 0..3
            const float4 wb = s_w[(k * 8 + c * 2 + 1) * 32 + lane];    // tools 4..7
            const unsigned long long w01 = pack2(wa.x, wa.y), w23 = pack2(wa.z, wa.w);
            const unsigned long long w45 = pack2(wb.x, wb.y), w67 = pack2(wb.z, wb.w);
#pragma unroll
            for (int qq = 0; qq < SW_ROUND_PIX; ++qq) {
              const float hc = c == 0 ? hv[qq][k].x : c == 1 ? hv[qq][k].y : c == 2 ? hv[qq][k].z : hv[qq][k].w;
              const unsigned long long h2 = pack2(hc, hc);
              fma2(v2[qq][0], h2, w01);
              fma2(v2[qq][1], h2, w23);
              fma2(v2[qq][2], h2, w45);
              fma2(v2[qq][3], h2, w67);
            }
          }
          if (p.conf_mode == TT_CONF_GAP_LINEAR) {
            gsum[k * 4 + 0] += (hv[0][k].x + hv[1][k].x) + (hv[2][k].x + hv[3][k].x);
            gsum[k * 4 + 1] += (hv[0][k].y + hv[1][k].y) + (hv[2][k].y + hv[3][k].y);
            gsum[k * 4 + 2] += (hv[0][k].z + hv[1][k].z) + (hv[2][k].z + hv[3][k].z);
            gsum[k * 4 + 3] += (hv[0][k].w + hv[1][k].w) + (hv[2][k].w + hv[3][k].w);
          }
        }
        float v[32];
#pragma unroll
        for (int qq = 0; qq < SW_ROUND_PIX; ++qq)
#pragma unroll
          for (int tp = 0; tp < 4; ++tp) unpack2(v2[qq][tp], v[qq * 8 + 2 * tp], v[qq * 8 + 2 * tp + 1]);
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
        s_out[t * SW_OUT_ROW + r * SW_ROUND_PIX + slot] = v[0] + bias;
      }
      if (!ok) break;
      stream_rounds += rounds;
      if (p.conf_mode == TT_CONF_GAP_LINEAR) {
#pragma unroll
        for (int i = 0; i < NCHUNK * 4; ++i) gap[i] += to_fixed(gsum[i]);
      }
      write_unit(n, unit_pix0, rounds);
    }
    if (ok && stream_rounds) flush_stream(cur_n);
  }

  // ---- the block's shared sums go to the global accumulators; the block that completes a
  // stream forms its result record
  __syncthreads();
#pragma unroll 1
  for (int bslot = 0; bslot < 2; ++bslot) {
    const unsigned int rounds = s_rounds[bslot];
    if (rounds == 0u) continue;                      // block-uniform
    const int n = n_block0 + bslot;
    long long* acc = reinterpret_cast<long long*>(scr + sl.off_acc + (size_t)n * sl.acc_stride);
    unsigned int* counter = reinterpret_cast<unsigned int*>(scr + sl.off_counter) + n;
    for (int i = tid; i < ACC_N; i += SW_THREADS) {
      const unsigned long long v = s_acc[bslot * ACC_N + i];
      if (v) atomicAdd(reinterpret_cast<unsigned long long*>(acc + i), v);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last[bslot] = (atomicAdd(counter, rounds) + rounds == (unsigned int)rpi);
    __syncthreads();
    if (!s_last[bslot]) continue;                    // block-uniform
    __threadfence();
    // result record of stream n, by the whole block: all loads of a step are in flight together
    const float inv_plane = 1.0f / (float)plane;
    if (p.conf_mode == TT_CONF_GAP_LINEAR)
      for (int c = tid; c < CH; c += SW_THREADS) s_gap_fin[c] = (float)((double)__ldcg(acc + c) * (double)FIX_INV) * inv_plane;
    __syncthreads();
    if (warp < T) {
      const int tt = warp;
      float a = 0.0f;
      if (p.conf_mode == TT_CONF_GAP_LINEAR) {
        float wv[CH / 32];
#pragma unroll
        for (int j = 0; j < CH / 32; ++j) wv[j] = __ldg(p.conf_w + tt * CH + lane + 32 * j);
#pragma unroll
        for (int j = 0; j < CH / 32; ++j) a = fmaf(wv[j], s_gap_fin[lane + 32 * j], a);
      }
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) a += __shfl_xor_sync(0xffffffffu, a, d);
      if (lane == 0) {
        const long long* st = acc + CH + tt * 4;
        const long long c = __ldcg(st + 0), x = __ldcg(st + 1), y = __ldcg(st + 2), spfin = __ldcg(st + 3);
        const float conf = p.conf_mode == TT_CONF_GAP_LINEAR ? sigmoid_acc(a + __ldg(p.conf_b + tt))
                                                            : (float)((double)spfin * (double)FIX_INV) * inv_plane;
        tt_result* r = p.results + n;
        r->conf[tt] = conf;
        r->count[tt] = (int32_t)c;
        r->cx[tt] = c ? (float)((double)x / (double)c) : -1.0f;
        r->cy[tt] = c ? (float)((double)y / (double)c) : -1.0f;
      }
    }
    __syncthreads();
    for (int i = tid; i < ACC_N; i += SW_THREADS) acc[i] = 0;
    if (tid == 0) *counter = 0u;
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

// Multiprocessor count of the current device (looked up once per device).
cudaError_t post_sm_count(int* out) {
  constexpr int MAX_DEV = 64;
  static int count[MAX_DEV] = {};
  static std::mutex mu;
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEV) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lk(mu);
  if (!count[dev]) {
    int v = 0;
    e = cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    count[dev] = v;
  }
  *out = count[dev];
  return cudaSuccess;
}

cudaError_t post_prepare() {
  cudaError_t e = cudaFuncSetAttribute(post_tile_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)post_smem_bytes(512));
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(post_stream_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, StreamCfg<1>::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(post_stream_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, StreamCfg<2>::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(post_stream_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, StreamCfg<4>::SMEM_BYTES);
}

cudaError_t launch_postprocess(const PostParams& p, cudaStream_t s) {
  const int plane = p.Hm * p.Wm;
  const int nb = post_blocks_per_img(plane);
  const bool direct = p.channels_last && (p.Ch == 128 || p.Ch == 256 || p.Ch == 512) &&
                      (((uintptr_t)p.h & 15) == 0) && ((p.img_stride & 3) == 0);
  if (direct) {
    int sms = 0;
    cudaError_t e = post_sm_count(&sms);
    if (e != cudaSuccess) return e;
    // persistent: one block per multiprocessor, fewer when there is less than a unit per warp
    const int unit_pix = sw_unit_rounds(plane) * SW_ROUND_PIX;
    const long long units = (long long)p.K * ((plane + unit_pix - 1) / unit_pix);
    const int warps = p.Ch == 512 ? StreamCfg<4>::WARPS : StreamCfg<1>::WARPS;
    const long long want = (units + warps - 1) / warps;
    const int grid = (int)(want < sms ? want : sms);
    const bool pdl = p.pdl != 0;
    if (p.Ch == 128) return launch_kernel(post_stream_kernel<1>, grid, StreamCfg<1>::THREADS, StreamCfg<1>::SMEM_BYTES, s, p, pdl);
    if (p.Ch == 256) return launch_kernel(post_stream_kernel<2>, grid, StreamCfg<2>::THREADS, StreamCfg<2>::SMEM_BYTES, s, p, pdl);
    return launch_kernel(post_stream_kernel<4>, grid, StreamCfg<4>::THREADS, StreamCfg<4>::SMEM_BYTES, s, p, pdl);
  } else {
    post_tile_kernel<<<p.K * nb, POST_THREADS, post_smem_bytes(p.Ch), s>>>(p);
  }
  return cudaGetLastError();
}

}  // namespace tt
