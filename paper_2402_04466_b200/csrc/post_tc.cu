// S4 + S5 of the bf16 path on the tensor cores.
//
// The mask head is a 1x1 convolution, i.e. a GEMM with M = pixels, K = hidden channels and a very
// small N (the tools); the pooled-state confidence sigmoid(W_c . mean_pixels(h') + b_c) equals, by
// linearity, sigmoid(mean_pixels(W_c . h') + b_c), so the confidence head is eight more columns of
// the same product, summed over the pixels afterwards.  One tcgen05.mma tile is 128 pixels x 16
// columns (rows 0..7 of the packed weights: head, rows 8..15: confidence head) x hidden channels,
// read from the bf16 channels-last hidden state that the ConvLSTM epilogue writes for the next
// step's convolution: half the bytes of the fp32 state, fetched by TMA in 128-pixel x 64-channel
// slabs (128-byte swizzle) through a ring of stages.  The stage is bound by HBM: the tensor work
// and the per-pixel epilogue (bias, sigmoid, threshold, outputs) are far below the copy time.
//
// Warp roles (192 threads, three blocks per multiprocessor): warp 0 = TMA producer (one lane),
// warp 1 = tensor-memory allocation and MMA issue (one lane), warps 2..5 = epilogue, one thread per
// pixel of the tile (tensor-memory lane = pixel).  Per tile every epilogue warp reduces its 32
// pixels' statistics (mask count, sum x, sum y by integer warp reductions; probability or
// confidence-head sums in a fixed shuffle order, then to fixed point); lane t keeps tool t's running
// sums in registers.  When the block moves on to another stream or ends, the warps' sums meet in
// shared memory and reach the per-stream accumulators in global memory through integer atomics;
// the block that completes a stream forms its result record and zeroes the accumulators again.  Integer additions commute,
// and the floating-point partial sums are formed over fixed groups of 32 pixels of one stream, so
// a stream's results do not depend on what else shares the launch.
// Every barrier wait is bounded (see tc_ptx.cuh).
#include "tt_internal.h"
#include "tc_ptx.cuh"

namespace tt {
namespace {

using namespace tc;

constexpr int PT_THREADS = 192;
constexpr int PT_STAGES = 3;                      // slabs in flight per block (a tile is hidden / 64 slabs)
constexpr int PT_SLAB_BYTES = 128 * 64 * 2;        // 128 pixels x 64 channels bf16
constexpr int PT_WSLAB_BYTES = 16 * 64 * 2;        // 16 weight rows x 64 channels bf16
constexpr int PT_MAX_SLABS = 8;                    // hidden <= 512
constexpr int PT_ACC = 8 + TT_MAX_TOOLS * 4;       // block accumulators: 8 confidence sums, then [tool][count, sx, sy, sum p]
constexpr float PT_FIX_SCALE = 1073741824.0f;      // 2^30, as in the other postprocess kernels
constexpr float PT_FIX_INV = 1.0f / 1073741824.0f;

__host__ __device__ inline int pt_smem_bytes(int kslabs) {
  return PT_STAGES * PT_SLAB_BYTES + kslabs * PT_WSLAB_BYTES + 1024 /*alignment slack*/ + 512 /*barriers, accumulators*/;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(tmap), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// 1 / (1 + e^-z) from the fast exponential and reciprocal (relative error about 1e-6, far inside
// this path's tolerance)
__device__ __forceinline__ float sigmoid_fast(float z) { return __fdividef(1.0f, 1.0f + __expf(-z)); }

__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

__global__ void __launch_bounds__(PT_THREADS, 3) post_tc_kernel(const __grid_constant__ PostTcParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* s_w = smem + PT_STAGES * PT_SLAB_BYTES;                       // [kslabs] weight slabs, 1024-byte aligned
  uint8_t* tail = s_w + p.kslabs * PT_WSLAB_BYTES;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(tail);                // [PT_STAGES]
  uint64_t* empty_bar = full_bar + PT_STAGES;                            // [PT_STAGES]
  uint64_t* tfull_bar = empty_bar + PT_STAGES;                           // [2]
  uint64_t* tempty_bar = tfull_bar + 2;                                  // [2]
  uint64_t* w_bar = tempty_bar + 2;                                      // [1]
  unsigned long long* s_acc = reinterpret_cast<unsigned long long*>(w_bar + 1);   // [PT_ACC]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_acc + PT_ACC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* s_last = const_cast<int*>(abort_flag) + 1;

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long wait_limit = p.wait_limit;
  const int plane = p.Hm * p.Wm;
  const int tpi = (plane + 127) >> 7;                                    // tiles per image
  const int total_tiles = p.K * tpi;
  const int t_begin = (int)((long long)blockIdx.x * total_tiles / gridDim.x);
  const int t_end = (int)((long long)(blockIdx.x + 1) * total_tiles / gridDim.x);
  const int kslabs = p.kslabs;

  if (threadIdx.x == 0) {
    for (int s = 0; s < PT_STAGES; ++s) {
      mbar_init(smem_u32(full_bar + s), 1);
      mbar_init(smem_u32(empty_bar + s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(tfull_bar + a), 1);
      mbar_init(smem_u32(tempty_bar + a), 4);
    }
    mbar_init(smem_u32(w_bar), 1);
    *abort_flag = 0;
    *s_last = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&p.map_h) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&p.map_w) : "memory");
  }
  if (threadIdx.x >= 64 && threadIdx.x < 64 + PT_ACC) s_acc[threadIdx.x - 64] = 0ull;
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(32u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0 && lane == 0) {
    // ------------------------------------------------------------------------ producer
    // the packed weights first (they are not the previous kernel's output), then the tiles
    mbar_arrive_expect_tx(smem_u32(w_bar), (uint32_t)(kslabs * PT_WSLAB_BYTES));
    for (int k = 0; k < kslabs; ++k) tma_load_2d(smem_u32(s_w + k * PT_WSLAB_BYTES), &p.map_w, smem_u32(w_bar), k * 64, 0);
    pdl_wait();
    uint32_t stage = 0, phase = 0;
    bool ok = true;
    for (int tile = t_begin; tile < t_end && ok; ++tile) {
      const int n = tile / tpi, pix0 = (tile - n * tpi) << 7;
      const int img = p.idx.v[n];
      for (int k = 0; k < kslabs; ++k) {
        ok = mbar_wait(smem_u32(empty_bar + stage), phase ^ 1u, abort_flag, p.status, 0xB00 + (int)stage, wait_limit);
        if (!ok) break;
        const uint32_t fb = smem_u32(full_bar + stage);
        mbar_arrive_expect_tx(fb, PT_SLAB_BYTES);
        // rows past the end of the image are zero-filled by the TMA unit
        tma_load_3d(smem_u32(smem + stage * PT_SLAB_BYTES), &p.map_h, fb, k * 64, pix0, img);
        if (++stage == PT_STAGES) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------------------------------------------------------------- MMA issuer
    constexpr uint32_t IDESC = make_idesc(128, 16);
    uint32_t stage = 0, phase = 0, acc_phase = 0;
    int acc = 0;
    bool ok = mbar_wait(smem_u32(w_bar), 0u, abort_flag, p.status, 0xB10, wait_limit);
    const uint64_t a_desc0 = make_smem_desc(smem_u32(smem), 1024u, 2u);
    const uint64_t b_desc0 = make_smem_desc(smem_u32(s_w), 1024u, 2u);
    for (int tile = t_begin; tile < t_end && ok; ++tile) {
      ok = mbar_wait(smem_u32(tempty_bar + acc), acc_phase ^ 1u, abort_flag, p.status, 0xB20 + acc, wait_limit);
      if (!ok) break;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + (uint32_t)(acc * 16);
      for (int k = 0; k < kslabs; ++k) {
        ok = mbar_wait(smem_u32(full_bar + stage), phase, abort_flag, p.status, 0xB30 + (int)stage, wait_limit);
        if (!ok) break;
        const uint64_t a_desc = a_desc0 + (uint64_t)(stage * (PT_SLAB_BYTES >> 4));
        const uint64_t b_desc = b_desc0 + (uint64_t)(k * (PT_WSLAB_BYTES >> 4));
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          umma_bf16(d_tmem, a_desc + (uint64_t)(2 * kk), b_desc + (uint64_t)(2 * kk), IDESC, (k | kk) != 0 ? 1u : 0u);
        umma_commit(smem_u32(empty_bar + stage));
        if (++stage == PT_STAGES) { stage = 0; phase ^= 1u; }
      }
      if (!ok) break;
      umma_commit(smem_u32(tfull_bar + acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  } else if (warp >= 2) {
    // ------------------------------------------------------------------------ epilogue
    pdl_wait();
    const int et = threadIdx.x - 64;               // 0..127
    const int quarter = warp & 3;                  // tensor-memory lanes 32*quarter .. +31
    const int T = p.T;
    const int Ch = kslabs * 64;
    uint8_t* scr = reinterpret_cast<uint8_t*>(p.scratch);
    float bias[TT_MAX_TOOLS];
#pragma unroll
    for (int t = 0; t < TT_MAX_TOOLS; ++t) bias[t] = t < T ? __ldg(p.head_b + t) : 0.0f;

    // block sums of stream n -> its global accumulators; the block that brings the stream's tile
    // count to tiles-per-image forms the result record and zeroes the accumulators again
    auto flush = [&](int n, int tiles_done) {
      long long* acc = reinterpret_cast<long long*>(scr + 256 + (size_t)n * ((size_t)Ch + TT_MAX_TOOLS * 4) * sizeof(long long));
      unsigned int* counter = reinterpret_cast<unsigned int*>(scr) + n;
      epi_bar();
      if (et < PT_ACC) {
        const unsigned long long v = s_acc[et];
        s_acc[et] = 0ull;
        if (v) atomicAdd(reinterpret_cast<unsigned long long*>(acc + (et < 8 ? et : Ch + et - 8)), v);
      }
      __threadfence();
      epi_bar();
      if (et == 0) *s_last = (atomicAdd(counter, (unsigned int)tiles_done) + (unsigned int)tiles_done == (unsigned int)tpi);
      epi_bar();
      if (*s_last) {
        __threadfence();
        if (et < T) {
          const float inv_plane = 1.0f / (float)plane;
          const long long* st = acc + Ch + et * 4;
          const long long c = __ldcg(st + 0), x = __ldcg(st + 1), y = __ldcg(st + 2), spf = __ldcg(st + 3);
          float conf;
          if (p.conf_mode == TT_CONF_GAP_LINEAR) {
            const float a = (float)((double)__ldcg(acc + et) * (double)PT_FIX_INV) * inv_plane + __ldg(p.conf_b + et);
            conf = 1.0f / (1.0f + expf(-a));
          } else {
            conf = (float)((double)spf * (double)PT_FIX_INV) * inv_plane;
          }
          tt_result* r = p.results + n;
          r->conf[et] = conf;
          r->count[et] = (int32_t)c;
          r->cx[et] = c ? (float)((double)x / (double)c) : -1.0f;
          r->cy[et] = c ? (float)((double)y / (double)c) : -1.0f;
        }
        epi_bar();
        if (et < PT_ACC) acc[et < 8 ? et : Ch + et - 8] = 0;
        if (et == 0) *counter = 0u;
      }
      epi_bar();
    };

    // Lane t < T of every epilogue warp carries tool t's running sums for the stream the block is
    // working on (mask count, sum x, sum y, and the fixed-point sum of probabilities or of the
    // confidence-head column); they meet in the block's shared accumulators only when the block
    // moves on to another stream or ends.
    long long r_cnt = 0, r_sx = 0, r_sy = 0, r_sum = 0;
    auto spill = [&]() {
      if (lane < T) {
        if (p.conf_mode == TT_CONF_MEAN_SIGMOID) atomicAdd(s_acc + 8 + lane * 4 + 3, (unsigned long long)r_sum);
        else atomicAdd(s_acc + lane, (unsigned long long)r_sum);
        atomicAdd(s_acc + 8 + lane * 4 + 0, (unsigned long long)r_cnt);
        atomicAdd(s_acc + 8 + lane * 4 + 1, (unsigned long long)r_sx);
        atomicAdd(s_acc + 8 + lane * 4 + 2, (unsigned long long)r_sy);
      }
      r_cnt = r_sx = r_sy = r_sum = 0;
    };

    uint32_t acc_phase = 0;
    int acc = 0;
    int cur_n = t_begin < t_end ? t_begin / tpi : 0, tiles_done = 0;
    bool ok = true;
    for (int tile = t_begin; tile < t_end; ++tile) {
      const int n = tile / tpi, pix0 = (tile - n * tpi) << 7;
      if (n != cur_n) {
        spill();
        flush(cur_n, tiles_done);
        cur_n = n;
        tiles_done = 0;
      }
      // the four warps agree on whether to go on, so that they meet at the same barriers afterwards
      ok = !named_barrier_or(2, 128, !mbar_wait(smem_u32(tfull_bar + acc), acc_phase, abort_flag, p.status, 0xB40 + acc, wait_limit));
      if (!ok) break;
      tc_fence_after();
      uint32_t v[16];
      tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * 16), v);
      // the accumulator is in registers: hand the buffer back before the arithmetic
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(tempty_bar + acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }

      const int pix = pix0 + quarter * 32 + lane;
      const bool live = pix < plane;
      const int px = live ? pix % p.Wm : 0, py = live ? pix / p.Wm : 0;
      const size_t o0 = (size_t)n * T * plane + pix;     // tool t's element: + t * plane
      uint32_t bits = 0;
#pragma unroll
      for (int t = 0; t < TT_MAX_TOOLS; ++t) {
        if (t < T) {
          const float z = __uint_as_float(v[t]) + bias[t];
          const float pr = sigmoid_fast(z);
          const bool m = live && (z > p.zthr);
          if (live) {
            const size_t o = o0 + (size_t)t * plane;
            p.logits[o] = z;
            p.probs[o] = pr;
            p.masks[o] = m ? 1 : 0;
          }
          bits |= (m ? 1u : 0u) << t;
          const int c1 = __popc(__ballot_sync(0xffffffffu, m));
          const int x1 = __reduce_add_sync(0xffffffffu, m ? px : 0);
          const int y1 = __reduce_add_sync(0xffffffffu, m ? py : 0);
          long long s1;
          if (p.conf_mode == TT_CONF_MEAN_SIGMOID) {
            // probabilities in units of 2^-26: 32 of them fit an unsigned 32-bit sum
            s1 = (long long)__reduce_add_sync(0xffffffffu, live ? __float2uint_rn(pr * 67108864.0f) : 0u) << 4;
          } else {
            // this pixel's share of the confidence head; rows past the image end were zero-filled
            float g = live ? __uint_as_float(v[8 + t]) : 0.0f;
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) g += __shfl_xor_sync(0xffffffffu, g, d);
            s1 = __float2ll_rn(g * PT_FIX_SCALE);
          }
          if (lane == t) { r_cnt += c1; r_sx += x1; r_sy += y1; r_sum += s1; }
        }
      }
      if (p.bits && live) p.bits[(size_t)n * plane + pix] = (uint8_t)bits;
      tiles_done += 1;
    }
    // hand on what the block has gathered (after a wait that ran out the tick's results are void anyway)
    if (ok && t_begin < t_end) {
      spill();
      flush(cur_n, tiles_done);
    }
  }

  // ------------------------------------------------------------------------------- teardown
  __syncwarp();
  if (*abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(16000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(32u) : "memory");
  }
}

}  // namespace

// hidden channels in whole 64-channel slabs; maps of at least one 128-pixel tile
bool post_tc_supported(int ch, int plane) { return ch >= 64 && ch <= 64 * PT_MAX_SLABS && ch % 64 == 0 && plane >= 128; }

cudaError_t launch_post_tc(const PostTcParams& p, int sm_count, cudaStream_t s) {
  if (p.kslabs < 1 || p.kslabs > PT_MAX_SLABS) return cudaErrorInvalidValue;
  const int smem = pt_smem_bytes(p.kslabs);
  cudaError_t e = cudaFuncSetAttribute(post_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, pt_smem_bytes(PT_MAX_SLABS));
  if (e != cudaSuccess) return e;
  const int plane = p.Hm * p.Wm;
  const int total = p.K * ((plane + 127) / 128);
  const int grid = total < 3 * sm_count ? total : 3 * sm_count;
  return launch_kernel(post_tc_kernel, grid, PT_THREADS, (size_t)smem, s, p, p.pdl != 0);
}

}  // namespace tt
