// First encoder layer of the bf16 path on the tensor cores: 3 input channels (planar fp32 from
// preprocess) -> COUT channels, 3x3, pad 1, stride 1 or 2, bias, ReLU, output bf16 channels-last.
//
// K = 27 (padded to 32) makes the arithmetic free on tcgen05; the layer is then bound by HBM
// (read the fp32 input once, write the bf16 output once).  The A operand cannot come straight
// from TMA (planar fp32 source, 3 channels), so four producer warps build it.  The input patch of
// a tile (all three planes, with halo) arrives in shared memory as one TMA box load; the box starts
// three columns left of the halo so that its first byte is 16-byte aligned, and everything outside
// the image is zero-filled by the TMA unit, which is the convolution's padding.  Two patch buffers
// keep the loads of the next two tiles in flight while the current one is used.  Each producer
// thread picks the 27 taps of one output pixel from
// shared memory, rounds them to bf16 and writes one 64-byte row of the
// [128 pixels][32] operand tile in the no-swizzle K-major core-matrix layout (8 rows x 16 bytes
// contiguous; neighbouring core matrices 128 bytes apart along K, 512 bytes apart along M).
// One warp issues two M128 x COUT x K16 MMAs per tile; four warps run the bias + ReLU epilogue
// from TMEM, write the bf16 tile into shared memory in the swizzled box layout and hand it to one
// TMA tile store (full 128-byte lines to L2 instead of 16-byte pieces per thread; the part of a
// border tile outside the image is clipped by the TMA unit).  The operand ring has 3 stages and the accumulator 2 buffers, so gather, MMA and
// epilogue of different tiles overlap.  All waits are bounded (see tc_ptx.cuh).
#include "tt_internal.h"
#include "tc_ptx.cuh"

namespace tt {
namespace {

using namespace tc;

constexpr int F_STAGES = 3;
constexpr int F_A_BYTES = 128 * 64;                 // 128 rows x 32 bf16
constexpr int F_THREADS = 288;                      // warps 0-3 gather, 4 MMA, 5-8 epilogue
constexpr int F_TMEM_COLS = 128;                    // two accumulator buffers of up to 64 columns

// Columns of the input patch box: 3 columns in front for alignment, the 15*stride + 3 columns of
// the patch, rounded up to a multiple of 4 (16 bytes).
__host__ __device__ constexpr int box_w(int stride) { return (15 * stride + 3 + 3 + 3) & ~3; }

template <int COUT, int STRIDE>
__global__ void __launch_bounds__(F_THREADS, 3) conv_first_tc_kernel(const __grid_constant__ ConvFirstTcParams p) {
  constexpr int PH = 7 * STRIDE + 3;                         // rows of the input patch of a 16 x 8 output tile
  constexpr int BW = box_w(STRIDE);                          // box columns: 3 alignment columns + the patch, rounded up to 4
  constexpr int PATCH_BYTES = 3 * PH * BW * 4;
  constexpr int PATCH_STRIDE = (PATCH_BYTES + 127) & ~127;   // patch buffers stay 128-byte aligned
  extern __shared__ uint8_t smem_raw[];
  uint8_t* s_out = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);  // one output tile, TMA box layout
  uint8_t* s_a = s_out + 128 * COUT * 2;                      // operand ring
  uint8_t* s_b = s_a + F_STAGES * F_A_BYTES;                  // weights in operand layout
  uint8_t* s_patch = s_b + COUT * 64;                         // [2] patches of [3][PH][BW] floats
  __shared__ __align__(8) uint64_t s_bar[2 * F_STAGES + 6];
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  uint64_t* a_full = s_bar;                 // [F_STAGES] 128 gather threads arrive
  uint64_t* a_empty = s_bar + F_STAGES;     // [F_STAGES] MMA commit
  uint64_t* t_full = s_bar + 2 * F_STAGES;  // [2] MMA commit
  uint64_t* t_empty = t_full + 2;           // [2] 4 epilogue warps arrive
  uint64_t* p_full = t_empty + 2;           // [2] patch landed (TMA transaction bytes)
  volatile int* abort_flag = &s_abort;

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long wait_limit = p.wait_limit;
  if (threadIdx.x == 0) {
    for (int s = 0; s < F_STAGES; ++s) {
      mbar_init(smem_u32(a_full + s), 128);
      mbar_init(smem_u32(a_empty + s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(t_full + a), 1);
      mbar_init(smem_u32(t_empty + a), 4);
      mbar_init(smem_u32(p_full + a), 1);
    }
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // weights: already packed in the operand layout, COUT * 64 bytes
  for (int i = threadIdx.x; i < COUT * 4; i += F_THREADS)
    reinterpret_cast<uint4*>(s_b)[i] = __ldg(reinterpret_cast<const uint4*>(p.w_packed) + i);
  fence_proxy_async_smem();
  if (warp == 4) {
    __syncwarp();   // the weight-staging loop may have left the lanes apart; the allocation is warp-collective
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)),
                 "r"((uint32_t)F_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = s_tmem;
  pdl_wait();   // the set-up above read weights only; the input tensor is the previous kernel's output

  const int tiles_per_img = p.tiles_x * p.tiles_y;
  const int total_tiles = p.K * tiles_per_img;

  if (warp < 4) {
    // ------------------------------------------------------------------ operand producers
    const int ptid = threadIdx.x;                 // 0..127
    const int row = ptid;
    const int py = row >> 4, px = row & 15;
    uint8_t* my_row = s_a + (row >> 3) * 512 + (row & 7) * 16;   // + kc * 128 per 16-byte chunk
    uint32_t stage = 0, phase = 0, pphase = 0;
    int buf = 0;

    // one thread starts the box load of a tile's input patch into patch buffer b
    auto fetch_patch = [&](int tile, int b) {
      const int tx = tile % p.tiles_x, ty = (tile / p.tiles_x) % p.tiles_y, img = tile / tiles_per_img;
      const uint32_t bar = smem_u32(p_full + b);
      mbar_arrive_expect_tx(bar, PATCH_BYTES);
      // column tx*16*STRIDE - 1 is the halo; the box starts 3 columns earlier, on a 16-byte boundary
      tma_load_4d(smem_u32(s_patch + b * PATCH_STRIDE), &p.map_in, bar, tx * 16 * STRIDE - 4, ty * 8 * STRIDE - 1, 0, img);
    };

    bool fail = false;   // a bounded wait ran out; the four warps learn of it together at the barrier
    if (ptid == 0) {
      if (blockIdx.x < total_tiles) fetch_patch(blockIdx.x, 0);
      if (blockIdx.x + gridDim.x < total_tiles) fetch_patch(blockIdx.x + gridDim.x, 1);
    }
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
      if (!fail && !mbar_wait(smem_u32(p_full + buf), pphase, abort_flag, p.status, 0x900 + buf, wait_limit)) fail = true;
      const float* patch = reinterpret_cast<const float*>(s_patch + buf * PATCH_STRIDE);
      float v[27];
#pragma unroll
      for (int c = 0; c < 3; ++c)
#pragma unroll
        for (int ky = 0; ky < 3; ++ky)
#pragma unroll
          for (int kx = 0; kx < 3; ++kx)
            v[(c * 3 + ky) * 3 + kx] = patch[(c * PH + py * STRIDE + ky) * BW + px * STRIDE + kx + 3];
      // the four producer warps meet here: everybody has read this patch buffer, it can be refilled
      if (named_barrier_or(1, 128, fail)) break;
      if (ptid == 0 && tile + 2 * (int)gridDim.x < total_tiles) {
        fence_proxy_async_smem();
        fetch_patch(tile + 2 * gridDim.x, buf);
      }
      if (buf) pphase ^= 1u;
      buf ^= 1;
      if (!mbar_wait(smem_u32(a_empty + stage), phase ^ 1u, abort_flag, p.status, 0x500 + (int)stage, wait_limit)) {
        fail = true;
        continue;
      }
      uint8_t* dst = my_row + stage * F_A_BYTES;
      uint4 u;
      u.x = pack_bf16(v[0], v[1]);   u.y = pack_bf16(v[2], v[3]);   u.z = pack_bf16(v[4], v[5]);   u.w = pack_bf16(v[6], v[7]);
      *reinterpret_cast<uint4*>(dst) = u;
      u.x = pack_bf16(v[8], v[9]);   u.y = pack_bf16(v[10], v[11]); u.z = pack_bf16(v[12], v[13]); u.w = pack_bf16(v[14], v[15]);
      *reinterpret_cast<uint4*>(dst + 128) = u;
      u.x = pack_bf16(v[16], v[17]); u.y = pack_bf16(v[18], v[19]); u.z = pack_bf16(v[20], v[21]); u.w = pack_bf16(v[22], v[23]);
      *reinterpret_cast<uint4*>(dst + 256) = u;
      u.x = pack_bf16(v[24], v[25]); u.y = pack_bf16(v[26], 0.f);   u.z = 0u;                      u.w = 0u;
      *reinterpret_cast<uint4*>(dst + 384) = u;
      fence_proxy_async_smem();
      mbar_arrive(smem_u32(a_full + stage));
      if (++stage == F_STAGES) { stage = 0; phase ^= 1u; }
    }
  } else if (warp == 4) {
    // ------------------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t IDESC = make_idesc(128, COUT);
      uint32_t stage = 0, phase = 0, acc_phase = 0;
      int acc = 0;
      for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        if (!mbar_wait(smem_u32(t_empty + acc), acc_phase ^ 1u, abort_flag, p.status, 0x600 + acc, wait_limit)) break;
        if (!mbar_wait(smem_u32(a_full + stage), phase, abort_flag, p.status, 0x700 + (int)stage, wait_limit)) break;
        tc_fence_after();
        const uint32_t a_addr = smem_u32(s_a + stage * F_A_BYTES), b_addr = smem_u32(s_b);
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * 64);
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          // K step k covers the 16-byte chunks 2k and 2k+1 of every row: 256 bytes further on
          const uint64_t a_desc = make_smem_desc_lbo(a_addr + k * 256, 128, 512, 0);
          const uint64_t b_desc = make_smem_desc_lbo(b_addr + k * 256, 128, 512, 0);
          umma_bf16(d_tmem, a_desc, b_desc, IDESC, k);
        }
        umma_commit(smem_u32(a_empty + stage));
        umma_commit(smem_u32(t_full + acc));
        if (++stage == F_STAGES) { stage = 0; phase ^= 1u; }
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // --------------------------------------------------------------------------- epilogue
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;            // tile row = pixel (row / 16, row % 16) of the patch
    const bool leader = (warp == 5 && lane == 0);   // issues and tracks the TMA stores
    constexpr int ROW_BYTES = COUT * 2;             // 128 (128-byte swizzle) or 64 (64-byte swizzle)
    const uint32_t sw = ROW_BYTES == 128 ? (uint32_t)(row & 7) : (uint32_t)((row >> 1) & 3);
    uint8_t* my_out = s_out + row * ROW_BYTES;
    uint32_t acc_phase = 0;
    int acc = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
      const int tx = tile % p.tiles_x, ty = (tile / p.tiles_x) % p.tiles_y, img = tile / tiles_per_img;
      const bool fail = !mbar_wait(smem_u32(t_full + acc), acc_phase, abort_flag, p.status, 0x800 + acc, wait_limit);
      // the previous tile's store must have finished reading s_out before it is overwritten
      if (leader) bulk_wait_group_read0();
      if (named_barrier_or(2, 128, fail)) break;   // all four warps stop together if any wait ran out
      tc_fence_after();
      const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * 64);
#pragma unroll
      for (int ck = 0; ck < COUT / 32; ++ck) {
        uint32_t v[32];
        tmem_ld32(t_addr + (uint32_t)(ck * 32), v);
#pragma unroll
        for (int i = 0; i < 32; i += 8) {
          const float4 ba = __ldg(reinterpret_cast<const float4*>(p.bias + ck * 32 + i));
          const float4 bb = __ldg(reinterpret_cast<const float4*>(p.bias + ck * 32 + i + 4));
          uint4 u;
          u.x = pack_bf16(fmaxf(__uint_as_float(v[i + 0]) + ba.x, 0.f), fmaxf(__uint_as_float(v[i + 1]) + ba.y, 0.f));
          u.y = pack_bf16(fmaxf(__uint_as_float(v[i + 2]) + ba.z, 0.f), fmaxf(__uint_as_float(v[i + 3]) + ba.w, 0.f));
          u.z = pack_bf16(fmaxf(__uint_as_float(v[i + 4]) + bb.x, 0.f), fmaxf(__uint_as_float(v[i + 5]) + bb.y, 0.f));
          u.w = pack_bf16(fmaxf(__uint_as_float(v[i + 6]) + bb.z, 0.f), fmaxf(__uint_as_float(v[i + 7]) + bb.w, 0.f));
          // 16-byte chunk c of this row sits at chunk position c ^ sw of the swizzled box
          const uint32_t c = (uint32_t)(ck * 4 + (i >> 3));
          *reinterpret_cast<uint4*>(my_out + ((c ^ sw) << 4)) = u;
        }
      }
      // the accumulator has been read: hand the TMEM buffer back to the MMA warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(t_empty + acc));
      fence_proxy_async_smem();
      asm volatile("bar.sync 3, 128;" ::: "memory");
      if (leader) {
        tma_store_4d(&p.map_out, smem_u32(s_out), 0, tx * 16, ty * 8, img);
        bulk_commit_group();
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (leader) bulk_wait_group0();
  }

  __syncwarp();
  if (*abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(16000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)F_TMEM_COLS)
                 : "memory");
  }
}

template <int COUT, int STRIDE>
cudaError_t launch_t(const ConvFirstTcParams& p, int grid, cudaStream_t s) {
  constexpr int PH = 7 * STRIDE + 3;
  constexpr int SMEM = 1024 + 128 * COUT * 2 + F_STAGES * F_A_BYTES + COUT * 64 + 2 * ((3 * PH * box_w(STRIDE) * 4 + 127) & ~127);
  auto kern = conv_first_tc_kernel<COUT, STRIDE>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
  if (e != cudaSuccess) return e;
  return launch_kernel(kern, grid, F_THREADS, SMEM, s, p, p.pdl != 0);
}

}  // namespace

bool conv_first_tc_supported(int cout) { return cout == 32 || cout == 64; }
int conv_first_tc_box_w(int stride) { return box_w(stride); }

// [cout][27] bf16 bit patterns (row-major, k = c*9 + ky*3 + kx) -> operand layout, cout*32 values
void conv_first_tc_pack(const uint16_t* w_bf16, int cout, uint16_t* packed) {
  for (int n = 0; n < cout; ++n)
    for (int k = 0; k < 32; ++k)
      packed[((n >> 3) * 4 + (k >> 3)) * 64 + (n & 7) * 8 + (k & 7)] = k < 27 ? w_bf16[n * 27 + k] : (uint16_t)0;
}

cudaError_t launch_conv_first_tc(const ConvFirstTcParams& p, int sm_count, cudaStream_t s) {
  const int total = p.K * p.tiles_x * p.tiles_y;
  const int grid = total < 3 * sm_count ? total : 3 * sm_count;
  if (p.cout == 32 && p.stride == 1) return launch_t<32, 1>(p, grid, s);
  if (p.cout == 32 && p.stride == 2) return launch_t<32, 2>(p, grid, s);
  if (p.cout == 64 && p.stride == 1) return launch_t<64, 1>(p, grid, s);
  if (p.cout == 64 && p.stride == 2) return launch_t<64, 2>(p, grid, s);
  return cudaErrorInvalidValue;
}

}  // namespace tt
