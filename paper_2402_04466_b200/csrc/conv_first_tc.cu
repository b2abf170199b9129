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
//
// FUSED form: the preprocessing stage runs inside this kernel, and the resized fp32 image is never written to
// or read from memory.  Four more warps build the patch instead of the TMA unit: bilinear resize +
// normalisation with the expressions of the stand-alone preprocess kernel, so the fp32 values are the same bits.
// They sample from frame rows staged in shared memory (rows are a byte stream: the 16-byte aligned range that
// covers a row's part is staged); the rows of the tile two ahead travel through the same threads' registers
// (128-bit loads issued before a tile is sampled, stored after it), so the memory latency hides behind the sampling.
#include "tt_internal.h"
#include "tc_ptx.cuh"
#include "pre_math.cuh"

namespace tt {
namespace {

using namespace tc;

constexpr int F_STAGES = 3;
constexpr int F_A_BYTES = 128 * 64;                 // 128 rows x 32 bf16
constexpr int F_THREADS = 288;                      // warps 0-3 gather, 4 MMA, 5-8 epilogue
constexpr int F_SAMPLER_WARPS = 8;                  // FUSED: warps 9.. stage frame rows and sample them into the patch buffers
constexpr int F_SAMPLERS = 32 * F_SAMPLER_WARPS;
constexpr int F_THREADS_FUSED = F_THREADS + F_SAMPLERS;
constexpr int F_SRC_STAGES = 3;
constexpr int F_SRC_ROWS = 32;                      // staged rows per tile at most, of up to 16 vectors (256 bytes) each
constexpr int F_SRC_PASSES = F_SRC_ROWS / (F_SAMPLERS / 16);   // a staging pass moves one vector per sampler thread
constexpr int F_SRC_BUDGET = 48 * 1024;             // shared memory the staged frame rows may take
constexpr int F_MAX_TILES = 128;                    // tile columns and tile rows the fused form keeps source ranges for
constexpr int F_TMEM_COLS = 128;                    // two accumulator buffers of up to 64 columns

// Columns of the input patch box: 3 columns in front for alignment, the 15*stride + 3 columns of
// the patch, rounded up to a multiple of 4 (16 bytes).
__host__ __device__ constexpr int box_w(int stride) { return (15 * stride + 3 + 3 + 3) & ~3; }

// Six bytes starting at byte offset `b` of a word-aligned shared buffer: the RGB triples of two
// neighbouring pixels.  lo = bytes b..b+3 (R0 G0 B0 R1), hi = bytes b+4..b+7 (G1 B1 . .).
__device__ __forceinline__ void fetch_pair(const uint32_t* s_words, int b, uint32_t& lo, uint32_t& hi) {
  const int w = b >> 2;
  const uint32_t sh = (uint32_t)(b & 3) * 8u;
  const uint32_t w0 = s_words[w], w1 = s_words[w + 1], w2 = s_words[w + 2];
  lo = __funnelshift_r(w0, w1, sh);
  hi = __funnelshift_r(w1, w2, sh);
}

struct TileAt {
  int tx, ty, img;
};
// tile index -> (tile column, tile row, image) without integer divisions
__device__ __forceinline__ TileAt tile_at(int tile, int tiles_x, int tiles_per_img, float inv_tiles_x, float inv_tiles_per_img) {
  TileAt t;
  t.img = pre::div_by(tile, tiles_per_img, inv_tiles_per_img);
  const int rem = tile - t.img * tiles_per_img;
  t.ty = pre::div_by(rem, tiles_x, inv_tiles_x);
  t.tx = rem - t.ty * tiles_x;
  return t;
}

template <int COUT, int STRIDE, bool FUSED>
__global__ void __launch_bounds__(FUSED ? F_THREADS_FUSED : F_THREADS, FUSED ? 2 : 3)
conv_first_tc_kernel(const __grid_constant__ ConvFirstTcParams p) {
  constexpr int PH = 7 * STRIDE + 3;                         // rows of the input patch of a 16 x 8 output tile
  constexpr int PW = 15 * STRIDE + 3;                        // its columns
  constexpr int BW = box_w(STRIDE);                          // box columns: 3 alignment columns + the patch, rounded up to 4
  constexpr int PATCH_BYTES = 3 * PH * BW * 4;
  constexpr int PATCH_STRIDE = (PATCH_BYTES + 127) & ~127;   // patch buffers stay 128-byte aligned
  extern __shared__ uint8_t smem_raw[];
  uint8_t* s_out = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);  // one output tile, TMA box layout
  uint8_t* s_a = s_out + 128 * COUT * 2;                      // operand ring
  uint8_t* s_b = s_a + F_STAGES * F_A_BYTES;                  // weights in operand layout
  uint8_t* s_patch = s_b + COUT * 64;                         // [2] patches of [3][PH][BW] floats
  uint8_t* s_src = s_patch + 2 * PATCH_STRIDE;                // FUSED: [F_SRC_STAGES] x src_rows_cap rows of src_row_cap bytes
  // FUSED: sample positions of every patch column of every tile column {3 * left source column or -1 outside the image, fx}
  // and of every patch row of every tile row {upper source row or -1, lower source row, fy, -}
  int2* s_xtab = reinterpret_cast<int2*>(s_src + F_SRC_STAGES * p.src_rows_cap * p.src_row_cap);
  int4* s_ytab = reinterpret_cast<int4*>(s_xtab + ((p.tiles_x * PW + 1) & ~1));
  __shared__ __align__(8) uint64_t s_bar[2 * F_STAGES + 8];
  __shared__ const uint8_t* s_frame[TT_MAX_STREAMS];          // the batch's frame pointers
  __shared__ int s_gx[F_MAX_TILES][2], s_gy[F_MAX_TILES][2];  // first and last source column / row under every tile column / row
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  uint64_t* a_full = s_bar;                 // [F_STAGES] 128 gather threads arrive
  uint64_t* a_empty = s_bar + F_STAGES;     // [F_STAGES] MMA commit
  uint64_t* t_full = s_bar + 2 * F_STAGES;  // [2] MMA commit
  uint64_t* t_empty = t_full + 2;           // [2] 4 epilogue warps arrive
  uint64_t* p_full = t_empty + 2;           // [2] patch landed (TMA transaction bytes; FUSED: 128 sampling threads arrive)
  uint64_t* p_empty = p_full + 2;           // [2] FUSED only: 128 gather threads have read the patch
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
      mbar_init(smem_u32(p_full + a), FUSED ? F_SAMPLERS : 1);
      mbar_init(smem_u32(p_empty + a), 128);
    }
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // weights: already packed in the operand layout, COUT * 64 bytes
  for (int i = threadIdx.x; i < COUT * 4; i += F_THREADS)
    reinterpret_cast<uint4*>(s_b)[i] = __ldg(reinterpret_cast<const uint4*>(p.w_packed) + i);
  if (FUSED) {
    if (threadIdx.x < TT_MAX_STREAMS) s_frame[threadIdx.x] = threadIdx.x < p.K ? (p.src_tab ? p.src_tab[threadIdx.x] : p.src.p[threadIdx.x]) : nullptr;
    // the source pixels under the part of every tile column's / tile row's patch that lies inside the resized image
    for (int i = threadIdx.x; i < p.tiles_x + p.tiles_y; i += F_THREADS_FUSED) {
      if (i < p.tiles_x) {
        const int first = max(i * 16 * STRIDE - 1, 0), last = min(i * 16 * STRIDE - 1 + PW - 1, p.W - 1);
        s_gx[i][0] = pre::axis_sample(first, p.src_w, p.W).i0;
        s_gx[i][1] = min(pre::axis_sample(last, p.src_w, p.W).i0 + 1, p.src_w - 1);
      } else {
        const int t = i - p.tiles_x;
        const int first = max(t * 8 * STRIDE - 1, 0), last = min(t * 8 * STRIDE - 1 + PH - 1, p.H - 1);
        s_gy[t][0] = pre::axis_sample(first, p.src_h, p.H).i0;
        s_gy[t][1] = pre::axis_sample(last, p.src_h, p.H).i1;
      }
    }
    const float inv_den_x = 1.0f / (float)(2 * p.W), inv_den_y = 1.0f / (float)(2 * p.H);
    for (int i = threadIdx.x; i < p.tiles_x * PW + p.tiles_y * PH; i += F_THREADS_FUSED) {
      if (i < p.tiles_x * PW) {
        const int t = i / PW, x = t * 16 * STRIDE - 1 + (i - t * PW);
        const bool in = x >= 0 && x < p.W;
        const pre::AxisSample sx = pre::axis_sample_fast(in ? x : 0, p.src_w, p.W, inv_den_x);
        s_xtab[i] = make_int2(in ? 3 * sx.i0 : -1, __float_as_int(sx.f));
      } else {
        const int k = i - p.tiles_x * PW, t = k / PH, y = t * 8 * STRIDE - 1 + (k - t * PH);
        const bool in = y >= 0 && y < p.H;
        const pre::AxisSample sy = pre::axis_sample_fast(in ? y : 0, p.src_h, p.H, inv_den_y);
        s_ytab[k] = make_int4(in ? sy.i0 : -1, sy.i1, __float_as_int(sy.f), 0);
      }
    }
  }
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
  const float inv_tiles_x = 1.0f / (float)p.tiles_x, inv_tiles_per_img = 1.0f / (float)tiles_per_img;

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
    if (!FUSED && ptid == 0) {
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
      if (FUSED) mbar_arrive(smem_u32(p_empty + buf));
      if (named_barrier_or(1, 128, fail)) break;
      if (!FUSED && ptid == 0 && tile + 2 * (int)gridDim.x < total_tiles) {
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
  } else if (FUSED && warp >= 9) {
    // ------------------------------------------------------- frame samplers (preprocessing)
    // Patch entry (c, r, j + 3) is pixel (y_base + r, x_base + j) of the resized image, zero outside it (the
    // convolution's padding).  Thread (g, j) of the first RG * PW owns patch column j and the rows g, g + RG, ...;
    // sample positions come from the tables made at the start of the kernel.
    //
    // Staging: in pass k thread t moves 16-byte vector t % 16 of footprint row t / 16 + (F_SAMPLERS / 16) k.  The
    // stage written while tile i is handled (for tile i + 2) was last read for tile i - 1, which every thread has
    // left behind at tile i's barrier; the same barrier, one tile later, makes the stores visible before they are read.
    constexpr int RG = (F_SAMPLERS / PW) < PH ? (F_SAMPLERS / PW) : PH;
    constexpr int ROWS = (PH + RG - 1) / RG;
    constexpr int VROWS = F_SAMPLERS / 16;
    const int bt = threadIdx.x - F_THREADS;
    const int g = bt / PW, j = bt - g * PW;
    const bool active = g < RG;
    const int stage_bytes = p.src_rows_cap * p.src_row_cap;
    const int vrow = bt >> 4, vcol = bt & 15;
    uint4 vreg[F_SRC_PASSES];
    uint32_t vmask = 0;
    uint32_t st = 0;   // stage of the current tile's rows

    // tile coordinates advance by the grid size without divisions: the step's own decomposition, then two carries
    const TileAt step = tile_at((int)gridDim.x, p.tiles_x, tiles_per_img, inv_tiles_x, inv_tiles_per_img);
    auto advance = [&](TileAt& c) {
      c.tx += step.tx;
      if (c.tx >= p.tiles_x) { c.tx -= p.tiles_x; ++c.ty; }
      c.ty += step.ty;
      if (c.ty >= p.tiles_y) { c.ty -= p.tiles_y; ++c.img; }
      c.img += step.img;
    };
    auto stage_load = [&](const TileAt& t) {
      const int sx_lo = s_gx[t.tx][0], sx_hi = s_gx[t.tx][1], sy_lo = s_gy[t.ty][0], sy_hi = s_gy[t.ty][1];
      const int n_rows = min(sy_hi - sy_lo + 1, p.src_rows_cap);
      const int span = 3 * (sx_hi - sx_lo) + 2;            // a row's bytes run from its first byte to first + span
      uintptr_t g_first = (uintptr_t)s_frame[t.img] + (size_t)(sy_lo + vrow) * p.src_pitch + (size_t)3 * sx_lo;
      vmask = 0;
#pragma unroll
      for (int k = 0; k < F_SRC_PASSES; ++k) {
        const uintptr_t a_vec = (g_first & ~(uintptr_t)15) + (uintptr_t)vcol * 16;
        // the vector starts at or before the row's last byte and inside the staged row
        if (vrow + VROWS * k < n_rows && a_vec <= g_first + span && vcol < (p.src_row_cap >> 4)) {
          vreg[k] = __ldg(reinterpret_cast<const uint4*>(a_vec));
          vmask |= 1u << k;
        }
        g_first += (size_t)VROWS * p.src_pitch;
      }
    };
    auto stage_store = [&](int st) {
      uint8_t* dst = s_src + st * stage_bytes + vrow * p.src_row_cap + vcol * 16;
#pragma unroll
      for (int k = 0; k < F_SRC_PASSES; ++k)
        if (vmask & (1u << k)) *reinterpret_cast<uint4*>(dst + VROWS * k * p.src_row_cap) = vreg[k];
    };

    TileAt cur = tile_at((int)blockIdx.x, p.tiles_x, tiles_per_img, inv_tiles_x, inv_tiles_per_img);
    TileAt ahd = cur;
    // the first two tiles' rows
    if (blockIdx.x < total_tiles) { stage_load(ahd); stage_store(0); }
    advance(ahd);
    if (blockIdx.x + gridDim.x < total_tiles) { stage_load(ahd); stage_store(1); }
    advance(ahd);
    uint32_t it = 0;
    bool fail = false;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++it) {
      const int b = (int)(it & 1u);
      const bool ahead = tile + 2 * (int)gridDim.x < total_tiles;
      if (ahead) stage_load(ahd);
      const int sx_lo = s_gx[cur.tx][0], sy_lo = s_gy[cur.ty][0];
      const int2 xe = active ? s_xtab[cur.tx * PW + j] : make_int2(-1, 0);
      const int xo = xe.x >= 0 ? xe.x - 3 * sx_lo : -1;   // byte offset of the left tap from the first staged column
      const float fx = __int_as_float(xe.y);
      // low bits of the address of the first staged column in source row 0: (that + row * pitch) & 15 is the byte
      // position of the column inside the staged row
      const uint32_t base_lo = (uint32_t)(uintptr_t)s_frame[cur.img] + (uint32_t)(3 * sx_lo);
      const int4* ytab = s_ytab + cur.ty * PH;
      if (!mbar_wait(smem_u32(p_empty + b), ((it >> 1) & 1u) ^ 1u, abort_flag, p.status, 0xA00 + b, wait_limit)) fail = true;
      if (named_barrier_or(4, F_SAMPLERS, fail)) break;
      if (active) {
        const uint32_t* words = reinterpret_cast<const uint32_t*>(s_src + st * stage_bytes);
        float* d = reinterpret_cast<float*>(s_patch + b * PATCH_STRIDE) + j + 3;
#pragma unroll
        for (int k = 0; k < ROWS; ++k) {
          // rows behind the patch's last are computed like the last one and not stored; samples outside the image
          // are computed from the first staged bytes and replaced by zero: no branch but the one on fy
          const int r = g + k * RG, rc = min(r, PH - 1);
          const int4 ye = ytab[rc];
          const float fy = __int_as_float(ye.z);
          const bool in = xo >= 0 && ye.x >= 0;
          const int off0 = (ye.x - sy_lo) * p.src_row_cap + (int)((base_lo + (uint32_t)(ye.x * p.src_pitch)) & 15u) + xo;
          float o0, o1, o2;
          uint32_t lo0, hi0;
          fetch_pair(words, in ? off0 : 0, lo0, hi0);
          if (fy == 0.0f) {
            pre::sample_row(lo0, hi0, fx, p.scale, p.shift, o0, o1, o2);
          } else {
            const int off1 = (ye.y - sy_lo) * p.src_row_cap + (int)((base_lo + (uint32_t)(ye.y * p.src_pitch)) & 15u) + xo;
            uint32_t lo1, hi1;
            fetch_pair(words, in ? off1 : 0, lo1, hi1);
            pre::sample_rows(lo0, hi0, lo1, hi1, fx, fy, p.scale, p.shift, o0, o1, o2);
          }
          if (r < PH) {
            d[r * BW] = in ? o0 : 0.f;
            d[(PH + r) * BW] = in ? o1 : 0.f;
            d[(2 * PH + r) * BW] = in ? o2 : 0.f;
          }
        }
      }
      mbar_arrive(smem_u32(p_full + b));
      if (ahead) stage_store((int)(st == 0 ? 2 : st - 1));   // (it + 2) mod 3
      st = st == 2 ? 0 : st + 1;
      advance(cur);
      advance(ahd);
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
      const TileAt t = tile_at(tile, p.tiles_x, tiles_per_img, inv_tiles_x, inv_tiles_per_img);
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
        tma_store_4d(&p.map_out, smem_u32(s_out), 0, t.tx * 16, t.ty * 8, t.img);
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

template <int COUT, int STRIDE, bool FUSED>
cudaError_t launch_t(const ConvFirstTcParams& p, int sm_count, cudaStream_t s) {
  constexpr int PH = 7 * STRIDE + 3;
  constexpr int SMEM = 1024 + 128 * COUT * 2 + F_STAGES * F_A_BYTES + COUT * 64 + 2 * ((3 * PH * box_w(STRIDE) * 4 + 127) & ~127);
  constexpr int PW = 15 * STRIDE + 3;
  const int smem = SMEM + (FUSED ? F_SRC_STAGES * p.src_rows_cap * p.src_row_cap + 8 * ((p.tiles_x * PW + 1) & ~1) + 16 * p.tiles_y * PH : 0);
  const int total = p.K * p.tiles_x * p.tiles_y;
  const int slots = (FUSED ? 2 : 3) * sm_count;
  const int grid = total < slots ? total : slots;
  auto kern = conv_first_tc_kernel<COUT, STRIDE, FUSED>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, FUSED ? SMEM + F_SRC_BUDGET : SMEM);
  if (e != cudaSuccess) return e;
  return launch_kernel(kern, grid, FUSED ? F_THREADS_FUSED : F_THREADS, smem, s, p, p.pdl != 0);
}

template <bool FUSED>
cudaError_t launch_f(const ConvFirstTcParams& p, int sm_count, cudaStream_t s) {
  if (p.cout == 32 && p.stride == 1) return launch_t<32, 1, FUSED>(p, sm_count, s);
  if (p.cout == 32 && p.stride == 2) return launch_t<32, 2, FUSED>(p, sm_count, s);
  if (p.cout == 64 && p.stride == 1) return launch_t<64, 1, FUSED>(p, sm_count, s);
  if (p.cout == 64 && p.stride == 2) return launch_t<64, 2, FUSED>(p, sm_count, s);
  return cudaErrorInvalidValue;
}

}  // namespace

bool conv_first_tc_supported(int cout) { return cout == 32 || cout == 64; }
int conv_first_tc_box_w(int stride) { return box_w(stride); }

bool conv_first_tc_staging(int stride, int src_w, int src_h, int net_w, int net_h, int* rows_cap, int* row_cap) {
  const int wo = (net_w + stride - 1) / stride, ho = (net_h + stride - 1) / stride;
  if ((wo + 15) / 16 > F_MAX_TILES || (ho + 7) / 8 > F_MAX_TILES) return false;
  // Worst-case footprint of a (7*stride+3) x (15*stride+3) patch: rows = ceil(PH * sh/nh) + 2; bytes per row =
  // 3 * (ceil(PW * sw/nw) + 2) + 15 (alignment at the front) + 15 (at the end) + 12 (the tap fetch reads three
  // whole words from its first byte), rounded up to 16.
  const long ph = 7 * stride + 3, pw = 15 * stride + 3;
  const long rows = (ph * src_h + net_h - 1) / net_h + 2;
  const long cols = (pw * src_w + net_w - 1) / net_w + 2;
  const long cap = ((3 * cols + 48 + 15) / 16) * 16;
  *rows_cap = (int)rows;
  *row_cap = (int)cap;
  if (rows > F_SRC_ROWS || cap > 256) return false;   // what the staging passes of the kernel cover
  // the sample positions are worked out with pre::div_by: numerators below 2^27
  if ((2L * net_w + 1) * src_w >= (1L << 27) || (2L * net_h + 1) * src_h >= (1L << 27)) return false;
  // staged rows plus the tables of sample positions
  const long tables = 8 * (((wo + 15) / 16 * pw + 1) & ~1L) + 16 * ((ho + 7) / 8) * ph;
  return F_SRC_STAGES * rows * cap + tables <= F_SRC_BUDGET;
}

// [cout][27] bf16 bit patterns (row-major, k = c*9 + ky*3 + kx) -> operand layout, cout*32 values
void conv_first_tc_pack(const uint16_t* w_bf16, int cout, uint16_t* packed) {
  for (int n = 0; n < cout; ++n)
    for (int k = 0; k < 32; ++k)
      packed[((n >> 3) * 4 + (k >> 3)) * 64 + (n & 7) * 8 + (k & 7)] = k < 27 ? w_bf16[n * 27 + k] : (uint16_t)0;
}

cudaError_t launch_conv_first_tc(const ConvFirstTcParams& p, int sm_count, cudaStream_t s) {
  return p.fused ? launch_f<true>(p, sm_count, s) : launch_f<false>(p, sm_count, s);
}

}  // namespace tt
