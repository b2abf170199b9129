// S2/S3 on the 5th-generation tensor cores: 3x3 convolution (pad 1, stride 1 or 2) as an
// implicit GEMM.  M = output pixels (a 16 x 8 patch = 128 rows per tile), N = output
// channels, K = 9 taps x input channels.  No im2col buffer exists anywhere: for every tap
// the producer issues one 4-D TMA box load of the shifted activation patch (NHWC bf16,
// 128-byte or 64-byte swizzle, out-of-range rows and columns zero-filled by the TMA unit,
// which is exactly the convolution's zero padding) and one 2-D TMA load of the matching
// K-slab of the packed weights.  tcgen05.mma accumulates in TMEM; two accumulator buffers
// let the epilogue of tile i overlap the main loop of tile i+1.  The epilogue reads TMEM
// with tcgen05.ld and applies bias + ReLU (encoder) or the whole ConvLSTM gate math
// (sigmoid/tanh, c' = f*c + i*g, h' = o*tanh(c')) so gate pre-activations never reach HBM.
//
// Stride-2 layers read four "parity views" of their input (even/odd rows x even/odd
// columns), each an ordinary tiled tensor map with doubled strides, so every tap is again
// a dense box.
//
// Warp roles (384 threads): warp 0 and warps 10, 11 = TMA producers (one lane each; producer j
// issues the loads of pipeline iterations j, j + n_prod, ... so that the cost of issuing a copy is
// spread over several instruction streams), warp 1 = TMEM allocation and MMA issue (one lane),
// warps 2..9 = epilogue (TMEM lane quarter = warp index mod 4, two warps per quarter, each taking
// half of the tile's columns).  The single threads that issue copies and MMAs are latency-bound
// instruction streams, so the roles are laid out so that each of them sits on a different warp
// scheduler (warp index mod 4).  What a pipeline iteration loads (tensor map, channel offset, tap
// shift) is the same for every tile, so it is tabulated in shared memory once per block.
// Every mbarrier wait is bounded: when a wait runs out the kernel records a status code,
// raises a block-wide abort flag, lets copies in flight land, frees its TMEM and returns.
#include "tt_internal.h"
#include "tc_ptx.cuh"

namespace tt {
namespace {

using namespace tc;

constexpr int BLOCK_M = 128;
constexpr int PATCH_W = 16, PATCH_H = 8;
constexpr int UMMA_K = 16;
constexpr int EPI_WARPS = 8;                       // two per TMEM lane quarter, each takes half of the columns
constexpr int N_PROD = 3;                          // producer warps: 0, 10, 11
constexpr int MMA_WARP = 1;
constexpr int EPI_WARP0 = 2;
constexpr int TC_THREADS = 32 * (2 + EPI_WARPS + (N_PROD - 1));
constexpr int MAX_K_ITERS = 9 * 16;                // 9 taps x up to 16 channel slabs

// PAIR: two CTAs of a cluster work on two neighbouring M-tiles with one MMA of 256 rows
// (cta_group::2).  Each CTA then stages its own activation box and only its own half of the
// weight slab's rows, so a stage holds a third less and the ring is half as deep again.
// CTAS: blocks per multiprocessor the configuration is sized for.  The small encoder layers are
// bound by the latency of their single-thread issue chains, not by bandwidth or arithmetic: two
// blocks per multiprocessor (half the ring each) run two such chains side by side.
template <int BLOCK_N, int SLAB_C, bool PAIR = false, int CTAS = 1>
struct TcCfg {
  static constexpr int A_BYTES = BLOCK_M * SLAB_C * 2;
  static constexpr int B_ROWS = PAIR ? BLOCK_N / 2 : BLOCK_N;     // weight rows staged by one CTA
  static constexpr int B_BYTES = B_ROWS * SLAB_C * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES_RAW = ((CTAS == 2 ? 104 : 192) * 1024) / STAGE_BYTES;
  static constexpr int STAGES = STAGES_RAW > 8 ? 8 : STAGES_RAW;
  static constexpr int TMEM_COLS = 2 * BLOCK_N < 32 ? 32 : 2 * BLOCK_N;
  static constexpr int BAR_BYTES = 256;
  static constexpr int TAB_BYTES = MAX_K_ITERS * 16 + 4 * TT_MAX_STREAMS * 4;   // iteration table + image index maps
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + BAR_BYTES + TAB_BYTES + 1024 /*alignment slack*/;
  // Halo mode (stride 1, 64-channel slabs): the activation ring holds haloed patches, one per
  // channel slab: 18 rows x 16 pixels x 64 channels for an 8 x 16 output patch (10 of the 16
  // columns are needed; a row pitch of 16 pixels = 2048 bytes keeps every 8-pixel operand group
  // of every tap at the same phase of the 1024-byte swizzle pattern).  The weight ring holds one
  // [BLOCK_N][64] slab per tap.
  static constexpr int HALO_PITCH = 10, HALO_ROWS = 18;
  static constexpr int HALO_A_BYTES = (HALO_ROWS * HALO_PITCH * SLAB_C * 2 + 1023) / 1024 * 1024;   // 23040 -> 23552
  static constexpr int HALO_A_TX = HALO_ROWS * HALO_PITCH * SLAB_C * 2;
  static constexpr int HALO_A_STAGES = 2;
  static constexpr int HALO_B_RAW = (210 * 1024 - HALO_A_STAGES * HALO_A_BYTES) / B_BYTES;
  static constexpr int HALO_B_STAGES = HALO_B_RAW > 8 ? 8 : HALO_B_RAW;
  static constexpr int HALO_SMEM_BYTES = HALO_B_STAGES * B_BYTES + HALO_A_STAGES * HALO_A_BYTES + BAR_BYTES + TAB_BYTES + 1024;
  static_assert(STAGES >= N_PROD, "every producer needs a stage of its own");
  static_assert((TMEM_COLS & (TMEM_COLS - 1)) == 0 && TMEM_COLS <= 512, "TMEM columns must be a power of two <= 512");
  static_assert(A_BYTES % 1024 == 0 && B_BYTES % 1024 == 0, "operand tiles must keep 1024-byte alignment");
};

// One special-function instruction each: tanh.approx (relative error about 2^-11, far inside
// the bf16 path's tolerance) and sigmoid(z) = 0.5 + 0.5 * tanh(z / 2).
__device__ __forceinline__ float fast_tanh(float z) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(z));
  return y;
}
__device__ __forceinline__ float fast_sigmoid(float z) { return fmaf(0.5f, fast_tanh(0.5f * z), 0.5f); }


// ------------------------------------------------------------------------------------ kernel
// WRES (weights resident): a layer whose whole packed weight matrix is at most WRES_BYTES fetches it once per
// block, before it waits for the previous kernel, and the ring then holds activation boxes only: one copy per
// iteration instead of two, and eight stages.
constexpr int WRES_BYTES = 40 * 1024;
constexpr int WRES_STAGES = 8;

template <int BLOCK_N, int SLAB_C, int EPI, bool PAIR, int CTAS = 1, bool HALO = false, bool WRES = false>
__global__ void __launch_bounds__(TC_THREADS, CTAS) conv_tc_kernel(const __grid_constant__ ConvTcParams p) {
  using Cfg = TcCfg<BLOCK_N, SLAB_C, PAIR, CTAS>;
  static_assert(!WRES || (!HALO && !PAIR && WRES_STAGES * Cfg::A_BYTES + WRES_BYTES + Cfg::BAR_BYTES + Cfg::TAB_BYTES + 1024 <= 112 * 1024),
                "resident weights: single-CTA tap-box form that still fits twice on a multiprocessor");
  static_assert(!HALO || (SLAB_C == 64 && !PAIR && CTAS == 1), "halo mode: 64-channel slabs, one block per multiprocessor");
  constexpr int PW = HALO ? 8 : PATCH_W;           // output patch: 8 x 16 pixels in halo mode, 16 x 8 otherwise
  constexpr int PH = HALO ? 16 : PATCH_H;
  static_assert(CTAS == 1 || (CTAS == 2 && !PAIR && Cfg::TMEM_COLS <= 256 && Cfg::SMEM_BYTES <= 112 * 1024),
                "two blocks per multiprocessor must fit its shared and tensor memory");
  // ring depth: stages of (A + B); in halo mode the weight ring, with the activation ring of its own behind it
  constexpr int STAGES = HALO ? Cfg::HALO_B_STAGES : WRES ? WRES_STAGES : Cfg::STAGES;
  constexpr int RING_STRIDE = HALO ? Cfg::B_BYTES : WRES ? Cfg::A_BYTES : Cfg::STAGE_BYTES;
  constexpr int A_STAGES = Cfg::HALO_A_STAGES;
  constexpr uint32_t LAYOUT = SLAB_C == 64 ? 2u : 4u;
  constexpr uint32_t SBO = 8u * SLAB_C * 2u;
  constexpr uint32_t IDESC = make_idesc(PAIR ? 2 * BLOCK_M : BLOCK_M, BLOCK_N);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* smem_a = smem + STAGES * RING_STRIDE;               // halo mode: activation ring behind the weight ring; WRES: the weights
  uint8_t* bar_mem = smem_a + (HALO ? A_STAGES * Cfg::HALO_A_BYTES : WRES ? WRES_BYTES : 0);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(bar_mem);   // [STAGES]
  uint64_t* empty_bar = full_bar + STAGES;                     // [STAGES]
  uint64_t* tfull_bar = empty_bar + STAGES;                    // [2]
  uint64_t* tempty_bar = tfull_bar + 2;                        // [2]
  uint64_t* afull_bar = tempty_bar + 2;                        // [2] halo mode: patch landed
  uint64_t* aempty_bar = afull_bar + 2;                        // [2] halo mode: all nine taps have read the patch
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aempty_bar + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int4* s_tab = reinterpret_cast<int4*>(bar_mem + Cfg::BAR_BYTES);            // [k_iters] {map slot, channel offset, dx, dy}
  int* s_img = reinterpret_cast<int*>(s_tab + MAX_K_ITERS);                   // [4][TT_MAX_STREAMS]: img0, img1, c_idx, h_out_idx

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long wait_limit = p.wait_limit;
  const int tiles_per_img = p.tiles_x * p.tiles_y;
  // Units of work: a tile (M-tile x N-tile), or for a CTA pair two neighbouring M-tiles x N-tile.
  // `worker` counts CTAs (or pairs), `rank` is this CTA's place in its pair, `m_tiles` the M-tiles.
  const int m_tiles = p.K * tiles_per_img;
  const int total_tiles = (PAIR ? (m_tiles + 1) / 2 : m_tiles) * p.n_tiles_n;
  const int rank = PAIR ? (int)cluster_ctarank() : 0;
  const int worker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int n_workers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  const int slabs_per_tap = p.slabs[0] + (p.n_src > 1 ? p.slabs[1] : 0);
  const int k_iters = 9 * slabs_per_tap;

  // What iteration `it` of a tile's main loop loads: tap it / slabs_per_tap, then source x
  // before source h, then the channel slab.
  for (int it = threadIdx.x; it < k_iters; it += TC_THREADS) {
    const int tap = it / slabs_per_tap, r = it % slabs_per_tap;
    const int src = r < p.slabs[0] ? 0 : 1;
    const int sl = src ? r - p.slabs[0] : r;
    const int ky = tap / 3, kx = tap % 3;
    int dx, dy, par;
    if (p.stride == 1) {
      dx = kx - 1;
      dy = ky - 1;
      par = 0;
    } else {
      // input column 2*xo + kx - 1: kx = 1 is the even view at xo, kx = 0 / 2 the odd view at xo-1 / xo
      const int xpar = (kx == 1) ? 0 : 1, ypar = (ky == 1) ? 0 : 1;
      dx = kx == 0 ? -1 : 0;
      dy = ky == 0 ? -1 : 0;
      par = ypar * 2 + xpar;
    }
    s_tab[it] = make_int4(src * 4 + par, sl * SLAB_C, dx, dy);
    asm volatile("prefetch.tensormap [%0];" ::"l"(&p.maps_a[src * 4 + par]) : "memory");
  }
  if (threadIdx.x < TT_MAX_STREAMS) {
    s_img[threadIdx.x] = p.img0.v[threadIdx.x];
    s_img[TT_MAX_STREAMS + threadIdx.x] = p.img1.v[threadIdx.x];
    s_img[2 * TT_MAX_STREAMS + threadIdx.x] = p.c_idx.v[threadIdx.x];
    s_img[3 * TT_MAX_STREAMS + threadIdx.x] = p.h_out_idx.v[threadIdx.x];
  }

  if (threadIdx.x == 0) {
    // in a pair the leader's "full" barriers collect one arrival per CTA and the bytes of both
    // CTAs' copies; its "accumulator free" barriers collect the epilogue warps of both CTAs
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(full_bar + s), PAIR ? 2 : 1);
      mbar_init(smem_u32(empty_bar + s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(tfull_bar + a), 1);
      mbar_init(smem_u32(tempty_bar + a), PAIR ? 2 * EPI_WARPS : EPI_WARPS);
      mbar_init(smem_u32(afull_bar + a), 1);
      mbar_init(smem_u32(aempty_bar + a), 1);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&p.map_b) : "memory");
    if (WRES) {
      // all weight slabs, in iteration order, behind the ring; they land on the first "patch landed" barrier
      const uint32_t wb = smem_u32(afull_bar);
      mbar_arrive_expect_tx(wb, (uint32_t)(k_iters * Cfg::B_BYTES));
      for (int it = 0; it < k_iters; ++it) tma_load_2d(smem_u32(smem_a + it * Cfg::B_BYTES), &p.map_b, wb, it * SLAB_C, 0);
    }
  }
  if (warp == MMA_WARP) {
    __syncwarp();   // the table loop above may have left the warp's lanes apart; the allocation is warp-collective
    if (PAIR) {
      // the same warp of both CTAs allocates the pair's columns
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"((uint32_t)Cfg::TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"((uint32_t)Cfg::TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();   // the peer's barriers exist before anything is signalled across the pair
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();   // everything above touched no activation; from here on the previous kernel's outputs are read

  const int n_prod = p.n_prod;
  const int prod = warp == 0 ? 0 : warp - (EPI_WARP0 + EPI_WARPS) + 1;   // producer index of warps 0, 10, 11
  if ((warp == 0 || warp >= EPI_WARP0 + EPI_WARPS) && prod < n_prod && lane == 0) {
    // ----------------------------------------------------------------- TMA producers
    // Producer `prod` owns iterations prod, prod + n_prod, ... of the block's sequence of
    // pipeline iterations (all tiles back to back); iteration g uses stage g % STAGES.
    uint32_t stage = (uint32_t)prod % STAGES, phase = 0;
    int it = prod;
    bool ok = true;
    const uint8_t* maps = reinterpret_cast<const uint8_t*>(p.maps_a);
    if (HALO) {
      // Iteration g = (slab, tap), slab-major: the weight slab of that tap and channel slab.  The
      // producer that owns a slab's first tap also fetches the slab's haloed activation patch
      // (x slabs first, then h slabs) into the activation ring, whose stage and phase follow from
      // the running slab count.
      const int cin_total = slabs_per_tap * SLAB_C;
      int slab_seq0 = 0;                               // slabs of all earlier tiles of this block
      for (int tile = worker; tile < total_tiles && ok; tile += n_workers) {
        const int nt = tile % p.n_tiles_n;
        const int m = tile / p.n_tiles_n;
        const int tx = m % p.tiles_x, ty = (m / p.tiles_x) % p.tiles_y, img = m / tiles_per_img;
        const int img_x = s_img[img], img_h = s_img[TT_MAX_STREAMS + img];
        for (; it < k_iters; it += n_prod) {
          const int sg = it / 9, tap = it - sg * 9;
          if (tap == 0) {
            const int seq = slab_seq0 + sg;
            const uint32_t a_stage = (uint32_t)seq & 1u, a_phase = ((uint32_t)seq >> 1) & 1u;
            ok = mbar_wait(smem_u32(aempty_bar + a_stage), a_phase ^ 1u, abort_flag, p.status, 0x900 + (int)a_stage, wait_limit);
            if (!ok) break;
            const int src = sg < p.slabs[0] ? 0 : 1;
            const uint32_t ab = smem_u32(afull_bar + a_stage);
            mbar_arrive_expect_tx(ab, Cfg::HALO_A_TX);
            tma_load_4d(smem_u32(smem_a + a_stage * Cfg::HALO_A_BYTES), &p.maps_halo[src], ab, (src ? sg - p.slabs[0] : sg) * SLAB_C,
                        tx * PW - 1, ty * PH - 1, src ? img_h : img_x);
          }
          ok = mbar_wait(smem_u32(empty_bar + stage), phase ^ 1u, abort_flag, p.status, 0x100 + (int)stage, wait_limit);
          if (!ok) break;
          const uint32_t fb = smem_u32(full_bar + stage);
          mbar_arrive_expect_tx(fb, Cfg::B_BYTES);
          tma_load_2d(smem_u32(smem + stage * Cfg::B_BYTES), &p.map_b, fb, tap * cin_total + sg * SLAB_C, nt * BLOCK_N);
          stage += (uint32_t)n_prod;
          if (stage >= (uint32_t)STAGES) { stage -= STAGES; phase ^= 1u; }
        }
        it -= k_iters;
        slab_seq0 += slabs_per_tap;
      }
    }
    // a pair's copies are counted on the leader's barriers
    const uint32_t full0c = PAIR ? map_to_cta(smem_u32(full_bar), 0u) : 0u;
    for (int tile = worker; tile < total_tiles && ok && !HALO; tile += n_workers) {
      const int nt = tile % p.n_tiles_n;
      // the second CTA of a pair takes the next M-tile; past the end it recomputes the last one (its epilogue stores nothing)
      const int m = PAIR ? min(2 * (tile / p.n_tiles_n) + rank, m_tiles - 1) : tile / p.n_tiles_n;
      const int tx = m % p.tiles_x, ty = (m / p.tiles_x) % p.tiles_y, img = m / tiles_per_img;
      const int x0 = tx * PATCH_W, y0 = ty * PATCH_H;
      // (two scalars, not an indexed array: an array would live in local memory, and a memory round
      // trip in this thread's loop delays every copy it issues)
      const int img_x = s_img[img], img_h = s_img[TT_MAX_STREAMS + img];
      for (; it < k_iters; it += n_prod) {
        const int4 e = s_tab[it];
        ok = mbar_wait(smem_u32(empty_bar + stage), phase ^ 1u, abort_flag, p.status, 0x100 + (int)stage, wait_limit);
        if (!ok) break;
        uint8_t* st = smem + stage * RING_STRIDE;
        if (PAIR) {
          const uint32_t fb = full0c + 8u * stage;
          mbar_arrive_expect_tx_cluster(fb, Cfg::STAGE_BYTES);
          tma_load_4d_pair(smem_u32(st), maps + e.x * (int)sizeof(TensorMap128), fb, e.y, x0 + e.z, y0 + e.w, e.x < 4 ? img_x : img_h);
          tma_load_2d_pair(smem_u32(st + Cfg::A_BYTES), &p.map_b, fb, it * SLAB_C, nt * BLOCK_N + rank * Cfg::B_ROWS);
        } else {
          const uint32_t fb = smem_u32(full_bar + stage);
          mbar_arrive_expect_tx(fb, WRES ? Cfg::A_BYTES : Cfg::STAGE_BYTES);
          tma_load_4d(smem_u32(st), maps + e.x * (int)sizeof(TensorMap128), fb, e.y, x0 + e.z, y0 + e.w, e.x < 4 ? img_x : img_h);
          if (!WRES) tma_load_2d(smem_u32(st + Cfg::A_BYTES), &p.map_b, fb, it * SLAB_C, nt * BLOCK_N);
        }
        stage += (uint32_t)n_prod;
        if (stage >= (uint32_t)STAGES) { stage -= STAGES; phase ^= 1u; }
      }
      it -= k_iters;
    }
  } else if (warp == MMA_WARP && lane == 0 && rank == 0) {
    // -------------------------------------------------------------------- MMA issuer
    // This loop is one thread's chain of dependent instructions and sets the pace of the whole
    // block, so everything that does not change is formed once: the operand descriptors differ
    // between stages only in their 14-bit address field (16-byte units; shared memory is far
    // below the field's range, so plain additions never carry out of it).
    uint32_t stage = 0, phase = 0, acc_phase = 0, a_stage = 0, a_phase = 0;
    int acc = 0;
    bool ok = true;
    const uint64_t a_desc0 = make_smem_desc(smem_u32(smem), SBO, LAYOUT);
    constexpr uint64_t STAGE_UNITS = RING_STRIDE >> 4, B_UNITS = Cfg::A_BYTES >> 4;
    const uint64_t w_desc0 = make_smem_desc(smem_u32(smem_a), SBO, LAYOUT);   // WRES: first resident weight slab
    if (WRES) ok = mbar_wait(smem_u32(afull_bar), 0u, abort_flag, p.status, 0xB00, wait_limit);
    const uint32_t full0 = smem_u32(full_bar), empty0 = smem_u32(empty_bar);
    uint64_t a_desc = a_desc0;
    for (int tile = worker; tile < total_tiles && ok; tile += n_workers) {
      ok = mbar_wait(smem_u32(tempty_bar + acc), acc_phase ^ 1u, abort_flag, p.status, 0x200 + acc, wait_limit);
      if (!ok) break;
      tc_fence_after();   // the epilogue's TMEM reads of this buffer come before the MMAs that overwrite it
      const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BLOCK_N);
      if (HALO) {
        // Output pixel (py, px) of the 8 x 16 patch reads halo pixel (py + ky, px + kx): the A operand
        // of a tap is the same shared-memory patch, entered (ky * 16 + kx) pixel rows of 128 bytes
        // further on.  The 8 pixels of one patch row are one 8-row operand group; groups are one halo
        // row = 2048 bytes apart.  The 128-byte swizzle is a function of the shared-memory address
        // (the TMA unit wrote the patch that way), so an operand that starts kx rows into a 1024-byte
        // pattern needs nothing but its start address.
        uint32_t first = 1;
        for (int sg = 0; sg < slabs_per_tap && ok; ++sg) {
          ok = mbar_wait(smem_u32(afull_bar + a_stage), a_phase, abort_flag, p.status, 0xA00 + (int)a_stage, wait_limit);
          if (!ok) break;
          const uint32_t a_base = smem_u32(smem_a + a_stage * Cfg::HALO_A_BYTES);
#pragma unroll 1
          for (int tap = 0; tap < 9; ++tap) {
            ok = mbar_wait(full0 + 8u * stage, phase, abort_flag, p.status, 0x300 + (int)stage, wait_limit);
            if (!ok) break;
            const int ky = tap / 3, kx = tap - ky * 3;
            const uint64_t a_tap = make_smem_desc(a_base + (uint32_t)((ky * Cfg::HALO_PITCH + kx) * 128), Cfg::HALO_PITCH * 128u, LAYOUT);
            const uint64_t b_tap = a_desc;               // a_desc walks the weight ring in this mode
            umma_bf16(d_tmem, a_tap, b_tap, IDESC, first ? 0u : 1u);
            first = 0;
#pragma unroll
            for (int k = 1; k < SLAB_C / UMMA_K; ++k) umma_bf16(d_tmem, a_tap + (uint64_t)(2 * k), b_tap + (uint64_t)(2 * k), IDESC, 1u);
            umma_commit(empty0 + 8u * stage);
            a_desc += (uint64_t)(Cfg::B_BYTES >> 4);
            if (++stage == STAGES) { stage = 0; phase ^= 1u; a_desc = a_desc0; }
          }
          if (!ok) break;
          umma_commit(smem_u32(aempty_bar + a_stage));   // the patch is free once all nine taps have read it
          if (++a_stage == (uint32_t)A_STAGES) { a_stage = 0; a_phase ^= 1u; }
        }
      }
      for (int it = 0; it < k_iters && !HALO; ++it) {
        // the copies complete on the barrier through the async proxy, which the MMAs read through too
        ok = mbar_wait(full0 + 8u * stage, phase, abort_flag, p.status, 0x300 + (int)stage, wait_limit);
        if (!ok) break;
        const uint64_t b_desc = WRES ? w_desc0 + (uint64_t)it * (uint64_t)(Cfg::B_BYTES >> 4) : a_desc + B_UNITS;
        // advance along K inside the swizzle atom: 16 bf16 = 32 bytes = 2 descriptor units
        if (PAIR) {
          umma_bf16_pair(d_tmem, a_desc, b_desc, IDESC, it != 0 ? 1u : 0u);
#pragma unroll
          for (int k = 1; k < SLAB_C / UMMA_K; ++k) umma_bf16_pair(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), IDESC, 1u);
          umma_commit_pair(empty0 + 8u * stage);     // frees the stage in both CTAs once the MMAs have read it
        } else {
          umma_bf16(d_tmem, a_desc, b_desc, IDESC, it != 0 ? 1u : 0u);
#pragma unroll
          for (int k = 1; k < SLAB_C / UMMA_K; ++k) umma_bf16(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), IDESC, 1u);
          umma_commit(empty0 + 8u * stage);          // frees the stage once the MMAs have read it
        }
        a_desc += STAGE_UNITS;
        if (++stage == STAGES) { stage = 0; phase ^= 1u; a_desc = a_desc0; }
      }
      if (!ok) break;
      if (PAIR) umma_commit_pair(smem_u32(tfull_bar + acc));   // accumulator complete, in both CTAs
      else umma_commit(smem_u32(tfull_bar + acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  } else if (warp >= EPI_WARP0 && warp < EPI_WARP0 + EPI_WARPS) {
    // ---------------------------------------------------------------------- epilogue
    constexpr int HALF_N = BLOCK_N / 2;           // columns handled by this warp
    constexpr int CHUNKS = HALF_N / 32;
    const int quarter = warp & 3;                 // TMEM lanes 32*quarter .. +31
    // 32-byte stores of bf16 values need 16 values per pixel row between sector boundaries
    const bool wide_out = EPI == TC_EPI_LSTM ? (p.hidden & 15) == 0 : (p.cout & 15) == 0;
    const int half = (warp - EPI_WARP0) >> 2;     // which half of the tile's columns
    const int row = quarter * 32 + lane;          // row of the 128-row tile = pixel of the patch
    const int py = row / PW, px = row % PW;
    uint32_t acc_phase = 0;
    int acc = 0;
    bool ok = true;
    const uint32_t tempty0c = PAIR ? map_to_cta(smem_u32(tempty_bar), 0u) : 0u;
    for (int tile = worker; tile < total_tiles; tile += n_workers) {
      const int nt = tile % p.n_tiles_n;
      const int m_raw = PAIR ? 2 * (tile / p.n_tiles_n) + rank : tile / p.n_tiles_n;
      const int m = min(m_raw, m_tiles - 1);
      const int tx = m % p.tiles_x, ty = (m / p.tiles_x) % p.tiles_y, img = m / tiles_per_img;
      const int x = tx * PW + px, y = ty * PH + py;
      const bool valid = x < p.Wo && y < p.Ho && m_raw < m_tiles;
      const size_t pix = (size_t)y * p.Wo + x;
      const int col0 = nt * BLOCK_N + half * HALF_N;  // first packed output column of this warp

      // The old cell state of this thread's pixel is fetched before the accumulator is
      // waited for, so its latency hides under the tile's main loop.
      float c_old[EPI == TC_EPI_LSTM ? CHUNKS * 8 : 1];
      size_t so = 0, ho = 0;
      if (EPI == TC_EPI_LSTM) {
        so = ((size_t)s_img[2 * TT_MAX_STREAMS + img] * p.Ho * p.Wo + pix) * p.hidden + (col0 >> 2);
        ho = ((size_t)s_img[3 * TT_MAX_STREAMS + img] * p.Ho * p.Wo + pix) * p.hidden + (col0 >> 2);
#pragma unroll
        for (int ck = 0; ck < CHUNKS; ++ck) {
          float c8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
          if (valid && (col0 >> 2) + ck * 8 < p.hidden) ld_global_v8(p.c_state + so + ck * 8, c8);
#pragma unroll
          for (int jj = 0; jj < 8; ++jj) c_old[ck * 8 + jj] = c8[jj];
        }
      }

      // the warp votes: its lanes leave the tile loop together or go on to the warp-collective TMEM loads together
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(tfull_bar + acc), acc_phase, abort_flag, p.status, 0x400 + acc, wait_limit));
      if (!ok) break;
      tc_fence_after();
      const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BLOCK_N + half * HALF_N);
      uint32_t hb[8];
#pragma unroll
      for (int ck = 0; ck < CHUNKS; ++ck) {
        uint32_t v[32];
        tmem_ld32(t_addr + (uint32_t)(ck * 32), v);
        const int n0 = col0 + ck * 32;            // first packed output column of this chunk
        if (EPI == TC_EPI_RELU_BF16) {
          if (valid && n0 < p.cout) {
            const float4* b4 = reinterpret_cast<const float4*>(p.bias + n0);
            __nv_bfloat16* dst = p.out + ((size_t)img * p.Ho * p.Wo + pix) * p.cout + n0;
#pragma unroll
            for (int i = 0; i < 32; i += 16) {
              uint32_t u[8];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float4 b = __ldg(b4 + i / 4 + j);
                u[2 * j + 0] = pack_bf16(fmaxf(__uint_as_float(v[i + 4 * j + 0]) + b.x, 0.f), fmaxf(__uint_as_float(v[i + 4 * j + 1]) + b.y, 0.f));
                u[2 * j + 1] = pack_bf16(fmaxf(__uint_as_float(v[i + 4 * j + 2]) + b.z, 0.f), fmaxf(__uint_as_float(v[i + 4 * j + 3]) + b.w, 0.f));
              }
              if (wide_out) {
                st_global_v8_b32(dst + i, u);        // 16 channels = one 32-byte sector
              } else {
                *reinterpret_cast<uint4*>(dst + i) = make_uint4(u[0], u[1], u[2], u[3]);
                *reinterpret_cast<uint4*>(dst + i + 8) = make_uint4(u[4], u[5], u[6], u[7]);
              }
            }
          }
        } else {
          // packed column = 4*jj + gate (i, f, g, o); 8 hidden units per 32-column chunk
          if (valid && (n0 >> 2) < p.hidden) {
            const float4* b4 = reinterpret_cast<const float4*>(p.bias + n0);
            float c_new[8], h_new[8];
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
              const float4 b = __ldg(b4 + jj);
              const float gi = __uint_as_float(v[4 * jj + 0]) + b.x;
              const float gf = __uint_as_float(v[4 * jj + 1]) + b.y;
              const float gg = __uint_as_float(v[4 * jj + 2]) + b.z;
              const float go = __uint_as_float(v[4 * jj + 3]) + b.w;
              c_new[jj] = fast_sigmoid(gf) * c_old[ck * 8 + jj] + fast_sigmoid(gi) * fast_tanh(gg);
              h_new[jj] = fast_sigmoid(go) * fast_tanh(c_new[jj]);
            }
            st_global_v8(p.c_state + so + ck * 8, c_new);
            if (p.h_f32) st_global_v8(p.h_f32 + so + ck * 8, h_new);
            // bf16 shadow of h': 8 values are half a sector, so two neighbouring chunks leave together
            const int hq = (ck & 1) * 4;
            hb[hq + 0] = pack_bf16(h_new[0], h_new[1]);
            hb[hq + 1] = pack_bf16(h_new[2], h_new[3]);
            hb[hq + 2] = pack_bf16(h_new[4], h_new[5]);
            hb[hq + 3] = pack_bf16(h_new[6], h_new[7]);
            if (wide_out && CHUNKS % 2 == 0) {
              if (ck & 1) st_global_v8_b32(p.h_bf16 + ho + (ck - 1) * 8, hb);
            } else {
              *reinterpret_cast<uint4*>(p.h_bf16 + ho + ck * 8) = make_uint4(hb[hq], hb[hq + 1], hb[hq + 2], hb[hq + 3]);
            }
          }
        }
      }
      // hand the accumulator buffer back to the MMA warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (PAIR) mbar_arrive_cluster(tempty0c + 8u * (uint32_t)acc);
        else mbar_arrive(smem_u32(tempty_bar + acc));
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  // ------------------------------------------------------------------------------- teardown
  __syncwarp();
  if (*abort_flag) {
    // a wait ran out somewhere: give copies and MMAs in flight time to land before the
    // shared memory and TMEM of this block are released
    for (int i = 0; i < 64; ++i) __nanosleep(16000);
  }
  tc_fence_before();
  __syncthreads();
  // neither CTA of a pair may go while the other can still signal its barriers or have its shared memory read by the pair's MMAs
  if (PAIR) cluster_sync_all();
  if (warp == MMA_WARP) {
    tc_fence_after();
    if (PAIR)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Cfg::TMEM_COLS) : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Cfg::TMEM_COLS) : "memory");
  }
}

template <int BLOCK_N, int SLAB_C, int EPI, int CTAS = 1>
cudaError_t launch_cfg(const ConvTcParams& p, int sm_count, cudaStream_t s) {
  using Cfg = TcCfg<BLOCK_N, SLAB_C, false, CTAS>;
  auto kern = conv_tc_kernel<BLOCK_N, SLAB_C, EPI, false, CTAS>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int total_tiles = p.K * p.tiles_x * p.tiles_y * p.n_tiles_n;
  const int slots = CTAS * sm_count;
  const int grid = total_tiles < slots ? total_tiles : slots;
  return launch_kernel(kern, grid, TC_THREADS, Cfg::SMEM_BYTES, s, p, p.pdl != 0);
}

// Weights resident: two blocks per multiprocessor, ring of activation boxes, the whole weight matrix behind it.
template <int BLOCK_N, int SLAB_C>
cudaError_t launch_wres(const ConvTcParams& p, int sm_count, cudaStream_t s) {
  using Cfg = TcCfg<BLOCK_N, SLAB_C, false, 2>;
  constexpr int SMEM = WRES_STAGES * Cfg::A_BYTES + WRES_BYTES + Cfg::BAR_BYTES + Cfg::TAB_BYTES + 1024;
  auto kern = conv_tc_kernel<BLOCK_N, SLAB_C, TC_EPI_RELU_BF16, false, 2, false, true>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
  if (e != cudaSuccess) return e;
  const int total_tiles = p.K * p.tiles_x * p.tiles_y;
  const int slots = 2 * sm_count;
  const int grid = total_tiles < slots ? total_tiles : slots;
  return launch_kernel(kern, grid, TC_THREADS, SMEM, s, p, p.pdl != 0);
}

// CTA pairs: clusters of two, one pair per unit of work, as many pairs as the device can hold at once.
template <int BLOCK_N, int SLAB_C, int EPI>
cudaError_t launch_pair(const ConvTcParams& p, int sm_count, cudaStream_t s) {
  using Cfg = TcCfg<BLOCK_N, SLAB_C, true>;
  auto kern = conv_tc_kernel<BLOCK_N, SLAB_C, EPI, true>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg{};
  cfg.blockDim = dim3(TC_THREADS);
  cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.pdl ? 2 : 1;
  // pairs that can be resident at once (a pair needs two multiprocessors of one cluster-capable group)
  static int max_pairs = 0;   // the same for every instantiation's launch shape: one block per multiprocessor
  if (max_pairs == 0) {
    cfg.gridDim = dim3((unsigned)(2 * (sm_count / 2)));
    int n = 0;
    e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
    if (e != cudaSuccess) return e;
    if (n < 1) return cudaErrorInvalidConfiguration;
    max_pairs = n;
  }
  const int m_tiles = p.K * p.tiles_x * p.tiles_y;
  const int units = ((m_tiles + 1) / 2) * p.n_tiles_n;
  const int pairs = units < max_pairs ? units : max_pairs;
  cfg.gridDim = dim3((unsigned)(2 * pairs));
  return cudaLaunchKernelEx(&cfg, kern, p);
}

// Halo mode: one haloed activation patch per channel slab instead of one box per tap.
template <int BLOCK_N, int EPI>
cudaError_t launch_halo(const ConvTcParams& p, int sm_count, cudaStream_t s) {
  using Cfg = TcCfg<BLOCK_N, 64>;
  auto kern = conv_tc_kernel<BLOCK_N, 64, EPI, false, 1, true>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::HALO_SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int total_tiles = p.K * p.tiles_x * p.tiles_y * p.n_tiles_n;
  const int grid = total_tiles < sm_count ? total_tiles : sm_count;
  return launch_kernel(kern, grid, TC_THREADS, Cfg::HALO_SMEM_BYTES, s, p, p.pdl != 0);
}

template <int EPI>
cudaError_t launch_shape(const ConvTcParams& p, int sm_count, cudaStream_t s) {
  if (p.halo) {
    if (EPI != TC_EPI_LSTM || p.slab_c != 64 || p.stride != 1 || p.pair) return cudaErrorInvalidValue;
    if (p.block_n == 256) return launch_halo<256, TC_EPI_LSTM>(p, sm_count, s);
    if (p.block_n == 128) return launch_halo<128, TC_EPI_LSTM>(p, sm_count, s);
    return cudaErrorInvalidValue;
  }
  if (p.pair) {
    if (p.slab_c == 64 && p.block_n == 256) return launch_pair<256, 64, EPI>(p, sm_count, s);
    return cudaErrorInvalidValue;
  }
  if (EPI == TC_EPI_RELU_BF16 && p.two_per_sm && p.wres) {
    const int k_iters = 9 * (p.slabs[0] + (p.n_src > 1 ? p.slabs[1] : 0));
    if (p.slab_c != 32 || p.block_n != 64 || p.n_tiles_n != 1 || k_iters * 64 * 32 * 2 > WRES_BYTES) return cudaErrorInvalidValue;
    return launch_wres<64, 32>(p, sm_count, s);
  }
  if (EPI == TC_EPI_RELU_BF16 && p.two_per_sm && p.block_n <= 128) {
    if (p.slab_c == 64 && p.block_n == 128) return launch_cfg<128, 64, TC_EPI_RELU_BF16, 2>(p, sm_count, s);
    if (p.slab_c == 64 && p.block_n == 64) return launch_cfg<64, 64, TC_EPI_RELU_BF16, 2>(p, sm_count, s);
    if (p.slab_c == 32 && p.block_n == 128) return launch_cfg<128, 32, TC_EPI_RELU_BF16, 2>(p, sm_count, s);
    if (p.slab_c == 32 && p.block_n == 64) return launch_cfg<64, 32, TC_EPI_RELU_BF16, 2>(p, sm_count, s);
  }
  if (p.slab_c == 64) {
    if (p.block_n == 256) return launch_cfg<256, 64, EPI>(p, sm_count, s);
    if (p.block_n == 128) return launch_cfg<128, 64, EPI>(p, sm_count, s);
    if (p.block_n == 64) return launch_cfg<64, 64, EPI>(p, sm_count, s);
  } else if (p.slab_c == 32) {
    if (p.block_n == 128) return launch_cfg<128, 32, EPI>(p, sm_count, s);
    if (p.block_n == 64) return launch_cfg<64, 32, EPI>(p, sm_count, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_conv_tc(const ConvTcParams& p, int sm_count, cudaStream_t s) {
  if (9 * (p.slabs[0] + (p.n_src > 1 ? p.slabs[1] : 0)) > MAX_K_ITERS || p.n_prod < 1 || p.n_prod > N_PROD) return cudaErrorInvalidValue;
  if (p.epilogue == TC_EPI_RELU_BF16) return launch_shape<TC_EPI_RELU_BF16>(p, sm_count, s);
  if (p.epilogue == TC_EPI_LSTM) return launch_shape<TC_EPI_LSTM>(p, sm_count, s);
  return cudaErrorInvalidValue;
}

}  // namespace tt
