// Internal launch interfaces shared by the translation units of libtt.so.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "tt.h"

namespace tt {

// Programmatic dependent launch.  A kernel launched with `pdl` set may start while its
// predecessor in the stream is still running: its blocks take multiprocessors as the
// predecessor's blocks leave them, do the set-up that touches no activation (barriers, tensor
// memory, weight staging) and then wait in pdl_wait() until the predecessor has completed and its
// writes are visible.  Without the launch attribute both device calls do nothing.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename Params>
inline cudaError_t launch_kernel(void (*kern)(const Params), int grid, int block, size_t smem, cudaStream_t s, const Params& p,
                                 bool pdl) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, p);
}

// Maps batch position n (0..K-1) of a launch to an image index inside a tensor that holds
// more images than the batch (state slots, ping-pong halves).
struct IdxMap {
  int32_t v[TT_MAX_STREAMS];
};

struct FramePtrs {
  const uint8_t* p[TT_MAX_STREAMS];
};

// ------------------------------------------------------------------------- S1 preprocess
struct PreprocessParams {
  FramePtrs src;                   // frame pointers by value (also used for host-side decisions)
  const uint8_t* const* src_tab;   // if non-null the kernel reads the pointers from this device table instead
  int32_t K, src_w, src_h, src_pitch, net_w, net_h;
  float inv_div, mean, inv_std;
  float* dst;  // [K][3][net_h][net_w]
};
cudaError_t launch_preprocess(const PreprocessParams& p, cudaStream_t s);

// ------------------------------------------------------------------ S2/S3 fp32 SIMT conv
enum ConvEpilogue : int32_t {
  EPI_RELU_F32_NCHW = 0,   // out fp32 [K][Cout][Ho][Wo]
  EPI_RELU_BF16_NHWC = 1,  // out bf16 [K][Ho][Wo][Cout]
  EPI_LSTM_F32_NCHW = 2    // gate math, c in place, h' to the "out" half of the ping-pong
};

struct ConvSimtParams {
  const float* in0;  // fp32 planar, image n at in0 + idx0.v[n]*img_stride0
  const float* in1;  // optional second source (recurrent h), channels follow in0's
  int64_t img_stride0, img_stride1;
  IdxMap idx0, idx1;
  int32_t C0, C1;
  int32_t H, W, Ho, Wo, stride, K;
  const float* wgt;   // packed [Cin][9][CoutPacked]
  const float* bias;  // packed [CoutPacked]
  int32_t cout, cout_packed, ocb;
  int32_t epilogue;
  // EPI_RELU_*: out; EPI_LSTM: c (in place), h_out
  void* out;
  int64_t out_img_stride;  // elements
  float* c_state;          // [slots][Ch][plane]
  float* h_state;          // [slots*2][Ch][plane]
  IdxMap c_idx, h_out_idx;
  int32_t hidden;
};
cudaError_t launch_conv_simt(const ConvSimtParams& p, cudaStream_t s);

// Opaque 128-byte TMA tensor map, passed inside __grid_constant__ kernel parameters.
struct alignas(64) TensorMap128 {
  uint8_t bytes[128];
};

// --------------------------------------- S2 first encoder layer of the bf16 path (Cin = 3)
// On the tensor cores (cout 32 or 64): operand tiles are built by producer threads.
struct ConvFirstTcParams {
  TensorMap128 map_out;       // output [K][Ho][Wo][cout] bf16, box [cout][16][8][1], 128B / 64B swizzle
  TensorMap128 map_in;        // input [K][3][H][W] fp32, box [conv_first_tc_box_w(stride)][7*stride+3][3][1], no swizzle
  const float* in;            // [K][3][H][W] fp32
  __nv_bfloat16* out;         // [K][Ho][Wo][cout] bf16
  int32_t H, W, Ho, Wo, stride, K, cout, tiles_x, tiles_y;
  int32_t pdl;                // launch as a programmatic dependent of the previous kernel in the stream
  const uint16_t* w_packed;   // device, cout*32 bf16 in the MMA operand layout
  const float* bias;          // device, [cout]
  int32_t* status;
  long long wait_limit;       // SM cycles after which a barrier wait gives up
  // fused preprocessing: the kernel samples the uint8 RGB frames itself (resize to W x H, then v * scale + shift)
  // and neither `in` nor map_in is used
  int32_t fused;
  FramePtrs src;                   // frame pointers by value ...
  const uint8_t* const* src_tab;   // ... or, if non-null, a device table of them
  int32_t src_w, src_h, src_pitch;
  float scale, shift;
  int32_t src_rows_cap, src_row_cap;   // staged frame rows per tile and bytes per staged row (conv_first_tc_staging)
};
bool conv_first_tc_supported(int cout);
// Shared-memory footprint of the frame rows one tile of the fused form stages: rows and bytes per row
// (a multiple of 16).  False if the resize factor makes it too large; the preprocessing then stays a kernel of its own.
bool conv_first_tc_staging(int stride, int src_w, int src_h, int net_w, int net_h, int* rows_cap, int* row_cap);
int conv_first_tc_box_w(int stride);   // columns of the input patch box (a multiple of 4)
void conv_first_tc_pack(const uint16_t* w_bf16, int cout, uint16_t* packed);
cudaError_t launch_conv_first_tc(const ConvFirstTcParams& p, int sm_count, cudaStream_t s);

// ------------------------------------------------- S2/S3 tcgen05 implicit-GEMM conv (bf16)
// One launch description; tensor maps live in device-visible constant storage owned by the
// caller (passed by value as __grid_constant__ kernel parameters).
enum TcEpilogue : int32_t { TC_EPI_RELU_BF16 = 0, TC_EPI_LSTM = 1 };

struct ConvTcParams {
  // A operand sources: up to two NHWC bf16 tensors (x then h); for stride 2 four parity
  // views of the single source.  maps_a[src*4 + parity] with parity = (ypar*2 + xpar).
  TensorMap128 maps_a[8];
  TensorMap128 maps_halo[2];// halo mode: the two sources again with a box of [64 channels][16][18][1] (haloed patch of an 8 x 16 tile)
  TensorMap128 map_b;       // packed weights [CoutPacked][Ktot] bf16, K-major
  int32_t n_src;            // 1 or 2
  int32_t slabs[2];         // channel slabs (of slab_c channels) per source
  int32_t slab_c;           // 64 or 32
  int32_t stride;           // 1 or 2
  int32_t K;                // images in the batch
  IdxMap img0, img1;        // image index of batch n inside source 0 / 1
  int32_t Ho, Wo;           // output extent
  int32_t tiles_x, tiles_y; // 16 x 8 pixel patches
  int32_t n_tiles_n;        // CoutPacked / block_n
  int32_t block_n;          // 64, 128 or 256
  int32_t n_prod;           // producer warps that issue loads, 1..3
  int32_t two_per_sm;       // encoder layers with tiles up to 128 wide: two blocks per multiprocessor, half the ring each
  int32_t wres;             // two_per_sm layer of 64 outputs and 32-channel slabs whose weights fit in 40 KB: fetched once per block
  int32_t halo;             // stride-1 layer of 64-channel slabs: one haloed patch per channel slab, 8 x 16 output patches
  int32_t pair;             // run as CTA pairs (cta_group::2): block_n 256, map_b's box then holds 128 rows
  int32_t pdl;              // launch as a programmatic dependent of the previous kernel in the stream
  int32_t cout;             // real output channels (RELU) or 4*hidden (LSTM)
  int32_t epilogue;
  const float* bias;        // packed order, [CoutPacked]
  // RELU epilogue
  __nv_bfloat16* out;       // [K][Ho][Wo][cout]
  // LSTM epilogue
  float* c_state;           // [slots][Hm][Wm][Ch] in place
  float* h_f32;             // [slots][Hm][Wm][Ch], or null: h' is written as its bf16 copy only
  __nv_bfloat16* h_bf16;    // [slots*2][Hm][Wm][Ch]
  IdxMap c_idx, h_out_idx;  // slot, slot*2+half
  int32_t hidden;
  int32_t* status;          // device word: 0 ok, else a code describing a wait that ran out
  long long wait_limit;     // SM cycles after which a barrier wait gives up
};
cudaError_t launch_conv_tc(const ConvTcParams& p, int sm_count, cudaStream_t s);
constexpr long long DEFAULT_WAIT_LIMIT_CYCLES = 4000000000ll;   // about 2 s of SM cycles

// Failure-path probe: one warp waits, through the same bounded wait as the tensor-core kernels, on
// a barrier that nothing ever completes; when `limit_cycles` have passed it records `code` in
// *status and returns normally.
cudaError_t launch_wait_probe(int32_t* status, long long limit_cycles, int code, cudaStream_t s);

// ------------------------------------------------------------------- S4/S5 postprocess
struct PostParams {
  const float* h;       // fp32, image n at h + idx.v[n]*img_stride
  int32_t channels_last;
  int64_t img_stride;
  IdxMap idx;
  int32_t K, Hm, Wm, Ch, T;
  const float* head_w;  // [T][Ch]
  const float* head_b;
  const float* conf_w;  // [T][Ch] or null
  const float* conf_b;
  int32_t conf_mode;
  float zthr;
  float* logits;        // [K][T][plane]
  float* probs;
  uint8_t* masks;
  uint8_t* bits;        // optional [K][plane], bit t = mask of tool t
  tt_result* results;   // device, [K]
  void* scratch;
  int32_t* status;      // optional device word: set non-zero when a bounded wait ran out
  long long wait_limit; // SM cycles after which a wait for a copy gives up (0: the default)
  int32_t pdl;          // launch as a programmatic dependent of the previous kernel in the stream (channels-last kernel only)
};
size_t post_scratch_bytes(int K, int hm, int wm, int ch, int T);
cudaError_t launch_postprocess(const PostParams& p, cudaStream_t s);
cudaError_t post_prepare();
cudaError_t post_static_scratch(void** ptr);  // device address of the library's built-in scratch array

// S4/S5 of the bf16 path on the tensor cores: reads the bf16 channels-last hidden state.
struct PostTcParams {
  TensorMap128 map_h;     // bf16 [n_img][plane][Ch], box [64 channels][128 pixels][1], 128-byte swizzle
  TensorMap128 map_w;     // bf16 [16][Ch]: rows 0..7 head weights, rows 8..15 confidence-head weights; box [64][16]
  IdxMap idx;             // image index of batch position n inside the hidden-state tensor
  int32_t K, Hm, Wm, T, kslabs;   // kslabs = Ch / 64
  const float* head_b;
  const float* conf_b;    // null for TT_CONF_MEAN_SIGMOID
  int32_t conf_mode;
  float zthr;
  float* logits;          // [K][T][plane]
  float* probs;
  uint8_t* masks;
  uint8_t* bits;          // optional [K][plane]
  tt_result* results;     // device, [K]
  void* scratch;          // post_scratch_bytes(...) bytes, zero on entry, zero again on exit
  int32_t* status;
  long long wait_limit;
  int32_t pdl;
};
bool post_tc_supported(int ch, int plane);
cudaError_t launch_post_tc(const PostTcParams& p, int sm_count, cudaStream_t s);

// -------------------------------------------------------------------------- S6 overlay
struct OverlayParams {
  FramePtrs src;
  const uint8_t* const* src_tab;   // as in PreprocessParams
  int32_t K, src_w, src_h, src_pitch, T, Hm, Wm;
  const uint8_t* masks;  // [K][T][plane] (used when bits == null)
  const uint8_t* bits;   // [K][plane] packed
  uint8_t palette[TT_MAX_TOOLS][3];
  uint8_t* dst;          // [K][src_h][src_w][4]
};
cudaError_t launch_overlay(const OverlayParams& p, cudaStream_t s);

// ------------------------------------------- scaled-up visualisation load (multi-layer blend)
struct RenderParams {
  FramePtrs src;
  int32_t K, src_w, src_h, src_pitch, T, Hm, Wm;
  const uint8_t* masks;   // [K][T][plane]
  uint8_t palette[TT_MAX_TOOLS][3];
  int32_t layers;         // the S6 blend is applied this many times, layer l with the palette rotated by l
  int32_t carve_ctas;     // 0: one block per 1024 pixels over the whole device; > 0: that many looping blocks
  uint8_t* dst;           // [K][src_h][src_w][4]
};
cudaError_t launch_render(const RenderParams& p, cudaStream_t s);

// ------------------------------------------------------------------------ layout helpers
// fp32 NCHW <-> internal layouts, used by state import/export and debug taps.
cudaError_t launch_nhwc_to_nchw_f32(const float* src, float* dst, int C, int plane, cudaStream_t s);
cudaError_t launch_nchw_to_nhwc_f32(const float* src, float* dst, int C, int plane, cudaStream_t s);
cudaError_t launch_nhwc_bf16_to_nchw_f32(const __nv_bfloat16* src, float* dst, int C, int plane, cudaStream_t s);
cudaError_t launch_nchw_f32_to_nhwc_bf16(const float* src, __nv_bfloat16* dst, int C, int plane, cudaStream_t s);

}  // namespace tt
