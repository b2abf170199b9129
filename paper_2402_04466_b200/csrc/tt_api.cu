// Context, weight repacking, tensor-map construction and the per-tick launch sequence behind
// the C ABI declared in tt.h.  Host code only; every stage of the path runs in the kernels
// of the other translation units.
#include <cuda.h>

#include <chrono>
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <thread>
#include <vector>

#include "tt_internal.h"
#include "pre_math.cuh"

using namespace tt;

// ------------------------------------------------------------------------------ data structures
struct tt_state {
  tt_ctx* ctx = nullptr;
  int slot = -1;
  int half = 0;       // which half of the h ping-pong holds the current h
  bool in_use = false;
  int last_pos = -1;  // batch position in the last submit that used this state
};

namespace {

struct SimtLayer {
  float* w = nullptr;  // [Cin][9][CoutPacked]
  float* b = nullptr;
  int cin = 0, cout = 0, cout_packed = 0, ocb = 16, stride = 1;
};

struct TcLayer {
  __nv_bfloat16* w = nullptr;  // [CoutPacked][9*Cin] K-major
  float* b = nullptr;          // packed order
  int cin0 = 0, cin1 = 0, cout = 0, slab_c = 64, stride = 1;
  TensorMap128 maps_a[8];
  TensorMap128 maps_halo[2];   // stride-1 layers of 64-channel slabs: haloed-patch boxes of the two sources
  bool has_halo = false;
  TensorMap128 map_b[3];       // block_n = 64, 128, 256
  bool has_b[3] = {false, false, false};
};

std::mutex g_err_mu;
std::string g_create_err;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  std::memcpy(&u, &f, 4);
  if ((u & 0x7F800000u) == 0x7F800000u) return (uint16_t)(u >> 16);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

int conv_out(int n, int s) { return (n + 2 - 3) / s + 1; }
int round_up(int a, int b) { return (a + b - 1) / b * b; }

}  // namespace

struct tt_ctx {
  tt_config cfg;
  int dev = 0;
  cudaStream_t stream = nullptr;
  bool own_stream = false;
  int sm_count = 148;
  bool bf16 = false;
  int n_enc = 0;
  int lay_c[TT_MAX_ENC + 1], lay_h[TT_MAX_ENC + 1], lay_w[TT_MAX_ENC + 1];  // [0] = network input
  int Hm = 0, Wm = 0, Ch = 0, T = 0, Cx = 0;
  size_t frame_bytes = 0;

  uint8_t* frames_stage = nullptr;
  float* pre = nullptr;
  void* enc_out[TT_MAX_ENC] = {nullptr, nullptr, nullptr, nullptr};
  float* c_state = nullptr;
  float* h_f32 = nullptr;             // fp32 path: [slots*2][Ch][plane]; bf16 path: [slots][plane][Ch]
  __nv_bfloat16* h_bf16 = nullptr;    // bf16 path: [slots*2][plane][Ch]
  float *logits = nullptr, *probs = nullptr;
  uint8_t *masks = nullptr, *bits = nullptr, *overlay = nullptr;
  tt_result* results_dev = nullptr;
  tt_result* results_host = nullptr;  // pinned
  int32_t* status_dev = nullptr;
  int32_t* status_host = nullptr;     // pinned
  void* post_scratch = nullptr;
  float* dbg_tmp = nullptr;
  size_t dbg_tmp_floats = 0;
  float *head_w = nullptr, *head_b = nullptr, *conf_w = nullptr, *conf_b = nullptr;
  float zthr = 0.f;

  PostTcParams post_tc{};       // bf16 path: mask and confidence heads on the tensor cores when the hidden width allows
  bool use_post_tc = false;
  ConvFirstTcParams first_tc{}; // bf16 path, first encoder layer on the tensor cores when its width (32 or 64) allows
  bool use_first_tc = false;
  bool fuse_pre = false;        // the first layer samples the frames itself; no preprocess launch, ctx->pre is not written
  FramePtrs fp_inflight{};      // device frame pointers of the submit being described (saved per slot)
  SimtLayer simt_enc[TT_MAX_ENC];
  SimtLayer simt_lstm;
  TcLayer tc_enc[TT_MAX_ENC];
  TcLayer tc_lstm;

  tt_state states[TT_MAX_STREAMS];
  // Up to TT_MAX_IN_FLIGHT submits may be in flight.  Everything a tick owns (frame staging, outputs,
  // result blocks, events) exists once per slot; the members above/below named like the slot's are the
  // slot that is currently bound (bind_slot / save_slot).
  struct Slot {
    uint8_t* frames_stage = nullptr;
    float *logits = nullptr, *probs = nullptr;
    uint8_t *masks = nullptr, *bits = nullptr, *overlay = nullptr;
    tt_result *results_dev = nullptr, *results_host = nullptr;
    int32_t* status_host = nullptr;
    cudaEvent_t ev_start = nullptr, ev_stop = nullptr, ev_copy = nullptr;
    cudaEvent_t stage_ev[TT_STAGE_COUNT + 1] = {};
    bool stage_ran[TT_STAGE_COUNT] = {};
    FramePtrs fp{};
    bool profiled = false;
    int K = 0;
    tt_frame frames[TT_MAX_STREAMS];
    tt_state* states[TT_MAX_STREAMS];
  } slots[TT_MAX_IN_FLIGHT];
  int q_head = 0, q_count = 0;      // oldest in-flight slot, number in flight
  int bound = 0;                    // slot whose resources the view members hold
  int last_done = -1;               // slot of the last completed submit (debug taps)
  // CUDA graphs of the tick's launch sequence, one per (stream count, slot, pointer table, state placement).
  // Frame pointers may change every tick, so the kernels read them from a small device table; a table that
  // does not yet hold the tick's pointers is refreshed by a 64-byte copy in front of the graph launch.
  struct TickGraph {
    int K = 0, slot = 0, flat = 0, tab = 0;
    int sig[TT_MAX_STREAMS] = {};   // state slot * 2 + half of every batch position
    int seen = 0;                   // direct executions of this key so far (capture happens on the second)
    uint64_t launches = 0;          // kernels inside the graph
    cudaGraphExec_t exec = nullptr;
  };
  std::vector<TickGraph> graphs;
  bool graphs_off = false;
  bool cta_pairs = false;           // TT_OPT_CTA_PAIRS
  bool enc_two_per_sm = true;       // !TT_OPT_ENC_ONE_PER_SM
  bool feed_forward = false;        // TT_OPT_FEED_FORWARD: no recurrent cell, the heads read the encoder output
  // Every slot owns a few device tables, each remembering the set of frame pointers it holds: a caller whose
  // frames arrive in a fixed set of buffers (a capture ring; the slot's own staging buffer for host frames) finds
  // its pointers already on the device and no copy is enqueued.
  static constexpr int FRAME_TABS = 8;
  const uint8_t** frame_tab_dev[TT_MAX_IN_FLIGHT] = {};   // device, [FRAME_TABS][TT_MAX_STREAMS] pointers per slot
  const uint8_t** frame_tab_host[TT_MAX_IN_FLIGHT] = {};  // pinned staging of one table
  const uint8_t* frame_tab_last[TT_MAX_IN_FLIGHT][FRAME_TABS][TT_MAX_STREAMS] = {};   // what each device table holds
  bool frame_tab_valid[TT_MAX_IN_FLIGHT][FRAME_TABS] = {};
  uint64_t frame_tab_used[TT_MAX_IN_FLIGHT][FRAME_TABS] = {};             // tick at which the table was last used (the oldest is replaced)
  const uint8_t* const* cur_tab = nullptr;                  // table the tick being enqueued reads
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_copy = nullptr;
  bool tick_profiled = false;
  int K_inflight = 0;
  tt_frame frames_inflight[TT_MAX_STREAMS];
  tt_state* states_inflight[TT_MAX_STREAMS];
  cudaEvent_t ev_start = nullptr, ev_stop = nullptr;
  bool profiling = false;
  cudaEvent_t stage_ev[TT_STAGE_COUNT + 1] = {};
  bool stage_ran[TT_STAGE_COUNT] = {};
  bool stage_valid = false;
  float stage_ms[TT_STAGE_COUNT];
  uint64_t n_launches = 0, n_ticks = 0;
  long long wait_limit = DEFAULT_WAIT_LIMIT_CYCLES;   // SM cycles a device-side barrier wait may take
  std::vector<void*> allocs;
  std::string err;
};

namespace {

tt_status fail(tt_ctx* ctx, tt_status st, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof(buf), fmt, ap);
  va_end(ap);
  if (ctx) {
    ctx->err = buf;
  } else {
    std::lock_guard<std::mutex> lk(g_err_mu);
    g_create_err = buf;
  }
  return st;
}

void bind_slot(tt_ctx* ctx, int i) {
  const tt_ctx::Slot& sl = ctx->slots[i];
  ctx->frames_stage = sl.frames_stage; ctx->logits = sl.logits; ctx->probs = sl.probs; ctx->masks = sl.masks;
  ctx->bits = sl.bits; ctx->overlay = sl.overlay; ctx->results_dev = sl.results_dev; ctx->results_host = sl.results_host;
  ctx->status_host = sl.status_host; ctx->ev_start = sl.ev_start; ctx->ev_stop = sl.ev_stop; ctx->ev_copy = sl.ev_copy;
  for (int k = 0; k <= TT_STAGE_COUNT; ++k) ctx->stage_ev[k] = sl.stage_ev[k];
  for (int k = 0; k < TT_STAGE_COUNT; ++k) ctx->stage_ran[k] = sl.stage_ran[k];
  ctx->tick_profiled = sl.profiled;
  ctx->K_inflight = sl.K;
  for (int k = 0; k < TT_MAX_STREAMS; ++k) { ctx->frames_inflight[k] = sl.frames[k]; ctx->states_inflight[k] = sl.states[k]; }
  ctx->fp_inflight = sl.fp;
  ctx->bound = i;
}

void save_slot(tt_ctx* ctx, int i) {
  tt_ctx::Slot& sl = ctx->slots[i];
  sl.frames_stage = ctx->frames_stage; sl.logits = ctx->logits; sl.probs = ctx->probs; sl.masks = ctx->masks;
  sl.bits = ctx->bits; sl.overlay = ctx->overlay; sl.results_dev = ctx->results_dev; sl.results_host = ctx->results_host;
  sl.status_host = ctx->status_host; sl.ev_start = ctx->ev_start; sl.ev_stop = ctx->ev_stop; sl.ev_copy = ctx->ev_copy;
  for (int k = 0; k <= TT_STAGE_COUNT; ++k) sl.stage_ev[k] = ctx->stage_ev[k];
  for (int k = 0; k < TT_STAGE_COUNT; ++k) sl.stage_ran[k] = ctx->stage_ran[k];
  sl.profiled = ctx->tick_profiled;
  sl.K = ctx->K_inflight;
  for (int k = 0; k < TT_MAX_STREAMS; ++k) { sl.frames[k] = ctx->frames_inflight[k]; sl.states[k] = ctx->states_inflight[k]; }
  sl.fp = ctx->fp_inflight;
}

#define TT_CUDA(ctx, expr)                                                                         \
  do {                                                                                             \
    cudaError_t e_ = (expr);                                                                       \
    if (e_ != cudaSuccess)                                                                         \
      return fail(ctx, e_ == cudaErrorMemoryAllocation ? TT_ERR_OOM : TT_ERR_CUDA, "%s: %s", #expr, \
                  cudaGetErrorString(e_));                                                         \
  } while (0)

template <typename T>
tt_status dev_alloc(tt_ctx* ctx, T** out, size_t count, bool zero = true) {
  void* p = nullptr;
  const size_t bytes = (count * sizeof(T) + 255) & ~(size_t)255;
  TT_CUDA(ctx, cudaMalloc(&p, bytes ? bytes : 256));
  ctx->allocs.push_back(p);
  if (zero) TT_CUDA(ctx, cudaMemsetAsync(p, 0, bytes ? bytes : 256, ctx->stream));
  *out = reinterpret_cast<T*>(p);
  return TT_OK;
}

template <typename T>
tt_status upload(tt_ctx* ctx, T** out, const std::vector<T>& host) {
  tt_status st = dev_alloc(ctx, out, host.size(), false);
  if (st != TT_OK) return st;
  TT_CUDA(ctx, cudaMemcpy(*out, host.data(), host.size() * sizeof(T), cudaMemcpyHostToDevice));
  return TT_OK;
}

// OIHW fp32 -> [Cin][9][CoutPacked]; with lstm_hidden > 0 the packed output order groups, per
// block of ocb outputs, the four gates of ocb/4 consecutive hidden units (gate-major inside).
tt_status pack_simt(tt_ctx* ctx, SimtLayer* L, const float* w, const float* b, int cin, int cout, int stride, int ocb,
                    int lstm_hidden, bool round_bf16) {
  L->cin = cin; L->cout = cout; L->stride = stride; L->ocb = ocb;
  const int hb = ocb / 4;
  const int packed = lstm_hidden ? round_up(lstm_hidden, hb) * 4 : round_up(cout, ocb);
  L->cout_packed = packed;
  std::vector<float> hw((size_t)cin * 9 * packed, 0.f), hbias((size_t)packed, 0.f);
  for (int pk = 0; pk < packed; ++pk) {
    int o;
    if (lstm_hidden) {
      const int grp = pk / ocb, local = pk % ocb, gate = local / hb, jj = local % hb, j = grp * hb + jj;
      o = j < lstm_hidden ? gate * lstm_hidden + j : -1;
    } else {
      o = pk < cout ? pk : -1;
    }
    if (o < 0) continue;
    hbias[pk] = b ? b[o] : 0.f;
    for (int c = 0; c < cin; ++c)
      for (int t = 0; t < 9; ++t) {
        float v = w[((size_t)o * cin + c) * 9 + t];
        if (round_bf16) {
          uint32_t u = (uint32_t)f32_to_bf16_rne(v) << 16;
          std::memcpy(&v, &u, 4);
        }
        hw[((size_t)c * 9 + t) * packed + pk] = v;
      }
  }
  tt_status st = upload(ctx, &L->w, hw);
  if (st != TT_OK) return st;
  return upload(ctx, &L->b, hbias);
}

tt_status encode_map(tt_ctx* ctx, TensorMap128* out, void* base, int rank, const cuuint64_t* dims,
                     const cuuint64_t* strides_bytes, const cuuint32_t* box, int inner_bytes) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return fail(ctx, TT_ERR_CUDA, "cuTensorMapEncodeTiled entry point unavailable");
  cuuint32_t ones[5] = {1, 1, 1, 1, 1};
  const CUtensorMapSwizzle sw = inner_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
  CUresult r = fn(reinterpret_cast<CUtensorMap*>(out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, base, dims,
                  strides_bytes, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(ctx, TT_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  return TT_OK;
}

// Plain (unswizzled) map of an fp32 tensor.
tt_status encode_map_f32(tt_ctx* ctx, TensorMap128* out, void* base, int rank, const cuuint64_t* dims,
                         const cuuint64_t* strides_bytes, const cuuint32_t* box) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return fail(ctx, TT_ERR_CUDA, "cuTensorMapEncodeTiled entry point unavailable");
  cuuint32_t ones[5] = {1, 1, 1, 1, 1};
  CUresult r = fn(reinterpret_cast<CUtensorMap*>(out), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, (cuuint32_t)rank, base, dims,
                  strides_bytes, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(ctx, TT_ERR_CUDA, "cuTensorMapEncodeTiled (fp32) failed with code %d", (int)r);
  return TT_OK;
}

// Activation maps for one NHWC bf16 source [n_img][H][W][C] consumed at the given stride.
// stride 1: one map (index 0).  stride 2: four parity views, index ypar*2 + xpar.
tt_status make_act_maps(tt_ctx* ctx, TensorMap128* maps4, __nv_bfloat16* base, int n_img, int H, int W, int C,
                        int stride, int slab_c) {
  const cuuint32_t box[4] = {(cuuint32_t)slab_c, 16, 8, 1};
  if (stride == 1) {
    const cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)n_img};
    const cuuint64_t str[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
    return encode_map(ctx, &maps4[0], base, 4, dims, str, box, slab_c * 2);
  }
  for (int yp = 0; yp < 2; ++yp)
    for (int xp = 0; xp < 2; ++xp) {
      const int wv = xp ? W / 2 : (W + 1) / 2, hv = yp ? H / 2 : (H + 1) / 2;
      if (wv < 1 || hv < 1) return fail(ctx, TT_ERR_UNSUPPORTED, "stride-2 layer input smaller than 2x2");
      const cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)wv, (cuuint64_t)hv, (cuuint64_t)n_img};
      const cuuint64_t str[3] = {(cuuint64_t)2 * C * 2, (cuuint64_t)2 * W * C * 2, (cuuint64_t)H * W * C * 2};
      tt_status st = encode_map(ctx, &maps4[yp * 2 + xp], base + ((size_t)yp * W + xp) * C, 4, dims, str, box, slab_c * 2);
      if (st != TT_OK) return st;
    }
  return TT_OK;
}

// OIHW fp32 -> bf16 [CoutPacked][9*Cin] with column k = tap*Cin + c.  lstm_hidden > 0: packed
// row 4*j + gate holds original output channel gate*hidden + j.
tt_status pack_tc(tt_ctx* ctx, TcLayer* L, const float* w, const float* b, int cin0, int cin1, int cout, int stride,
                  int lstm_hidden) {
  const int cin = cin0 + cin1;
  L->cin0 = cin0; L->cin1 = cin1; L->cout = cout; L->stride = stride;
  const bool c64 = (cin0 % 64 == 0) && (cin1 % 64 == 0);
  const bool c32 = (cin0 % 32 == 0) && (cin1 % 32 == 0);
  if (!c32) return fail(ctx, TT_ERR_UNSUPPORTED, "bf16 tensor-core layers need input channels in multiples of 32 (got %d+%d)", cin0, cin1);
  L->slab_c = c64 ? 64 : 32;
  if (cout % 64 != 0) return fail(ctx, TT_ERR_UNSUPPORTED, "bf16 tensor-core layers need output channels in multiples of 64 (got %d)", cout);
  if (lstm_hidden && lstm_hidden % 16 != 0) return fail(ctx, TT_ERR_UNSUPPORTED, "bf16 ConvLSTM needs hidden in multiples of 16");
  const size_t ktot = (size_t)9 * cin;
  std::vector<uint16_t> hw((size_t)cout * ktot);
  std::vector<float> hb((size_t)cout);
  for (int pk = 0; pk < cout; ++pk) {
    const int o = lstm_hidden ? (pk & 3) * lstm_hidden + (pk >> 2) : pk;
    hb[pk] = b ? b[o] : 0.f;
    for (int c = 0; c < cin; ++c)
      for (int t = 0; t < 9; ++t) hw[(size_t)pk * ktot + (size_t)t * cin + c] = f32_to_bf16_rne(w[((size_t)o * cin + c) * 9 + t]);
  }
  uint16_t* dw = nullptr;
  tt_status st = upload(ctx, &dw, hw);
  if (st != TT_OK) return st;
  L->w = reinterpret_cast<__nv_bfloat16*>(dw);
  st = upload(ctx, &L->b, hb);
  if (st != TT_OK) return st;
  const int bns[3] = {64, 128, 256};
  for (int i = 0; i < 3; ++i) {
    L->has_b[i] = (cout % bns[i] == 0) && !(L->slab_c == 32 && bns[i] == 256);
    if (!L->has_b[i]) continue;
    const cuuint64_t dims[2] = {(cuuint64_t)ktot, (cuuint64_t)cout};
    const cuuint64_t str[1] = {(cuuint64_t)ktot * 2};
    const cuuint32_t box[2] = {(cuuint32_t)L->slab_c, (cuuint32_t)bns[i]};
    st = encode_map(ctx, &L->map_b[i], L->w, 2, dims, str, box, L->slab_c * 2);
    if (st != TT_OK) return st;
  }
  return TT_OK;
}

// two_per_sm: tiles up to 128 wide run two blocks per multiprocessor (encoder layers)
int pick_block_n(const TcLayer& L, int m_tiles, int sm_count, bool two_per_sm) {
  const int bns[3] = {64, 128, 256};
  int best = -1;
  double best_cost = 0;
  for (int i = 0; i < 3; ++i) {
    if (!L.has_b[i]) continue;
    const long tiles = (long)m_tiles * (L.cout / bns[i]);
    const int per_sm = (two_per_sm && bns[i] <= 128) ? 2 : 1;
    const long slots = (long)per_sm * sm_count;
    const long waves = (tiles + slots - 1) / slots;
    // Time of a tile: its main loop is paced by the thread that issues the MMAs (about 600 cycles
    // per K slab whatever the width) until the tensor pipe itself needs longer (2 cycles per
    // column and K slab of 64 at 128 rows, shared by the blocks of a multiprocessor).
    const double cost = (double)waves * std::max(600.0, 2.5 * bns[i] * per_sm);
    if (best < 0 || cost < best_cost - 1e-9 || (std::fabs(cost - best_cost) < 1e-9 && bns[i] > bns[best])) {
      best = i;
      best_cost = cost;
    }
  }
  return best;
}

tt_status validate(const tt_config* c, const tt_weights* w) {
  if (!c || !w) return fail(nullptr, TT_ERR_INVALID_ARG, "null config or weights");
  if (c->struct_size != sizeof(tt_config) || c->abi_version != TT_ABI_VERSION)
    return fail(nullptr, TT_ERR_INVALID_ARG, "tt_config struct_size/abi_version mismatch (%u/%u, expected %zu/%u)",
                c->struct_size, c->abi_version, sizeof(tt_config), TT_ABI_VERSION);
  if (c->max_streams < 1 || c->max_streams > TT_MAX_STREAMS) return fail(nullptr, TT_ERR_INVALID_ARG, "max_streams out of range");
  if (c->src_w < 2 || c->src_h < 2 || c->src_w > 16384 || c->src_h > 16384 || c->src_pitch < 3 * c->src_w)
    return fail(nullptr, TT_ERR_INVALID_ARG, "bad source frame geometry");
  if (c->net_w < 2 || c->net_h < 2 || c->net_w > 16384 || c->net_h > 16384) return fail(nullptr, TT_ERR_INVALID_ARG, "bad network input size");
  if (!(c->norm_div != 0.f) || !(c->norm_std != 0.f)) return fail(nullptr, TT_ERR_INVALID_ARG, "norm_div and norm_std must be non-zero");
  if (c->n_enc < 1 || c->n_enc > TT_MAX_ENC) return fail(nullptr, TT_ERR_INVALID_ARG, "n_enc out of range");
  for (int l = 0; l < c->n_enc; ++l) {
    if (c->enc_cout[l] < 1 || c->enc_cout[l] > 1024) return fail(nullptr, TT_ERR_INVALID_ARG, "enc_cout out of range");
    if (c->enc_stride[l] != 1 && c->enc_stride[l] != 2) return fail(nullptr, TT_ERR_INVALID_ARG, "enc_stride must be 1 or 2");
    if (!w->enc_w[l] || !w->enc_b[l]) return fail(nullptr, TT_ERR_INVALID_ARG, "missing encoder weights");
  }
  if (c->hidden < 4 || c->hidden > 512 || c->hidden % 4) return fail(nullptr, TT_ERR_UNSUPPORTED, "hidden must be a multiple of 4 in [4, 512]");
  if (c->n_tools < 1 || c->n_tools > TT_MAX_TOOLS) return fail(nullptr, TT_ERR_INVALID_ARG, "n_tools out of range");
  if (c->precision != TT_FP32 && c->precision != TT_BF16) return fail(nullptr, TT_ERR_INVALID_ARG, "bad precision");
  if (c->conf_mode != TT_CONF_MEAN_SIGMOID && c->conf_mode != TT_CONF_GAP_LINEAR) return fail(nullptr, TT_ERR_INVALID_ARG, "bad conf_mode");
  if (!(c->threshold > 0.f && c->threshold < 1.f)) return fail(nullptr, TT_ERR_INVALID_ARG, "threshold must lie in (0,1)");
  const bool ff = c->options[TT_OPT_FEED_FORWARD] != 0;
  if ((!ff && (!w->lstm_w || !w->lstm_b)) || !w->head_w || !w->head_b) return fail(nullptr, TT_ERR_INVALID_ARG, "missing weights");
  if (ff && c->hidden != c->enc_cout[c->n_enc - 1])
    return fail(nullptr, TT_ERR_INVALID_ARG, "a feed-forward model's `hidden` must equal its last encoder width (the heads read the encoder output)");
  if (c->conf_mode == TT_CONF_GAP_LINEAR && (!w->conf_w || !w->conf_b)) return fail(nullptr, TT_ERR_INVALID_ARG, "missing confidence-head weights");
  return TT_OK;
}

tt_status build(tt_ctx* ctx, const tt_weights* w) {
  const tt_config& c = ctx->cfg;
  cudaDeviceProp prop;
  TT_CUDA(ctx, cudaGetDeviceProperties(&prop, ctx->dev));
  if (prop.major != 10) return fail(ctx, TT_ERR_UNSUPPORTED, "device %d is sm_%d%d; this library is built for sm_100a only", ctx->dev, prop.major, prop.minor);
  ctx->sm_count = prop.multiProcessorCount;
  // multiprocessors left to another workload (TT_OPT_RESERVED_SMS): the persistent kernels size their grids for the rest
  if (c.options[TT_OPT_RESERVED_SMS] != 0) {
    if ((int)c.options[TT_OPT_RESERVED_SMS] > ctx->sm_count / 2)
      return fail(ctx, TT_ERR_INVALID_ARG, "at most half of the device's %d multiprocessors can be reserved", ctx->sm_count);
    ctx->sm_count -= (int)c.options[TT_OPT_RESERVED_SMS];
  }
  if (c.cuda_stream) {
    ctx->stream = reinterpret_cast<cudaStream_t>(c.cuda_stream);
  } else {
    TT_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->stream, cudaStreamNonBlocking));
    ctx->own_stream = true;
  }
  TT_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
  for (int i = 0; i < TT_STAGE_COUNT; ++i) ctx->stage_ms[i] = -1.f;
  TT_CUDA(ctx, post_prepare());

  const int S = c.max_streams;
  ctx->bf16 = c.precision == TT_BF16;
  ctx->n_enc = c.n_enc;
  ctx->lay_c[0] = 3; ctx->lay_h[0] = c.net_h; ctx->lay_w[0] = c.net_w;
  for (int l = 0; l < c.n_enc; ++l) {
    ctx->lay_c[l + 1] = c.enc_cout[l];
    ctx->lay_h[l + 1] = conv_out(ctx->lay_h[l], c.enc_stride[l]);
    ctx->lay_w[l + 1] = conv_out(ctx->lay_w[l], c.enc_stride[l]);
  }
  ctx->Hm = ctx->lay_h[c.n_enc]; ctx->Wm = ctx->lay_w[c.n_enc];
  ctx->Cx = ctx->lay_c[c.n_enc]; ctx->Ch = c.hidden; ctx->T = c.n_tools;
  if (ctx->Hm < 1 || ctx->Wm < 1) return fail(ctx, TT_ERR_INVALID_ARG, "encoder output is empty");
  const size_t plane = (size_t)ctx->Hm * ctx->Wm;
  ctx->frame_bytes = (size_t)c.src_h * c.src_pitch;
  ctx->zthr = (float)std::log((double)c.threshold / (1.0 - (double)c.threshold));

  tt_status st;
  if ((st = dev_alloc(ctx, &ctx->pre, (size_t)S * 3 * c.net_h * c.net_w)) != TT_OK) return st;
  size_t max_floats = (size_t)3 * c.net_h * c.net_w;
  for (int l = 0; l < c.n_enc; ++l) {
    const size_t n = (size_t)ctx->lay_c[l + 1] * ctx->lay_h[l + 1] * ctx->lay_w[l + 1];
    if (n > max_floats) max_floats = n;
    if (ctx->bf16) {
      __nv_bfloat16* p = nullptr;
      if ((st = dev_alloc(ctx, &p, (size_t)S * n)) != TT_OK) return st;
      ctx->enc_out[l] = p;
    } else {
      float* p = nullptr;
      if ((st = dev_alloc(ctx, &p, (size_t)S * n)) != TT_OK) return st;
      ctx->enc_out[l] = p;
    }
  }
  if ((size_t)ctx->Ch * plane > max_floats) max_floats = (size_t)ctx->Ch * plane;
  if ((size_t)ctx->T * plane > max_floats) max_floats = (size_t)ctx->T * plane;
  ctx->dbg_tmp_floats = max_floats;
  if ((st = dev_alloc(ctx, &ctx->dbg_tmp, max_floats)) != TT_OK) return st;
  if ((st = dev_alloc(ctx, &ctx->c_state, (size_t)S * ctx->Ch * plane)) != TT_OK) return st;
  if (ctx->bf16) {
    if ((st = dev_alloc(ctx, &ctx->h_f32, (size_t)S * ctx->Ch * plane)) != TT_OK) return st;
    if ((st = dev_alloc(ctx, &ctx->h_bf16, (size_t)S * 2 * ctx->Ch * plane)) != TT_OK) return st;
  } else {
    if ((st = dev_alloc(ctx, &ctx->h_f32, (size_t)S * 2 * ctx->Ch * plane)) != TT_OK) return st;
  }
  if ((st = dev_alloc(ctx, &ctx->status_dev, 1)) != TT_OK) return st;
  {
    uint8_t* scr = nullptr;
    if ((st = dev_alloc(ctx, &scr, post_scratch_bytes(S, ctx->Hm, ctx->Wm, ctx->Ch, ctx->T))) != TT_OK) return st;
    ctx->post_scratch = scr;
  }
  // per-slot resources
  for (int i = 0; i < TT_MAX_IN_FLIGHT; ++i) {
    tt_ctx::Slot& sl = ctx->slots[i];
    if ((st = dev_alloc(ctx, &sl.frames_stage, (size_t)S * ctx->frame_bytes + 16)) != TT_OK) return st;
    if ((st = dev_alloc(ctx, &sl.logits, (size_t)S * ctx->T * plane)) != TT_OK) return st;
    if ((st = dev_alloc(ctx, &sl.probs, (size_t)S * ctx->T * plane)) != TT_OK) return st;
    if ((st = dev_alloc(ctx, &sl.masks, (size_t)S * ctx->T * plane)) != TT_OK) return st;
    if ((st = dev_alloc(ctx, &sl.bits, (size_t)S * plane)) != TT_OK) return st;
    if (c.overlay && (st = dev_alloc(ctx, &sl.overlay, (size_t)S * c.src_w * c.src_h * 4)) != TT_OK) return st;
    if ((st = dev_alloc(ctx, &sl.results_dev, (size_t)S)) != TT_OK) return st;
    TT_CUDA(ctx, cudaHostAlloc(reinterpret_cast<void**>(&sl.results_host), sizeof(tt_result) * S, cudaHostAllocDefault));
    TT_CUDA(ctx, cudaHostAlloc(reinterpret_cast<void**>(&sl.status_host), sizeof(int32_t), cudaHostAllocDefault));
    *sl.status_host = 0;
    {
      uint64_t* tab = nullptr;
      if ((st = dev_alloc(ctx, &tab, (size_t)tt_ctx::FRAME_TABS * TT_MAX_STREAMS)) != TT_OK) return st;
      ctx->frame_tab_dev[i] = reinterpret_cast<const uint8_t**>(tab);
      TT_CUDA(ctx, cudaHostAlloc(reinterpret_cast<void**>(&ctx->frame_tab_host[i]), sizeof(void*) * TT_MAX_STREAMS, cudaHostAllocDefault));
    }
    TT_CUDA(ctx, cudaEventCreate(&sl.ev_start));
    TT_CUDA(ctx, cudaEventCreate(&sl.ev_stop));
    TT_CUDA(ctx, cudaEventCreateWithFlags(&sl.ev_copy, cudaEventDisableTiming));
    for (int k = 0; k <= TT_STAGE_COUNT; ++k) TT_CUDA(ctx, cudaEventCreate(&sl.stage_ev[k]));
  }
  bind_slot(ctx, 0);
  ctx->graphs_off = c.options[TT_OPT_PLAIN_LAUNCHES] != 0;
  ctx->cta_pairs = c.options[TT_OPT_CTA_PAIRS] != 0;
  ctx->enc_two_per_sm = c.options[TT_OPT_ENC_ONE_PER_SM] == 0;
  ctx->feed_forward = c.options[TT_OPT_FEED_FORWARD] != 0;
  const bool no_post_tc = c.options[TT_OPT_NO_POST_TC] != 0;

  // ---- weights
  const bool r = ctx->bf16;  // round weights to bf16 on the bf16 path
  {
    std::vector<float> hw(w->head_w, w->head_w + (size_t)ctx->T * ctx->Ch), hb(w->head_b, w->head_b + ctx->T);
    if (r) for (auto& v : hw) { uint32_t u = (uint32_t)f32_to_bf16_rne(v) << 16; std::memcpy(&v, &u, 4); }
    if ((st = upload(ctx, &ctx->head_w, hw)) != TT_OK) return st;
    if ((st = upload(ctx, &ctx->head_b, hb)) != TT_OK) return st;
    if (c.conf_mode == TT_CONF_GAP_LINEAR) {
      std::vector<float> cw(w->conf_w, w->conf_w + (size_t)ctx->T * ctx->Ch), cb(w->conf_b, w->conf_b + ctx->T);
      if (r) for (auto& v : cw) { uint32_t u = (uint32_t)f32_to_bf16_rne(v) << 16; std::memcpy(&v, &u, 4); }
      if ((st = upload(ctx, &ctx->conf_w, cw)) != TT_OK) return st;
      if ((st = upload(ctx, &ctx->conf_b, cb)) != TT_OK) return st;
    }
  }
  if (!ctx->bf16) {
    for (int l = 0; l < c.n_enc; ++l)
      if ((st = pack_simt(ctx, &ctx->simt_enc[l], w->enc_w[l], w->enc_b[l], ctx->lay_c[l], ctx->lay_c[l + 1],
                          c.enc_stride[l], ctx->lay_c[l + 1] > 16 ? 32 : 16, 0, false)) != TT_OK)
        return st;
    if (!ctx->feed_forward &&
        (st = pack_simt(ctx, &ctx->simt_lstm, w->lstm_w, w->lstm_b, ctx->Cx + ctx->Ch, 4 * ctx->Ch, 1,
                        ctx->Ch >= 8 ? 32 : 16, ctx->Ch, false)) != TT_OK)
      return st;
  } else {
    if (ctx->lay_c[1] % 8) return fail(ctx, TT_ERR_UNSUPPORTED, "bf16 path needs enc_cout[0] in multiples of 8");
    // the tensor-core first layer fetches its input patches with TMA: rows of the planar fp32 input must be 16-byte multiples
    if (conv_first_tc_supported(ctx->lay_c[1]) && c.net_w % 4 == 0 && (c.enc_stride[0] == 1 || c.enc_stride[0] == 2)) {
      const int co = ctx->lay_c[1];
      std::vector<uint16_t> wb((size_t)co * 27), packed((size_t)co * 32);
      for (size_t i = 0; i < wb.size(); ++i) wb[i] = f32_to_bf16_rne(w->enc_w[0][i]);
      conv_first_tc_pack(wb.data(), co, packed.data());
      std::vector<float> hb(w->enc_b[0], w->enc_b[0] + co);
      uint16_t* dw = nullptr;
      float* db = nullptr;
      if ((st = upload(ctx, &dw, packed)) != TT_OK) return st;
      if ((st = upload(ctx, &db, hb)) != TT_OK) return st;
      ConvFirstTcParams& f = ctx->first_tc;
      f.in = ctx->pre; f.out = reinterpret_cast<__nv_bfloat16*>(ctx->enc_out[0]);
      f.H = c.net_h; f.W = c.net_w; f.Ho = ctx->lay_h[1]; f.Wo = ctx->lay_w[1]; f.stride = c.enc_stride[0]; f.cout = co;
      f.tiles_x = (f.Wo + 15) / 16; f.tiles_y = (f.Ho + 7) / 8;
      f.w_packed = dw; f.bias = db; f.status = ctx->status_dev; f.wait_limit = ctx->wait_limit;
      {
        const cuuint64_t dims[4] = {(cuuint64_t)co, (cuuint64_t)f.Wo, (cuuint64_t)f.Ho, (cuuint64_t)S};
        const cuuint64_t str[3] = {(cuuint64_t)co * 2, (cuuint64_t)f.Wo * co * 2, (cuuint64_t)f.Ho * f.Wo * co * 2};
        const cuuint32_t box[4] = {(cuuint32_t)co, 16, 8, 1};
        if ((st = encode_map(ctx, &f.map_out, ctx->enc_out[0], 4, dims, str, box, co * 2)) != TT_OK) return st;
      }
      {
        const cuuint64_t dims[4] = {(cuuint64_t)f.W, (cuuint64_t)f.H, 3, (cuuint64_t)S};
        const cuuint64_t str[3] = {(cuuint64_t)f.W * 4, (cuuint64_t)f.H * f.W * 4, (cuuint64_t)3 * f.H * f.W * 4};
        const cuuint32_t box[4] = {(cuuint32_t)conv_first_tc_box_w(f.stride), (cuuint32_t)(7 * f.stride + 3), 3, 1};
        if ((st = encode_map_f32(ctx, &f.map_in, ctx->pre, 4, dims, str, box)) != TT_OK) return st;
      }
      ctx->use_first_tc = true;
      ctx->fuse_pre = c.options[TT_OPT_FUSED_PRE] != 0 &&
                      conv_first_tc_staging(f.stride, c.src_w, c.src_h, c.net_w, c.net_h, &f.src_rows_cap, &f.src_row_cap);
      f.fused = ctx->fuse_pre ? 1 : 0;
      f.src_w = c.src_w; f.src_h = c.src_h; f.src_pitch = c.src_pitch;
      f.scale = pre::norm_scale(1.0f / c.norm_div, 1.0f / c.norm_std);
      f.shift = pre::norm_shift(c.norm_mean, 1.0f / c.norm_std);
    } else if ((st = pack_simt(ctx, &ctx->simt_enc[0], w->enc_w[0], w->enc_b[0], 3, ctx->lay_c[1], c.enc_stride[0],
                               ctx->lay_c[1] > 16 ? 32 : 16, 0, true)) != TT_OK) {
      return st;
    }
    for (int l = 1; l < c.n_enc; ++l) {
      TcLayer& L = ctx->tc_enc[l];
      if ((st = pack_tc(ctx, &L, w->enc_w[l], w->enc_b[l], ctx->lay_c[l], 0, ctx->lay_c[l + 1], c.enc_stride[l], 0)) != TT_OK) return st;
      if ((st = make_act_maps(ctx, &L.maps_a[0], reinterpret_cast<__nv_bfloat16*>(ctx->enc_out[l - 1]), S, ctx->lay_h[l],
                              ctx->lay_w[l], ctx->lay_c[l], c.enc_stride[l], L.slab_c)) != TT_OK)
        return st;
    }
    TcLayer& L = ctx->tc_lstm;
    if (!ctx->feed_forward) {
      if ((st = pack_tc(ctx, &L, w->lstm_w, w->lstm_b, ctx->Cx, ctx->Ch, 4 * ctx->Ch, 1, ctx->Ch)) != TT_OK) return st;
      if ((st = make_act_maps(ctx, &L.maps_a[0], reinterpret_cast<__nv_bfloat16*>(ctx->enc_out[c.n_enc - 1]), S, ctx->Hm,
                              ctx->Wm, ctx->Cx, 1, L.slab_c)) != TT_OK)
        return st;
      if ((st = make_act_maps(ctx, &L.maps_a[4], ctx->h_bf16, 2 * S, ctx->Hm, ctx->Wm, ctx->Ch, 1, L.slab_c)) != TT_OK) return st;
      if (L.slab_c == 64 && !c.options[TT_OPT_NO_HALO]) {
        // haloed patch of an 8 x 16 output tile: 18 rows of 16 pixels (10 are needed; the pitch keeps the swizzle phase)
        const cuuint32_t box[4] = {64, 10, 18, 1};
        struct { __nv_bfloat16* base; int n_img, C; } srcs[2] = {{reinterpret_cast<__nv_bfloat16*>(ctx->enc_out[c.n_enc - 1]), S, ctx->Cx},
                                                                {ctx->h_bf16, 2 * S, ctx->Ch}};
        for (int i = 0; i < 2; ++i) {
          const cuuint64_t dims[4] = {(cuuint64_t)srcs[i].C, (cuuint64_t)ctx->Wm, (cuuint64_t)ctx->Hm, (cuuint64_t)srcs[i].n_img};
          const cuuint64_t str[3] = {(cuuint64_t)srcs[i].C * 2, (cuuint64_t)ctx->Wm * srcs[i].C * 2, (cuuint64_t)ctx->Hm * ctx->Wm * srcs[i].C * 2};
          if ((st = encode_map(ctx, &L.maps_halo[i], srcs[i].base, 4, dims, str, box, 128)) != TT_OK) return st;
        }
        L.has_halo = true;
      }
    } else if (no_post_tc || !post_tc_supported(ctx->Ch, (int)plane)) {
      return fail(ctx, TT_ERR_UNSUPPORTED, "a bf16 feed-forward model needs a last encoder width in multiples of 64 (at most 512) and "
                                           "a map of at least 128 pixels: its heads run on the tensor cores only");
    }
    if (!no_post_tc && post_tc_supported(ctx->Ch, (int)plane)) {
      // packed weights of both heads, bf16 [16][Ch] (the context's head weights are bf16 values already)
      std::vector<uint16_t> pw((size_t)16 * ctx->Ch, 0);
      for (int t = 0; t < ctx->T; ++t)
        for (int ch = 0; ch < ctx->Ch; ++ch) {
          pw[(size_t)t * ctx->Ch + ch] = f32_to_bf16_rne(w->head_w[(size_t)t * ctx->Ch + ch]);
          if (c.conf_mode == TT_CONF_GAP_LINEAR) pw[(size_t)(8 + t) * ctx->Ch + ch] = f32_to_bf16_rne(w->conf_w[(size_t)t * ctx->Ch + ch]);
        }
      uint16_t* dpw = nullptr;
      if ((st = upload(ctx, &dpw, pw)) != TT_OK) return st;
      PostTcParams& q = ctx->post_tc;
      {
        // the heads' input: the bf16 copy of the new hidden state, or a feed-forward model's last encoder output
        const cuuint64_t dims[3] = {(cuuint64_t)ctx->Ch, (cuuint64_t)plane, (cuuint64_t)(ctx->feed_forward ? S : 2 * S)};
        const cuuint64_t str[2] = {(cuuint64_t)ctx->Ch * 2, (cuuint64_t)plane * ctx->Ch * 2};
        const cuuint32_t box[3] = {64, 128, 1};
        void* src = ctx->feed_forward ? ctx->enc_out[c.n_enc - 1] : static_cast<void*>(ctx->h_bf16);
        if ((st = encode_map(ctx, &q.map_h, src, 3, dims, str, box, 128)) != TT_OK) return st;
      }
      {
        const cuuint64_t dims[2] = {(cuuint64_t)ctx->Ch, 16};
        const cuuint64_t str[1] = {(cuuint64_t)ctx->Ch * 2};
        const cuuint32_t box[2] = {64, 16};
        if ((st = encode_map(ctx, &q.map_w, dpw, 2, dims, str, box, 128)) != TT_OK) return st;
      }
      q.Hm = ctx->Hm; q.Wm = ctx->Wm; q.T = ctx->T; q.kslabs = ctx->Ch / 64;
      q.head_b = ctx->head_b; q.conf_b = ctx->conf_b; q.conf_mode = c.conf_mode; q.zthr = ctx->zthr;
      q.scratch = ctx->post_scratch; q.status = ctx->status_dev; q.wait_limit = ctx->wait_limit;
      ctx->use_post_tc = true;
    }
  }
  for (int i = 0; i < TT_MAX_STREAMS; ++i) {
    ctx->states[i].ctx = ctx;
    ctx->states[i].slot = i;
  }
  TT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  return TT_OK;
}

void release(tt_ctx* ctx) {
  if (!ctx) return;
  cudaSetDevice(ctx->dev);
  if (ctx->stream) cudaStreamSynchronize(ctx->stream);
  for (void* p : ctx->allocs) cudaFree(p);
  if (ctx->copy_stream) cudaStreamSynchronize(ctx->copy_stream);
  for (int i = 0; i < TT_MAX_IN_FLIGHT; ++i) {
    tt_ctx::Slot& sl = ctx->slots[i];
    if (sl.results_host) cudaFreeHost(sl.results_host);
    if (sl.status_host) cudaFreeHost(sl.status_host);
    if (sl.ev_start) cudaEventDestroy(sl.ev_start);
    if (sl.ev_stop) cudaEventDestroy(sl.ev_stop);
    if (sl.ev_copy) cudaEventDestroy(sl.ev_copy);
    for (int k = 0; k <= TT_STAGE_COUNT; ++k)
      if (sl.stage_ev[k]) cudaEventDestroy(sl.stage_ev[k]);
  }
  for (auto& g : ctx->graphs)
    if (g.exec) cudaGraphExecDestroy(g.exec);
  for (int i = 0; i < TT_MAX_IN_FLIGHT; ++i)
    if (ctx->frame_tab_host[i]) cudaFreeHost(ctx->frame_tab_host[i]);
  if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  if (ctx->own_stream && ctx->stream) cudaStreamDestroy(ctx->stream);
  delete ctx;
}

bool owns_state(const tt_ctx* ctx, const tt_state* st) {
  return st && st->ctx == ctx && st->slot >= 0 && st->slot < ctx->cfg.max_streams && st == &ctx->states[st->slot] && st->in_use;
}

// With profiling on, stage_ev[i + 1] is recorded right after stage i was enqueued; the stage's
// time is the span from the previous recorded event.
tt_status mark_stage(tt_ctx* ctx, int stage, int launches) {
  ctx->n_launches += (uint64_t)launches;
  if (!ctx->profiling) return TT_OK;
  TT_CUDA(ctx, cudaEventRecord(ctx->stage_ev[stage + 1], ctx->stream));
  ctx->stage_ran[stage] = true;
  return TT_OK;
}

PreprocessParams preprocess_params(const tt_ctx* ctx, int K, const FramePtrs& frames, const uint8_t* const* tab) {
  const tt_config& c = ctx->cfg;
  PreprocessParams pp;
  pp.src = frames; pp.src_tab = tab; pp.K = K; pp.src_w = c.src_w; pp.src_h = c.src_h; pp.src_pitch = c.src_pitch;
  pp.net_w = c.net_w; pp.net_h = c.net_h;
  pp.inv_div = 1.0f / c.norm_div; pp.mean = c.norm_mean; pp.inv_std = 1.0f / c.norm_std;
  pp.dst = ctx->pre;
  return pp;
}

// Launch sequence of one tick.  Everything is enqueued on ctx->stream.
tt_status enqueue_tick(tt_ctx* ctx, int K, const FramePtrs& frames, tt_state* const* states) {
  const tt_config& c = ctx->cfg;
  cudaStream_t s = ctx->stream;
  tt_status ms_;
  const size_t plane = (size_t)ctx->Hm * ctx->Wm;
  IdxMap ident, c_idx, h_in, h_out;
  for (int n = 0; n < TT_MAX_STREAMS; ++n) {
    ident.v[n] = n;
    const int slot = n < K ? states[n]->slot : 0, half = n < K ? states[n]->half : 0;
    c_idx.v[n] = slot;
    h_in.v[n] = slot * 2 + half;
    h_out.v[n] = slot * 2 + (1 - half);
  }

  if (!ctx->fuse_pre) {
    TT_CUDA(ctx, launch_preprocess(preprocess_params(ctx, K, frames, ctx->cur_tab), s));
    if ((ms_ = mark_stage(ctx, TT_STAGE_PREPROCESS, 1)) != TT_OK) return ms_;
  }

  if (!ctx->bf16) {
    const float* in = ctx->pre;
    for (int l = 0; l < ctx->n_enc; ++l) {
      const SimtLayer& L = ctx->simt_enc[l];
      ConvSimtParams q{};
      q.in0 = in; q.img_stride0 = (int64_t)ctx->lay_c[l] * ctx->lay_h[l] * ctx->lay_w[l]; q.idx0 = ident;
      q.C0 = ctx->lay_c[l]; q.C1 = 0;
      q.H = ctx->lay_h[l]; q.W = ctx->lay_w[l]; q.Ho = ctx->lay_h[l + 1]; q.Wo = ctx->lay_w[l + 1];
      q.stride = L.stride; q.K = K; q.wgt = L.w; q.bias = L.b; q.cout = L.cout; q.cout_packed = L.cout_packed; q.ocb = L.ocb;
      q.epilogue = EPI_RELU_F32_NCHW; q.out = ctx->enc_out[l];
      q.out_img_stride = (int64_t)L.cout * q.Ho * q.Wo;
      TT_CUDA(ctx, launch_conv_simt(q, s));
      if ((ms_ = mark_stage(ctx, TT_STAGE_ENC0 + l, 1)) != TT_OK) return ms_;
      in = reinterpret_cast<const float*>(ctx->enc_out[l]);
    }
    if (!ctx->feed_forward) {
    const SimtLayer& L = ctx->simt_lstm;
    ConvSimtParams q{};
    q.in0 = in; q.img_stride0 = (int64_t)ctx->Cx * plane; q.idx0 = ident; q.C0 = ctx->Cx;
    q.in1 = ctx->h_f32; q.img_stride1 = (int64_t)ctx->Ch * plane; q.idx1 = h_in; q.C1 = ctx->Ch;
    q.H = ctx->Hm; q.W = ctx->Wm; q.Ho = ctx->Hm; q.Wo = ctx->Wm; q.stride = 1; q.K = K;
    q.wgt = L.w; q.bias = L.b; q.cout = L.cout; q.cout_packed = L.cout_packed; q.ocb = L.ocb;
    q.epilogue = EPI_LSTM_F32_NCHW; q.c_state = ctx->c_state; q.h_state = ctx->h_f32; q.c_idx = c_idx; q.h_out_idx = h_out;
    q.hidden = ctx->Ch;
    TT_CUDA(ctx, launch_conv_simt(q, s));
    if ((ms_ = mark_stage(ctx, TT_STAGE_CONVLSTM, 1)) != TT_OK) return ms_;
    }
  } else {
    if (ctx->use_first_tc) {
      ctx->first_tc.K = K;
      // with the preprocessing inside it the kernel is the first of the tick and may follow a copy: launched normally
      ctx->first_tc.pdl = (ctx->profiling || ctx->fuse_pre) ? 0 : 1;
      ctx->first_tc.src = frames; ctx->first_tc.src_tab = ctx->cur_tab;
      TT_CUDA(ctx, launch_conv_first_tc(ctx->first_tc, ctx->sm_count, s));
      if ((ms_ = mark_stage(ctx, TT_STAGE_ENC0, 1)) != TT_OK) return ms_;
    } else {
      const SimtLayer& L = ctx->simt_enc[0];
      ConvSimtParams q{};
      q.in0 = ctx->pre; q.img_stride0 = (int64_t)3 * c.net_h * c.net_w; q.idx0 = ident; q.C0 = 3; q.C1 = 0;
      q.H = c.net_h; q.W = c.net_w; q.Ho = ctx->lay_h[1]; q.Wo = ctx->lay_w[1];
      q.stride = L.stride; q.K = K; q.wgt = L.w; q.bias = L.b; q.cout = L.cout; q.cout_packed = L.cout_packed; q.ocb = L.ocb;
      q.epilogue = EPI_RELU_BF16_NHWC; q.out = ctx->enc_out[0];
      q.out_img_stride = (int64_t)L.cout * q.Ho * q.Wo;
      TT_CUDA(ctx, launch_conv_simt(q, s));
      if ((ms_ = mark_stage(ctx, TT_STAGE_ENC0, 1)) != TT_OK) return ms_;
    }
    auto fill_common = [&](ConvTcParams& q, const TcLayer& L, int Ho, int Wo, bool encoder) -> tt_status {
      std::memcpy(q.maps_a, L.maps_a, sizeof(q.maps_a));
      q.slab_c = L.slab_c; q.stride = L.stride; q.K = K; q.Ho = Ho; q.Wo = Wo;
      q.tiles_x = (Wo + 15) / 16; q.tiles_y = (Ho + 7) / 8;
      const int bi = pick_block_n(L, K * q.tiles_x * q.tiles_y, ctx->sm_count, encoder && ctx->enc_two_per_sm);
      if (bi < 0) return fail(ctx, TT_ERR_UNSUPPORTED, "no tensor-core tile shape fits this layer");
      const int bns[3] = {64, 128, 256};
      q.block_n = bns[bi]; q.map_b = L.map_b[bi]; q.n_tiles_n = L.cout / q.block_n;
      // on request 256-wide tiles run on CTA pairs: each CTA stages its own activation box and half of the weight slab
      q.pair = (bi == 2 && L.slab_c == 64 && L.has_b[1] && ctx->cta_pairs && K * q.tiles_x * q.tiles_y >= 2) ? 1 : 0;
      if (q.pair) q.map_b = L.map_b[1];
      q.two_per_sm = (encoder && ctx->enc_two_per_sm) ? 1 : 0;
      if (!encoder && L.has_halo && !q.pair && (bi == 2 || bi == 1)) {
        q.halo = 1;
        q.maps_halo[0] = L.maps_halo[0];
        q.maps_halo[1] = L.maps_halo[1];
        q.tiles_x = (Wo + 7) / 8; q.tiles_y = (Ho + 15) / 16;
      }
      q.cout = L.cout; q.bias = L.b; q.status = ctx->status_dev; q.wait_limit = ctx->wait_limit;
      q.n_prod = 3;
      q.pdl = ctx->profiling ? 0 : 1;
      return TT_OK;
    };
    for (int l = 1; l < ctx->n_enc; ++l) {
      const TcLayer& L = ctx->tc_enc[l];
      ConvTcParams q{};
      tt_status st = fill_common(q, L, ctx->lay_h[l + 1], ctx->lay_w[l + 1], true);
      if (st != TT_OK) return st;
      q.n_src = 1; q.slabs[0] = L.cin0 / L.slab_c; q.slabs[1] = 0; q.img0 = ident; q.img1 = ident;
      // a weight matrix of at most 40 KB (64 outputs, up to 32 inputs x 9 taps) stays in shared memory for the whole launch
      q.wres = (q.two_per_sm && q.block_n == 64 && L.slab_c == 32 && q.n_tiles_n == 1 && 9 * q.slabs[0] * 64 * 32 * 2 <= 40 * 1024) ? 1 : 0;
      q.epilogue = TC_EPI_RELU_BF16; q.out = reinterpret_cast<__nv_bfloat16*>(ctx->enc_out[l]);
      TT_CUDA(ctx, launch_conv_tc(q, ctx->sm_count, s));
      if ((ms_ = mark_stage(ctx, TT_STAGE_ENC0 + l, 1)) != TT_OK) return ms_;
    }
    if (!ctx->feed_forward) {
    const TcLayer& L = ctx->tc_lstm;
    ConvTcParams q{};
    tt_status st = fill_common(q, L, ctx->Hm, ctx->Wm, false);
    if (st != TT_OK) return st;
    q.n_src = 2; q.slabs[0] = L.cin0 / L.slab_c; q.slabs[1] = L.cin1 / L.slab_c; q.img0 = ident; q.img1 = h_in;
    // with the heads on the tensor cores nothing on the path reads an fp32 copy of h': its consumers (the next
    // step's convolution and the heads) take the bf16 copy, so only that copy is written
    q.epilogue = TC_EPI_LSTM; q.c_state = ctx->c_state; q.h_f32 = ctx->use_post_tc ? nullptr : ctx->h_f32; q.h_bf16 = ctx->h_bf16;
    q.c_idx = c_idx; q.h_out_idx = h_out; q.hidden = ctx->Ch;
    TT_CUDA(ctx, launch_conv_tc(q, ctx->sm_count, s));
    if ((ms_ = mark_stage(ctx, TT_STAGE_CONVLSTM, 1)) != TT_OK) return ms_;
    }
  }

  if (ctx->use_post_tc) {
    PostTcParams& q = ctx->post_tc;
    q.idx = ctx->feed_forward ? ident : h_out; q.K = K;
    q.logits = ctx->logits; q.probs = ctx->probs; q.masks = ctx->masks; q.bits = ctx->bits; q.results = ctx->results_dev;
    q.pdl = ctx->profiling ? 0 : 1;
    TT_CUDA(ctx, launch_post_tc(q, ctx->sm_count, s));
    if ((ms_ = mark_stage(ctx, TT_STAGE_POSTPROCESS, 1)) != TT_OK) return ms_;
  } else {
  PostParams po{};
  po.h = ctx->h_f32; po.channels_last = ctx->bf16 ? 1 : 0; po.img_stride = (int64_t)ctx->Ch * plane;
  po.idx = ctx->bf16 ? c_idx : h_out;
  if (ctx->feed_forward) {   // fp32 path: the heads read the planar output of the last encoder layer
    po.h = reinterpret_cast<const float*>(ctx->enc_out[ctx->n_enc - 1]);
    po.idx = ident;
  }
  po.K = K; po.Hm = ctx->Hm; po.Wm = ctx->Wm; po.Ch = ctx->Ch; po.T = ctx->T;
  po.head_w = ctx->head_w; po.head_b = ctx->head_b; po.conf_w = ctx->conf_w; po.conf_b = ctx->conf_b;
  po.conf_mode = c.conf_mode; po.zthr = ctx->zthr;
  po.logits = ctx->logits; po.probs = ctx->probs; po.masks = ctx->masks; po.bits = ctx->bits;
  po.results = ctx->results_dev; po.scratch = ctx->post_scratch; po.status = ctx->status_dev; po.wait_limit = ctx->wait_limit;
  po.pdl = (ctx->bf16 && !ctx->profiling) ? 1 : 0;
  TT_CUDA(ctx, launch_postprocess(po, s));
  if ((ms_ = mark_stage(ctx, TT_STAGE_POSTPROCESS, 1)) != TT_OK) return ms_;
  }

  if (c.overlay) {
    OverlayParams ov{};
    ov.src = frames; ov.src_tab = ctx->cur_tab; ov.K = K; ov.src_w = c.src_w; ov.src_h = c.src_h; ov.src_pitch = c.src_pitch;
    ov.T = ctx->T; ov.Hm = ctx->Hm; ov.Wm = ctx->Wm; ov.masks = ctx->masks; ov.bits = ctx->bits;
    std::memcpy(ov.palette, c.palette, sizeof(ov.palette));
    ov.dst = ctx->overlay;
    TT_CUDA(ctx, launch_overlay(ov, s));
    if ((ms_ = mark_stage(ctx, TT_STAGE_OVERLAY, 1)) != TT_OK) return ms_;
  }
  ctx->n_ticks += 1;
  return TT_OK;
}

}  // namespace

// ====================================================================================== C ABI
extern "C" {

uint32_t tt_abi_version(void) { return TT_ABI_VERSION; }

const char* tt_last_error(const tt_ctx* ctx) {
  if (ctx) return ctx->err.c_str();
  std::lock_guard<std::mutex> lk(g_err_mu);
  return g_create_err.c_str();
}

tt_status tt_create(const tt_config* cfg, const tt_weights* weights, tt_ctx** out) {
  if (!out) return fail(nullptr, TT_ERR_INVALID_ARG, "null output pointer");
  *out = nullptr;
  tt_status st = validate(cfg, weights);
  if (st != TT_OK) return st;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev < 1) return fail(nullptr, TT_ERR_CUDA, "no CUDA device available");
  if (cfg->device < 0 || cfg->device >= n_dev) return fail(nullptr, TT_ERR_INVALID_ARG, "device ordinal out of range");
  tt_ctx* ctx = new (std::nothrow) tt_ctx();
  if (!ctx) return fail(nullptr, TT_ERR_OOM, "host allocation failed");
  ctx->cfg = *cfg;
  ctx->dev = cfg->device;
  if (cudaSetDevice(ctx->dev) != cudaSuccess) {
    delete ctx;
    return fail(nullptr, TT_ERR_CUDA, "cudaSetDevice failed");
  }
  st = build(ctx, weights);
  if (st != TT_OK) {
    fail(nullptr, st, "%s", ctx->err.c_str());
    release(ctx);
    return st;
  }
  *out = ctx;
  return TT_OK;
}

tt_status tt_destroy(tt_ctx* ctx) {
  release(ctx);
  return TT_OK;
}

tt_status tt_map_size(const tt_ctx* ctx, int32_t* hm, int32_t* wm) {
  if (!ctx || !hm || !wm) return TT_ERR_INVALID_ARG;
  *hm = ctx->Hm;
  *wm = ctx->Wm;
  return TT_OK;
}

static tt_status zero_state(tt_ctx* ctx, tt_state* st) {
  const size_t n = (size_t)ctx->Ch * ctx->Hm * ctx->Wm;
  TT_CUDA(ctx, cudaSetDevice(ctx->dev));
  TT_CUDA(ctx, cudaMemsetAsync(ctx->c_state + (size_t)st->slot * n, 0, n * sizeof(float), ctx->stream));
  if (ctx->bf16) {
    TT_CUDA(ctx, cudaMemsetAsync(ctx->h_f32 + (size_t)st->slot * n, 0, n * sizeof(float), ctx->stream));
    TT_CUDA(ctx, cudaMemsetAsync(ctx->h_bf16 + (size_t)st->slot * 2 * n, 0, 2 * n * sizeof(__nv_bfloat16), ctx->stream));
  } else {
    TT_CUDA(ctx, cudaMemsetAsync(ctx->h_f32 + (size_t)st->slot * 2 * n, 0, 2 * n * sizeof(float), ctx->stream));
  }
  st->half = 0;
  st->last_pos = -1;
  return TT_OK;
}

tt_status tt_state_create(tt_ctx* ctx, tt_state** out) {
  if (!ctx || !out) return TT_ERR_INVALID_ARG;
  *out = nullptr;
  if (ctx->q_count) return fail(ctx, TT_ERR_NOT_READY, "a submit is in flight");
  for (int i = 0; i < ctx->cfg.max_streams; ++i)
    if (!ctx->states[i].in_use) {
      ctx->states[i].in_use = true;
      tt_status st = zero_state(ctx, &ctx->states[i]);
      if (st != TT_OK) { ctx->states[i].in_use = false; return st; }
      *out = &ctx->states[i];
      return TT_OK;
    }
  return fail(ctx, TT_ERR_ADMISSION, "all %d state slots of this context are in use", ctx->cfg.max_streams);
}

tt_status tt_state_reset(tt_ctx* ctx, tt_state* st) {
  if (!ctx || !owns_state(ctx, st)) return ctx ? fail(ctx, TT_ERR_INVALID_ARG, "state does not belong to this context") : TT_ERR_INVALID_ARG;
  if (ctx->q_count) return fail(ctx, TT_ERR_NOT_READY, "a submit is in flight");
  return zero_state(ctx, st);
}

tt_status tt_state_export(tt_ctx* ctx, tt_state* st, float* h_host, float* c_host) {
  if (!ctx || !owns_state(ctx, st) || !h_host || !c_host) return ctx ? fail(ctx, TT_ERR_INVALID_ARG, "bad state or null buffer") : TT_ERR_INVALID_ARG;
  if (ctx->q_count) return fail(ctx, TT_ERR_NOT_READY, "a submit is in flight");
  if (ctx->feed_forward) return fail(ctx, TT_ERR_UNSUPPORTED, "a feed-forward model has no recurrent state");
  TT_CUDA(ctx, cudaSetDevice(ctx->dev));
  const int plane = ctx->Hm * ctx->Wm;
  const size_t n = (size_t)ctx->Ch * plane;
  if (ctx->bf16) {
    if (ctx->use_post_tc)   // h' exists as its bf16 copy only; every bf16 value is an fp32 value
      TT_CUDA(ctx, launch_nhwc_bf16_to_nchw_f32(ctx->h_bf16 + ((size_t)st->slot * 2 + st->half) * n, ctx->dbg_tmp, ctx->Ch, plane, ctx->stream));
    else
      TT_CUDA(ctx, launch_nhwc_to_nchw_f32(ctx->h_f32 + (size_t)st->slot * n, ctx->dbg_tmp, ctx->Ch, plane, ctx->stream));
    TT_CUDA(ctx, cudaMemcpyAsync(h_host, ctx->dbg_tmp, n * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
    TT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    TT_CUDA(ctx, launch_nhwc_to_nchw_f32(ctx->c_state + (size_t)st->slot * n, ctx->dbg_tmp, ctx->Ch, plane, ctx->stream));
    TT_CUDA(ctx, cudaMemcpyAsync(c_host, ctx->dbg_tmp, n * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
  } else {
    TT_CUDA(ctx, cudaMemcpyAsync(h_host, ctx->h_f32 + ((size_t)st->slot * 2 + st->half) * n, n * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
    TT_CUDA(ctx, cudaMemcpyAsync(c_host, ctx->c_state + (size_t)st->slot * n, n * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
  }
  TT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  return TT_OK;
}

tt_status tt_state_import(tt_ctx* ctx, tt_state* st, const float* h_host, const float* c_host) {
  if (!ctx || !owns_state(ctx, st) || !h_host || !c_host) return ctx ? fail(ctx, TT_ERR_INVALID_ARG, "bad state or null buffer") : TT_ERR_INVALID_ARG;
  if (ctx->q_count) return fail(ctx, TT_ERR_NOT_READY, "a submit is in flight");
  if (ctx->feed_forward) return fail(ctx, TT_ERR_UNSUPPORTED, "a feed-forward model has no recurrent state");
  TT_CUDA(ctx, cudaSetDevice(ctx->dev));
  const int plane = ctx->Hm * ctx->Wm;
  const size_t n = (size_t)ctx->Ch * plane;
  if (ctx->bf16) {
    TT_CUDA(ctx, cudaMemcpyAsync(ctx->dbg_tmp, h_host, n * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
    TT_CUDA(ctx, launch_nchw_to_nhwc_f32(ctx->dbg_tmp, ctx->h_f32 + (size_t)st->slot * n, ctx->Ch, plane, ctx->stream));
    TT_CUDA(ctx, launch_nchw_f32_to_nhwc_bf16(ctx->dbg_tmp, ctx->h_bf16 + ((size_t)st->slot * 2 + st->half) * n, ctx->Ch, plane, ctx->stream));
    TT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    TT_CUDA(ctx, cudaMemcpyAsync(ctx->dbg_tmp, c_host, n * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
    TT_CUDA(ctx, launch_nchw_to_nhwc_f32(ctx->dbg_tmp, ctx->c_state + (size_t)st->slot * n, ctx->Ch, plane, ctx->stream));
  } else {
    TT_CUDA(ctx, cudaMemcpyAsync(ctx->h_f32 + ((size_t)st->slot * 2 + st->half) * n, h_host, n * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
    TT_CUDA(ctx, cudaMemcpyAsync(ctx->c_state + (size_t)st->slot * n, c_host, n * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
  }
  TT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  return TT_OK;
}

tt_status tt_submit_frames(tt_ctx* ctx, int32_t K, const tt_frame* frames, tt_state* const* states) {
  if (!ctx) return TT_ERR_INVALID_ARG;
  if (!frames || !states || K < 1) return fail(ctx, TT_ERR_INVALID_ARG, "null frames/states or K < 1");
  if (K > ctx->cfg.max_streams)
    return fail(ctx, TT_ERR_ADMISSION, "K = %d streams exceed the %d this context was sized for", K, ctx->cfg.max_streams);
  if (ctx->q_count >= TT_MAX_IN_FLIGHT)
    return fail(ctx, TT_ERR_NOT_READY, "%d submits are already in flight; call tt_sync first", TT_MAX_IN_FLIGHT);
  for (int n = 0; n < K; ++n) {
    if (!owns_state(ctx, states[n])) return fail(ctx, TT_ERR_INVALID_ARG, "states[%d] is null or belongs to another context", n);
    if (!frames[n].data) return fail(ctx, TT_ERR_INVALID_ARG, "frames[%d].data is null", n);
    for (int m = 0; m < n; ++m)
      if (states[m] == states[n]) return fail(ctx, TT_ERR_INVALID_ARG, "states[%d] and states[%d] are the same state", m, n);
  }
  TT_CUDA(ctx, cudaSetDevice(ctx->dev));
  const int slot = (ctx->q_head + ctx->q_count) % TT_MAX_IN_FLIGHT;   // the oldest slot that is not in flight
  bind_slot(ctx, slot);
  cudaStream_t s = ctx->stream;
  for (int i = 0; i < TT_STAGE_COUNT; ++i) ctx->stage_ran[i] = false;
  ctx->stage_valid = false;
  ctx->tick_profiled = ctx->profiling;
  // The tick's start event goes in front of the first thing the tick enqueues.  With host frames or stage events that
  // is here; a tick of device-resident frames records it only when its launch is ready, so that the host work in
  // between (table look-ups, a graph capture) does not sit inside the device interval that gpu_ms reports.
  bool start_pending = true;
  auto record_start = [&]() -> cudaError_t {
    if (!start_pending) return cudaSuccess;
    start_pending = false;
    return cudaEventRecord(ctx->ev_start, s);
  };
  bool any_host = ctx->profiling;
  for (int n = 0; n < K; ++n) any_host |= !frames[n].on_device;
  if (any_host) TT_CUDA(ctx, record_start());
  if (ctx->profiling) TT_CUDA(ctx, cudaEventRecord(ctx->stage_ev[0], s));
  FramePtrs fp{};
  bool any_h2d = false;
  for (int n = 0; n < K; ++n) {
    if (frames[n].on_device) {
      fp.p[n] = frames[n].data;
    } else {
      // host frames go over a copy stream of their own, so the copy of this tick can run while the
      // previous tick still computes; the compute stream waits for the copy below
      uint8_t* dst = ctx->frames_stage + (size_t)n * ctx->frame_bytes;
      TT_CUDA(ctx, cudaMemcpyAsync(dst, frames[n].data, ctx->frame_bytes, cudaMemcpyHostToDevice, ctx->copy_stream));
      fp.p[n] = dst;
      any_h2d = true;
    }
  }
  tt_status st = TT_OK;
  if (any_h2d) {
    TT_CUDA(ctx, cudaEventRecord(ctx->ev_copy, ctx->copy_stream));
    TT_CUDA(ctx, cudaStreamWaitEvent(s, ctx->ev_copy, 0));
  }
  // frame pointers of this tick -> the slot's device table (the kernels read them from there).  The copy is
  // skipped when the table already holds these pointers: always the case for host frames (they are staged in
  // the slot's own buffer) and for callers whose frames arrive in a fixed set of device buffers.
  int tab = -1, oldest = 0;
  for (int i = 0; i < tt_ctx::FRAME_TABS && tab < 0; ++i) {
    bool same = ctx->frame_tab_valid[slot][i];
    for (int n = 0; n < TT_MAX_STREAMS && same; ++n) same = ctx->frame_tab_last[slot][i][n] == (n < K ? fp.p[n] : nullptr);
    if (same) tab = i;
    if (ctx->frame_tab_used[slot][i] < ctx->frame_tab_used[slot][oldest]) oldest = i;
  }
  const bool tab_miss = tab < 0;
  if (tab_miss) tab = oldest;
  ctx->frame_tab_used[slot][tab] = ctx->n_ticks + 1;
  ctx->cur_tab = ctx->frame_tab_dev[slot] + tab * TT_MAX_STREAMS;
  // refreshes the chosen table; called in front of the tick's launch (a graph capture, which enqueues nothing,
  // comes before it, so that its host time stays outside the interval between the tick's events)
  auto refresh_table = [&]() -> tt_status {
    TT_CUDA(ctx, record_start());
    if (tab_miss) {
      for (int n = 0; n < TT_MAX_STREAMS; ++n) ctx->frame_tab_last[slot][tab][n] = ctx->frame_tab_host[slot][n] = n < K ? fp.p[n] : nullptr;
      ctx->frame_tab_valid[slot][tab] = false;   // stays so if the copy cannot be enqueued
      TT_CUDA(ctx, cudaMemcpyAsync(ctx->frame_tab_dev[slot] + tab * TT_MAX_STREAMS, ctx->frame_tab_host[slot],
                                   sizeof(void*) * TT_MAX_STREAMS, cudaMemcpyHostToDevice, s));
      ctx->frame_tab_valid[slot][tab] = true;
    }
    // everything that moves host data to the device (frames, pointer table) counts as the H2D stage
    return mark_stage(ctx, TT_STAGE_H2D, 0);
  };

  // The launch sequence of a tick is replayed from a CUDA graph.  Which kernel variants a tick launches depends
  // on the stream count and the frames' alignment alone, so the first tick of such a family runs as plain
  // launches (modules load, attributes are set outside any capture); after it, every new (slot, pointer
  // table, state placement) of the family is captured the first time it shows up.  With stage events
  // requested the tick always runs as plain launches.
  tt_ctx::TickGraph* tg = nullptr;
  bool family_warm = false;
  if (!ctx->graphs_off && !ctx->profiling) {
    int flat = 1;
    // the overlay launch picks its word-wise variant from the frames' 4-byte alignment: part of the key
    for (int n = 0; n < K; ++n) flat &= (((uintptr_t)fp.p[n] & 3) == 0) ? 1 : 0;
    for (auto& g : ctx->graphs) {
      family_warm |= g.K == K && g.flat == flat && (g.seen >= 1 || g.exec);
      bool same = g.K == K && g.slot == slot && g.flat == flat && g.tab == tab;
      for (int n = 0; n < K && same; ++n) same = g.sig[n] == states[n]->slot * 2 + states[n]->half;
      if (same) { tg = &g; break; }
    }
    if (!tg) {
      if (ctx->graphs.size() >= 256) {            // bounded cache: drop everything and start over
        for (auto& g : ctx->graphs)
          if (g.exec) cudaGraphExecDestroy(g.exec);
        ctx->graphs.clear();
      }
      tt_ctx::TickGraph g;
      g.K = K; g.slot = slot; g.flat = flat; g.tab = tab;
      for (int n = 0; n < K; ++n) g.sig[n] = states[n]->slot * 2 + states[n]->half;
      ctx->graphs.push_back(g);
      tg = &ctx->graphs.back();
    }
  }
  if (tg && tg->exec) {
    if ((st = refresh_table()) != TT_OK) return st;
    TT_CUDA(ctx, cudaGraphLaunch(tg->exec, s));
    ctx->n_launches += tg->launches;
    ctx->n_ticks += 1;
  } else if (tg && (tg->seen >= 1 || family_warm)) {
    // capture the sequence (kernels plus the two result copies), then launch it
    const uint64_t launches_before = ctx->n_launches;
    cudaGraph_t graph = nullptr;
    cudaError_t ce = cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal);
    if (ce == cudaSuccess) {
      st = enqueue_tick(ctx, K, fp, states);
      if (st == TT_OK) {
        ce = cudaMemcpyAsync(ctx->results_host, ctx->results_dev, sizeof(tt_result) * K, cudaMemcpyDeviceToHost, s);
        if (ce == cudaSuccess) ce = cudaMemcpyAsync(ctx->status_host, ctx->status_dev, sizeof(int32_t), cudaMemcpyDeviceToHost, s);
      }
      cudaError_t ee = cudaStreamEndCapture(s, &graph);
      if (ce == cudaSuccess) ce = ee;
    }
    if (st == TT_OK && ce == cudaSuccess && graph) ce = cudaGraphInstantiate(&tg->exec, graph, 0);
    if (graph) cudaGraphDestroy(graph);
    if (st != TT_OK || ce != cudaSuccess || !tg->exec) {
      // capture is an optimisation only: clear the error, switch it off and run this tick directly
      cudaGetLastError();
      tg->exec = nullptr;
      ctx->graphs_off = true;
      ctx->n_launches = launches_before;
      ctx->n_ticks -= (st == TT_OK) ? 1 : 0;
      if ((st = refresh_table()) != TT_OK) return st;
      st = enqueue_tick(ctx, K, fp, states);
      if (st != TT_OK) return st;
      TT_CUDA(ctx, cudaMemcpyAsync(ctx->results_host, ctx->results_dev, sizeof(tt_result) * K, cudaMemcpyDeviceToHost, s));
      TT_CUDA(ctx, cudaMemcpyAsync(ctx->status_host, ctx->status_dev, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    } else {
      tg->launches = ctx->n_launches - launches_before;
      if ((st = refresh_table()) != TT_OK) return st;
      TT_CUDA(ctx, cudaGraphLaunch(tg->exec, s));
    }
  } else {
    if ((st = refresh_table()) != TT_OK) return st;
    st = enqueue_tick(ctx, K, fp, states);
    if (st != TT_OK) return st;
    TT_CUDA(ctx, cudaMemcpyAsync(ctx->results_host, ctx->results_dev, sizeof(tt_result) * K, cudaMemcpyDeviceToHost, s));
    TT_CUDA(ctx, cudaMemcpyAsync(ctx->status_host, ctx->status_dev, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    if (tg) tg->seen += 1;
  }
  TT_CUDA(ctx, cudaEventRecord(ctx->ev_stop, s));
  for (int n = 0; n < TT_MAX_STREAMS; ++n) ctx->states[n].last_pos = -1;
  for (int n = 0; n < K; ++n) {
    ctx->frames_inflight[n] = frames[n];
    ctx->states_inflight[n] = states[n];
    states[n]->half ^= 1;
    states[n]->last_pos = n;
  }
  ctx->K_inflight = K;
  ctx->fp_inflight = fp;
  save_slot(ctx, slot);
  ctx->q_count += 1;
  return TT_OK;
}

tt_status tt_sync(tt_ctx* ctx, tt_result* results) {
  if (!ctx) return TT_ERR_INVALID_ARG;
  if (ctx->q_count == 0) return fail(ctx, TT_ERR_NOT_READY, "nothing has been submitted");
  if (!results) return fail(ctx, TT_ERR_INVALID_ARG, "null results");
  TT_CUDA(ctx, cudaSetDevice(ctx->dev));
  const int slot = ctx->q_head;
  bind_slot(ctx, slot);
  if (ctx->cfg.sync_timeout_ns == 0) {
    TT_CUDA(ctx, cudaEventSynchronize(ctx->ev_stop));
  } else {
    const auto t0 = std::chrono::steady_clock::now();
    for (;;) {
      cudaError_t e = cudaEventQuery(ctx->ev_stop);
      if (e == cudaSuccess) break;
      if (e != cudaErrorNotReady) return fail(ctx, TT_ERR_CUDA, "cudaEventQuery: %s", cudaGetErrorString(e));
      const auto dt = std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now() - t0).count();
      if ((uint64_t)dt > ctx->cfg.sync_timeout_ns) return fail(ctx, TT_ERR_TIMEOUT, "tt_sync timed out after %llu ns", (unsigned long long)dt);
      std::this_thread::yield();
    }
  }
  ctx->q_head = (ctx->q_head + 1) % TT_MAX_IN_FLIGHT;
  ctx->q_count -= 1;
  ctx->last_done = slot;
  float ms = 0.f;
  TT_CUDA(ctx, cudaEventElapsedTime(&ms, ctx->ev_start, ctx->ev_stop));
  if (ctx->tick_profiled) {
    int prev = 0;  // index into stage_ev of the last recorded event
    for (int i = 0; i < TT_STAGE_COUNT; ++i) {
      ctx->stage_ms[i] = -1.f;
      if (!ctx->stage_ran[i]) continue;
      TT_CUDA(ctx, cudaEventElapsedTime(&ctx->stage_ms[i], ctx->stage_ev[prev], ctx->stage_ev[i + 1]));
      prev = i + 1;
    }
    ctx->stage_valid = true;
  }
  const size_t plane = (size_t)ctx->Hm * ctx->Wm;
  for (int n = 0; n < ctx->K_inflight; ++n) {
    tt_result r = ctx->results_host[n];
    r.frame_index = ctx->frames_inflight[n].frame_index;
    r.arrival_ns = ctx->frames_inflight[n].arrival_ns;
    r.masks_dev = ctx->masks + (size_t)n * ctx->T * plane;
    r.probs_dev = ctx->probs + (size_t)n * ctx->T * plane;
    r.overlay_dev = ctx->cfg.overlay ? ctx->overlay + (size_t)n * ctx->cfg.src_w * ctx->cfg.src_h * 4 : nullptr;
    r.gpu_ms = ms;
    r.reserved_ = 0;
    results[n] = r;
  }
  if (*ctx->status_host != 0) {
    const int code = *ctx->status_host;
    *ctx->status_host = 0;
    cudaMemsetAsync(ctx->status_dev, 0, sizeof(int32_t), ctx->stream);
    // a tick that gave up may have left partial sums in the post-processing accumulators
    cudaMemsetAsync(ctx->post_scratch, 0, post_scratch_bytes(ctx->cfg.max_streams, ctx->Hm, ctx->Wm, ctx->Ch, ctx->T), ctx->stream);
    return fail(ctx, TT_ERR_DEVICE_STATUS, "a kernel gave up a bounded wait (code 0x%x); results of this tick are invalid", code);
  }
  return TT_OK;
}

tt_status tt_query(tt_ctx* ctx) {
  if (!ctx) return TT_ERR_INVALID_ARG;
  if (ctx->q_count == 0) return TT_ERR_NOT_READY;
  cudaError_t e = cudaEventQuery(ctx->slots[ctx->q_head].ev_stop);
  if (e == cudaSuccess) return TT_OK;
  if (e == cudaErrorNotReady) return TT_ERR_NOT_READY;
  return fail(ctx, TT_ERR_CUDA, "cudaEventQuery: %s", cudaGetErrorString(e));
}

tt_status tt_debug_tensor(tt_ctx* ctx, tt_state* st, int32_t which, float* host_dst, size_t cap) {
  if (!ctx || !owns_state(ctx, st) || !host_dst) return ctx ? fail(ctx, TT_ERR_INVALID_ARG, "bad state or null buffer") : TT_ERR_INVALID_ARG;
  if (ctx->q_count) return fail(ctx, TT_ERR_NOT_READY, "a submit is in flight");
  TT_CUDA(ctx, cudaSetDevice(ctx->dev));
  const int plane = ctx->Hm * ctx->Wm;
  const int pos = st->last_pos;
  const float* src = nullptr;  // NCHW fp32 device source
  size_t n = 0;
  cudaStream_t s = ctx->stream;
  if (which == TT_TENSOR_H || which == TT_TENSOR_C) {
    n = (size_t)ctx->Ch * plane;
    if (cap < n) return fail(ctx, TT_ERR_INVALID_ARG, "buffer too small");
    std::vector<float> other(n);
    tt_status r = which == TT_TENSOR_H ? tt_state_export(ctx, st, host_dst, other.data()) : tt_state_export(ctx, st, other.data(), host_dst);
    return r;
  }
  if (pos < 0 || ctx->last_done < 0) return fail(ctx, TT_ERR_NOT_READY, "this state was not part of the last submit");
  bind_slot(ctx, ctx->last_done);
  if (which == TT_TENSOR_PRE) {
    n = (size_t)3 * ctx->cfg.net_h * ctx->cfg.net_w;
    if (ctx->fuse_pre) {
      // the resized image never reached memory: make it now, from the frame buffers of that submit
      TT_CUDA(ctx, launch_preprocess(preprocess_params(ctx, ctx->K_inflight, ctx->fp_inflight, nullptr), s));
    }
    src = ctx->pre + (size_t)pos * n;
  } else if (which >= TT_TENSOR_ENC0 && which < TT_TENSOR_ENC0 + ctx->n_enc) {
    const int l = which - TT_TENSOR_ENC0;
    const int C = ctx->lay_c[l + 1], pl = ctx->lay_h[l + 1] * ctx->lay_w[l + 1];
    n = (size_t)C * pl;
    if (ctx->bf16) {
      TT_CUDA(ctx, launch_nhwc_bf16_to_nchw_f32(reinterpret_cast<__nv_bfloat16*>(ctx->enc_out[l]) + (size_t)pos * n, ctx->dbg_tmp, C, pl, s));
      src = ctx->dbg_tmp;
    } else {
      src = reinterpret_cast<float*>(ctx->enc_out[l]) + (size_t)pos * n;
    }
  } else if (which == TT_TENSOR_LOGITS || which == TT_TENSOR_PROB) {
    n = (size_t)ctx->T * plane;
    src = (which == TT_TENSOR_LOGITS ? ctx->logits : ctx->probs) + (size_t)pos * n;
  } else {
    return fail(ctx, TT_ERR_INVALID_ARG, "unknown tensor id %d", which);
  }
  if (cap < n) return fail(ctx, TT_ERR_INVALID_ARG, "buffer too small: need %zu floats", n);
  TT_CUDA(ctx, cudaMemcpyAsync(host_dst, src, n * sizeof(float), cudaMemcpyDeviceToHost, s));
  TT_CUDA(ctx, cudaStreamSynchronize(s));
  return TT_OK;
}

tt_status tt_set_profiling(tt_ctx* ctx, int32_t on) {
  if (!ctx) return TT_ERR_INVALID_ARG;
  if (ctx->q_count) return fail(ctx, TT_ERR_NOT_READY, "a submit is in flight");
  ctx->profiling = on != 0;
  ctx->stage_valid = false;
  return TT_OK;
}

tt_status tt_get_stage_times(tt_ctx* ctx, float* ms) {
  if (!ctx || !ms) return TT_ERR_INVALID_ARG;
  for (int i = 0; i < TT_STAGE_COUNT; ++i) ms[i] = ctx->stage_valid ? ctx->stage_ms[i] : -1.f;
  return TT_OK;
}

tt_status tt_get_counters(const tt_ctx* ctx, uint64_t* kernel_launches, uint64_t* ticks) {
  if (!ctx || !kernel_launches || !ticks) return TT_ERR_INVALID_ARG;
  *kernel_launches = ctx->n_launches;
  *ticks = ctx->n_ticks;
  return TT_OK;
}

tt_status tt_debug_expire_wait(tt_ctx* ctx, uint64_t limit_cycles) {
  if (!ctx) return TT_ERR_INVALID_ARG;
  if (limit_cycles == 0 || limit_cycles > (uint64_t)DEFAULT_WAIT_LIMIT_CYCLES)
    return fail(ctx, TT_ERR_INVALID_ARG, "limit_cycles must lie in [1, %lld]", DEFAULT_WAIT_LIMIT_CYCLES);
  TT_CUDA(ctx, cudaSetDevice(ctx->dev));
  TT_CUDA(ctx, launch_wait_probe(ctx->status_dev, (long long)limit_cycles, 0xA00, ctx->stream));
  return TT_OK;
}

// ------------------------------------------------------------------------- stage-level calls
namespace {
inline bool misaligned(const void* p, uintptr_t a) { return ((uintptr_t)p & (a - 1)) != 0; }

// Argument checks shared by tt_postprocess and tt_postprocess_static.  Everything the kernels
// assume about sizes and alignment is checked here, on the host, so that a bad argument comes
// back as a status and never as a device fault.
tt_status check_post_args(const char* who, const float* h_dev, int32_t channels_last, int32_t K, int32_t hm, int32_t wm,
                          int32_t hidden, int32_t n_tools, const float* head_w_dev, const float* head_b_dev,
                          const float* conf_w_dev, const float* conf_b_dev, int32_t conf_mode, float threshold,
                          float* logits_dev, float* probs_dev, uint8_t* masks_dev, tt_result* results_dev) {
  if (!h_dev || !head_w_dev || !head_b_dev || !logits_dev || !probs_dev || !masks_dev || !results_dev || K < 1 ||
      K > TT_MAX_STREAMS || hm < 1 || wm < 1 || hm > 16384 || wm > 16384 || n_tools < 1 || n_tools > TT_MAX_TOOLS ||
      !(threshold > 0.f && threshold < 1.f) || (conf_mode != TT_CONF_MEAN_SIGMOID && conf_mode != TT_CONF_GAP_LINEAR) ||
      (conf_mode == TT_CONF_GAP_LINEAR && (!conf_w_dev || !conf_b_dev)))
    return fail(nullptr, TT_ERR_INVALID_ARG, "%s: bad argument", who);
  if (hidden < 4 || hidden > 512 || hidden % 4) return fail(nullptr, TT_ERR_UNSUPPORTED, "%s: hidden must be a multiple of 4 in [4, 512]", who);
  // channels-last rows are read with 128-bit loads; every fp32 tensor with 32-bit accesses; the result records hold 64-bit members
  if (misaligned(h_dev, channels_last ? 16 : 4) || misaligned(head_w_dev, 4) || misaligned(head_b_dev, 4) ||
      misaligned(conf_w_dev, 4) || misaligned(conf_b_dev, 4) || misaligned(logits_dev, 4) || misaligned(probs_dev, 4) ||
      misaligned(results_dev, 8))
    return fail(nullptr, TT_ERR_INVALID_ARG,
                "%s: misaligned pointer (h_dev needs %d-byte alignment, other fp32 tensors 4, results_dev 8)", who,
                channels_last ? 16 : 4);
  return TT_OK;
}
}  // namespace

tt_status tt_preprocess(const uint8_t* src_dev, int32_t K, int64_t src_frame_stride, int32_t src_w, int32_t src_h,
                        int32_t src_pitch, float* dst_dev, int32_t net_w, int32_t net_h, float norm_div,
                        float norm_mean, float norm_std, void* cuda_stream) {
  if (!src_dev || !dst_dev || K < 1 || K > TT_MAX_STREAMS || src_w < 1 || src_h < 1 || net_w < 1 || net_h < 1 ||
      src_w > 16384 || src_h > 16384 || net_w > 16384 || net_h > 16384 || src_pitch < 3 * src_w || norm_div == 0.f ||
      norm_std == 0.f)
    return fail(nullptr, TT_ERR_INVALID_ARG, "tt_preprocess: bad argument");
  if (misaligned(dst_dev, 4)) return fail(nullptr, TT_ERR_INVALID_ARG, "tt_preprocess: dst_dev must be 4-byte aligned");
  PreprocessParams p{};
  for (int n = 0; n < K; ++n) p.src.p[n] = src_dev + (size_t)n * src_frame_stride;
  p.K = K; p.src_w = src_w; p.src_h = src_h; p.src_pitch = src_pitch; p.net_w = net_w; p.net_h = net_h;
  p.inv_div = 1.0f / norm_div; p.mean = norm_mean; p.inv_std = 1.0f / norm_std; p.dst = dst_dev;
  cudaError_t e = launch_preprocess(p, reinterpret_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) return fail(nullptr, TT_ERR_CUDA, "tt_preprocess: %s", cudaGetErrorString(e));
  return TT_OK;
}

size_t tt_postprocess_scratch_bytes(int32_t K, int32_t hm, int32_t wm, int32_t hidden, int32_t n_tools) {
  if (K < 1 || hm < 1 || wm < 1 || hidden < 1 || n_tools < 1) return 0;
  return post_scratch_bytes(K, hm, wm, hidden, n_tools);
}

tt_status tt_postprocess(const float* h_dev, int32_t channels_last, int32_t K, int32_t hm, int32_t wm, int32_t hidden,
                         int32_t n_tools, const float* head_w_dev, const float* head_b_dev, const float* conf_w_dev,
                         const float* conf_b_dev, int32_t conf_mode, float threshold, float* logits_dev, float* probs_dev,
                         uint8_t* masks_dev, tt_result* results_dev, void* scratch_dev, void* cuda_stream) {
  tt_status a = check_post_args("tt_postprocess", h_dev, channels_last, K, hm, wm, hidden, n_tools, head_w_dev, head_b_dev,
                                conf_w_dev, conf_b_dev, conf_mode, threshold, logits_dev, probs_dev, masks_dev, results_dev);
  if (a != TT_OK) return a;
  if (!scratch_dev || misaligned(scratch_dev, 8))
    return fail(nullptr, TT_ERR_INVALID_ARG, "tt_postprocess: scratch_dev is null or not 8-byte aligned");
  cudaError_t e = post_prepare();
  if (e != cudaSuccess) return fail(nullptr, TT_ERR_CUDA, "tt_postprocess: %s", cudaGetErrorString(e));
  PostParams p{};
  p.h = h_dev; p.channels_last = channels_last; p.img_stride = (int64_t)hidden * hm * wm;
  for (int n = 0; n < TT_MAX_STREAMS; ++n) p.idx.v[n] = n;
  p.K = K; p.Hm = hm; p.Wm = wm; p.Ch = hidden; p.T = n_tools;
  p.head_w = head_w_dev; p.head_b = head_b_dev; p.conf_w = conf_w_dev; p.conf_b = conf_b_dev; p.conf_mode = conf_mode;
  p.zthr = (float)std::log((double)threshold / (1.0 - (double)threshold));
  p.logits = logits_dev; p.probs = probs_dev; p.masks = masks_dev; p.bits = nullptr; p.results = results_dev;
  p.scratch = scratch_dev;
  e = cudaMemsetAsync(scratch_dev, 0, post_scratch_bytes(K, hm, wm, hidden, n_tools), reinterpret_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) return fail(nullptr, TT_ERR_CUDA, "tt_postprocess: %s", cudaGetErrorString(e));
  e = launch_postprocess(p, reinterpret_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) return fail(nullptr, TT_ERR_CUDA, "tt_postprocess: %s", cudaGetErrorString(e));
  return TT_OK;
}

// Variant of tt_postprocess for callers that cannot allocate: same kernels, scratch taken from
// the array built into the library.  No allocation or free happens on this path.
tt_status tt_postprocess_static(const float* h_dev, int32_t channels_last, int32_t K, int32_t hm, int32_t wm,
                                int32_t hidden, int32_t n_tools, const float* head_w_dev, const float* head_b_dev,
                                const float* conf_w_dev, const float* conf_b_dev, int32_t conf_mode, float threshold,
                                float* logits_dev, float* probs_dev, uint8_t* masks_dev, tt_result* results_dev,
                                void* cuda_stream) {
  tt_status a = check_post_args("tt_postprocess_static", h_dev, channels_last, K, hm, wm, hidden, n_tools, head_w_dev,
                                head_b_dev, conf_w_dev, conf_b_dev, conf_mode, threshold, logits_dev, probs_dev, masks_dev,
                                results_dev);
  if (a != TT_OK) return a;
  const size_t need = post_scratch_bytes(K, hm, wm, hidden, n_tools);
  if (need > (size_t)TT_POSTPROCESS_STATIC_SCRATCH_BYTES)
    return fail(nullptr, TT_ERR_UNSUPPORTED,
                "tt_postprocess_static: this problem needs %zu bytes of scratch, the built-in array holds %u; "
                "use tt_postprocess with caller-provided scratch",
                need, (unsigned)TT_POSTPROCESS_STATIC_SCRATCH_BYTES);
  void* scratch = nullptr;
  cudaError_t e = post_static_scratch(&scratch);
  if (e != cudaSuccess) return fail(nullptr, TT_ERR_CUDA, "tt_postprocess_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
  e = post_prepare();
  if (e != cudaSuccess) return fail(nullptr, TT_ERR_CUDA, "tt_postprocess_static: %s", cudaGetErrorString(e));
  PostParams p{};
  p.h = h_dev; p.channels_last = channels_last; p.img_stride = (int64_t)hidden * hm * wm;
  for (int n = 0; n < TT_MAX_STREAMS; ++n) p.idx.v[n] = n;
  p.K = K; p.Hm = hm; p.Wm = wm; p.Ch = hidden; p.T = n_tools;
  p.head_w = head_w_dev; p.head_b = head_b_dev; p.conf_w = conf_w_dev; p.conf_b = conf_b_dev; p.conf_mode = conf_mode;
  p.zthr = (float)std::log((double)threshold / (1.0 - (double)threshold));
  p.logits = logits_dev; p.probs = probs_dev; p.masks = masks_dev; p.bits = nullptr; p.results = results_dev;
  p.scratch = scratch;
  // the accumulators in the shared array must start at zero, whatever an earlier call left there
  e = cudaMemsetAsync(scratch, 0, need, reinterpret_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) return fail(nullptr, TT_ERR_CUDA, "tt_postprocess_static: %s", cudaGetErrorString(e));
  e = launch_postprocess(p, reinterpret_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) return fail(nullptr, TT_ERR_CUDA, "tt_postprocess_static: %s", cudaGetErrorString(e));
  return TT_OK;
}

tt_status tt_overlay(const uint8_t* src_dev, int32_t K, int64_t src_frame_stride, int32_t src_w, int32_t src_h,
                     int32_t src_pitch, const uint8_t* masks_dev, int32_t n_tools, int32_t hm, int32_t wm,
                     const uint8_t* palette_host, uint8_t* dst_dev, void* cuda_stream) {
  if (!src_dev || !masks_dev || !palette_host || !dst_dev || K < 1 || K > TT_MAX_STREAMS || src_w < 1 || src_h < 1 ||
      src_w > 16384 || src_h > 16384 || src_pitch < 3 * src_w || n_tools < 1 || n_tools > TT_MAX_TOOLS || hm < 1 || wm < 1 ||
      hm > 16384 || wm > 16384)
    return fail(nullptr, TT_ERR_INVALID_ARG, "tt_overlay: bad argument");
  if (misaligned(dst_dev, 4)) return fail(nullptr, TT_ERR_INVALID_ARG, "tt_overlay: dst_dev must be 4-byte aligned (RGBA8 pixels are stored as words)");
  OverlayParams p{};
  for (int n = 0; n < K; ++n) p.src.p[n] = src_dev + (size_t)n * src_frame_stride;
  p.K = K; p.src_w = src_w; p.src_h = src_h; p.src_pitch = src_pitch; p.T = n_tools; p.Hm = hm; p.Wm = wm;
  p.masks = masks_dev; p.bits = nullptr;
  std::memcpy(p.palette, palette_host, (size_t)n_tools * 3);
  p.dst = dst_dev;
  cudaError_t e = launch_overlay(p, reinterpret_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) return fail(nullptr, TT_ERR_CUDA, "tt_overlay: %s", cudaGetErrorString(e));
  return TT_OK;
}

tt_status tt_render_layers(const uint8_t* src_dev, int32_t K, int64_t src_frame_stride, int32_t src_w, int32_t src_h,
                           int32_t src_pitch, const uint8_t* masks_dev, int32_t n_tools, int32_t hm, int32_t wm,
                           const uint8_t* palette_host, int32_t layers, int32_t carve_ctas, uint8_t* dst_dev,
                           void* cuda_stream) {
  if (!src_dev || !masks_dev || !palette_host || !dst_dev || K < 1 || K > TT_MAX_STREAMS || src_w < 1 || src_h < 1 ||
      src_w > 16384 || src_h > 16384 || src_pitch < 3 * src_w || n_tools < 1 || n_tools > TT_MAX_TOOLS || hm < 1 || wm < 1 ||
      hm > 16384 || wm > 16384 || layers < 1 || layers > 4096 || carve_ctas < 0 || carve_ctas > 65535)
    return fail(nullptr, TT_ERR_INVALID_ARG, "tt_render_layers: bad argument");
  if (misaligned(dst_dev, 4)) return fail(nullptr, TT_ERR_INVALID_ARG, "tt_render_layers: dst_dev must be 4-byte aligned");
  RenderParams p{};
  for (int n = 0; n < K; ++n) p.src.p[n] = src_dev + (size_t)n * src_frame_stride;
  p.K = K; p.src_w = src_w; p.src_h = src_h; p.src_pitch = src_pitch; p.T = n_tools; p.Hm = hm; p.Wm = wm;
  p.masks = masks_dev; p.layers = layers; p.carve_ctas = carve_ctas; p.dst = dst_dev;
  std::memcpy(p.palette, palette_host, (size_t)n_tools * 3);
  cudaError_t e = launch_render(p, reinterpret_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) return fail(nullptr, TT_ERR_CUDA, "tt_render_layers: %s", cudaGetErrorString(e));
  return TT_OK;
}

}  // extern "C"
