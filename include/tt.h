/*
 * tt.h — C ABI of the B200-native per-frame hot path for K concurrent tool-tracking streams.
 *
 * Problem statement (paper, Sections I and V-B): N identical applications run at once,
 * each consuming its own frame stream through a recurrent model and producing per-frame
 * tracking output under an end-to-end latency budget.  Here the N applications become K
 * stream slots of one context on one GPU; every tick the K frames are batched into one
 * sequence of launches so that per-frame latency stays flat as K grows.
 *
 * The per-frame operator chain is the one of the paper's Endoscopy Tool Tracking
 * application (Section III-A): format conversion -> recurrent (LSTM) inference ->
 * tool-tracking post-processing -> overlay.  The paper does not give the arithmetic of
 * these operators; the definitions are stated with each call below.
 *
 * Conventions
 *   - plain C99 types only; every call returns tt_status and never aborts or throws;
 *   - "host" / "device" is stated for every pointer; device pointers must belong to the
 *     context's CUDA device;
 *   - all work is enqueued on the context's CUDA stream (paper Section III-A: one stream
 *     is allocated at format conversion and reused by the operators after it);
 *   - no entry point has a CPU fallback: without a usable sm_100 device calls fail with
 *     TT_ERR_CUDA / TT_ERR_UNSUPPORTED.
 */
#ifndef TT_H_
#define TT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TT_ABI_VERSION 1u
#define TT_MAX_STREAMS 8
#define TT_MAX_TOOLS 8
#define TT_MAX_ENC 4
#define TT_MAX_IN_FLIGHT 3   /* submits that may be in flight in one context */

typedef enum {
  TT_OK = 0,
  TT_ERR_INVALID_ARG = 1,   /* null pointer, bad size, duplicate state, wrong struct_size */
  TT_ERR_UNSUPPORTED = 2,   /* shape / precision combination the kernels do not cover */
  TT_ERR_OOM = 3,           /* device or host allocation failed */
  TT_ERR_CUDA = 4,          /* a CUDA runtime/driver call failed; see tt_last_error */
  TT_ERR_ADMISSION = 5,     /* more streams than the context was sized for (Section IV-A, admission control) */
  TT_ERR_NOT_READY = 6,     /* submit while TT_MAX_IN_FLIGHT submits are in flight, sync with nothing submitted, state access while in flight */
  TT_ERR_TIMEOUT = 7,       /* bounded wait expired; the device is left usable */
  TT_ERR_DEVICE_STATUS = 8  /* a kernel reported a bounded device-side wait that ran out */
} tt_status;

typedef enum { TT_FP32 = 0, TT_BF16 = 1 } tt_precision;
/* Indices into tt_config.options; a non-zero byte switches the option on. */
typedef enum {
  TT_OPT_PLAIN_LAUNCHES = 0, /* launch every tick as plain kernel launches, never from a CUDA graph */
  TT_OPT_FEED_FORWARD = 1,   /* the model has no recurrent cell: encoder -> mask/confidence heads (the paper's second
                                workload class, a feed-forward segmentation network, Section V-B); `hidden` must equal the
                                last encoder width, lstm_w/lstm_b are ignored, states carry nothing */
  TT_OPT_CTA_PAIRS = 2,      /* run 256-wide tensor-core tiles on CTA pairs (cta_group::2).  Off by default: measured
                                11-15 % slower than single-CTA tiles on the benchmark shapes */
  TT_OPT_RESERVED_SMS = 4,   /* value = number of multiprocessors left free for another workload (at most half of the
                                device): the persistent tensor-core and post-processing kernels size their grids for the
                                rest.  With tt_render_layers' carved-out form this gives the visualisation load its own
                                multiprocessors (the single-GPU isolation the paper leaves as future work, Section VIII) */
  TT_OPT_ENC_ONE_PER_SM = 5, /* run the tensor-core encoder layers with one block per multiprocessor instead of two
                                (for A/B measurements) */
  TT_OPT_NO_HALO = 6,        /* ConvLSTM fetches one activation box per tap instead of one haloed patch per channel
                                slab (for A/B measurements) */
  TT_OPT_FUSED_PRE = 7,      /* bf16 path: run the preprocessing inside the first encoder layer instead of as a kernel of its
                                own that writes the resized fp32 image (same bits; slower as measured, kept for A/B
                                measurements; ignored where the layer or the resize factor does not allow it) */
  TT_OPT_NO_POST_TC = 3      /* bf16 path: post-process from the fp32 hidden state, not from its bf16 copy on the
                                tensor cores (for A/B measurements; not available for feed-forward models) */
} tt_option;
typedef enum { TT_CONF_MEAN_SIGMOID = 0, TT_CONF_GAP_LINEAR = 1 } tt_conf_mode;

/* Which intermediate tensor tt_debug_tensor copies out (always NCHW fp32 on the host). */
typedef enum {
  TT_TENSOR_PRE = 0,      /* [3][net_h][net_w]                       */
  TT_TENSOR_ENC0 = 1,     /* [enc_cout[l]][H_l][W_l], l = which - 1  */
  TT_TENSOR_ENC1 = 2,
  TT_TENSOR_ENC2 = 3,
  TT_TENSOR_ENC3 = 4,
  TT_TENSOR_H = 8,        /* [hidden][Hm][Wm] state after the last step */
  TT_TENSOR_C = 9,
  TT_TENSOR_LOGITS = 10,  /* [n_tools][Hm][Wm] */
  TT_TENSOR_PROB = 11     /* [n_tools][Hm][Wm] */
} tt_tensor_id;

typedef struct {
  uint32_t struct_size;            /* = sizeof(tt_config) */
  uint32_t abi_version;            /* = TT_ABI_VERSION */
  int32_t device;                  /* CUDA device ordinal */
  int32_t max_streams;             /* K_max, 1..TT_MAX_STREAMS; also the number of state slots */
  int32_t src_w, src_h, src_pitch; /* uint8 RGB interleaved frames, pitch in bytes >= 3*src_w */
  int32_t net_w, net_h;            /* resize target */
  float norm_div, norm_mean, norm_std; /* out = ((v / div) - mean) / std */
  int32_t n_enc;                   /* 1..TT_MAX_ENC encoder layers: 3x3 conv, pad 1, bias, ReLU */
  int32_t enc_cout[TT_MAX_ENC];
  int32_t enc_stride[TT_MAX_ENC];  /* 1 or 2 */
  int32_t hidden;                  /* ConvLSTM hidden channels; 3x3, stride 1, pad 1 */
  int32_t n_tools;                 /* 1..TT_MAX_TOOLS */
  int32_t precision;               /* tt_precision */
  int32_t conf_mode;               /* tt_conf_mode */
  float threshold;                 /* on the sigmoid, in (0,1) */
  int32_t overlay;                 /* non-zero: also produce the RGBA8 overlay per frame */
  uint8_t palette[TT_MAX_TOOLS][3];
  uint8_t options[8];              /* indexed by tt_option; all zero = defaults */
  void* cuda_stream;               /* cudaStream_t owned by the caller, or NULL: the library creates one */
  uint64_t sync_timeout_ns;        /* 0: wait without limit in tt_sync */
} tt_config;

/* Host pointers, fp32, framework-conventional layouts.  Copied and repacked by tt_create;
 * the caller may free them afterwards.  On a TT_BF16 context every weight tensor is
 * rounded to bf16 (nearest even) while repacking; biases stay fp32. */
typedef struct {
  const float* enc_w[TT_MAX_ENC];  /* [Cout][Cin][3][3] */
  const float* enc_b[TT_MAX_ENC];  /* [Cout] */
  const float* lstm_w;             /* [4*hidden][Cx+hidden][3][3]; output blocks i|f|g|o, input channels x then h */
  const float* lstm_b;             /* [4*hidden] */
  const float* head_w;             /* [n_tools][hidden] */
  const float* head_b;             /* [n_tools] */
  const float* conf_w;             /* [n_tools][hidden]; NULL for TT_CONF_MEAN_SIGMOID */
  const float* conf_b;             /* [n_tools] */
} tt_weights;

typedef struct tt_ctx tt_ctx;     /* opaque, library-owned */
typedef struct tt_state tt_state; /* opaque recurrent state (h, c) of one stream, owned by its context */

typedef struct {
  const uint8_t* data;   /* [src_h][src_pitch] bytes; device memory if on_device != 0, else pinned host memory */
  int32_t on_device;
  int32_t reserved_;
  uint64_t frame_index;  /* echoed into the result */
  uint64_t arrival_ns;   /* caller's clock; echoed, not interpreted */
} tt_frame;

typedef struct {
  uint64_t frame_index;
  uint64_t arrival_ns;
  float conf[TT_MAX_TOOLS];
  float cx[TT_MAX_TOOLS];      /* mask centroid in mask-grid index coordinates; -1 when the mask is empty */
  float cy[TT_MAX_TOOLS];
  int32_t count[TT_MAX_TOOLS]; /* pixels above threshold */
  const uint8_t* masks_dev;    /* device, [n_tools][Hm][Wm] 0/1; valid until submit number TT_MAX_IN_FLIGHT after this one */
  const float* probs_dev;      /* device, [n_tools][Hm][Wm]; same lifetime */
  const uint8_t* overlay_dev;  /* device, [src_h][src_w][4] RGBA8, or NULL when overlay is off */
  float gpu_ms;                /* device time of the whole batch this frame was part of: from the first thing the tick
                                  enqueued (the host->device copies, for host frames) to its last */
  int32_t reserved_;
} tt_result;

uint32_t tt_abi_version(void);

/*
 * tt_create — build a context for one model and up to max_streams concurrent streams
 * (the paper's N concurrent application instances, Section V-B, all running the same
 * model).  Validates the configuration, allocates every activation, state and output
 * buffer for max_streams on cfg->device, repacks the weights into the kernels' internal
 * layouts and builds the TMA tensor maps.  On error *out is NULL; tt_last_error(NULL)
 * describes a failed create.
 */
tt_status tt_create(const tt_config* cfg, const tt_weights* weights, tt_ctx** out);

/* Frees everything the context owns, states included.  NULL is accepted. */
tt_status tt_destroy(tt_ctx* ctx);

/* Last error text of the context (or of the last failed tt_create when ctx is NULL).
 * The pointer stays valid until the next failing call on the same context. */
const char* tt_last_error(const tt_ctx* ctx);

/* Mask-grid (= encoder output = recurrent state) extent of the context. */
tt_status tt_map_size(const tt_ctx* ctx, int32_t* hm, int32_t* wm);

/*
 * Recurrent state of one stream.  The paper keeps it inside the inference operator
 * (Section III-A); here it is an explicit object so that streams can be reset, exported
 * and re-imported.  A context holds at most max_streams states (TT_ERR_ADMISSION beyond).
 * create/reset zero h and c.  export/import use host fp32 buffers [hidden][Hm][Wm]
 * (NCHW) and are synchronous with the context's stream.
 */
tt_status tt_state_create(tt_ctx* ctx, tt_state** out);
tt_status tt_state_reset(tt_ctx* ctx, tt_state* st);
tt_status tt_state_export(tt_ctx* ctx, tt_state* st, float* h_host, float* c_host);
tt_status tt_state_import(tt_ctx* ctx, tt_state* st, const float* h_host, const float* c_host);

/*
 * tt_submit_frames — enqueue one tick: the newest frame of K streams, each with its own
 * recurrent state, goes through the whole per-frame chain (Section III-A):
 *   S1 preprocess   bilinear resize (half-pixel centres, edge clamp, no antialias) of the
 *                   uint8 RGB frame to net_w x net_h, normalise, planar fp32;
 *   S2 encoder      n_enc x [3x3 conv, pad 1, stride enc_stride[l], bias, ReLU];
 *   S3 ConvLSTM     gates = W (*) concat[x, h] + b; c' = s(f) c + s(i) tanh(g); h' = s(o) tanh(c');
 *   S4 mask head    z = 1x1 conv(h') + b; p = sigmoid(z); mask = z > logit(threshold);
 *   S5 per tool     confidence (mean of p, or sigmoid(linear(global-average-pool(h')))),
 *                   count and centroid of the mask;
 *   S6 overlay      (if enabled) alpha-0.4 integer blend of the masks onto an RGBA8 copy.
 * Asynchronous: returns once the work is enqueued.  Up to TT_MAX_IN_FLIGHT submits may be in flight (the
 * host->device copies of the later ones overlap the compute of the first: with three, the copy engine
 * need not wait for the host between ticks; ticks execute in submit order, so a state may be used by
 * all of them); tt_sync returns them oldest first.  frames[k].data must
 * stay valid until the tt_sync of its submit returns.  Errors: K < 1 or null/duplicate/foreign states -> TT_ERR_INVALID_ARG;
 * K > max_streams -> TT_ERR_ADMISSION; TT_MAX_IN_FLIGHT submits already in flight -> TT_ERR_NOT_READY.
 * Nothing is enqueued when one of these argument errors is returned.
 */
tt_status tt_submit_frames(tt_ctx* ctx, int32_t K, const tt_frame* frames, tt_state* const* states);

/*
 * tt_sync — wait for the oldest submit in flight and fill results[0..K-1] (host, caller-owned,
 * same order as the submitted frames).  This is the "departure from the leaf operator" of
 * the paper's end-to-end latency definition (Section II-C).  With a non-zero
 * sync_timeout_ns the wait is bounded: TT_ERR_TIMEOUT leaves the submit in flight and the
 * call may be repeated.  TT_ERR_DEVICE_STATUS: a kernel gave up a bounded device-side
 * wait; results are invalid, the context stays usable.
 */
tt_status tt_sync(tt_ctx* ctx, tt_result* results);

/*
 * tt_debug_tensor — copy one intermediate tensor of the last completed submit for the
 * stream that used `st` into host_dst as NCHW fp32 (cap = capacity in floats).
 * Synchronous; for tests and parity checks only.
 */
tt_status tt_debug_tensor(tt_ctx* ctx, tt_state* st, int32_t which, float* host_dst, size_t cap);

/*
 * tt_query — non-blocking: TT_OK when the oldest submit in flight has finished (tt_sync will not
 * block), TT_ERR_NOT_READY when it is still running or nothing is in flight.
 */
tt_status tt_query(tt_ctx* ctx);

/*
 * Batch planner for unsynchronised arrivals (host logic only, no CUDA calls, no context needed).
 * The paper's N applications run unsynchronised (Section V-B) and are protected from each other
 * by an admission control that refuses a client the GPU cannot accommodate (Section IV-A,
 * "Admission Control").  With one shared launch sequence the same questions become: which
 * waiting frames go into the next tick, and may another stream join?
 *   - tt_sched_admit: a new stream is refused (TT_ERR_ADMISSION) when all max_streams slots are
 *     taken or when the predicted tick time with one more stream exceeds budget_fraction *
 *     deadline_ns.  The prediction is tick_ms_base + tick_ms_per_stream * K until ticks of that
 *     size have been observed, then an exponential average of the observed times.
 *   - tt_sched_arrive: a frame of an admitted stream arrived at t_ns (caller's monotonic clock).
 *     If the stream's previous frame is still waiting the new frame is dropped: TT_ERR_ADMISSION.
 *   - tt_sched_next: at time now_ns, returns in K / stream_ids / frame_indices / arrival_ns
 *     (arrays of max_streams entries) the batch to launch now, or K = 0 and in *wake_ns the time
 *     to ask again (UINT64_MAX: nothing waiting, or max_in_flight batches already launched — ask
 *     again after a completion).  With nothing in flight a waiting frame is released at once.
 *     While a batch is in flight, frames are held to coalesce and released as soon as every
 *     admitted stream has a frame waiting, or the oldest waiting frame has waited window_ns, or
 *     waiting longer would push the oldest frame past budget_fraction * deadline_ns given the
 *     predicted tick time.
 *   - tt_sched_complete: the oldest launched batch finished (device time gpu_ms, at done_ns);
 *     updates the cost model and counts frames that finished later than arrival + deadline_ns.
 */
typedef struct tt_sched tt_sched;
typedef struct {
  uint32_t struct_size;       /* = sizeof(tt_sched_config) */
  int32_t max_streams;        /* 1..TT_MAX_STREAMS */
  int32_t max_in_flight;      /* 1 or 2 batches launched and not yet completed */
  float budget_fraction;      /* share of deadline_ns one tick may take, in (0, 1] */
  uint64_t window_ns;         /* coalescing window */
  uint64_t deadline_ns;       /* per-frame latency budget, e.g. 16 666 667 */
  float tick_ms_base;         /* prior of the tick-time model */
  float tick_ms_per_stream;
} tt_sched_config;
tt_status tt_sched_create(const tt_sched_config* cfg, tt_sched** out);
tt_status tt_sched_destroy(tt_sched* s);
tt_status tt_sched_admit(tt_sched* s, int32_t* stream_id);
tt_status tt_sched_release(tt_sched* s, int32_t stream_id);
tt_status tt_sched_arrive(tt_sched* s, int32_t stream_id, uint64_t frame_index, uint64_t t_ns);
tt_status tt_sched_next(tt_sched* s, uint64_t now_ns, int32_t* K, int32_t* stream_ids, uint64_t* frame_indices,
                        uint64_t* arrival_ns, uint64_t* wake_ns);
tt_status tt_sched_complete(tt_sched* s, float gpu_ms, uint64_t done_ns);
tt_status tt_sched_predict_ms(const tt_sched* s, int32_t K, float* ms);
tt_status tt_sched_stats(const tt_sched* s, uint64_t* batches, uint64_t* frames, uint64_t* dropped, uint64_t* missed);

/*
 * Measurement hooks (the paper times every operator's input and output, Section II-C, data
 * flow tracking; here CUDA events on the context's stream bracket each stage of a tick).
 * tt_set_profiling(on != 0) makes every following submit record stage events.
 * tt_get_stage_times fills ms[TT_STAGE_COUNT] (host) with the device time of each stage of
 * the last completed submit, -1 for stages that did not run or when profiling was off.
 * tt_get_counters reports how many of the library's kernels and ticks this context has
 * launched since creation.
 */
typedef enum {
  TT_STAGE_H2D = 0,        /* host->device frame copies (frames with on_device == 0) */
  TT_STAGE_PREPROCESS = 1,
  TT_STAGE_ENC0 = 2,       /* encoder layer l = stage 2 + l */
  TT_STAGE_ENC1 = 3,
  TT_STAGE_ENC2 = 4,
  TT_STAGE_ENC3 = 5,
  TT_STAGE_CONVLSTM = 6,
  TT_STAGE_POSTPROCESS = 7,
  TT_STAGE_OVERLAY = 8,
  TT_STAGE_COUNT = 9
} tt_stage;
tt_status tt_set_profiling(tt_ctx* ctx, int32_t on);
tt_status tt_get_stage_times(tt_ctx* ctx, float* ms);
tt_status tt_get_counters(const tt_ctx* ctx, uint64_t* kernel_launches, uint64_t* ticks);

/*
 * tt_debug_expire_wait — failure-path probe, for tests.  Every barrier wait inside the kernels is
 * bounded: when one runs out the kernel records a code in the context's status word and returns,
 * and the tt_sync of that tick answers TT_ERR_DEVICE_STATUS (the paper's systems have no such
 * path; it is this library's reading of "a failed client must not take the GPU down with it",
 * Section IV-A).  This call enqueues, on the context's stream, one warp that waits through that
 * same bounded wait on a barrier nothing ever completes, with a limit of limit_cycles SM cycles
 * (1 .. 4e9; about 2e6 is a millisecond), records its code and returns.  The next tt_sync
 * therefore reports TT_ERR_DEVICE_STATUS, clears the status word, and the context is usable as before.
 * Nothing traps, faults or waits without bound.
 */
tt_status tt_debug_expire_wait(tt_ctx* ctx, uint64_t limit_cycles);

/* ---------------------------------------------------------------------------------------
 * Stage-level entry points on caller-owned device buffers (no context needed).  They run
 * the same kernels as the corresponding stage of tt_submit_frames and are asynchronous on
 * `cuda_stream` (a cudaStream_t, NULL = default stream).
 * ------------------------------------------------------------------------------------ */

/*
 * tt_preprocess — S1, the format-conversion operator of Section III-A.
 * src_dev: K frames, frame k at src_dev + k*src_frame_stride bytes, uint8 RGB interleaved,
 * row pitch src_pitch bytes (any alignment).  dst_dev: fp32 [K][3][net_h][net_w], 4-byte aligned
 * (16-byte alignment with net_w a multiple of 4 lets the kernel use 128-bit stores).  For output sample o of
 * an axis resized from `in` to `out`: s = clamp((o+1/2)*in/out - 1/2, 0, in-1) evaluated in
 * exact integer arithmetic, i0 = floor(s), i1 = min(i0+1, in-1), weight s - i0.
 */
tt_status tt_preprocess(const uint8_t* src_dev, int32_t K, int64_t src_frame_stride, int32_t src_w,
                        int32_t src_h, int32_t src_pitch, float* dst_dev, int32_t net_w, int32_t net_h,
                        float norm_div, float norm_mean, float norm_std, void* cuda_stream);

/*
 * tt_postprocess — S4+S5, the tool-tracking post-processing operator of Section III-A.
 * h_dev: fp32 hidden state of K streams, channels-last [K][Hm][Wm][hidden] when
 * channels_last != 0 (16-byte aligned), else planar [K][hidden][Hm][Wm] (4-byte aligned).  head_w/head_b (and conf_w/conf_b
 * for TT_CONF_GAP_LINEAR) are device fp32 [n_tools][hidden] / [n_tools].
 * Outputs (device): logits, probs fp32 [K][n_tools][Hm][Wm]; masks uint8 same shape;
 * results: K tt_result records (8-byte aligned) of which conf, cx, cy, count are written.
 * scratch_dev: tt_postprocess_scratch_bytes(...) bytes of device memory, 8-byte aligned; the call
 * clears it first, contents on entry are ignored.
 * hidden must be a multiple of 4 and at most 512; hm, wm at most 16384.  A misaligned or null
 * pointer is answered with TT_ERR_INVALID_ARG before anything is launched.  The stage-level calls
 * have no status word: a bounded device-side wait that ran out inside them (which no healthy
 * device produces) leaves the outputs incomplete without an error code; contexts report it
 * through tt_sync.
 */
size_t tt_postprocess_scratch_bytes(int32_t K, int32_t hm, int32_t wm, int32_t hidden, int32_t n_tools);
tt_status tt_postprocess(const float* h_dev, int32_t channels_last, int32_t K, int32_t hm, int32_t wm,
                         int32_t hidden, int32_t n_tools, const float* head_w_dev, const float* head_b_dev,
                         const float* conf_w_dev, const float* conf_b_dev, int32_t conf_mode, float threshold,
                         float* logits_dev, float* probs_dev, uint8_t* masks_dev, tt_result* results_dev,
                         void* scratch_dev, void* cuda_stream);

/*
 * tt_postprocess_static — the same computation as tt_postprocess for callers that must not
 * allocate device memory.  The paper has no counterpart for this call; it exists for users of
 * this library that run where cudaMalloc is off limits: code inside a real-time frame loop
 * that promised its host application a fixed memory footprint, plug-ins that are handed their
 * buffers by a framework's own allocator, and callers that keep a whole device reserved by
 * another pool.  Nothing is allocated or freed here, neither through CUDA nor through any
 * library (one exception: the very first call on a device makes the CUDA runtime load the
 * library's device code, which the runtime does with allocations of its own; see below): the partial sums that tt_postprocess keeps in caller-provided scratch live in a
 * fixed array of TT_POSTPROCESS_STATIC_SCRATCH_BYTES that is part of the library image (each
 * GPU that loads the library holds that much memory until the process ends).  Inputs and
 * outputs are still the caller's.
 *
 * Limits and rules:
 *   - tt_postprocess_scratch_bytes(K, hm, wm, hidden, n_tools) must not exceed
 *     TT_POSTPROCESS_STATIC_SCRATCH_BYTES, else TT_ERR_UNSUPPORTED is returned and nothing runs
 *     (32 KiB: 256 + K * 8 * (hidden + 32) bytes rounded up to 256, so 8 streams fit with up to 476
 *     hidden channels whatever the grid size; 8 streams of 512 hidden channels need 35 KB and are
 *     refused, 7 such streams fit);
 *   - the first call on a device looks up the array's device address and sets the kernels'
 *     shared-memory attributes (with that device current); make that first call, once, in a
 *     set-up phase and before starting any stream capture;
 *   - all calls on a device share the one array.  It keeps whatever the previous call left; the
 *     accumulators in it must start at zero, so every call clears the part it uses (a memset on
 *     `cuda_stream`) before its kernel runs.  Two calls whose kernels overlap on the GPU
 *     (different streams without an ordering between them) race on the array.  Serialise them.
 * Everything else (arguments, layouts, outputs, errors) is as for tt_postprocess.
 */
#define TT_POSTPROCESS_STATIC_SCRATCH_BYTES (32u << 10)
tt_status tt_postprocess_static(const float* h_dev, int32_t channels_last, int32_t K, int32_t hm, int32_t wm,
                                int32_t hidden, int32_t n_tools, const float* head_w_dev, const float* head_b_dev,
                                const float* conf_w_dev, const float* conf_b_dev, int32_t conf_mode, float threshold,
                                float* logits_dev, float* probs_dev, uint8_t* masks_dev, tt_result* results_dev,
                                void* cuda_stream);

/*
 * tt_overlay — S6, the stand-in for the visualisation operator of Section II-B / III-A
 * (mask overlay on the frame).  src_dev as in tt_preprocess; masks_dev uint8
 * [K][n_tools][Hm][Wm]; palette: n_tools RGB triples (host); dst_dev uint8
 * [K][src_h][src_w][4], 4-byte aligned.  Mask sample for source pixel (x, y): (floor(x*Wm/src_w),
 * floor(y*Hm/src_h)); tools blended in ascending order as (153*rgb + 102*colour + 127)/255.
 */
tt_status tt_overlay(const uint8_t* src_dev, int32_t K, int64_t src_frame_stride, int32_t src_w, int32_t src_h,
                     int32_t src_pitch, const uint8_t* masks_dev, int32_t n_tools, int32_t hm, int32_t wm,
                     const uint8_t* palette_host, uint8_t* dst_dev, void* cuda_stream);

/*
 * tt_render_layers — a scaled-up stand-in for the visualisation load.  The paper finds that the
 * visualisation work sharing a GPU with the inference work is what spreads the latencies
 * (Section VI) and names single-GPU isolation of the two as future work (Section VIII).  This
 * call is the "graphics" side of that experiment in CUDA: a full-resolution blend of `layers`
 * layers; layer l applies tt_overlay's blend with tool t drawn in palette colour (t + l) mod
 * n_tools, on the result of layer l - 1.  Arguments as for tt_overlay.
 * carve_ctas == 0: time-shared form, one block per 1024 pixels spread over the whole device.
 * carve_ctas  > 0: carved-out form, that many blocks loop over the batch, each claiming 64 KB of
 * shared memory so that the inference path's large blocks are not placed beside it; give the
 * inference context TT_OPT_RESERVED_SMS = carve_ctas so that it leaves those multiprocessors free.
 * The arithmetic per pixel does not depend on the mask values.
 */
tt_status tt_render_layers(const uint8_t* src_dev, int32_t K, int64_t src_frame_stride, int32_t src_w, int32_t src_h,
                           int32_t src_pitch, const uint8_t* masks_dev, int32_t n_tools, int32_t hm, int32_t wm,
                           const uint8_t* palette_host, int32_t layers, int32_t carve_ctas, uint8_t* dst_dev,
                           void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* TT_H_ */
