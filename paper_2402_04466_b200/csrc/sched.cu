// Host-side batch planner for unsynchronised stream arrivals (no CUDA calls in this file).
//
// The paper runs N independent application processes whose frames arrive unsynchronised and
// keeps them from interfering with an admission control that refuses a client the GPU cannot
// accommodate (Section IV-A, "Admission Control").  Here the K streams share one launch
// sequence, so the planner's job is (1) to coalesce frames that arrive while the GPU is busy into
// one tick without holding any frame longer than a small window (an idle GPU takes a frame at once), (2) to refuse a new stream when the
// predicted tick time with one more stream would eat more than the allowed share of the frame
// budget, and (3) to refuse a frame whose stream still has an older frame waiting (the stream has
// overrun its period; the newer frame is dropped and counted).  It plans only: the caller
// launches what tt_sched_next returns with tt_submit_frames and reports completion back.
#include <algorithm>
#include <cstring>
#include <deque>
#include <new>

#include "tt.h"

struct tt_sched {
  tt_sched_config cfg;
  bool admitted[TT_MAX_STREAMS];
  bool waiting[TT_MAX_STREAMS];
  uint64_t wait_index[TT_MAX_STREAMS];
  uint64_t wait_arrival[TT_MAX_STREAMS];
  int n_admitted = 0;
  struct Batch {
    int K;
    uint64_t arrival[TT_MAX_STREAMS];
  };
  std::deque<Batch> in_flight;
  float ewma_ms[TT_MAX_STREAMS + 1];
  bool seen[TT_MAX_STREAMS + 1];
  uint64_t n_batches = 0, n_frames = 0, n_dropped = 0, n_missed = 0;
};

namespace {

float predict(const tt_sched* s, int K) {
  if (K < 1) return 0.f;
  if (K > TT_MAX_STREAMS) K = TT_MAX_STREAMS;
  if (s->seen[K]) return s->ewma_ms[K];
  // nearest observed K, shifted by the prior's slope; the prior alone if nothing was observed yet
  int best = -1;
  for (int k = 1; k <= TT_MAX_STREAMS; ++k)
    if (s->seen[k] && (best < 0 || std::abs(k - K) < std::abs(best - K))) best = k;
  if (best < 0) return s->cfg.tick_ms_base + s->cfg.tick_ms_per_stream * (float)K;
  // extrapolating downwards with the prior's slope could cross zero; a tick of K streams never
  // costs less than the K/best share of an observed tick of `best` streams
  const float shifted = s->ewma_ms[best] + s->cfg.tick_ms_per_stream * (float)(K - best);
  const float floor_ms = K < best ? s->ewma_ms[best] * (float)K / (float)best : s->ewma_ms[best];
  return std::max(shifted, floor_ms);
}

}  // namespace

extern "C" {

tt_status tt_sched_create(const tt_sched_config* cfg, tt_sched** out) {
  if (!out) return TT_ERR_INVALID_ARG;
  *out = nullptr;
  if (!cfg || cfg->struct_size != sizeof(tt_sched_config)) return TT_ERR_INVALID_ARG;
  if (cfg->max_streams < 1 || cfg->max_streams > TT_MAX_STREAMS || cfg->max_in_flight < 1 || cfg->max_in_flight > 2 ||
      cfg->deadline_ns == 0 || !(cfg->budget_fraction > 0.f && cfg->budget_fraction <= 1.f) || cfg->tick_ms_base < 0.f ||
      cfg->tick_ms_per_stream < 0.f)
    return TT_ERR_INVALID_ARG;
  tt_sched* s = new (std::nothrow) tt_sched();
  if (!s) return TT_ERR_OOM;
  s->cfg = *cfg;
  for (int i = 0; i < TT_MAX_STREAMS; ++i) s->admitted[i] = s->waiting[i] = false;
  for (int i = 0; i <= TT_MAX_STREAMS; ++i) { s->seen[i] = false; s->ewma_ms[i] = 0.f; }
  *out = s;
  return TT_OK;
}

tt_status tt_sched_destroy(tt_sched* s) {
  delete s;
  return TT_OK;
}

tt_status tt_sched_admit(tt_sched* s, int32_t* stream_id) {
  if (!s || !stream_id) return TT_ERR_INVALID_ARG;
  *stream_id = -1;
  if (s->n_admitted >= s->cfg.max_streams) return TT_ERR_ADMISSION;
  const float budget_ms = (float)((double)s->cfg.deadline_ns * 1e-6) * s->cfg.budget_fraction;
  if (predict(s, s->n_admitted + 1) > budget_ms) return TT_ERR_ADMISSION;
  for (int i = 0; i < s->cfg.max_streams; ++i)
    if (!s->admitted[i]) {
      s->admitted[i] = true;
      s->waiting[i] = false;
      s->n_admitted += 1;
      *stream_id = i;
      return TT_OK;
    }
  return TT_ERR_ADMISSION;
}

tt_status tt_sched_release(tt_sched* s, int32_t stream_id) {
  if (!s || stream_id < 0 || stream_id >= s->cfg.max_streams || !s->admitted[stream_id]) return TT_ERR_INVALID_ARG;
  s->admitted[stream_id] = false;
  s->waiting[stream_id] = false;
  s->n_admitted -= 1;
  return TT_OK;
}

tt_status tt_sched_arrive(tt_sched* s, int32_t stream_id, uint64_t frame_index, uint64_t t_ns) {
  if (!s || stream_id < 0 || stream_id >= s->cfg.max_streams || !s->admitted[stream_id]) return TT_ERR_INVALID_ARG;
  if (s->waiting[stream_id]) {
    s->n_dropped += 1;  // the stream overran its period: its older frame is still waiting
    return TT_ERR_ADMISSION;
  }
  s->waiting[stream_id] = true;
  s->wait_index[stream_id] = frame_index;
  s->wait_arrival[stream_id] = t_ns;
  return TT_OK;
}

tt_status tt_sched_next(tt_sched* s, uint64_t now_ns, int32_t* K, int32_t* stream_ids, uint64_t* frame_indices,
                        uint64_t* arrival_ns, uint64_t* wake_ns) {
  if (!s || !K || !stream_ids || !frame_indices || !arrival_ns || !wake_ns) return TT_ERR_INVALID_ARG;
  *K = 0;
  *wake_ns = UINT64_MAX;
  int n_wait = 0;
  uint64_t oldest = UINT64_MAX;
  for (int i = 0; i < s->cfg.max_streams; ++i)
    if (s->admitted[i] && s->waiting[i]) {
      n_wait += 1;
      oldest = std::min(oldest, s->wait_arrival[i]);
    }
  if (n_wait == 0) return TT_OK;
  if ((int)s->in_flight.size() >= s->cfg.max_in_flight) return TT_OK;  // caller wakes on completion
  // Work-conserving: with nothing in flight a waiting frame launches at once (holding it back
  // would only add latency).  While a tick is in flight, frames are held so that they coalesce:
  // release when every admitted stream has a frame, when the oldest frame has waited out the
  // coalescing window, or when waiting any longer would push the oldest frame past its budget.
  const uint64_t tick_ns = (uint64_t)((double)predict(s, n_wait) * 1e6);
  const uint64_t budget_ns = (uint64_t)((double)s->cfg.deadline_ns * (double)s->cfg.budget_fraction);
  const bool idle = s->in_flight.empty();
  const bool all_present = n_wait == s->n_admitted;
  const bool window_over = now_ns >= oldest + s->cfg.window_ns;
  const bool deadline_near = now_ns + tick_ns >= oldest + budget_ns;
  if (!(idle || all_present || window_over || deadline_near)) {
    *wake_ns = std::min(oldest + s->cfg.window_ns, oldest + budget_ns > tick_ns ? oldest + budget_ns - tick_ns : oldest);
    return TT_OK;
  }
  tt_sched::Batch b;
  b.K = 0;
  for (int i = 0; i < s->cfg.max_streams; ++i)
    if (s->admitted[i] && s->waiting[i]) {
      stream_ids[b.K] = i;
      frame_indices[b.K] = s->wait_index[i];
      arrival_ns[b.K] = s->wait_arrival[i];
      b.arrival[b.K] = s->wait_arrival[i];
      s->waiting[i] = false;
      b.K += 1;
    }
  *K = b.K;
  s->in_flight.push_back(b);
  s->n_batches += 1;
  s->n_frames += (uint64_t)b.K;
  return TT_OK;
}

tt_status tt_sched_complete(tt_sched* s, float gpu_ms, uint64_t done_ns) {
  if (!s || !(gpu_ms >= 0.f)) return TT_ERR_INVALID_ARG;
  if (s->in_flight.empty()) return TT_ERR_NOT_READY;
  const tt_sched::Batch b = s->in_flight.front();
  s->in_flight.pop_front();
  if (!s->seen[b.K]) {
    s->seen[b.K] = true;
    s->ewma_ms[b.K] = gpu_ms;
  } else {
    s->ewma_ms[b.K] += 0.125f * (gpu_ms - s->ewma_ms[b.K]);
  }
  for (int i = 0; i < b.K; ++i)
    if (done_ns > b.arrival[i] + s->cfg.deadline_ns) s->n_missed += 1;
  return TT_OK;
}

tt_status tt_sched_predict_ms(const tt_sched* s, int32_t K, float* ms) {
  if (!s || !ms || K < 1 || K > TT_MAX_STREAMS) return TT_ERR_INVALID_ARG;
  *ms = predict(s, K);
  return TT_OK;
}

tt_status tt_sched_stats(const tt_sched* s, uint64_t* batches, uint64_t* frames, uint64_t* dropped, uint64_t* missed) {
  if (!s || !batches || !frames || !dropped || !missed) return TT_ERR_INVALID_ARG;
  *batches = s->n_batches;
  *frames = s->n_frames;
  *dropped = s->n_dropped;
  *missed = s->n_missed;
  return TT_OK;
}

}  // extern "C"
