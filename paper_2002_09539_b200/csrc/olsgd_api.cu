// C ABI of libolsgd: context, argument checks, workspace carving, stream and
// event choreography of one Overlap-Local-SGD period.  No arithmetic of the
// method happens on the host; every step is a kernel launch.
#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <utility>
#include <vector>

#include "olsgd_internal.h"

using namespace olsgd;

namespace {

thread_local std::string g_last_error;

constexpr size_t kAlign = 256;
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct ProfRec {
  int cls, tag;
  cudaEvent_t start, stop;
};

}  // namespace

struct olsgd_ctx {
  olsgd_model_spec spec;
  olsgd_hparams hp;
  olsgd_data data;
  int64_t P = 0, ld = 0;

  // device state, carved from the caller's workspace
  float* x[2] = {nullptr, nullptr};  // ping-pong worker models [m][ld]
  int cur = 0;                       // x[cur] holds x_k
  float* u = nullptr;                // local momentum [m][ld]
  float* g = nullptr;                // stacked gradients [m][ld] (model modes)
  float* z = nullptr;                // anchor [ld]
  float* v = nullptr;                // anchor momentum [ld]
  float* tmp = nullptr;              // [ld] scratch for olsgd_get_params
  __nv_bfloat16* shadow = nullptr;   // bf16 copy of x_k [m][ld] (tensor-core path)
  int32_t* idx = nullptr;            // [m][batch]
  int32_t* idx_next = nullptr;       // [m][batch], indices of the minibatch staged ahead
  int32_t* ident = nullptr;          // [m][batch], ident[i][j] = j
  int* dev_status = nullptr;         // one word: a kernel's bounded wait gave up
  int64_t* dev_k = nullptr;          // iteration number read by the index kernel inside a graph
  float* loss_ring = nullptr;        // [graph_block][m] losses of one replayed block
  float* stage_x[2] = {nullptr, nullptr};  // host-fed minibatches [m][batch][d_in]
  void* stage_y[2] = {nullptr, nullptr};   // [m][batch] targets / labels
  ModelBuffers mb;

  cudaStream_t main = nullptr, side = nullptr;
  cudaStream_t copy = nullptr;       // owned: host-to-device staging copies
  cudaStream_t aux = nullptr;        // owned: backward-pass work beside the critical path
  cudaEvent_t aux_fork = nullptr, aux_join = nullptr;
  // Staging of the next iteration's minibatch beside the current iteration (bf16 path, index
  // rule with replacement): the rows of iteration pre_k are, or are being, staged into set
  // pre_k % 2 on stream `pre`; pre_pending: the main stream has not yet waited for pre_done.
  cudaStream_t pre = nullptr;
  cudaEvent_t pre_begin = nullptr, pre_done = nullptr;
  // recorded on the main stream when an iteration has finished reading staged-minibatch set b
  cudaEvent_t set_free[2] = {nullptr, nullptr};
  bool set_free_valid[2] = {false, false};   // false: the event does not cover the set's last reader
  bool pre_pending = false;
  int64_t pre_k = -1;
  cudaEvent_t pullback_done = nullptr, reduce_done = nullptr;
  cudaEvent_t h2d_done[2] = {nullptr, nullptr}, stage_free[2] = {nullptr, nullptr};
  // host-fed steps hand their losses to the host on stream `pre`, off the main stream (a copy
  // between two steps' kernels would hold up the next step's first launch): loss_read marks
  // the end of that copy, which the next kernel that writes the loss buffer must wait for
  cudaEvent_t loss_read = nullptr;
  bool loss_read_pending = false;
  int host_slot = 0;
  bool reduce_pending = false;  // an anchor refresh was launched and not yet waited for
  int reduce_reads = -1;        // which x buffer that refresh reads
  // Sync steps form the worker sum inside the launches that write x_{k+1} (the fused
  // weight-gradient launch, the stand-alone update kernel on long ranges): sum_part is the
  // [S][ld] scratch of partial sums, `summed` the ranges (offset, length) of a row that the
  // sync step which closed this period covered that way; the anchor refresh takes those from
  // the partial sums and the rest of the row from the worker models.
  bool anchor_fusion = false;
  float* sum_part = nullptr;
  std::vector<std::pair<int64_t, int64_t>> summed;
  int64_t last_summed = 0;   // parameters per row the most recent refresh took from sum_part
  bool need_sync = false;       // a period ended; olsgd_period_sync is due
  bool sync_begun = false;      // olsgd_period_sync_begin ran; _finish is due

  // graph_block: default length of a captured block; graph_len: length of the block that
  // graph_exec holds (a short run that is repeated is captured whole, up to kMaxGraphBlock);
  // plain_steps: iterations launched kernel by kernel so far (one-time kernel set-up happens
  // there, never inside a capture).
  int graph_len = 0;
  int64_t plain_steps = 0, plain_syncs = 0;
  // olsgd_run replays a captured CUDA graph of `graph_block` iterations (a whole number of
  // periods, an even number of steps so that the ping-pong buffers return to their places)
  int graph_block = 0;
  cudaGraphExec_t graph_exec = nullptr;
  int graph_cur = -1;            // c->cur at capture time
  int graph_kpar = -1;           // parity of k at capture time (selects the staged-minibatch set)
  bool graph_staged = false;     // the captured block starts from rows staged ahead
  bool graph_off = false;        // capture failed once: stay on the plain path
  bool capturing = false;        // the index kernel reads k from dev_k
  int64_t capture_k0 = 0;        // k at the start of the block being captured
  int64_t graph_launches = 0;    // kernel launches of one block
  int64_t graph_replays = 0;

  int device = -1;              // ordinal of the device the context was created on
  int64_t k = 0;
  int64_t launches = 0;
  bool prof = false;
  std::vector<ProfRec> prof_pending;
  std::vector<cudaEvent_t> prof_pool;
  // per kernel class and, inside a class, per tag (the layer a launch belongs to, else 0)
  int64_t prof_launches[OLSGD_N_KERNEL_CLASSES][OLSGD_MAX_DIMS] = {{0}};
  double prof_ms[OLSGD_N_KERNEL_CLASSES][OLSGD_MAX_DIMS] = {{0}};
  std::string err;
};

namespace {

olsgd_status fail(olsgd_ctx* ctx, olsgd_status st, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (ctx) ctx->err = buf;
  g_last_error = buf;
  return st;
}

#define OLSGD_CUDA(ctx, call)                                                             \
  do {                                                                                    \
    cudaError_t e_ = (call);                                                              \
    if (e_ != cudaSuccess)                                                                \
      return fail(ctx, OLSGD_ECUDA, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(e_), \
                  __FILE__, __LINE__);                                                    \
  } while (0)

// A context belongs to the device that was current in olsgd_init: its workspace, streams and
// events live there, and kernel attributes are configured per device.
olsgd_status check_device(olsgd_ctx* c) {
  const int dev = current_device();
  if (dev != c->device)
    return fail(c, OLSGD_ESTATE, "the context was created on device %d but device %d is current",
                c->device, dev);
  return OLSGD_OK;
}
#define OLSGD_ON_DEVICE(c)                          \
  do {                                              \
    olsgd_status ds_ = check_device(c);             \
    if (ds_ != OLSGD_OK) return ds_;                \
  } while (0)

// Brackets one kernel launch: counts it and, when profiling, times it with
// events on the launching stream.
struct Launch {
  olsgd_ctx* c;
  cudaStream_t s;
  ProfRec rec{};
  bool timed = false;
  // code = kernel class + 256 * tag
  Launch(olsgd_ctx* ctx, int code, cudaStream_t stream) : c(ctx), s(stream) {
    const int cls = code & 0xFF;
    c->launches++;
    if (!c->prof) return;
    auto get = [&]() {
      cudaEvent_t e = nullptr;
      if (!c->prof_pool.empty()) {
        e = c->prof_pool.back();
        c->prof_pool.pop_back();
      } else if (cudaEventCreate(&e) != cudaSuccess) {
        e = nullptr;
      }
      return e;
    };
    rec.cls = cls;
    rec.tag = (code >> 8) & (OLSGD_MAX_DIMS - 1);
    rec.start = get();
    rec.stop = get();
    if (rec.start && rec.stop) {
      timed = true;
      cudaEventRecord(rec.start, s);
    }
  }
  ~Launch() {
    if (timed) {
      cudaEventRecord(rec.stop, s);
      c->prof_pending.push_back(rec);
    }
  }
};

void free_host_side(olsgd_ctx* c) {
  for (auto& r : c->prof_pending) {
    cudaEventDestroy(r.start);
    cudaEventDestroy(r.stop);
  }
  for (auto e : c->prof_pool) cudaEventDestroy(e);
  if (c->pullback_done) cudaEventDestroy(c->pullback_done);
  if (c->reduce_done) cudaEventDestroy(c->reduce_done);
  for (int b = 0; b < 2; ++b) {
    if (c->h2d_done[b]) cudaEventDestroy(c->h2d_done[b]);
    if (c->stage_free[b]) cudaEventDestroy(c->stage_free[b]);
  }
  if (c->copy) cudaStreamDestroy(c->copy);
  if (c->aux_fork) cudaEventDestroy(c->aux_fork);
  if (c->aux_join) cudaEventDestroy(c->aux_join);
  if (c->aux) cudaStreamDestroy(c->aux);
  if (c->pre_begin) cudaEventDestroy(c->pre_begin);
  if (c->pre_done) cudaEventDestroy(c->pre_done);
  if (c->loss_read) cudaEventDestroy(c->loss_read);
  for (int b = 0; b < 2; ++b)
    if (c->set_free[b]) cudaEventDestroy(c->set_free[b]);
  if (c->pre) cudaStreamDestroy(c->pre);
  if (c->graph_exec) cudaGraphExecDestroy(c->graph_exec);
  delete c;
}

ProfHook make_hook(olsgd_ctx* c) {
  ProfHook hook;
  hook.ctx = c;
  hook.begin = [](void* ctx, int cls, cudaStream_t s) -> void* {
    return new (std::nothrow) Launch(static_cast<olsgd_ctx*>(ctx), cls, s);
  };
  hook.end = [](void* h) { delete static_cast<Launch*>(h); };
  return hook;
}

// Iterations in one captured block: whole periods, an even count, at least eight steps.
constexpr int kMaxGraphBlock = 64;   // iterations in one captured block, at most
int graph_block_len(int tau) {
  int periods = (8 + tau - 1) / tau;
  if ((periods * tau) % 2) periods *= 2;
  return periods * tau;
}

struct Plan {
  int64_t P = 0, ld = 0;
  size_t off_x0 = 0, off_x1 = 0, off_u = 0, off_g = 0, off_z = 0, off_v = 0, off_tmp = 0,
         off_shadow = 0, off_idx = 0, off_idx_next = 0, off_ident = 0, off_status = 0, off_dev_k = 0,
         off_loss_ring = 0, off_sum_part = 0, off_stage_x[2] = {0, 0},
         off_stage_y[2] = {0, 0}, off_model = 0, total = 0;
  bool has_u = false, has_g = false, has_shadow = false, has_sum_part = false;
  ModelPlan mp;
};

olsgd_status check_spec(const olsgd_model_spec* spec, int64_t* P) {
  if (!spec) return fail(nullptr, OLSGD_EINVAL, "model spec is NULL");
  switch (spec->kind) {
    case OLSGD_FLAT:
      if (spec->flat_P < 1) return fail(nullptr, OLSGD_EINVAL, "flat_P must be >= 1");
      *P = spec->flat_P;
      return OLSGD_OK;
    case OLSGD_LINREG:
      if (spec->n_dims != 1 || spec->dims[0] < 1)
        return fail(nullptr, OLSGD_EINVAL, "LINREG needs n_dims == 1 and dims[0] >= 1");
      *P = spec->dims[0];
      return OLSGD_OK;
    case OLSGD_SOFTMAX:
    case OLSGD_MLP: {
      if (spec->kind == OLSGD_SOFTMAX && spec->n_dims != 2)
        return fail(nullptr, OLSGD_EINVAL, "SOFTMAX needs n_dims == 2");
      if (spec->n_dims < 2 || spec->n_dims > OLSGD_MAX_DIMS)
        return fail(nullptr, OLSGD_EINVAL, "MLP needs 2 <= n_dims <= %d", OLSGD_MAX_DIMS);
      int64_t p = 0;
      for (int l = 0; l < spec->n_dims; ++l)
        if (spec->dims[l] < 1) return fail(nullptr, OLSGD_EINVAL, "dims[%d] must be >= 1", l);
      for (int l = 0; l + 1 < spec->n_dims; ++l)
        p += (int64_t)spec->dims[l + 1] * spec->dims[l] + spec->dims[l + 1];
      if (spec->dims[spec->n_dims - 1] > kMaxClasses)
        return fail(nullptr, OLSGD_EINVAL, "at most %d classes are supported", kMaxClasses);
      *P = p;
      return OLSGD_OK;
    }
    default:
      return fail(nullptr, OLSGD_EINVAL, "unknown model kind %d", spec->kind);
  }
}

olsgd_status check_hp(const olsgd_hparams* hp) {
  if (!hp) return fail(nullptr, OLSGD_EINVAL, "hyper-parameters are NULL");
  if (hp->m < 1 || hp->m > 65535) return fail(nullptr, OLSGD_EINVAL, "m must be in [1, 65535]");
  if (hp->tau < 1) return fail(nullptr, OLSGD_EINVAL, "tau must be >= 1");
  if (hp->batch < 1) return fail(nullptr, OLSGD_EINVAL, "batch must be >= 1");
  if (!(hp->gamma > 0.f)) return fail(nullptr, OLSGD_EINVAL, "gamma must be > 0");
  if (!(hp->alpha >= 0.f && hp->alpha <= 1.f))
    return fail(nullptr, OLSGD_EINVAL, "alpha must be in [0, 1]");
  if (!(hp->beta >= 0.f && hp->beta < 1.f))
    return fail(nullptr, OLSGD_EINVAL, "beta must be in [0, 1)");
  if (!(hp->mu >= 0.f && hp->mu < 1.f)) return fail(nullptr, OLSGD_EINVAL, "mu must be in [0, 1)");
  if (hp->m_total != 0 && (hp->worker_offset < 0 || hp->worker_offset + hp->m > hp->m_total))
    return fail(nullptr, OLSGD_EINVAL, "worker_offset + m must not exceed m_total");
  if (hp->m_total == 0 && hp->worker_offset != 0)
    return fail(nullptr, OLSGD_EINVAL, "worker_offset needs m_total");
  if (hp->m_total != 0 && hp->mode != OLSGD_MODE_OVERLAP)
    return fail(nullptr, OLSGD_EINVAL, "sharded contexts support OLSGD_MODE_OVERLAP only");
  if (hp->sampling != 0 && hp->sampling != 1)
    return fail(nullptr, OLSGD_EINVAL, "sampling must be 0 (with replacement) or 1 (epoch rule)");
  if (hp->mode != OLSGD_MODE_OVERLAP && hp->mode != OLSGD_MODE_LOCAL_SGD)
    return fail(nullptr, OLSGD_EINVAL, "mode must be OLSGD_MODE_OVERLAP or OLSGD_MODE_LOCAL_SGD");
  return OLSGD_OK;
}

olsgd_status make_plan(const olsgd_model_spec* spec, const olsgd_hparams* hp, Plan* pl) {
  olsgd_status st = check_spec(spec, &pl->P);
  if (st != OLSGD_OK) return st;
  st = check_hp(hp);
  if (st != OLSGD_OK) return st;
  const int64_t m = hp->m;
  pl->ld = (int64_t)align_up((size_t)pl->P, 64);  // rows start on 256-byte boundaries
  const size_t row = (size_t)pl->ld * sizeof(float);
  pl->has_u = hp->mu != 0.f;
  pl->has_g = spec->kind != OLSGD_FLAT;
  pl->has_shadow = spec->kind == OLSGD_MLP && spec->gemm_bf16 != 0;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, kAlign);
    return o;
  };
  pl->off_x0 = take(row * m);
  pl->off_x1 = take(row * m);
  pl->off_u = pl->has_u ? take(row * m) : 0;
  pl->off_g = pl->has_g ? take(row * m) : 0;
  pl->off_z = take(row);
  pl->off_v = take(row);
  pl->off_tmp = take(row);
  pl->off_status = take(sizeof(int));
  pl->off_dev_k = take(sizeof(int64_t));
  {
    const int base = graph_block_len(hp->tau);
    pl->off_loss_ring = take((size_t)(base > kMaxGraphBlock ? base : kMaxGraphBlock) * m * sizeof(float));
  }
  pl->off_shadow = pl->has_shadow ? take((size_t)pl->ld * m * sizeof(__nv_bfloat16)) : 0;
  pl->off_idx = pl->has_g ? take((size_t)m * hp->batch * sizeof(int32_t)) : 0;
  pl->off_idx_next = pl->has_g ? take((size_t)m * hp->batch * sizeof(int32_t)) : 0;
  if (pl->has_g) {
    pl->off_ident = take((size_t)m * hp->batch * sizeof(int32_t));
    for (int b = 0; b < 2; ++b) {
      pl->off_stage_x[b] = take((size_t)m * hp->batch * spec->dims[0] * sizeof(float));
      pl->off_stage_y[b] = take((size_t)m * hp->batch * sizeof(int32_t));
    }
  }
  pl->off_model = off;
  if (pl->has_g) {
    if (!plan_model(*spec, *hp, &pl->mp)) return fail(nullptr, OLSGD_EINVAL, "%s", pl->mp.error);
    off = align_up(off + pl->mp.bytes, kAlign);
  }
  // partial worker sums of the sync steps (Eq. 5's sum formed where x_{k+1} is written)
  pl->has_sum_part = hp->mode == OLSGD_MODE_OVERLAP && m >= 2;
  pl->off_sum_part = pl->has_sum_part ? take((size_t)worker_sum_slices(hp->m) * row) : 0;
  pl->total = off;
  return OLSGD_OK;
}

olsgd_status drain_profile(olsgd_ctx* c) {
  // launches are bracketed on every stream the context uses: all of them must be idle
  // before the events are read, or the sample of a launch still in flight would be lost
  if (c->copy) OLSGD_CUDA(c, cudaStreamSynchronize(c->copy));
  if (c->aux) OLSGD_CUDA(c, cudaStreamSynchronize(c->aux));
  if (c->pre) OLSGD_CUDA(c, cudaStreamSynchronize(c->pre));
  OLSGD_CUDA(c, cudaStreamSynchronize(c->main));
  OLSGD_CUDA(c, cudaStreamSynchronize(c->side));
  for (auto& r : c->prof_pending) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, r.start, r.stop) == cudaSuccess) {
      c->prof_ms[r.cls][r.tag] += ms;
      c->prof_launches[r.cls][r.tag] += 1;
    }
    c->prof_pool.push_back(r.start);
    c->prof_pool.push_back(r.stop);
  }
  c->prof_pending.clear();
  return OLSGD_OK;
}

// Eq. 3 / Eq. 4 for all workers: reads x[cur], writes x[1-cur], flips.
olsgd_status apply_update(olsgd_ctx* c, const float* g, int64_t ldg) {
  const bool period_end = (c->k + 1) % c->hp.tau == 0;
  const bool local_sgd = c->hp.mode == OLSGD_MODE_LOCAL_SGD;
  const bool sync = period_end && !local_sgd;   // Eq. 4 belongs to the overlap method only
  const int nxt = 1 - c->cur;
  // The anchor refresh of the previous period runs on the side stream.  It must
  // have finished before a pull-back reads z, and before its input buffer is
  // overwritten.
  if (c->reduce_pending && (sync || c->reduce_reads == nxt)) {
    OLSGD_CUDA(c, cudaStreamWaitEvent(c->main, c->reduce_done, 0));
    c->reduce_pending = false;
  }
  // the whole row, or (when hidden-layer weights were updated inside their weight-gradient
  // GEMM) the ranges that are left: biases and the output layer
  const bool model = c->spec.kind != OLSGD_FLAT;
  const int n_ranges = model ? c->mb.n_ranges : 1;
  for (int r = 0; r < n_ranges; ++r) {
    const int64_t off = model ? c->mb.range_off[r] : 0;
    const int64_t len = model ? c->mb.range_len[r] : c->P;
    UpdateArgs a;
    if (sync && c->anchor_fusion && update_sums_workers(len, c->hp.m)) {
      a.sum_part = c->sum_part + off;
      a.sum_slices = worker_sum_slices(c->hp.m);
      c->summed.emplace_back(off, len);
    }
    a.x_in = c->x[c->cur] + off;
    a.x_out = c->x[nxt] + off;
    a.g = g + off;
    a.u = c->u ? c->u + off : nullptr;
    a.z = c->z + off;
    a.shadow = c->shadow ? c->shadow + off : nullptr;
    a.P = len;
    a.ld = c->ld;
    a.ldg = ldg;
    a.m = c->hp.m;
    a.gamma = c->hp.gamma;
    a.mu = c->hp.mu;
    a.alpha = c->hp.alpha;
    a.sync = sync;
    // tagged 1 on sync steps (Eq. 4 applied too, and the worker sum where the range is long)
    Launch l(c, OLSGD_KC_UPDATE | ((sync ? 1 : 0) << 8), c->main);
    OLSGD_CUDA(c, launch_fused_update(a, c->main));
  }
  if (period_end && local_sgd) {
    // Eq. 2: blocking average of all worker models, in place, on the main stream
    Launch l(c, OLSGD_KC_ANCHOR, c->main);
    OLSGD_CUDA(c, launch_worker_mean_broadcast(c->x[nxt], c->shadow, c->z, c->P, c->ld, c->hp.m,
                                               c->main));
  }
  c->cur = nxt;
  c->k += 1;
  if (sync) c->need_sync = true;
  return OLSGD_OK;
}

// S1: the minibatch indices of iteration k into c->idx, by the context's sampling rule.
cudaError_t draw_indices(olsgd_ctx* c, int64_t k) {
  // while a graph is being captured the kernel gets the offset inside the block and adds
  // the block's first iteration from device memory, so that every replay draws new batches
  const int64_t* k_ptr = c->capturing ? c->dev_k : nullptr;
  if (c->capturing) k -= c->capture_k0;
  if (c->hp.sampling == 1)
    return launch_minibatch_indices_epoch(c->idx, c->hp.seed, c->hp.m, k, c->hp.batch,
                                          c->data.n_per_worker, c->hp.worker_offset, k_ptr,
                                          c->dev_status, c->main);
  return launch_minibatch_indices(c->idx, c->hp.seed, c->hp.m, k, c->hp.batch,
                                  c->data.n_per_worker, c->hp.worker_offset, k_ptr, c->main);
}

// S2-S6 of one iteration on the main stream, reading the minibatch rows
// idx[i][:] of `data`.  stage_slot >= 0 marks a host-fed staging slot to release.
olsgd_status step_body(olsgd_ctx* c, const olsgd_data& data, int32_t* idx,
                       float* loss_device, int stage_slot, const __nv_bfloat16* xb16_in = nullptr,
                       const IndexRule* rule = nullptr, bool batch_staged = false,
                       cudaEvent_t mid_event = nullptr) {
  if (c->loss_read_pending && !c->capturing) {
    // the losses of the last host-fed step are still being copied out of the buffer this
    // step's kernels write again
    OLSGD_CUDA(c, cudaStreamWaitEvent(c->main, c->loss_read, 0));
    c->loss_read_pending = false;
  }
  StepIO io;
  io.mid_event = mid_event;
  io.xb16_in = xb16_in;
  io.rule = rule;
  io.batch_set = (int)(c->k & 1);
  io.batch_staged = batch_staged;
  io.x = c->x[c->cur];
  io.shadow = c->shadow;
  io.g = c->g;
  io.ld = c->ld;
  io.idx = idx;
  io.loss = loss_device;
  io.status = c->dev_status;
  memset(&io.upd, 0, sizeof io.upd);
  io.wait_before_update = nullptr;
  // with the two streams of the context serialised (side == main) nothing runs beside the
  // main stream either
  const bool beside = c->aux != nullptr && c->side != c->main;
  io.aux = beside ? c->aux : nullptr;
  io.aux_fork = c->aux_fork;
  io.aux_join = c->aux_join;
  if ((c->spec.kind == OLSGD_MLP && c->spec.gemm_bf16 == 1) ||
      ((c->spec.kind == OLSGD_SOFTMAX || c->spec.kind == OLSGD_LINREG) && c->mb.fused_head)) {
    const bool sync = (c->k + 1) % c->hp.tau == 0 && c->hp.mode == OLSGD_MODE_OVERLAP;
    const int nxt = 1 - c->cur;
    io.upd.enabled = 1;
    io.upd.x_in = c->x[c->cur];
    io.upd.x_out = c->x[nxt];
    io.upd.u = c->u;
    io.upd.z = c->z;
    io.upd.shadow = c->shadow;
    io.upd.ld = c->ld;
    io.upd.gamma = c->hp.gamma;
    io.upd.mu = c->hp.mu;
    io.upd.alpha = c->hp.alpha;
    io.upd.sync = sync ? 1 : 0;
    if (sync && c->anchor_fusion && c->mb.n_summed > 0) {
      // the worker sums of the weight matrices whose update is fused are formed by the same
      // launch; the anchor refresh finishes Eq. 5 / Eq. 10-11 from them
      io.upd.sum_part = c->sum_part;
      io.upd.sum_slices = worker_sum_slices(c->hp.m);
      for (int r = 0; r < c->mb.n_summed; ++r)
        c->summed.emplace_back(c->mb.summed_off[r], c->mb.summed_len[r]);
    }
    // same rule as in apply_update, applied before the first kernel that writes x[nxt]
    if (c->reduce_pending && (sync || c->reduce_reads == nxt)) {
      io.wait_before_update = c->reduce_done;
      c->reduce_pending = false;
    }
  }
  const ProfHook hook = make_hook(c);
  cudaError_t e = model_forward_backward(c->spec, c->hp, data, c->mb, io, c->main, hook);
  if (e != cudaSuccess)
    return fail(c, OLSGD_ECUDA, "forward/backward failed: %s", cudaGetErrorString(e));
  if (stage_slot >= 0) OLSGD_CUDA(c, cudaEventRecord(c->stage_free[stage_slot], c->main));
  if (c->set_free[0] && !c->capturing && c->spec.kind == OLSGD_MLP && c->spec.gemm_bf16 != 0) {
    OLSGD_CUDA(c, cudaEventRecord(c->set_free[io.batch_set], c->main));
    c->set_free_valid[io.batch_set] = true;
  }
  // S5-S6
  olsgd_status st = apply_update(c, c->g, c->ld);
  if (st != OLSGD_OK) return st;
  return OLSGD_OK;
}

olsgd_status copy_out(olsgd_ctx* c, void* dst, const void* src, size_t bytes) {
  OLSGD_CUDA(c, cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDefault, c->main));
  OLSGD_CUDA(c, cudaStreamSynchronize(c->main));
  return OLSGD_OK;
}

// Reads the device status word; both streams must be idle.
olsgd_status check_device_status(olsgd_ctx* c) {
  int st = 0;
  OLSGD_CUDA(c, cudaMemcpy(&st, c->dev_status, sizeof(int), cudaMemcpyDeviceToHost));
  if (st != 0)
    return fail(c, (olsgd_status)st, "a kernel gave up waiting on a barrier (status %d)", st);
  return OLSGD_OK;
}

}  // namespace

namespace olsgd {
void set_thread_error(const char* text) { g_last_error = text ? text : ""; }
int g_launch_overlap = 1;
int g_gemm_pairs = 0;
std::atomic<int64_t> g_tc_launches{0};
thread_local bool g_launch_plain = false;

int current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  return dev;
}

int sm_count() {
  static int cached[kMaxDevices] = {0};
  const int dev = current_device();
  if (dev >= 0 && dev < kMaxDevices && cached[dev] > 0) return cached[dev];
  int n = 0;
  if (dev < 0 || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
    cudaGetLastError();
    return 1;
  }
  if (dev < kMaxDevices) cached[dev] = n;
  return n;
}
}  // namespace olsgd

extern "C" {

olsgd_status olsgd_param_count(const olsgd_model_spec* spec, int64_t* out_P) {
  if (!out_P) return fail(nullptr, OLSGD_EINVAL, "out_P is NULL");
  return check_spec(spec, out_P);
}

olsgd_status olsgd_workspace_bytes(const olsgd_model_spec* spec, const olsgd_hparams* hp,
                                   size_t* out_bytes) {
  if (!out_bytes) return fail(nullptr, OLSGD_EINVAL, "out_bytes is NULL");
  Plan pl;
  olsgd_status st = make_plan(spec, hp, &pl);
  if (st != OLSGD_OK) return st;
  *out_bytes = pl.total;
  return OLSGD_OK;
}

olsgd_status olsgd_init(olsgd_ctx** out, const olsgd_model_spec* spec, const olsgd_hparams* hp,
                        const olsgd_data* data, const float* x0_device, void* workspace_device,
                        size_t workspace_bytes, void* main_stream, void* side_stream) {
  if (!out) return fail(nullptr, OLSGD_EINVAL, "out is NULL");
  *out = nullptr;
  Plan pl;
  olsgd_status st = make_plan(spec, hp, &pl);
  if (st != OLSGD_OK) return st;
  if (!x0_device || (reinterpret_cast<uintptr_t>(x0_device) & 15))
    return fail(nullptr, OLSGD_EINVAL, "x0_device must be non-null and 16-byte aligned");
  if (!workspace_device || (reinterpret_cast<uintptr_t>(workspace_device) & (kAlign - 1)))
    return fail(nullptr, OLSGD_EINVAL, "workspace_device must be non-null and 256-byte aligned");
  if (workspace_bytes < pl.total)
    return fail(nullptr, OLSGD_ENOMEM, "workspace too small: %zu bytes given, %zu needed",
                workspace_bytes, pl.total);
  if (spec->kind != OLSGD_FLAT) {
    if (!data || !data->X || !data->y) return fail(nullptr, OLSGD_EINVAL, "data is required");
    if (data->n_per_worker < 1 || data->n_per_worker > 0x7FFFFFFF)
      return fail(nullptr, OLSGD_EINVAL, "n_per_worker must be in [1, 2^31)");
    if ((reinterpret_cast<uintptr_t>(data->X) & 15) || (reinterpret_cast<uintptr_t>(data->y) & 3))
      return fail(nullptr, OLSGD_EINVAL, "data pointers are misaligned");
  }
  olsgd_ctx* c = new (std::nothrow) olsgd_ctx();
  if (!c) return fail(nullptr, OLSGD_ENOMEM, "host allocation failed");
  c->spec = *spec;
  c->hp = *hp;
  c->device = current_device();
  if (data) c->data = *data; else memset(&c->data, 0, sizeof c->data);
  c->P = pl.P;
  c->ld = pl.ld;
  c->main = static_cast<cudaStream_t>(main_stream);
  c->side = static_cast<cudaStream_t>(side_stream);
  char* ws = static_cast<char*>(workspace_device);
  c->x[0] = reinterpret_cast<float*>(ws + pl.off_x0);
  c->x[1] = reinterpret_cast<float*>(ws + pl.off_x1);
  c->u = pl.has_u ? reinterpret_cast<float*>(ws + pl.off_u) : nullptr;
  c->g = pl.has_g ? reinterpret_cast<float*>(ws + pl.off_g) : nullptr;
  c->z = reinterpret_cast<float*>(ws + pl.off_z);
  c->v = reinterpret_cast<float*>(ws + pl.off_v);
  c->tmp = reinterpret_cast<float*>(ws + pl.off_tmp);
  c->dev_status = reinterpret_cast<int*>(ws + pl.off_status);
  c->dev_k = reinterpret_cast<int64_t*>(ws + pl.off_dev_k);
  c->loss_ring = reinterpret_cast<float*>(ws + pl.off_loss_ring);
  c->graph_block = graph_block_len(hp->tau);
  c->shadow = pl.has_shadow ? reinterpret_cast<__nv_bfloat16*>(ws + pl.off_shadow) : nullptr;
  c->sum_part = pl.has_sum_part ? reinterpret_cast<float*>(ws + pl.off_sum_part) : nullptr;
  c->anchor_fusion = c->sum_part != nullptr;
  c->idx = pl.has_g ? reinterpret_cast<int32_t*>(ws + pl.off_idx) : nullptr;
  c->idx_next = pl.has_g ? reinterpret_cast<int32_t*>(ws + pl.off_idx_next) : nullptr;
  if (pl.has_g) {
    c->ident = reinterpret_cast<int32_t*>(ws + pl.off_ident);
    for (int b = 0; b < 2; ++b) {
      c->stage_x[b] = reinterpret_cast<float*>(ws + pl.off_stage_x[b]);
      c->stage_y[b] = ws + pl.off_stage_y[b];
    }
  }

  auto bail = [&](olsgd_status s) {
    g_last_error = c->err;
    free_host_side(c);
    return s;
  };
#define OLSGD_INIT_CUDA(call)                                                               \
  do {                                                                                      \
    cudaError_t e_ = (call);                                                                \
    if (e_ != cudaSuccess)                                                                  \
      return bail(fail(c, OLSGD_ECUDA, "%s failed: %s", #call, cudaGetErrorString(e_)));    \
  } while (0)

  OLSGD_INIT_CUDA(cudaEventCreateWithFlags(&c->pullback_done, cudaEventDisableTiming));
  OLSGD_INIT_CUDA(cudaEventCreateWithFlags(&c->reduce_done, cudaEventDisableTiming));
  if (pl.has_g) {
    OLSGD_INIT_CUDA(cudaStreamCreateWithFlags(&c->copy, cudaStreamNonBlocking));
    OLSGD_INIT_CUDA(cudaStreamCreateWithFlags(&c->aux, cudaStreamNonBlocking));
    OLSGD_INIT_CUDA(cudaEventCreateWithFlags(&c->aux_fork, cudaEventDisableTiming));
    OLSGD_INIT_CUDA(cudaEventCreateWithFlags(&c->aux_join, cudaEventDisableTiming));
    {
      // staging ahead must not take SMs from the kernels on the critical path
      int lo = 0, hi = 0;
      OLSGD_INIT_CUDA(cudaDeviceGetStreamPriorityRange(&lo, &hi));
      OLSGD_INIT_CUDA(cudaStreamCreateWithPriority(&c->pre, cudaStreamNonBlocking, lo));
    }
    OLSGD_INIT_CUDA(cudaEventCreateWithFlags(&c->pre_begin, cudaEventDisableTiming));
    OLSGD_INIT_CUDA(cudaEventCreateWithFlags(&c->pre_done, cudaEventDisableTiming));
    OLSGD_INIT_CUDA(cudaEventCreateWithFlags(&c->loss_read, cudaEventDisableTiming));
    for (int b = 0; b < 2; ++b)
      OLSGD_INIT_CUDA(cudaEventCreateWithFlags(&c->set_free[b], cudaEventDisableTiming));
    for (int b = 0; b < 2; ++b) {
      OLSGD_INIT_CUDA(cudaEventCreateWithFlags(&c->h2d_done[b], cudaEventDisableTiming));
      OLSGD_INIT_CUDA(cudaEventCreateWithFlags(&c->stage_free[b], cudaEventDisableTiming));
    }
  }
  // zero everything once (padding, momentum buffers, gradient padding), then
  // x_0^(i) = z_0 = x0
  OLSGD_INIT_CUDA(cudaMemsetAsync(ws, 0, pl.total, c->main));
  const size_t pbytes = (size_t)c->P * sizeof(float);
  for (int i = 0; i < c->hp.m; ++i)
    OLSGD_INIT_CUDA(cudaMemcpyAsync(c->x[0] + (int64_t)i * c->ld, x0_device, pbytes,
                                    cudaMemcpyDeviceToDevice, c->main));
  OLSGD_INIT_CUDA(cudaMemcpyAsync(c->z, x0_device, pbytes, cudaMemcpyDeviceToDevice, c->main));
  if (pl.has_g) {
    {
      Launch l(c, OLSGD_KC_INDEX, c->main);
      OLSGD_INIT_CUDA(launch_identity_indices(c->ident, c->hp.m, c->hp.batch, c->main));
    }
    if (!bind_model(c->spec, c->hp, pl.mp, ws + pl.off_model, &c->mb)) {
      return bail(fail(c, OLSGD_EINVAL, "%s", c->mb.error));
    }
    if (c->shadow) {
      Launch l(c, OLSGD_KC_OTHER, c->main);
      OLSGD_INIT_CUDA(launch_cast_bf16(c->x[0], c->shadow, (int64_t)c->hp.m * c->ld, c->main));
    }
  }
  OLSGD_INIT_CUDA(cudaStreamSynchronize(c->main));
#undef OLSGD_INIT_CUDA
  *out = c;
  return OLSGD_OK;
}

olsgd_status olsgd_local_step_with_grads(olsgd_ctx* c, const float* g_device) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  OLSGD_ON_DEVICE(c);
  if (c->spec.kind != OLSGD_FLAT)
    return fail(c, OLSGD_ESTATE, "olsgd_local_step_with_grads is for OLSGD_FLAT contexts");
  if (!g_device || (reinterpret_cast<uintptr_t>(g_device) & 3))
    return fail(c, OLSGD_EINVAL, "g_device must be non-null and 4-byte aligned");
  if (c->need_sync) return fail(c, OLSGD_ESTATE, "a period ended: call olsgd_period_sync first");
  return apply_update(c, g_device, c->P);
}

olsgd_status olsgd_local_step(olsgd_ctx* c, float* loss_device) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  OLSGD_ON_DEVICE(c);
  if (c->spec.kind == OLSGD_FLAT)
    return fail(c, OLSGD_ESTATE, "OLSGD_FLAT contexts take olsgd_local_step_with_grads");
  if (c->need_sync) return fail(c, OLSGD_ESTATE, "a period ended: call olsgd_period_sync first");
  // S1: minibatch indices xi_k^(i).  Where the minibatch is staged by the gather kernel and
  // the rule is the with-replacement one, that kernel draws them itself.
  const bool staged = c->spec.kind == OLSGD_MLP && c->spec.gemm_bf16 != 0;
  auto rule_for = [&](int64_t k) {
    IndexRule rule;
    rule.key0 = (uint32_t)(c->hp.seed & 0xFFFFFFFFu);
    rule.key1 = (uint32_t)(c->hp.seed >> 32);
    // while a graph is being captured: the offset inside the block, added on the device to
    // the block's first iteration
    rule.k_base = (uint64_t)(c->capturing ? k - c->capture_k0 : k);
    rule.k_ptr = c->capturing ? reinterpret_cast<const long long*>(c->dev_k) : nullptr;
    rule.worker_offset = (uint32_t)c->hp.worker_offset;
    return rule;
  };
  if (staged && c->hp.sampling == 0 && gather_draws_indices(c->hp.batch, c->spec.dims[0])) {
    // Were this iteration's rows staged beside the previous one?
    bool have = c->pre_k == c->k;
    if (c->pre_pending) {
      // also when they were not: the staging in flight must not outlive its buffers' next use
      OLSGD_CUDA(c, cudaStreamWaitEvent(c->main, c->pre_done, 0));
      c->pre_pending = false;
    }
    // Stage the rows of iteration k + 1 on the context's own stream while iteration k runs,
    // from the point where iteration k's forward GEMMs are launched (pre_begin, recorded on
    // the main stream inside the step): set (k + 1) % 2 was last read by iteration k - 1,
    // which precedes that point.  Not with the two streams of the context serialised.
    const bool ahead = c->pre && c->side != c->main;
    const int64_t k_now = c->k;
    const IndexRule rule = rule_for(k_now), next = rule_for(k_now + 1);
    olsgd_status st = step_body(c, c->data, c->idx, loss_device, -1, nullptr, &rule, have,
                                ahead ? c->pre_begin : nullptr);
    if (st != OLSGD_OK) return st;
    if (ahead) {
      OLSGD_CUDA(c, cudaStreamWaitEvent(c->pre, c->pre_begin, 0));
      g_launch_plain = true;
      const cudaError_t e = model_stage_batch(c->spec, c->hp, c->data, c->mb, c->idx_next, next,
                                              (int)((k_now + 1) & 1), c->pre, make_hook(c));
      g_launch_plain = false;
      if (e != cudaSuccess)
        return fail(c, OLSGD_ECUDA, "staging the next minibatch failed: %s", cudaGetErrorString(e));
      OLSGD_CUDA(c, cudaEventRecord(c->pre_done, c->pre));
      c->pre_pending = true;
      c->pre_k = k_now + 1;
    }
    return OLSGD_OK;
  }
  if (!staged && c->hp.sampling == 0) {
    // linear and softmax regression read their rows straight from the data set: their first
    // kernel draws the indices of the with-replacement rule itself
    const IndexRule rule = rule_for(c->k);
    return step_body(c, c->data, c->idx, loss_device, -1, nullptr, &rule);
  }
  {
    Launch l(c, OLSGD_KC_INDEX, c->main);
    OLSGD_CUDA(c, draw_indices(c, c->k));
  }
  return step_body(c, c->data, c->idx, loss_device, -1);
}

// Shared body of the two host-fed entry points; elem = bytes per input element (4 or 2).
static olsgd_status local_step_host_impl(olsgd_ctx* c, const void* Xb_host, const void* yb_host,
                                         float* loss_host, size_t elem) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  OLSGD_ON_DEVICE(c);
  if (c->spec.kind == OLSGD_FLAT)
    return fail(c, OLSGD_ESTATE, "OLSGD_FLAT contexts take olsgd_local_step_with_grads");
  if (!Xb_host || !yb_host) return fail(c, OLSGD_EINVAL, "host minibatch pointers are NULL");
  if (elem == 2 && !(c->spec.kind == OLSGD_MLP && c->spec.gemm_bf16 != 0))
    return fail(c, OLSGD_ESTATE, "bf16 minibatches are for models whose GEMM operands are bf16 "
                                 "(OLSGD_MLP with gemm_bf16 != 0)");
  if (elem == 2 && (c->spec.dims[0] % 64 != 0 || c->hp.batch % 8 != 0))
    return fail(c, OLSGD_ESTATE, "bf16 minibatches need dims[0] %% 64 == 0 and batch %% 8 == 0 "
                                 "(16-byte pieces of a row are moved): use olsgd_local_step_host");
  if (c->need_sync) return fail(c, OLSGD_ESTATE, "a period ended: call olsgd_period_sync first");
  // this step writes the staged-minibatch set of iteration k itself (bf16 rows: on the copy
  // stream)
  if (c->pre_pending) {
    OLSGD_CUDA(c, cudaStreamWaitEvent(c->main, c->pre_done, 0));
    OLSGD_CUDA(c, cudaStreamWaitEvent(c->copy, c->pre_done, 0));
    c->pre_pending = false;
  }
  if (c->pre_k == c->k) c->pre_k = -1;
  const int slot = c->host_slot;
  c->host_slot ^= 1;
  const size_t rows = (size_t)c->hp.m * c->hp.batch;
  // the kernels that read this slot two steps ago must be done before it is refilled
  OLSGD_CUDA(c, cudaStreamWaitEvent(c->copy, c->stage_free[slot], 0));
  OLSGD_CUDA(c, cudaMemcpyAsync(c->stage_x[slot], Xb_host, rows * c->spec.dims[0] * elem,
                                cudaMemcpyHostToDevice, c->copy));
  OLSGD_CUDA(c, cudaMemcpyAsync(c->stage_y[slot], yb_host, rows * 4, cudaMemcpyHostToDevice, c->copy));
  // bf16 rows need only their transposed copy and the label copy: both are made on the copy
  // stream, right behind the transfer, into the set of iteration k, once the last iteration
  // that read that set (normally k - 2) is done.
  const bool stage_on_copy = elem == 2 && c->side != c->main;
  if (stage_on_copy) {
    const int set = (int)(c->k & 1);
    if (!c->set_free_valid[set]) {
      // unknown (graph replays do not record it): everything issued so far
      OLSGD_CUDA(c, cudaEventRecord(c->set_free[set], c->main));
      c->set_free_valid[set] = true;
    }
    OLSGD_CUDA(c, cudaStreamWaitEvent(c->copy, c->set_free[set], 0));
    g_launch_plain = true;
    const cudaError_t e = model_stage_host_rows(
        c->spec, c->hp, reinterpret_cast<const __nv_bfloat16*>(c->stage_x[slot]),
        reinterpret_cast<const int32_t*>(c->stage_y[slot]), c->mb, set, c->copy, make_hook(c));
    g_launch_plain = false;
    if (e != cudaSuccess)
      return fail(c, OLSGD_ECUDA, "staging the host rows failed: %s", cudaGetErrorString(e));
  }
  OLSGD_CUDA(c, cudaEventRecord(c->h2d_done[slot], c->copy));
  OLSGD_CUDA(c, cudaStreamWaitEvent(c->main, c->h2d_done[slot], 0));
  olsgd_data staged;
  staged.X = c->stage_x[slot];
  staged.y = c->stage_y[slot];
  staged.n_per_worker = c->hp.batch;
  const __nv_bfloat16* direct =
      elem == 2 ? reinterpret_cast<const __nv_bfloat16*>(c->stage_x[slot]) : nullptr;
  olsgd_status st = step_body(c, staged, c->ident, nullptr, slot, direct, nullptr, stage_on_copy);
  if (st != OLSGD_OK) return st;
  if (loss_host) {
    // stage_free[slot] was recorded on the main stream behind the kernel that wrote the losses
    OLSGD_CUDA(c, cudaStreamWaitEvent(c->pre, c->stage_free[slot], 0));
    OLSGD_CUDA(c, cudaMemcpyAsync(loss_host, c->mb.loss, (size_t)c->hp.m * sizeof(float),
                                  cudaMemcpyDeviceToHost, c->pre));
    OLSGD_CUDA(c, cudaEventRecord(c->loss_read, c->pre));
    c->loss_read_pending = true;
  }
  return OLSGD_OK;
}

olsgd_status olsgd_local_step_host(olsgd_ctx* c, const float* Xb_host, const void* yb_host,
                                   float* loss_host) {
  return local_step_host_impl(c, Xb_host, yb_host, loss_host, sizeof(float));
}

olsgd_status olsgd_local_step_host_bf16(olsgd_ctx* c, const void* Xb_host_bf16, const void* yb_host,
                                        float* loss_host) {
  return local_step_host_impl(c, Xb_host_bf16, yb_host, loss_host, 2);
}

olsgd_status olsgd_selftest_wait_timeout(olsgd_ctx* c, int32_t limit_ms) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  OLSGD_ON_DEVICE(c);
  if (limit_ms < 1 || limit_ms > 2000) return fail(c, OLSGD_EINVAL, "limit_ms must be in [1, 2000]");
  Launch l(c, OLSGD_KC_OTHER, c->main);
  OLSGD_CUDA(c, launch_wait_selftest(c->dev_status, (uint64_t)limit_ms * 1000000ull, c->main));
  return OLSGD_OK;
}

olsgd_status olsgd_clear_status(olsgd_ctx* c) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  OLSGD_CUDA(c, cudaStreamSynchronize(c->side));
  OLSGD_CUDA(c, cudaMemsetAsync(c->dev_status, 0, sizeof(int), c->main));
  OLSGD_CUDA(c, cudaStreamSynchronize(c->main));
  c->err.clear();
  return OLSGD_OK;
}

olsgd_status olsgd_join(olsgd_ctx* c) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  OLSGD_ON_DEVICE(c);
  if (c->copy) OLSGD_CUDA(c, cudaStreamSynchronize(c->copy));
  if (c->aux) OLSGD_CUDA(c, cudaStreamSynchronize(c->aux));
  if (c->pre) OLSGD_CUDA(c, cudaStreamSynchronize(c->pre));
  OLSGD_CUDA(c, cudaStreamSynchronize(c->side));
  OLSGD_CUDA(c, cudaStreamSynchronize(c->main));
  c->reduce_pending = false;
  return check_device_status(c);
}

// S7 on the side stream for one row.  The ranges whose worker sums the sync step left in
// sum_part are finished from those S rows; what lies between them (biases, output layer, or
// the whole row when nothing was summed) goes through the worker-mean kernel.  With `partial`
// non-null both only write this context's undivided column sums there (sharded sync).
static olsgd_status launch_anchor_refresh(olsgd_ctx* c, float* partial) {
  std::sort(c->summed.begin(), c->summed.end());
  c->last_summed = 0;
  // the long ranges first: the next sync step's launches wait for all of this anyway, and
  // the short kernels then run in the shadow of the next period's first GEMMs
  for (const auto& r : c->summed) {
    // tagged 1: the refresh from partial sums (0: the worker-mean kernel)
    Launch l(c, OLSGD_KC_ANCHOR | (1 << 8), c->side);
    OLSGD_CUDA(c, launch_anchor_from_slices(c->sum_part + r.first, worker_sum_slices(c->hp.m),
                                            c->ld, c->z + r.first, c->v + r.first, r.second,
                                            c->hp.beta, c->hp.m,
                                            partial ? partial + r.first : nullptr, c->side));
    c->last_summed += r.second;
  }
  int64_t from = 0;
  auto rest = [&](int64_t end) -> cudaError_t {
    if (end <= from) return cudaSuccess;
    AnchorArgs a;
    a.x = c->x[c->cur] + from;
    a.z = c->z + from;
    a.v = c->v + from;
    a.P = end - from;
    a.ld = c->ld;
    a.m = c->hp.m;
    a.beta = c->hp.beta;
    a.partial = partial ? partial + from : nullptr;
    Launch l(c, OLSGD_KC_ANCHOR, c->side);
    return launch_worker_mean_anchor(a, c->side);
  };
  for (const auto& r : c->summed) {
    OLSGD_CUDA(c, rest(r.first));
    from = r.first + r.second;
  }
  OLSGD_CUDA(c, rest(c->P));
  c->summed.clear();
  return OLSGD_OK;
}

olsgd_status olsgd_period_sync(olsgd_ctx* c) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  OLSGD_ON_DEVICE(c);
  if (!c->need_sync || c->sync_begun)
    return fail(c, OLSGD_ESTATE, "olsgd_period_sync is legal once, right after a period ends (k=%lld, tau=%d)",
                (long long)c->k, c->hp.tau);
  if (c->hp.m_total != 0 && c->hp.m_total != c->hp.m)
    return fail(c, OLSGD_ESTATE, "this context holds a shard of the workers: use "
                                 "olsgd_period_sync_begin / olsgd_period_sync_finish");
  // S7 on the side stream, ordered after the pull-back that closed the period
  OLSGD_CUDA(c, cudaEventRecord(c->pullback_done, c->main));
  OLSGD_CUDA(c, cudaStreamWaitEvent(c->side, c->pullback_done, 0));
  const olsgd_status st = launch_anchor_refresh(c, nullptr);
  if (st != OLSGD_OK) return st;
  OLSGD_CUDA(c, cudaEventRecord(c->reduce_done, c->side));
  c->reduce_pending = true;
  c->reduce_reads = c->cur;
  c->need_sync = false;
  return OLSGD_OK;
}

olsgd_status olsgd_set_anchor_fusion(olsgd_ctx* c, int32_t on) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  if (c->need_sync || c->sync_begun)
    return fail(c, OLSGD_ESTATE, "a period ended: call olsgd_period_sync first");
  const bool want = on != 0 && c->sum_part != nullptr;
  if (want != c->anchor_fusion) {
    c->anchor_fusion = want;
    // a captured block carries the old choice
    if (c->graph_exec) {
      cudaGraphExecDestroy(c->graph_exec);
      c->graph_exec = nullptr;
    }
  }
  return OLSGD_OK;
}

int32_t olsgd_anchor_fusion(const olsgd_ctx* c) { return c && c->anchor_fusion ? 1 : 0; }
int64_t olsgd_summed_floats(const olsgd_ctx* c) { return c ? c->last_summed : -1; }

olsgd_status olsgd_period_sync_begin(olsgd_ctx* c, float* partial_sum_device) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  OLSGD_ON_DEVICE(c);
  if (!partial_sum_device || (reinterpret_cast<uintptr_t>(partial_sum_device) & 15))
    return fail(c, OLSGD_EINVAL, "partial_sum_device must be non-null and 16-byte aligned");
  if (!c->need_sync || c->sync_begun)
    return fail(c, OLSGD_ESTATE, "olsgd_period_sync_begin is legal once, right after a period ends");
  OLSGD_CUDA(c, cudaEventRecord(c->pullback_done, c->main));
  OLSGD_CUDA(c, cudaStreamWaitEvent(c->side, c->pullback_done, 0));
  const olsgd_status st = launch_anchor_refresh(c, partial_sum_device);
  if (st != OLSGD_OK) return st;
  // from here on the worker models are no longer read by the refresh, but z is not ready:
  // the main stream must still wait for reduce_done (recorded by _finish) before it reads z
  c->sync_begun = true;
  return OLSGD_OK;
}

olsgd_status olsgd_period_sync_finish(olsgd_ctx* c, const float* total_sum_device) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  OLSGD_ON_DEVICE(c);
  if (!total_sum_device || (reinterpret_cast<uintptr_t>(total_sum_device) & 15))
    return fail(c, OLSGD_EINVAL, "total_sum_device must be non-null and 16-byte aligned");
  if (!c->sync_begun)
    return fail(c, OLSGD_ESTATE, "olsgd_period_sync_finish needs olsgd_period_sync_begin first");
  const int m_total = c->hp.m_total ? c->hp.m_total : c->hp.m;
  {
    Launch l(c, OLSGD_KC_ANCHOR, c->side);
    OLSGD_CUDA(c, launch_anchor_from_sum(total_sum_device, c->z, c->v, c->P, c->hp.beta, m_total,
                                         c->side));
  }
  OLSGD_CUDA(c, cudaEventRecord(c->reduce_done, c->side));
  c->reduce_pending = true;
  c->reduce_reads = c->cur;
  c->need_sync = false;
  c->sync_begun = false;
  return OLSGD_OK;
}

int64_t olsgd_row_floats(const olsgd_ctx* c) { return c ? c->ld : -1; }

// One iteration of olsgd_run: a local step and, when a period ends, the anchor refresh.
static olsgd_status run_one(olsgd_ctx* c, float* loss) {
  olsgd_status st = olsgd_local_step(c, loss);
  if (st != OLSGD_OK) return st;
  if (c->need_sync) {
    st = olsgd_period_sync(c);
    if (!c->capturing) c->plain_syncs += 1;
  }
  if (!c->capturing) c->plain_steps += 1;
  return st;
}

// Captures one block of iterations (starting at the current, period-aligned state) into a
// graph.  The block ends with the side stream joined and with the device counter advanced,
// so that replaying it continues the run.  On any failure the context falls back to plain
// launches for good; the run itself is never affected because a capture executes nothing.
static bool capture_block(olsgd_ctx* c, int len) {
  if (c->graph_exec) {
    cudaGraphExecDestroy(c->graph_exec);
    c->graph_exec = nullptr;
  }
  const int64_t k0 = c->k, launches0 = c->launches, pre_k0 = c->pre_k;
  const int cur0 = c->cur;
  cudaGraph_t graph = nullptr;
  if (cudaStreamBeginCapture(c->main, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
    cudaGetLastError();
    c->graph_off = true;
    return false;
  }
  c->capturing = true;
  c->capture_k0 = k0;
  bool ok = true;
  for (int j = 0; j < len && ok; ++j)
    ok = run_one(c, c->loss_ring + (int64_t)j * c->hp.m) == OLSGD_OK;
  if (ok && c->reduce_pending) {
    ok = cudaStreamWaitEvent(c->main, c->reduce_done, 0) == cudaSuccess;
    c->reduce_pending = false;
  }
  // the staging of the iteration after the block joins the main stream before the counter
  // it reads is advanced (and every stream of a capture must rejoin its origin)
  if (ok && c->pre_pending) ok = cudaStreamWaitEvent(c->main, c->pre_done, 0) == cudaSuccess;
  c->pre_pending = false;
  if (ok) ok = launch_counter(c->dev_k, 0, len, false, c->main) == cudaSuccess;
  c->capturing = false;
  const cudaError_t e = cudaStreamEndCapture(c->main, &graph);
  // nothing ran: put the host-side state back to the start of the block
  c->graph_launches = c->launches - launches0 + 1;
  c->launches = launches0;
  c->k = k0;
  c->cur = cur0;
  c->pre_k = pre_k0;
  c->need_sync = false;
  c->reduce_pending = false;
  if (!ok || e != cudaSuccess || !graph) {
    if (graph) cudaGraphDestroy(graph);
    cudaGetLastError();
    c->graph_off = true;
    return false;
  }
  const cudaError_t ie = cudaGraphInstantiate(&c->graph_exec, graph, 0);
  cudaGraphDestroy(graph);
  if (ie != cudaSuccess) {
    cudaGetLastError();
    c->graph_exec = nullptr;
    c->graph_off = true;
    return false;
  }
  c->graph_cur = cur0;
  c->graph_kpar = (int)(k0 & 1);
  c->graph_staged = pre_k0 == k0;
  c->graph_len = len;
  return true;
}

olsgd_status olsgd_run(olsgd_ctx* c, int64_t n_iters, float* loss_device) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  OLSGD_ON_DEVICE(c);
  if (n_iters < 0) return fail(c, OLSGD_EINVAL, "n_iters must be >= 0");
  if (c->spec.kind == OLSGD_FLAT)
    return fail(c, OLSGD_ESTATE, "OLSGD_FLAT contexts take olsgd_local_step_with_grads");
  if (c->loss_read_pending) {
    // (a replayed graph cannot wait for an event from outside it: settle this one first)
    OLSGD_CUDA(c, cudaStreamWaitEvent(c->main, c->loss_read, 0));
    c->loss_read_pending = false;
  }
  int64_t t = 0;
  auto plain = [&](int64_t count) -> olsgd_status {
    for (int64_t j = 0; j < count; ++j, ++t) {
      olsgd_status st = run_one(c, loss_device ? loss_device + t * c->hp.m : nullptr);
      if (st != OLSGD_OK) return st;
    }
    return OLSGD_OK;
  };
  // the legacy default stream cannot be captured
  const bool real_stream = c->main != nullptr && c->main != cudaStreamLegacy &&
                           c->main != cudaStreamPerThread;
  // Which block this run is executed in.  A run of at most kMaxGraphBlock iterations, on a
  // context that has already launched an ordinary and a sync step kernel by kernel, is
  // captured whole (whole periods, an even count): a caller that repeats olsgd_run(n) with a
  // small n then pays one graph launch per call.  A long run (three default blocks or more)
  // uses the default block: one block of plain launches, the capture, then replays.  Anything
  // else that is at least as long as the block of an existing graph replays that graph.
  const int base = c->graph_block;
  const int unit = (c->hp.tau % 2) ? 2 * c->hp.tau : c->hp.tau;
  if (!real_stream || c->graph_off || c->prof || base <= 0 || n_iters < base) return plain(n_iters);
  olsgd_status st = OLSGD_OK;
  // reach a period boundary
  while (c->k % c->hp.tau != 0 && t < n_iters)
    if ((st = plain(1)) != OLSGD_OK) return st;
  const int64_t left = n_iters - t, whole = left / unit * unit;
  const bool plain_seen = c->plain_syncs >= 1 && (c->hp.tau == 1 || c->plain_steps > c->plain_syncs);
  int block = 0;
  bool first_plain = true;     // run one block with plain launches before a capture
  if (whole >= base && whole <= kMaxGraphBlock && plain_seen) {
    block = (int)whole;
    first_plain = false;       // every kernel of a period has been launched before
  } else if (left >= 3 * (int64_t)base) {
    block = base;
  } else if (c->graph_exec && left >= c->graph_len) {
    block = c->graph_len;
  }
  if (block <= 0) return plain(left);
  // A block starts with the side stream joined and with the minibatch staged ahead by plain
  // steps (if any) joined too, outside any capture: from "the rows of iteration k are staged"
  // or from "none are".
  auto settle = [&]() -> olsgd_status {
    if (c->reduce_pending) {
      OLSGD_CUDA(c, cudaStreamWaitEvent(c->main, c->reduce_done, 0));
      c->reduce_pending = false;
    }
    if (c->pre_pending) {
      OLSGD_CUDA(c, cudaStreamWaitEvent(c->main, c->pre_done, 0));
      c->pre_pending = false;
    }
    return OLSGD_OK;
  };
  auto graph_fits = [&]() {
    return c->graph_exec && c->graph_len == block && c->graph_cur == c->cur &&
           c->graph_kpar == (int)(c->k & 1) && c->graph_staged == (c->pre_k == c->k);
  };
  if ((st = settle()) != OLSGD_OK) return st;
  if (!graph_fits()) {
    if (first_plain) {
      // one block with plain launches first (this also performs every one-time kernel attribute
      // set-up, which must not happen inside a capture), then the capture
      if (n_iters - t < 2 * (int64_t)block) return plain(n_iters - t);
      if ((st = plain(block)) != OLSGD_OK) return st;
      if ((st = settle()) != OLSGD_OK) return st;
    }
    if (!graph_fits() && !capture_block(c, block)) return plain(n_iters - t);
  }
  {
    Launch l(c, OLSGD_KC_INDEX, c->main);
    OLSGD_CUDA(c, launch_counter(c->dev_k, c->k, 0, true, c->main));
  }
  while (n_iters - t >= block) {
    OLSGD_CUDA(c, cudaGraphLaunch(c->graph_exec, c->main));
    if (loss_device)
      OLSGD_CUDA(c, cudaMemcpyAsync(loss_device + t * c->hp.m, c->loss_ring,
                                    (size_t)block * c->hp.m * sizeof(float),
                                    cudaMemcpyDeviceToDevice, c->main));
    c->k += block;
    if (c->graph_staged) c->pre_k = c->k;   // the block's last iteration staged the next rows
    c->set_free_valid[0] = c->set_free_valid[1] = false;
    c->graph_replays += 1;
    c->launches += c->graph_launches;
    t += block;
  }
  return plain(n_iters - t);
}

olsgd_status olsgd_get_params(olsgd_ctx* c, int32_t which, float* dst, size_t n_floats) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  OLSGD_ON_DEVICE(c);
  if (!dst) return fail(c, OLSGD_EINVAL, "dst is NULL");
  if (n_floats != (size_t)c->P)
    return fail(c, OLSGD_EINVAL, "n_floats is %zu but P is %lld", n_floats, (long long)c->P);
  const int m = c->hp.m;
  if (which >= m || which < -5 - (m - 1))
    return fail(c, OLSGD_EINVAL, "which = %d is out of range", which);
  if (which <= -5 && !c->u) return fail(c, OLSGD_EINVAL, "no local momentum buffer (mu = 0)");
  OLSGD_CUDA(c, cudaStreamSynchronize(c->side));
  c->reduce_pending = false;
  OLSGD_CUDA(c, cudaStreamSynchronize(c->main));
  {
    olsgd_status ds = check_device_status(c);
    if (ds != OLSGD_OK) return ds;
  }
  const size_t bytes = (size_t)c->P * sizeof(float);
  const float* xk = c->x[c->cur];
  if (which >= 0) return copy_out(c, dst, xk + (int64_t)which * c->ld, bytes);
  if (which == -1) return copy_out(c, dst, c->z, bytes);
  if (which == -2) return copy_out(c, dst, c->v, bytes);
  if (which <= -5) return copy_out(c, dst, c->u + (int64_t)(-5 - which) * c->ld, bytes);
  {
    Launch l(c, OLSGD_KC_OTHER, c->main);
    OLSGD_CUDA(c, launch_virtual_sequence(xk, c->z, c->tmp, c->P, c->ld, m,
                                          which == -3 ? c->hp.alpha : 0.f, c->main));
  }
  return copy_out(c, dst, c->tmp, bytes);
}

olsgd_status olsgd_set_params(olsgd_ctx* c, int32_t which, const float* src, size_t n_floats) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  OLSGD_ON_DEVICE(c);
  if (!src) return fail(c, OLSGD_EINVAL, "src is NULL");
  if (n_floats != (size_t)c->P)
    return fail(c, OLSGD_EINVAL, "n_floats is %zu but P is %lld", n_floats, (long long)c->P);
  const int m = c->hp.m;
  if (which >= m || which < -5 - (m - 1) || which == -3 || which == -4)
    return fail(c, OLSGD_EINVAL, "which = %d cannot be set", which);
  if (which <= -5 && !c->u) return fail(c, OLSGD_EINVAL, "no local momentum buffer (mu = 0)");
  OLSGD_CUDA(c, cudaStreamSynchronize(c->side));
  c->reduce_pending = false;
  OLSGD_CUDA(c, cudaStreamSynchronize(c->main));
  float* dst = which >= 0   ? c->x[c->cur] + (int64_t)which * c->ld
               : which == -1 ? c->z
               : which == -2 ? c->v
                             : c->u + (int64_t)(-5 - which) * c->ld;
  OLSGD_CUDA(c, cudaMemcpyAsync(dst, src, (size_t)c->P * sizeof(float), cudaMemcpyDefault, c->main));
  if (which >= 0 && c->shadow) {
    Launch l(c, OLSGD_KC_OTHER, c->main);
    OLSGD_CUDA(c, launch_cast_bf16(dst, c->shadow + (int64_t)which * c->ld, c->ld, c->main));
  }
  OLSGD_CUDA(c, cudaStreamSynchronize(c->main));
  return OLSGD_OK;
}

olsgd_status olsgd_set_iteration(olsgd_ctx* c, int64_t k) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  if (k < 0 || k % c->hp.tau != 0)
    return fail(c, OLSGD_EINVAL, "k must be a non-negative multiple of tau");
  if (c->need_sync) return fail(c, OLSGD_ESTATE, "a period ended: call olsgd_period_sync first");
  c->k = k;
  return OLSGD_OK;
}

olsgd_status olsgd_consensus_distance(olsgd_ctx* c, double* out_host) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  OLSGD_ON_DEVICE(c);
  if (!out_host) return fail(c, OLSGD_EINVAL, "out_host is NULL");
  OLSGD_CUDA(c, cudaStreamSynchronize(c->side));
  c->reduce_pending = false;
  OLSGD_CUDA(c, cudaStreamSynchronize(c->main));
  // the scratch row holds ld floats = ld / 2 doubles: slot 0 the result, then the partials
  int n_partials = (int)(c->ld / 2 - 1);
  if (n_partials > 592) n_partials = 592;
  double* scratch = reinterpret_cast<double*>(c->tmp);
  {
    Launch l(c, OLSGD_KC_OTHER, c->main);
    OLSGD_CUDA(c, launch_consensus_distance(c->x[c->cur], c->z, scratch, n_partials, c->P, c->ld,
                                            c->hp.m, c->main));
    c->launches++;
  }
  return copy_out(c, out_host, scratch, sizeof(double));
}

olsgd_status olsgd_get_indices(olsgd_ctx* c, int64_t k, int32_t* dst) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  OLSGD_ON_DEVICE(c);
  if (!dst) return fail(c, OLSGD_EINVAL, "dst is NULL");
  if (c->spec.kind == OLSGD_FLAT) return fail(c, OLSGD_ESTATE, "OLSGD_FLAT draws no minibatches");
  if (k < 0) return fail(c, OLSGD_EINVAL, "k must be >= 0");
  OLSGD_CUDA(c, cudaStreamSynchronize(c->main));
  {
    Launch l(c, OLSGD_KC_INDEX, c->main);
    OLSGD_CUDA(c, draw_indices(c, k));
  }
  return copy_out(c, dst, c->idx, (size_t)c->hp.m * c->hp.batch * sizeof(int32_t));
}

olsgd_status olsgd_class_pairs(uint64_t seed, int32_t m, int32_t* dst, void* stream) {
  if (m < 1 || m > 65535) return fail(nullptr, OLSGD_EINVAL, "m must be in [1, 65535]");
  if (!dst) return fail(nullptr, OLSGD_EINVAL, "dst is NULL");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaPointerAttributes attr;
  OLSGD_CUDA(nullptr, cudaPointerGetAttributes(&attr, dst));
  if (attr.type == cudaMemoryTypeDevice || attr.type == cudaMemoryTypeManaged) {
    OLSGD_CUDA(nullptr, launch_class_pairs(dst, seed, m, s));
    OLSGD_CUDA(nullptr, cudaStreamSynchronize(s));
    return OLSGD_OK;
  }
  // host destination: the table is tiny, stage it through pinned host memory
  // that the device writes directly
  int32_t* pinned = nullptr;
  OLSGD_CUDA(nullptr, cudaHostAlloc(reinterpret_cast<void**>(&pinned), sizeof(int32_t) * 2 * m,
                                    cudaHostAllocMapped));
  int32_t* dev_view = nullptr;
  cudaError_t e = cudaHostGetDevicePointer(reinterpret_cast<void**>(&dev_view), pinned, 0);
  if (e == cudaSuccess) e = launch_class_pairs(dev_view, seed, m, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e == cudaSuccess) memcpy(dst, pinned, sizeof(int32_t) * 2 * m);
  cudaFreeHost(pinned);
  if (e != cudaSuccess)
    return fail(nullptr, OLSGD_ECUDA, "class-pair kernel failed: %s", cudaGetErrorString(e));
  return OLSGD_OK;
}

olsgd_status olsgd_selftest_per_device_table(void) {
  // host only: the table the launch wrappers consult, driven with made-up device ordinals
  olsgd::PerDeviceSmem t;
  bool ok = t.needs(0, 100);                  // nothing configured yet
  t.set(0, 100);
  ok = ok && !t.needs(0, 100) && !t.needs(0, 64);   // device 0 is configured for up to 100 bytes
  ok = ok && t.needs(1, 100);                 // ... which says nothing about device 1
  ok = ok && t.needs(0, 200);                 // a larger request configures again
  t.set(0, 200);
  t.set(0, 150);                              // and the table only ever grows
  ok = ok && !t.needs(0, 200);
  t.set(1, 100);
  ok = ok && !t.needs(1, 100) && !t.needs(0, 200);
  ok = ok && t.needs(-1, 1) && t.needs(olsgd::kMaxDevices, 1);   // unknown ordinals: always
  t.set(olsgd::kMaxDevices, 1);
  ok = ok && t.needs(olsgd::kMaxDevices, 1);
  if (!ok) return fail(nullptr, OLSGD_ESTATE, "per-device attribute table is inconsistent");
  return OLSGD_OK;
}

int32_t olsgd_epoch_rule_half_bits(int64_t n) {
  if (n < 1 || n > 0x7FFFFFFF) return -1;
  return olsgd::epoch_rule_half_bits(n);
}

int64_t olsgd_iteration(const olsgd_ctx* c) { return c ? c->k : -1; }
int64_t olsgd_launch_count(const olsgd_ctx* c) { return c ? c->launches : -1; }
int64_t olsgd_graph_replays(const olsgd_ctx* c) { return c ? c->graph_replays : -1; }
int64_t olsgd_graph_block(const olsgd_ctx* c) { return c ? c->graph_block : -1; }

int olsgd_set_launch_overlap(int on) {
  const int before = olsgd::g_launch_overlap;
  olsgd::g_launch_overlap = on ? 1 : 0;
  return before;
}

int64_t olsgd_tensor_core_launches(void) { return olsgd::g_tc_launches.load(); }

int olsgd_set_gemm_pairs(int on) {
  const int before = olsgd::g_gemm_pairs;
  olsgd::g_gemm_pairs = on ? 1 : 0;
  return before;
}

olsgd_status olsgd_profile_enable(olsgd_ctx* c, int32_t on) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  olsgd_status st = drain_profile(c);
  if (st != OLSGD_OK) return st;
  c->prof = on != 0;
  return OLSGD_OK;
}

olsgd_status olsgd_profile_read(olsgd_ctx* c, int64_t* launches, double* millis, int32_t reset) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  if (!launches || !millis) return fail(c, OLSGD_EINVAL, "output arrays are NULL");
  olsgd_status st = drain_profile(c);
  if (st != OLSGD_OK) return st;
  for (int i = 0; i < OLSGD_N_KERNEL_CLASSES; ++i) {
    launches[i] = 0;
    millis[i] = 0.0;
    for (int t = 0; t < OLSGD_MAX_DIMS; ++t) {
      launches[i] += c->prof_launches[i][t];
      millis[i] += c->prof_ms[i][t];
      if (reset) {
        c->prof_launches[i][t] = 0;
        c->prof_ms[i][t] = 0.0;
      }
    }
  }
  return OLSGD_OK;
}

olsgd_status olsgd_profile_read_layers(olsgd_ctx* c, int64_t* launches, double* millis,
                                       int32_t reset) {
  if (!c) return fail(nullptr, OLSGD_EINVAL, "ctx is NULL");
  if (!launches || !millis) return fail(c, OLSGD_EINVAL, "output arrays are NULL");
  olsgd_status st = drain_profile(c);
  if (st != OLSGD_OK) return st;
  for (int i = 0; i < OLSGD_N_KERNEL_CLASSES; ++i)
    for (int t = 0; t < OLSGD_MAX_DIMS; ++t) {
      launches[i * OLSGD_MAX_DIMS + t] = c->prof_launches[i][t];
      millis[i * OLSGD_MAX_DIMS + t] = c->prof_ms[i][t];
      if (reset) {
        c->prof_launches[i][t] = 0;
        c->prof_ms[i][t] = 0.0;
      }
    }
  return OLSGD_OK;
}

const char* olsgd_last_error(const olsgd_ctx* c) {
  return c ? c->err.c_str() : g_last_error.c_str();
}

olsgd_status olsgd_destroy(olsgd_ctx* c) {
  if (!c) return OLSGD_OK;
  if (c->copy) cudaStreamSynchronize(c->copy);
  if (c->aux) cudaStreamSynchronize(c->aux);
  if (c->pre) cudaStreamSynchronize(c->pre);
  cudaStreamSynchronize(c->side);
  cudaStreamSynchronize(c->main);
  free_host_side(c);
  return OLSGD_OK;
}

}  // extern "C"
