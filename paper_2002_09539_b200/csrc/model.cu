// Forward/backward orchestration of the model families: which kernels run, in
// which order, on which staging buffers.  Host code only.
#include <cstdio>
#include <cstring>

#include "olsgd_internal.h"

namespace olsgd {
namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Scope {
  const ProfHook& h;
  void* handle;
  Scope(const ProfHook& hook, int cls, cudaStream_t s) : h(hook), handle(hook.begin(hook.ctx, cls, s)) {}
  ~Scope() { if (handle) h.end(handle); }
};

#define OLSGD_TRY(call)                    \
  do {                                     \
    cudaError_t e_ = (call);               \
    if (e_ != cudaSuccess) return e_;      \
  } while (0)

inline int n_layers(const olsgd_model_spec& s) { return s.n_dims - 1; }

// gemm_bf16: 0 = fp32 CUDA cores, 1 = tcgen05 tensor cores, 2 = the same bf16
// data flow on CUDA cores (validation of the tensor-core kernels)
inline bool bf16_path(const olsgd_model_spec& s) { return s.kind == OLSGD_MLP && s.gemm_bf16 != 0; }
inline bool tensor_path(const olsgd_model_spec& s) {
  return s.kind == OLSGD_MLP && (s.gemm_bf16 == 1 || s.gemm_bf16 == 3);
}

// Is the update of parameter layer p (a hidden layer's weights and bias) applied inside its
// weight-gradient GEMM?
bool layer_update_is_fused(const olsgd_model_spec& spec, const olsgd_hparams& hp, int p) {
  // the layer's weights must start on a 32-byte boundary of a parameter row (tensor maps over
  // x, u and the bf16 copy): earlier layers of odd sizes can push them off it
  int64_t w_off = 0;
  for (int q = 0; q < p; ++q) w_off += (int64_t)spec.dims[q + 1] * spec.dims[q] + spec.dims[q + 1];
  return spec.gemm_bf16 == 1 && spec.dims[p + 1] % 128 == 0 && spec.dims[p] % 128 == 0 &&
         hp.batch % 64 == 0 && hp.batch <= 128 && w_off % 8 == 0;
}

// One GEMM of the bf16 path.  On the tensor-core modes a GEMM whose shape or alignment the
// tcgen05 kernels do not take (row pitches that are not multiples of 16 bytes, i.e. widths
// or batches off the grid of 8, operands off a 16-byte boundary) runs on the CUDA-core kernel
// instead: same operand rounding, fp32 accumulation in another order.
cudaError_t run_gemm(const olsgd_model_spec& spec, GemmArgs ga, int* status, cudaStream_t s) {
  ga.status = status;
  if (tensor_path(spec)) {
    if (wgrad_tc_supported(ga)) return launch_wgrad_tc(ga, s);
    if (gemm_tc_supported(ga)) return launch_gemm_tc(ga, s);
  }
  return launch_gemm_simt(ga, s);
}

}  // namespace

bool plan_model(const olsgd_model_spec& spec, const olsgd_hparams& hp, ModelPlan* mp) {
  const size_t m = hp.m, B = hp.batch;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  };
  mp->off_loss = take(m * sizeof(float));
  if (spec.kind == OLSGD_LINREG) {
    mp->bytes = off;
    return true;
  }
  const int L = n_layers(spec);
  const size_t d0 = spec.dims[0], C = spec.dims[L];
  mp->off_yb[0] = mp->off_yb[1] = take(m * B * sizeof(int32_t));
  mp->off_dlogits = take(m * B * C * sizeof(float));
  mp->off_rowloss = take(m * B * sizeof(float));
  if (!bf16_path(spec)) {
    if (L != 1) {
      snprintf(mp->error, sizeof mp->error,
               "hidden layers need gemm_bf16 = 1 (tensor cores) or 2 (CUDA-core check)");
      return false;
    }
    mp->off_xb32 = take(m * B * d0 * sizeof(float));
    mp->bytes = off;
    return true;
  }
  if (L < 2) {
    snprintf(mp->error, sizeof mp->error, "gemm_bf16 needs at least one hidden layer");
    return false;
  }
  const size_t e = sizeof(__nv_bfloat16);
  mp->off_yb[1] = take(m * B * sizeof(int32_t));
  for (int b = 0; b < 2; ++b) {
    mp->off_xb16[b] = take(m * B * d0 * e);
    mp->off_xb16t[b] = take(m * B * d0 * e);
  }
  for (int l = 1; l < L; ++l) {
    const size_t w = spec.dims[l];
    mp->off_h[l] = take(m * B * w * e);
    mp->off_ht[l] = take(m * B * w * e);
    mp->off_da[l] = take(m * B * w * e);
    mp->off_dat[l] = take(m * B * w * e);
  }
  mp->bytes = off;
  return true;
}

bool bind_model(const olsgd_model_spec& spec, const olsgd_hparams& hp, const ModelPlan& mp,
                char* base, ModelBuffers* mb) {
  mb->loss = reinterpret_cast<float*>(base + mp.off_loss);
  mb->n_ranges = 1;
  mb->range_off[0] = 0;
  if (spec.kind == OLSGD_LINREG) {
    // the model kernel applies the update itself: nothing is left for the update kernel
    mb->range_len[0] = spec.dims[0];
    mb->fused_head = true;
    mb->n_ranges = 0;
    return true;
  }
  const int L = n_layers(spec);
  int64_t off = 0;
  for (int l = 0; l < L; ++l) {
    mb->w_off[l] = off;
    off += (int64_t)spec.dims[l + 1] * spec.dims[l];
    mb->b_off[l] = off;
    off += spec.dims[l + 1];
  }
  for (int b = 0; b < 2; ++b) mb->yb[b] = reinterpret_cast<int32_t*>(base + mp.off_yb[b]);
  mb->dlogits = reinterpret_cast<float*>(base + mp.off_dlogits);
  mb->rowloss = reinterpret_cast<float*>(base + mp.off_rowloss);
  mb->range_len[0] = off;
  if (!bf16_path(spec)) {
    mb->xb32 = reinterpret_cast<float*>(base + mp.off_xb32);
    // softmax regression: where the output-layer weight-gradient kernel can apply the update
    // itself, nothing is left for the update kernel
    HeadArgs probe{};
    probe.K = spec.dims[0];
    probe.C = spec.dims[1];
    probe.w_off = 0;
    probe.ld = 4;
    mb->fused_head = spec.kind == OLSGD_SOFTMAX && L == 1 && head_wgrad_can_update(probe);
    if (mb->fused_head) mb->n_ranges = 0;
    return true;
  }
  auto bp = [&](size_t o) { return reinterpret_cast<__nv_bfloat16*>(base + o); };
  for (int b = 0; b < 2; ++b) {
    mb->xb16[b] = bp(mp.off_xb16[b]);
    mb->xb16t[b] = bp(mp.off_xb16t[b]);
  }
  for (int l = 1; l < L; ++l) {
    mb->h[l] = bp(mp.off_h[l]);
    mb->ht[l] = bp(mp.off_ht[l]);
    mb->da[l] = bp(mp.off_da[l]);
    mb->dat[l] = bp(mp.off_dat[l]);
  }
  // gemm_bf16 == 1: hidden-layer weight matrices whose shape the weight-gradient kernel
  // takes are updated in its epilogue; everything else goes to the update kernel
  int64_t P = off;
  for (int p = 0; p < L - 1; ++p) mb->fused_layer[p] = layer_update_is_fused(spec, hp, p);
  {
    HeadArgs probe{};
    probe.K = spec.dims[L - 1];
    probe.C = spec.dims[L];
    probe.w_off = mb->w_off[L - 1];
    probe.ld = 4;   // every row pitch the context uses is a multiple of 64 floats
    mb->fused_head = spec.gemm_bf16 == 1 && head_wgrad_can_update(probe);
  }
  int64_t start = 0;
  mb->n_ranges = 0;
  auto close_range = [&](int64_t end) {
    if (end > start) {
      mb->range_off[mb->n_ranges] = start;
      mb->range_len[mb->n_ranges] = end - start;
      mb->n_ranges++;
    }
  };
  // what is left for the update kernel: the layers that no weight-gradient kernel updates
  for (int p = 0; p < L; ++p) {
    const bool in_kernel = p < L - 1 ? mb->fused_layer[p] : mb->fused_head;
    if (in_kernel) {
      close_range(mb->w_off[p]);
      start = mb->b_off[p] + spec.dims[p + 1];
    }
  }
  close_range(P);
  // the ranges of a row whose worker sums the sync-step weight-gradient launch can form: the
  // fused layers' weight matrices
  mb->n_summed = 0;
  for (int p = 0; p < L - 1; ++p) {
    if (!mb->fused_layer[p]) continue;
    mb->summed_off[mb->n_summed] = mb->w_off[p];
    mb->summed_len[mb->n_summed] = mb->b_off[p] - mb->w_off[p];
    mb->n_summed++;
  }
  return true;
}

cudaError_t model_forward_backward(const olsgd_model_spec& spec, const olsgd_hparams& hp,
                                   const olsgd_data& data, const ModelBuffers& mb,
                                   const StepIO& io, cudaStream_t s, const ProfHook& hook) {
  const int m = hp.m, B = hp.batch;
  const int64_t n = data.n_per_worker;
  float* loss = io.loss ? io.loss : mb.loss;
  const float* X = static_cast<const float*>(data.X);

  if (spec.kind == OLSGD_LINREG) {
    // the kernel writes x_{k+1} and, on sync steps, reads the anchor
    if (io.upd.enabled && io.wait_before_update)
      OLSGD_TRY(cudaStreamWaitEvent(s, io.wait_before_update, 0));
    Scope sc(hook, OLSGD_KC_FORWARD, s);
    return launch_linreg(X, static_cast<const float*>(data.y), io.idx, io.x, io.g, loss, m, B, n,
                         spec.dims[0], io.ld, io.upd.enabled ? &io.upd : nullptr, io.rule, s);
  }

  const int L = n_layers(spec);
  const int d0 = spec.dims[0], C = spec.dims[L];
  const bool bf = bf16_path(spec);

  // softmax regression in fp32 reads its rows straight from the data set (gather fused into
  // the two output-layer kernels); every other model stages the minibatch
  const bool fused_gather = !bf && L == 1;
  const bool rows_in_bf16 = bf && io.xb16_in != nullptr;
  const int set = bf ? io.batch_set : 0;
  if (rows_in_bf16 && io.batch_staged) {
    // transposed copy and labels were made on the copy stream (model_stage_host_rows)
  } else if (rows_in_bf16) {
    Scope sc(hook, OLSGD_KC_GATHER, s);
    OLSGD_TRY(launch_transpose_bf16(io.xb16_in, static_cast<const int32_t*>(data.y), mb.xb16t[set],
                                    mb.yb[set], m, B, d0, s));
  } else if (bf && io.batch_staged) {
    // the rows of this iteration were staged ahead of time (model_stage_batch)
  } else if (!fused_gather) {
    Scope sc(hook, OLSGD_KC_GATHER, s);
    OLSGD_TRY(launch_gather(X, static_cast<const int32_t*>(data.y), io.idx, bf ? nullptr : mb.xb32,
                            bf ? mb.xb16[set] : nullptr, bf ? mb.xb16t[set] : nullptr, mb.yb[set], m,
                            B, n, d0, io.rule, s));
  }

  // hidden layers, forward: H_l^T [d_l][B] = relu(W_l [d_l][d_{l-1}] * H_{l-1} [B][d_{l-1}]^T + b)
  for (int l = 1; l < L; ++l) {
    GemmArgs ga{};
    ga.A = io.shadow + mb.w_off[l - 1];
    ga.lda = spec.dims[l - 1];
    ga.a_batch = io.ld;
    ga.B = (l == 1) ? (rows_in_bf16 ? io.xb16_in : mb.xb16[set]) : mb.h[l - 1];
    ga.ldb = spec.dims[l - 1];
    ga.b_batch = (int64_t)B * spec.dims[l - 1];
    ga.m = m;
    ga.Ma = spec.dims[l];
    ga.Nb = B;
    ga.K = spec.dims[l - 1];
    // W_1 is not read again in this iteration (no input gradient is formed for the data);
    // the weights of the other layers are read again by their input-gradient GEMM
    ga.a_read_once = (l == 1) ? 1 : 0;
    // the weights' bf16 copy is written by the update at the end of an iteration: the kernel
    // ahead of the first layer's GEMM may be that update, the one ahead of any later layer's
    // GEMM is the previous layer's GEMM
    ga.a_ready_early = (l >= 2) ? 1 : 0;
    ga.epilogue = GEMM_EPI_BIAS_RELU;
    ga.bias = io.x + mb.b_off[l - 1];
    ga.bias_batch = io.ld;
    ga.out_t = mb.ht[l];
    ga.out_n = mb.h[l];
    {
      Scope sc(hook, OLSGD_KC_FORWARD | (l << 8), s);   // tagged with the layer it produces
      OLSGD_TRY(run_gemm(spec, ga, io.status, s));
    }
  }
  // From here the next iteration's rows may be staged beside this iteration: measured on
  // config 3, a gather started here (beside the output-layer kernels and the input-gradient
  // GEMM) costs the step 6 us less than one started beside the forward GEMMs.
  if (io.mid_event) OLSGD_TRY(cudaEventRecord(io.mid_event, s));

  // output layer: forward, loss, and backward to its input
  HeadArgs ha{};
  ha.in32 = bf ? nullptr : (fused_gather ? X : mb.xb32);
  ha.row_idx = fused_gather ? io.idx : nullptr;
  ha.n_rows = n;
  ha.y_all = static_cast<const int32_t*>(data.y);
  ha.in16 = bf ? mb.h[L - 1] : nullptr;
  ha.x = io.x;
  ha.ld = io.ld;
  ha.w_off = mb.w_off[L - 1];
  ha.b_off = mb.b_off[L - 1];
  ha.yb = mb.yb[set];
  ha.dlogits = mb.dlogits;
  ha.rowloss = mb.rowloss;
  ha.din32 = nullptr;
  ha.din16 = bf ? mb.da[L - 1] : nullptr;
  ha.din16t = bf ? mb.dat[L - 1] : nullptr;
  ha.m = m;
  ha.batch = B;
  ha.K = spec.dims[L - 1];
  ha.C = C;
  ha.round_w_bf16 = bf;
  {
    // with the fused gather and the with-replacement rule the forward kernel draws the rows
    // of the minibatch itself and leaves them in io.idx for the weight-gradient kernel
    HeadArgs fwd = ha;
    if (fused_gather && io.rule) {
      fwd.draw = 1;
      fwd.rule = *io.rule;
      fwd.idx_out = io.idx;
    }
    Scope sc(hook, OLSGD_KC_LOSS, s);
    OLSGD_TRY(launch_head_forward(fwd, s));
  }

  // From here on kernels may write x_{k+1} and, on sync steps, read the anchor: the anchor
  // refresh of the previous period must have finished.
  bool waited = false;
  const bool head_updates = io.upd.enabled && mb.fused_head;
  if (head_updates && io.wait_before_update) {
    OLSGD_TRY(cudaStreamWaitEvent(s, io.wait_before_update, 0));
    waited = true;
  }
  // The output layer's weight gradient (and update) depends only on the output-layer forward
  // kernel, and nothing before the end of the backward pass depends on it: with hidden layers
  // it runs on the second stream, beside the input-gradient and weight-gradient GEMMs.
  const bool beside = io.aux != nullptr && L >= 2;
  {
    FusedUpdateArgs hu = io.upd;
    hu.b_off = -1;
    cudaStream_t hs = s;
    if (beside) {
      OLSGD_TRY(cudaEventRecord(io.aux_fork, s));
      OLSGD_TRY(cudaStreamWaitEvent(io.aux, io.aux_fork, 0));
      hs = io.aux;
      g_launch_plain = true;
    }
    cudaError_t he;
    {
      Scope sc(hook, OLSGD_KC_BACKWARD, hs);
      he = launch_head_wgrad(ha, io.g, loss, head_updates ? &hu : nullptr, hs);
    }
    g_launch_plain = false;
    OLSGD_TRY(he);
    if (beside) OLSGD_TRY(cudaEventRecord(io.aux_join, io.aux));
  }

  // hidden layers, backward.  The weight-gradient GEMMs that carry their own update are
  // collected and launched together after the input-gradient chain (they depend on nothing
  // else in it, and every input-gradient GEMM still reads its layer's bf16 shadow before the
  // launch that overwrites it).
  GemmArgs pending[OLSGD_MAX_DIMS];
  int n_pending = 0;
  auto flush = [&]() -> cudaError_t {
    if (n_pending == 0) return cudaSuccess;
    if (io.wait_before_update && !waited) {
      OLSGD_TRY(cudaStreamWaitEvent(s, io.wait_before_update, 0));
      waited = true;
    }
    // tagged 1 on sync steps (the launch that also applies Eq. 4 and, with the worker sum
    // inside, forms the partial sums), 0 on ordinary steps
    Scope sc(hook, OLSGD_KC_WGRAD_UPDATE | ((pending[0].upd.sync ? 1 : 0) << 8), s);
    const cudaError_t e = launch_wgrad_tc_batch(pending, n_pending, s);
    n_pending = 0;
    return e;
  };
  for (int l = L - 1; l >= 1; --l) {
    if (l >= 2) {
      // dA_{l-1}^T [d_{l-1}][B] = (W_l^T [d_{l-1}][d_l] * dA_l [B][d_l]^T) .* (H_{l-1}^T > 0).
      // W_l^T is read in place from the bf16 shadow of W_l [d_l][d_{l-1}] as an MN-major
      // operand, and BEFORE the weight-gradient GEMM of this layer, whose fused epilogue
      // overwrites that shadow with W_l of the next iteration.
      GemmArgs gd{};
      gd.A = io.shadow + mb.w_off[l - 1];
      gd.a_mn_major = 1;
      gd.a_ready_early = 1;   // ahead of it runs the output-layer forward kernel or an input-
                              // gradient GEMM; the launch that rewrites the bf16 copy comes later
      gd.lda = spec.dims[l - 1];
      gd.a_batch = io.ld;
      gd.B = mb.da[l];
      gd.ldb = spec.dims[l];
      gd.b_batch = (int64_t)B * spec.dims[l];
      gd.m = m;
      gd.Ma = spec.dims[l - 1];
      gd.Nb = B;
      gd.K = spec.dims[l];
      gd.epilogue = GEMM_EPI_RELU_MASK;
      gd.mask = mb.ht[l - 1];
      gd.out_t = mb.dat[l - 1];
      gd.out_n = mb.da[l - 1];
      Scope sc(hook, OLSGD_KC_BACKWARD | ((l - 1) << 8), s);   // gradient of hidden layer l - 1
      OLSGD_TRY(run_gemm(spec, gd, io.status, s));
    }
    // dW_l [d_l][d_{l-1}] = dA_l^T [d_l][B] * (H_{l-1}^T [d_{l-1}][B])^T
    GemmArgs gw{};
    gw.A = mb.dat[l];
    gw.lda = B;
    gw.a_batch = (int64_t)spec.dims[l] * B;
    gw.B = (l == 1) ? mb.xb16t[set] : mb.ht[l - 1];
    gw.ldb = B;
    gw.b_batch = (int64_t)spec.dims[l - 1] * B;
    gw.m = m;
    gw.Ma = spec.dims[l];
    gw.Nb = spec.dims[l - 1];
    gw.K = B;
    gw.epilogue = GEMM_EPI_STORE_F32;
    gw.out_f = io.g + mb.w_off[l - 1];
    gw.ldo = spec.dims[l - 1];
    gw.out_batch = io.ld;
    const bool fused = io.upd.enabled && mb.fused_layer[l - 1];
    if (fused) {
      // the update of W_l happens in this GEMM's epilogue: no gradient is stored
      gw.upd = io.upd;
      gw.upd.w_off = mb.w_off[l - 1];
      gw.upd.b_off = mb.b_off[l - 1];   // and of its bias, from the row sums of dA_l^T
    }
    // the tensor-core weight-gradient kernel also adds up the rows of dA_l^T: the bias gradient
    const bool rowsum_in_gemm = tensor_path(spec) && wgrad_tc_supported(gw);
    if (rowsum_in_gemm && !fused) {
      gw.rowsum_out = io.g + mb.b_off[l - 1];
      gw.rowsum_batch = io.ld;
    }
    if (fused) {
      gw.status = io.status;
      pending[n_pending++] = gw;
      if (n_pending == wgrad_tc_batch_limit()) OLSGD_TRY(flush());
    } else {
      Scope sc(hook, OLSGD_KC_BACKWARD, s);
      OLSGD_TRY(run_gemm(spec, gw, io.status, s));
    }
    if (!rowsum_in_gemm) {
      Scope sc(hook, OLSGD_KC_BACKWARD, s);
      OLSGD_TRY(launch_bias_grad(mb.dat[l], io.g, io.ld, mb.b_off[l - 1], m, spec.dims[l], B, s));
    }
  }
  OLSGD_TRY(flush());
  if (beside) OLSGD_TRY(cudaStreamWaitEvent(s, io.aux_join, 0));
  // no kernel above took the update: the update kernel that follows needs the same ordering
  if (io.wait_before_update && !waited) OLSGD_TRY(cudaStreamWaitEvent(s, io.wait_before_update, 0));
  return cudaSuccess;
}

cudaError_t model_stage_batch(const olsgd_model_spec& spec, const olsgd_hparams& hp,
                              const olsgd_data& data, const ModelBuffers& mb, int32_t* idx,
                              const IndexRule& rule, int set, cudaStream_t s, const ProfHook& hook) {
  if (!bf16_path(spec)) return cudaErrorInvalidValue;
  Scope sc(hook, OLSGD_KC_GATHER, s);
  return launch_gather(static_cast<const float*>(data.X), static_cast<const int32_t*>(data.y), idx,
                       nullptr, mb.xb16[set], mb.xb16t[set], mb.yb[set], hp.m, hp.batch,
                       data.n_per_worker, spec.dims[0], &rule, s);
}

cudaError_t model_stage_host_rows(const olsgd_model_spec& spec, const olsgd_hparams& hp,
                                  const __nv_bfloat16* rows, const int32_t* labels,
                                  const ModelBuffers& mb, int set, cudaStream_t s,
                                  const ProfHook& hook) {
  if (!bf16_path(spec)) return cudaErrorInvalidValue;
  Scope sc(hook, OLSGD_KC_GATHER, s);
  return launch_transpose_bf16(rows, labels, mb.xb16t[set], mb.yb[set], hp.m, hp.batch, spec.dims[0], s);
}

}  // namespace olsgd
