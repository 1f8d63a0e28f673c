// Internal declarations shared by the translation units of libolsgd.
// Host-side launch wrappers only; every kernel lives in its own .cu file.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "olsgd.h"

namespace olsgd {

// ---- overlapped launches -----------------------------------------------------
// The kernels of one iteration form a chain on the main stream, most of them short.  They
// are launched with programmatic stream serialization: the blocks of a kernel may become
// resident while the kernel before it is still draining, and each block executes
// launch_gate() before its first access to global memory.  The gate returns once every
// earlier kernel of the stream has completed and its writes are visible, then lets the
// kernel after this one start its own launch.  A kernel launched the ordinary way passes
// through the gate at once.
extern int g_launch_overlap;   // olsgd_set_launch_overlap
extern int g_gemm_pairs;       // olsgd_set_gemm_pairs: long-K GEMMs on CTA pairs (cta_group::2)
extern std::atomic<int64_t> g_tc_launches;  // launches of the tcgen05 kernels so far
                                            // (olsgd_tensor_core_launches)
// Set around a launch that goes to a stream whose previous operation is an event wait, not a
// kernel: such a launch is an ordinary one (its kernel passes the gate at once).
extern thread_local bool g_launch_plain;

#ifdef __CUDACC__
__device__ __forceinline__ void launch_gate() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem,
                           cudaStream_t s, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (g_launch_overlap && !g_launch_plain) ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
#endif

// ---- olsgd_api.cu -------------------------------------------------------------
// Records the text olsgd_last_error(NULL) returns for context-free calls of this thread.
void set_thread_error(const char* text);

// ---- per-device bookkeeping ---------------------------------------------------
// Kernel attributes set with cudaFuncSetAttribute and the number of multiprocessors belong to
// a device, not to the process: one process may drive several GPUs (one context each), so
// "already configured" is remembered per device ordinal.
constexpr int kMaxDevices = 64;
struct PerDeviceSmem {
  size_t bytes[kMaxDevices] = {0};   // largest dynamic shared-memory size configured so far
  // does a launch with `smem` bytes on device `dev` need the attribute (re)set first?  An
  // ordinal outside the table is never remembered: it is configured on every launch.
  bool needs(int dev, size_t smem) const {
    return dev < 0 || dev >= kMaxDevices || smem > bytes[dev];
  }
  void set(int dev, size_t smem) {
    if (dev >= 0 && dev < kMaxDevices && smem > bytes[dev]) bytes[dev] = smem;
  }
};
int current_device();   // ordinal of the current device, -1 if it cannot be read
int sm_count();         // multiprocessors of the current device (cached per device; >= 1)
#ifdef __CUDACC__
// Raises the kernel's dynamic shared-memory limit on the current device when this launch
// needs more than that device was configured for.  Not to be called inside a stream capture
// for the first time (olsgd_run launches its first block outside the capture for this reason).
template <typename Kern>
cudaError_t ensure_dynamic_smem(PerDeviceSmem& table, Kern kern, size_t smem) {
  const int dev = current_device();
  if (!table.needs(dev, smem)) return cudaSuccess;
  const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e == cudaSuccess) table.set(dev, smem);
  return e;
}
#endif

// ---- update_kernels.cu ------------------------------------------------------
// Eq. 3 (+ local Nesterov buffer) and, when `sync`, Eq. 4, for all m workers.
// x_in/x_out/u/shadow rows have stride `ld` floats (multiple of 4, 16-byte
// aligned rows); g rows have stride `ldg`.  z may be null unless `sync`.
struct UpdateArgs {
  const float* x_in;
  float* x_out;
  const float* g;
  float* u;              // null when mu == 0
  const float* z;        // anchor, read on sync steps
  __nv_bfloat16* shadow; // bf16 copy of x_out, or null
  int64_t P, ld, ldg;
  int m;
  float gamma, mu, alpha;
  bool sync;
  // sync steps only, sum_slices > 0: the launch also adds up x_{k+1} over the workers in the
  // order of the worker-mean kernel and leaves slice s's column sums in row s of sum_part
  // (row pitch ld); launch_anchor_from_slices finishes the anchor refresh from there.
  float* sum_part = nullptr;
  int sum_slices = 0;
};
cudaError_t launch_fused_update(const UpdateArgs& a, cudaStream_t s);
// Whether a sync-step update launch over P parameters of m workers should form the worker
// sums itself: only when its one-thread-per-column-strip grid of worker_sum_slices(m) rows
// still fills the GPU (the choice changes the launches, never the bits).
bool update_sums_workers(int64_t P, int m);

// Eq. 5 (beta == 0) or Eq. 10-11: worker mean in a fixed order, then z (and v).
struct AnchorArgs {
  const float* x;
  float* z;
  float* v;
  int64_t P, ld;
  int m;
  float beta;
  float* partial;   // non-null: only write the undivided column sums there (sharded sync)
};
cudaError_t launch_worker_mean_anchor(const AnchorArgs& a, cudaStream_t s);
// The number S of interleaved slices the worker sum is formed in (slice s adds the workers
// s, s + S, ... in order, the slices are combined in order): a function of m alone, used by
// every kernel that forms the sum so that all of them give the same bits.
int worker_sum_slices(int m);
// Eq. 5 / Eq. 10-11 from column sums over all m_total workers (sum is padded like a state row).
cudaError_t launch_anchor_from_sum(const float* sum, float* z, float* v, int64_t P, float beta,
                                   int m_total, cudaStream_t s);
// Eq. 5 / Eq. 10-11 for P entries from `slices` rows of partial worker sums (row pitch ld):
// the rows are added in slice order, which completes the summation order of the worker-mean
// kernel, then divided by m.  With `partial` non-null only the undivided totals are written,
// there, and z, v are left alone (sharded sync, as in AnchorArgs).
cudaError_t launch_anchor_from_slices(const float* part, int slices, int64_t ld, float* z, float* v,
                                      int64_t P, float beta, int m, float* partial, cudaStream_t s);

// Eq. 2 on a sync step: every worker row of x (and of its bf16 shadow, if any) and z are
// replaced by the worker mean, summed in worker order.
cudaError_t launch_worker_mean_broadcast(float* x, __nv_bfloat16* shadow, float* z, int64_t P,
                                         int64_t ld, int m, cudaStream_t s);

// *out = sum_i ||x_i - z||^2 in double; scratch holds at least 2 * n_partials floats.
cudaError_t launch_consensus_distance(const float* x, const float* z, double* scratch,
                                      int n_partials, int64_t P, int64_t ld, int m,
                                      cudaStream_t s);

// dst[j] = (1-alpha) * mean_i x_i[j] + alpha * z[j]   (alpha = 0: mean model)
cudaError_t launch_virtual_sequence(const float* x, const float* z, float* dst, int64_t P,
                                    int64_t ld, int m, float alpha, cudaStream_t s);

// ---- sampling_kernels.cu ----------------------------------------------------
// worker_offset: global id of this context's first worker (the rule is a function of the
// global worker id, so a sharded run draws the same minibatches as an unsharded one)
// k_ptr: if non-null the iteration number is k + *k_ptr, read on the device (captured graphs)
cudaError_t launch_minibatch_indices(int32_t* idx, uint64_t seed, int m, int64_t k, int batch,
                                     int64_t n, int worker_offset, const int64_t* k_ptr,
                                     cudaStream_t s);
// *p = value (set) or *p += by
cudaError_t launch_counter(int64_t* p, int64_t value, int64_t by, bool set, cudaStream_t s);
// The epoch rule (one pass over the worker's samples per epoch, Feistel permutation).
// status: device word that receives OLSGD_ETIMEOUT if the cycle walk of a slot runs out.
cudaError_t launch_minibatch_indices_epoch(int32_t* idx, uint64_t seed, int m, int64_t k, int batch,
                                           int64_t n, int worker_offset, const int64_t* k_ptr,
                                           int* status, cudaStream_t s);
// h of the epoch rule: the Feistel network permutes 2^(2h) values, h = ceil(ceil(log2 n) / 2).
int epoch_rule_half_bits(int64_t n);
cudaError_t launch_class_pairs(int32_t* dst, uint64_t seed, int m, cudaStream_t s);
// idx[i][j] = j: the "indices" of a minibatch that is already contiguous
cudaError_t launch_identity_indices(int32_t* idx, int m, int batch, cudaStream_t s);

// ---- simt_kernels.cu --------------------------------------------------------
constexpr int kMaxClasses = 32;  // the output layer is handled by one warp per row

cudaError_t launch_cast_bf16(const float* src, __nv_bfloat16* dst, int64_t n, cudaStream_t s);

// Linear regression, one block per worker: r = X_b w - y_b, loss = sum r^2 / 2B,
// g = X_b^T r / B, reading the batch rows straight from the worker's partition.  With upd
// non-null and enabled the gradient is not stored: the kernel applies Eq. 3 / Eq. 4 itself.
// With rule non-null the kernel draws the minibatch indices itself (S1 inside the model kernel,
// the with-replacement rule) and writes them to idx; otherwise it reads them from idx.
struct FusedUpdateArgs;
struct IndexRule;
cudaError_t launch_linreg(const float* X, const float* y, int32_t* idx, const float* x,
                          float* g, float* loss, int m, int batch, int64_t n, int d, int64_t ld,
                          const FusedUpdateArgs* upd, const IndexRule* rule, cudaStream_t s);

// S2: copy the minibatch rows of every worker into contiguous staging.
//   xb32  float [m][B][d]   (or null)
//   xb16  bf16  [m][B][d]   (or null), xb16t bf16 [m][d][B] (or null)
//   yb    int32 [m][B]
// bf16 minibatch rows [m][batch][d] -> their transposed copy [m][d][batch], and the labels
// y[m][batch] -> yb (d % 64 == 0, batch % 8 == 0)
cudaError_t launch_transpose_bf16(const __nv_bfloat16* xb16, const int32_t* y, __nv_bfloat16* xb16t,
                                  int32_t* yb, int m, int batch, int d, cudaStream_t s);
// With `rule` non-null (only where gather_draws_indices says so) the kernel draws the
// with-replacement minibatch indices of iteration k itself (and stores them to idx) instead
// of reading idx.
struct IndexRule {
  uint32_t key0, key1;        // seed, low and high word
  uint64_t k_base;            // iteration number, or its offset from *k_ptr
  const long long* k_ptr;     // device-resident iteration number of a captured graph, or null
  uint32_t worker_offset;     // global id of local worker 0
};
bool gather_draws_indices(int batch, int d);
cudaError_t launch_gather(const float* X, const int32_t* y, int32_t* idx, float* xb32,
                          __nv_bfloat16* xb16, __nv_bfloat16* xb16t, int32_t* yb, int m, int batch,
                          int64_t n, int d, const IndexRule* rule, cudaStream_t s);

// Output layer, forward + loss + backward to its input, one warp per batch row.
//   in32 / in16   the layer's input [m][B][K], exactly one non-null
//   W, b          this layer's fp32 weights [C][K] and bias [C] inside row i of x (stride ld)
//   dlogits       float [m][B][C]  (p - onehot) / B
//   rowloss       float [m][B]
//   din32 / din16 / din16t   gradient w.r.t. the layer's input, already multiplied by the
//                 ReLU mask (input > 0); any may be null ([m][B][K], [m][B][K], [m][K][B])
struct HeadArgs {
  const float* in32;
  const __nv_bfloat16* in16;
  const float* x;        // parameters [m][ld]
  int64_t ld, w_off, b_off;
  const int32_t* yb;
  float* dlogits;
  float* rowloss;
  float* din32;
  __nv_bfloat16* din16;
  __nv_bfloat16* din16t;
  int m, batch, K, C;
  bool round_w_bf16;     // round W to bf16 before use (tensor-core path's operand rule)
  // Gather fused in (fp32 input only): when row_idx is non-null, in32 is the whole data set
  // [m][n_rows][K], batch row b of worker i is its row row_idx[i * batch + b], and the label
  // comes from y_all [m][n_rows] instead of yb.
  const int32_t* row_idx;
  int64_t n_rows;
  const int32_t* y_all;
  // Forward kernel only, with the fused gather: draw != 0 makes the kernel compute the rows
  // of its batch slots by the with-replacement index rule (S1 inside the kernel) instead of
  // reading row_idx, and write them to idx_out for the weight-gradient kernel that follows.
  int draw;
  IndexRule rule;
  int32_t* idx_out;
};
cudaError_t launch_head_forward(const HeadArgs& a, cudaStream_t s);

// Output layer weight/bias gradient and the mean loss:
//   g[i][w_off + c*K + j] = sum_b dlogits[i][b][c] * in[i][b][j];  g[i][b_off + c] = sum_b dlogits
//   loss[i] = mean_b rowloss[i][b]   (loss may be null)
// With upd non-null and upd->enabled (only where head_wgrad_can_update says so) the gradient
// is not stored: the kernel applies Eq. 3 / Eq. 4 to the layer's weights and bias on the spot.
struct FusedUpdateArgs;
bool head_wgrad_can_update(const HeadArgs& a);
cudaError_t launch_head_wgrad(const HeadArgs& a, float* g, float* loss, const FusedUpdateArgs* upd,
                              cudaStream_t s);

// g[i][b_off + r] = sum_c dat[i][r][c]   (bias gradient of a hidden layer from dA^T [m][R][B])
cudaError_t launch_bias_grad(const __nv_bfloat16* dat, float* g, int64_t ld, int64_t b_off, int m,
                             int R, int batch, cudaStream_t s);

// ---- gemm --------------------------------------------------------------------
// Worker-batched D[i] = A[i] * B[i]^T with both operands K-major bf16:
//   A [m][Ma][K] (row pitch lda, batch pitch a_batch, in elements); with a_mn_major the
//     same operand is stored transposed, [m][K][Ma] (row pitch lda), and read in place
//   B [m][Nb][K] (row pitch ldb, batch pitch b_batch)
// D is [Ma][Nb] per worker, fp32 accumulate, consumed by one of three epilogues.
enum GemmEpilogue {
  // out = relu(D + bias[row]); written bf16 as [Ma][Nb] (out_t) and [Nb][Ma] (out_n)
  GEMM_EPI_BIAS_RELU = 0,
  // out = D * (mask[row][col] > 0); written bf16 as [Ma][Nb] (out_t) and [Nb][Ma] (out_n)
  GEMM_EPI_RELU_MASK = 1,
  // out = D, written fp32 to out_f [row * ldo + col]
  GEMM_EPI_STORE_F32 = 2
};
// Parameter update applied inside the weight-gradient GEMM's epilogue instead of
// storing the gradient: the tile D[row][col] updates parameter w_off + row * Nb + col
// of every worker row (stride ld) of x_in/x_out/u/shadow.
struct FusedUpdateArgs {
  int enabled;
  const float* x_in;
  float* x_out;
  float* u;               // null or mu == 0: plain SGD
  const float* z;
  __nv_bfloat16* shadow;
  int64_t ld, w_off;
  float gamma, mu, alpha;
  int sync;
  // weight-gradient GEMM only: >= 0 makes the kernel update the layer's bias (parameters
  // b_off .. b_off + Ma - 1 of every worker row) from the row sums it forms, instead of
  // storing them as a gradient
  int64_t b_off;
  // weight-gradient GEMM on sync steps only, sum_slices > 0: the launch also adds up
  // x_{k+1} over the workers, in the order of the worker-mean kernel (sum_slices interleaved
  // slices, each in worker order), and leaves slice s's sums of the layer's weight matrix in
  // row s of sum_part; launch_anchor_from_slices finishes the anchor refresh from there.
  float* sum_part;     // [sum_slices][ld] floats of scratch
  int sum_slices;      // worker_sum_slices(m), or 0: no sum
};
struct GemmArgs {
  const __nv_bfloat16* A;
  const __nv_bfloat16* B;
  int64_t lda, a_batch, ldb, b_batch;
  int m, Ma, Nb, K;
  int a_mn_major;            // A is stored [K][Ma]
  int a_read_once;           // nothing reads A again soon: L2 may give its lines up first
  // A was last written by a kernel that had completed before the kernel launched just ahead
  // of this one started: with chained launches the first A tiles may then be loaded while
  // that kernel still drains
  int a_ready_early;
  int epilogue;
  const float* bias;         // BIAS_RELU: bias[i * bias_batch + row]
  int64_t bias_batch;
  const __nv_bfloat16* mask; // RELU_MASK: [m][Ma][Nb], same layout as out_t
  __nv_bfloat16* out_t;      // [m][Ma][Nb]
  __nv_bfloat16* out_n;      // [m][Nb][Ma]
  float* out_f;              // STORE_F32: out_f[i * out_batch + row * ldo + col]
  int64_t ldo, out_batch;
  int* status;               // device word that receives OLSGD_ETIMEOUT if a bounded wait gives up
  FusedUpdateArgs upd;       // weight-gradient kernel only
  // weight-gradient kernel only, or null: rowsum_out[i * rowsum_batch + row] = sum_k A[i][row][k],
  // the bias gradient of the layer (A = dA^T), summed in the order of the bias-gradient kernel
  float* rowsum_out;
  int64_t rowsum_batch;
};
// Plain CUDA-core version, used to validate the tensor-core kernel.
cudaError_t launch_gemm_simt(const GemmArgs& a, cudaStream_t s);
// tcgen05 / TMEM / TMA version.  Needs Ma % 128 == 0, K % 64 == 0, Nb % 16 == 0.
bool gemm_tc_supported(const GemmArgs& a);
cudaError_t launch_gemm_tc(const GemmArgs& a, cudaStream_t s);
// One thread waits (bounded by limit_ns) on a barrier nothing arrives on and reports the time-out.
cudaError_t launch_wait_selftest(int* status, uint64_t limit_ns, cudaStream_t s);
// Weight-gradient specialisation (short K, fp32 store): needs Ma % 128 == 0, Nb % 128 == 0,
// K in {64, 128, 192, 256}, epilogue GEMM_EPI_STORE_F32.
bool wgrad_tc_supported(const GemmArgs& a);
cudaError_t launch_wgrad_tc(const GemmArgs& a, cudaStream_t s);
// The same for n <= wgrad_tc_batch_limit() layers in ONE launch (all fused or all plain, same
// workers, same K, same status word); the layers must not depend on one another.
int wgrad_tc_batch_limit();
cudaError_t launch_wgrad_tc_batch(const GemmArgs* args, int n, cudaStream_t s);

// ---- model.cu ------------------------------------------------------------------
struct ModelPlan {
  size_t bytes = 0;
  char error[160] = {0};
  // offsets inside the model area
  size_t off_yb[2] = {0, 0}, off_xb32 = 0, off_xb16[2] = {0, 0}, off_xb16t[2] = {0, 0},
         off_dlogits = 0, off_rowloss = 0, off_loss = 0;
  size_t off_h[OLSGD_MAX_DIMS] = {0}, off_ht[OLSGD_MAX_DIMS] = {0};    // hidden activations
  size_t off_da[OLSGD_MAX_DIMS] = {0}, off_dat[OLSGD_MAX_DIMS] = {0};  // their gradients
  // worker sum inside the sync-step weight-gradient launch: partial sums [slices][ld]
};
struct ModelBuffers {
  char error[160] = {0};
  // The staged minibatch exists twice on the bf16 path (iteration k uses set k % 2), so that
  // the rows of iteration k + 1 can be staged while iteration k still reads its own; every
  // other model has one set and both entries point at it.
  int32_t* yb[2] = {nullptr, nullptr};
  float* xb32 = nullptr;
  __nv_bfloat16 *xb16[2] = {nullptr, nullptr}, *xb16t[2] = {nullptr, nullptr};
  float *dlogits = nullptr, *rowloss = nullptr, *loss = nullptr;
  __nv_bfloat16* h[OLSGD_MAX_DIMS] = {nullptr};
  __nv_bfloat16* ht[OLSGD_MAX_DIMS] = {nullptr};
  __nv_bfloat16* da[OLSGD_MAX_DIMS] = {nullptr};
  __nv_bfloat16* dat[OLSGD_MAX_DIMS] = {nullptr};
  int64_t w_off[OLSGD_MAX_DIMS] = {0}, b_off[OLSGD_MAX_DIMS] = {0};
  // weights and bias of parameter layer p are updated inside their weight-gradient kernel
  bool fused_layer[OLSGD_MAX_DIMS] = {false};
  // the output layer's weights and bias are updated inside its weight-gradient kernel
  bool fused_head = false;
  // what is left for the stand-alone update kernel: ranges [off, off + len) of a worker row
  int n_ranges = 0;
  int64_t range_off[OLSGD_MAX_DIMS + 1] = {0}, range_len[OLSGD_MAX_DIMS + 1] = {0};
  // Worker sum inside the sync-step weight-gradient launch: the ranges of a row it covers
  // (the fused layers' weight matrices).
  int n_summed = 0;
  int64_t summed_off[OLSGD_MAX_DIMS] = {0}, summed_len[OLSGD_MAX_DIMS] = {0};
};
struct StepIO {
  const float* x;                // x_k, [m][ld]
  const __nv_bfloat16* shadow;   // bf16 copy of x_k or null
  float* g;                      // out: [m][ld]
  int64_t ld;
  int32_t* idx;                  // [m][batch]
  const IndexRule* rule;         // if non-null, idx is an output: the gather draws the indices
  const __nv_bfloat16* xb16_in;  // if non-null: this step's rows, already bf16, [m][batch][dims[0]]
                                 // (data.y then holds their labels [m][batch]); idx is unused
  int batch_set;                 // which staged-minibatch set this iteration uses (0 or 1)
  bool batch_staged;             // the set already holds this iteration's rows (or, with
                                 // xb16_in, their transposed copy and labels): no staging kernel
  float* loss;                   // out: [m] or null
  int* status;                   // device status word (see GemmArgs::status)
  FusedUpdateArgs upd;           // state pointers and factors for the fused epilogue (w_off unset)
  cudaEvent_t wait_before_update;  // if non-null, the stream waits for it before x_out is written
  // Optional second stream (with two events) for work that does not lie on the critical
  // path of the backward pass; null: everything runs on the main stream.
  cudaStream_t aux;
  cudaEvent_t aux_fork, aux_join;
  // If non-null: recorded on the main stream once the forward GEMMs are launched, the point
  // from which the next iteration's rows may be staged beside this iteration.
  cudaEvent_t mid_event;
};
// Lets model.cu count and time its launches without knowing the context type.  `cls` is a
// kernel class, optionally plus 256 * (the layer the launch belongs to).
struct ProfHook {
  void* ctx;
  void* (*begin)(void* ctx, int cls, cudaStream_t s);
  void (*end)(void* handle);
};
bool plan_model(const olsgd_model_spec& spec, const olsgd_hparams& hp, ModelPlan* mp);
bool bind_model(const olsgd_model_spec& spec, const olsgd_hparams& hp, const ModelPlan& mp,
                char* base, ModelBuffers* mb);
cudaError_t model_forward_backward(const olsgd_model_spec& spec, const olsgd_hparams& hp,
                                   const olsgd_data& data, const ModelBuffers& mb,
                                   const StepIO& io, cudaStream_t s, const ProfHook& hook);
// S1 + S2 of the bf16 path for one iteration, by themselves: draws the indices by `rule` and
// stages the rows into set `set` on stream s.
cudaError_t model_stage_batch(const olsgd_model_spec& spec, const olsgd_hparams& hp,
                              const olsgd_data& data, const ModelBuffers& mb, int32_t* idx,
                              const IndexRule& rule, int set, cudaStream_t s, const ProfHook& hook);
// The staging of host-fed bf16 rows by itself: transposed copy and labels into set `set`.
cudaError_t model_stage_host_rows(const olsgd_model_spec& spec, const olsgd_hparams& hp,
                                  const __nv_bfloat16* rows, const int32_t* labels,
                                  const ModelBuffers& mb, int set, cudaStream_t s,
                                  const ProfHook& hook);

}  // namespace olsgd
