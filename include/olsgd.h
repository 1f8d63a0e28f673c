/*
 * olsgd.h -- C ABI of the Overlap-Local-SGD hot path for m simulated workers
 * stacked on one GPU (Wang, Liang, Joshi, "Overlap Local-SGD", arXiv
 * 2002.09539, Section 2 "Proposed Algorithm").
 *
 * One context holds the m worker models x^(1..m), their local momentum
 * buffers, the anchor z and the anchor momentum buffer v, all resident in
 * device memory that the CALLER allocates and hands over as one workspace.
 * A context owns host memory, CUDA events and three small streams of its
 * own: one for host-to-device staging copies, one on which the output layer's
 * weight gradient runs beside the hidden layers' backward pass, and one
 * (low priority) on which the next iteration's minibatch rows are staged
 * while the current iteration computes; all of them are joined by
 * olsgd_join and olsgd_destroy, and the borrowed data set must stay valid
 * until then.  The library never allocates device memory, never throws,
 * never aborts: every call returns a status and `olsgd_last_error` gives the
 * reason as text.
 *
 * Conventions
 *   - "device pointer": memory on the current CUDA device, 16-byte aligned.
 *   - Flat parameter layout: for each layer in order, the weight matrix
 *     W_l row-major as [out][in] followed by its bias b_l [out]; linear
 *     regression is one weight vector w [d] without bias.
 *   - Iterations k are 0-based.  Iteration k is a "sync step" when
 *     (k + 1) mod tau == 0.
 *   - Calls are asynchronous with respect to the host unless stated.  All
 *     calls on one context must come from one host thread at a time.
 */
#ifndef OLSGD_H
#define OLSGD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct olsgd_ctx olsgd_ctx; /* opaque, host side */

typedef enum {
  OLSGD_OK = 0,
  OLSGD_EINVAL = 1,   /* bad argument; nothing was changed                */
  OLSGD_ESTATE = 2,   /* call out of order; nothing was changed           */
  OLSGD_ENOMEM = 3,   /* workspace too small / host allocation failed     */
  OLSGD_ECUDA = 4,    /* a CUDA runtime or driver call failed             */
  OLSGD_ETIMEOUT = 5  /* a bounded device-side wait gave up               */
} olsgd_status;

typedef enum {
  OLSGD_LINREG = 0,   /* loss (1/2B) sum (x_s . w - y_s)^2, dims = {d}             */
  OLSGD_SOFTMAX = 1,  /* softmax regression, dims = {d_in, n_classes}              */
  OLSGD_MLP = 2,      /* ReLU MLP + mean cross-entropy, dims = {d_in, h.., classes} */
  OLSGD_FLAT = 3      /* flat parameter vector, gradients supplied by the caller   */
} olsgd_model;

#define OLSGD_MAX_DIMS 8

typedef struct {
  int32_t kind;                 /* olsgd_model                                        */
  int32_t n_dims;               /* entries used in dims (1 for LINREG, 0 for FLAT)    */
  int32_t dims[OLSGD_MAX_DIMS]; /* e.g. {3072, 1024, 1024, 10}                        */
  int32_t gemm_bf16;            /* MLP only.  1 = bf16 operands on the tensor cores, fp32
                                   accumulate, fp32 master weights, the parameter update
                                   of the hidden-layer weights fused into the weight-
                                   gradient GEMM; 3 = the same GEMMs with the update as a
                                   separate kernel; 2 = the same bf16 data flow on CUDA
                                   cores (a check of the tensor-core kernels); 0 = fp32
                                   (models without hidden layers).  Any layer widths and
                                   batch sizes are accepted.  In modes 1 and 3 the
                                   tensor-core kernels take batches and layer widths in
                                   multiples of 8 (16-byte row pitches; partial last tiles
                                   are padded with zeros by TMA and clipped on the way
                                   out); any other GEMM runs on the CUDA-core kernel of
                                   mode 2.  The update is fused into
                                   the weight-gradient GEMM of layers whose two widths are
                                   multiples of 128 at a batch of 64 or 128; the other
                                   layers go through the update kernel.
                                   olsgd_tensor_core_launches counts what ran where.   */
  int32_t reserved;
  int64_t flat_P;               /* FLAT only: number of parameters                    */
} olsgd_model_spec;

/* The paper's symbols (Section 2): m workers, tau local steps per period,
 * gamma learning rate (Eq. 3), alpha pull-back rate (Eq. 4), beta anchor
 * momentum factor (Eq. 10).  mu is the factor of the "common Nesterov
 * momentum" of the local step (u <- mu u + g, x <- x - gamma (g + mu u));
 * mu = 0 is plain SGD, beta = 0 is the vanilla anchor refresh of Eq. 5.     */
typedef enum {
  OLSGD_MODE_OVERLAP = 0,    /* Overlap-Local-SGD: Eq. 3-5 (and Eq. 10-11)                 */
  OLSGD_MODE_LOCAL_SGD = 1   /* Local SGD / periodic averaging, Eq. 2: on a sync step every
                                worker model is replaced by the average of all of them,
                                on the main stream (blocking); tau = 1 is fully synchronous
                                SGD.  alpha and beta are ignored, olsgd_period_sync is
                                never due, and z reports the last average                */
} olsgd_mode;

typedef struct {
  int32_t m, tau, batch, mode /* olsgd_mode */;
  float gamma, alpha, beta, mu;
  uint64_t seed;                /* seeds the minibatch index rule                    */
  /* Sharding of the worker dimension over several contexts (one per GPU).  This context
   * holds the workers worker_offset .. worker_offset + m - 1 of m_total; the minibatch rule
   * uses the global worker id and the anchor is the mean over all m_total workers, formed
   * with olsgd_period_sync_begin / _finish around the caller's all-reduce.  m_total = 0
   * means "not sharded" (m_total = m, worker_offset = 0).                              */
  int32_t worker_offset, m_total;
  /* Minibatch rule.  0: independent uniform draws with replacement (see olsgd_get_indices).
   * 1: one pass over D_i per epoch without replacement: draw t = k * batch + j of worker i
   * takes sample pi(t mod n) of epoch e = t div n, where pi is a four-round balanced Feistel
   * permutation of 0..n-1 with cycle walking (Black and Rogaway, CT-RSA 2002) on two halves
   * of h = ceil(ceil(log2 n) / 2) bits; round r maps (L, R) to (R, L xor F) with F the low h
   * bits of word 0 of the Philox4x32-10 block of counter (R, 4 e + r, i, 3) and the same
   * key; the network is applied again while the value is >= n.                          */
  int32_t sampling, reserved2;
} olsgd_hparams;

/* Worker i's data set D_i (Eq. 1).  Device pointers, borrowed for the life of
 * the context, never written, never freed.
 *   X  float32 [m][n_per_worker][dims[0]]
 *   y  float32 [m][n_per_worker]  (LINREG targets)  or
 *      int32   [m][n_per_worker]  (class labels in [0, dims[last]))         */
typedef struct {
  const void* X;
  const void* y;
  int64_t n_per_worker;
} olsgd_data;

/* Number of parameters P of one model copy in the flat layout.              */
olsgd_status olsgd_param_count(const olsgd_model_spec* spec, int64_t* out_P);

/* Bytes of device workspace `olsgd_init` needs for this model and these
 * hyper-parameters (state, gradients, batch staging, activations).          */
olsgd_status olsgd_workspace_bytes(const olsgd_model_spec* spec, const olsgd_hparams* hp,
                                   size_t* out_bytes);

/* Create a context.  Sets x_0^(i) = z_0 = x0 for every worker (the initial
 * condition of Theorem 1), zeroes the momentum buffers u_i and v, k = 0.
 *   x0_device        P floats, device; copied, not kept
 *   workspace_device at least olsgd_workspace_bytes bytes, 256-byte aligned;
 *                    owned by the caller, must outlive the context
 *   main_stream      cudaStream_t on which the local steps run
 *   side_stream      cudaStream_t on which the anchor refresh runs; may equal
 *                    main_stream (then nothing overlaps)
 *   data             may be NULL for OLSGD_FLAT
 * The context belongs to the CUDA device that is current during this call (the workspace,
 * the data set and both streams must live there); every later call on it must be made with
 * the same device current and returns OLSGD_ESTATE otherwise.
 * Checks: m, tau, batch >= 1; gamma > 0; 0 <= alpha <= 1; 0 <= beta < 1;
 * 0 <= mu < 1; pointers non-null and aligned.  On error *out is NULL.       */
olsgd_status olsgd_init(olsgd_ctx** out, const olsgd_model_spec* spec, const olsgd_hparams* hp,
                        const olsgd_data* data, const float* x0_device, void* workspace_device,
                        size_t workspace_bytes, void* main_stream, void* side_stream);

/* One iteration k -> k+1 for all m workers on the main stream: draw the
 * minibatches xi_k^(i), evaluate g_i(x_k^(i); xi_k^(i)), apply Eq. 3 (with
 * the local Nesterov buffer when mu > 0) and, on a sync step, Eq. 4 against
 * the anchor produced by the previous period (the one-period lag stated after
 * Eq. 5), all on the device.
 *   loss_device  m floats, device: mean minibatch loss per worker at x_k; or NULL
 * Returns OLSGD_ESTATE if a period ended and olsgd_period_sync has not been
 * called since.                                                             */
olsgd_status olsgd_local_step(olsgd_ctx* ctx, float* loss_device);

/* The same iteration, with this step's minibatches supplied from HOST memory
 * instead of being drawn from the resident data set: for a caller whose data
 * loader lives on the host.  The rows are copied to the device on a copy stream
 * owned by the context (double-buffered, so the copy of step k+1 overlaps the
 * kernels of step k), then the step runs exactly as olsgd_local_step does.
 *   Xb_host    float32 [m][batch][dims[0]], host (pinned memory for a truly
 *              asynchronous copy); must stay valid and unchanged until a later
 *              call has joined the streams (olsgd_get_params, olsgd_join)
 *   yb_host    float32 [m][batch] (LINREG) or int32 [m][batch]
 *   loss_host  m floats, host: written asynchronously with the per-worker
 *              minibatch losses, valid after the streams are joined; or NULL
 * The minibatch index rule is not used by this call.                         */
olsgd_status olsgd_local_step_host(olsgd_ctx* ctx, const float* Xb_host, const void* yb_host,
                                   float* loss_host);

/* olsgd_local_step_host for models whose GEMM operands are bf16 (OLSGD_MLP with
 * gemm_bf16 != 0): the caller hands over the rows already rounded to bf16
 * (round-to-nearest-even, the rounding the device applies to fp32 rows), which
 * halves the host-to-device bytes of a step.  The result has the bits of
 * olsgd_local_step_host on the fp32 rows they were rounded from.
 *   Xb_host_bf16  bf16 (uint16 storage) [m][batch][dims[0]], host, same lifetime
 *                 rule as Xb_host above
 *   yb_host       int32 [m][batch]
 *   loss_host     as above
 * Returns OLSGD_ESTATE for any other model, and where dims[0] is not a
 * multiple of 64 or the batch not a multiple of 8 (the rows are moved in
 * 16-byte pieces; olsgd_local_step_host takes every shape).                 */
olsgd_status olsgd_local_step_host_bf16(olsgd_ctx* ctx, const void* Xb_host_bf16,
                                        const void* yb_host, float* loss_host);

/* Block the host until every stream of the context is idle.                 */
olsgd_status olsgd_join(olsgd_ctx* ctx);

/* Every wait a kernel of this library performs on a barrier is bounded; a wait that runs
 * out makes the kernel return early and the next joining call (olsgd_join,
 * olsgd_get_params) return OLSGD_ETIMEOUT.  olsgd_selftest_wait_timeout exercises that
 * path without any fault: it launches a kernel whose one thread waits, for at most
 * limit_ms milliseconds, on a barrier that nothing ever arrives on.  After it, olsgd_join
 * returns OLSGD_ETIMEOUT until olsgd_clear_status is called; the context and the GPU
 * stay usable throughout.  limit_ms must be in [1, 2000].                        */
olsgd_status olsgd_selftest_wait_timeout(olsgd_ctx* ctx, int32_t limit_ms);
olsgd_status olsgd_clear_status(olsgd_ctx* ctx);

/* Host-only self-test of the table that remembers, per device ordinal, which dynamic
 * shared-memory limit each kernel has been configured for (kernel attributes belong to a
 * device: a process that opens contexts on two GPUs must configure both).  Launches
 * nothing and needs no GPU.  OLSGD_OK, or OLSGD_ESTATE if the table misbehaves.          */
olsgd_status olsgd_selftest_per_device_table(void);

/* Same iteration for OLSGD_FLAT: the stacked gradients G_k (Eq. 7 without its
 * zero column) come from the caller.
 *   g_device  float32 [m][P], device, row stride P; read on the main stream */
olsgd_status olsgd_local_step_with_grads(olsgd_ctx* ctx, const float* g_device);

/* Anchor refresh at the end of a period: Eq. 5 (beta = 0) or Eq. 10-11, as a
 * reduction over the worker dimension launched on the side stream after the
 * pull-back that closed the period.  Returns at once; the next period's local
 * steps overlap with it and its result is first read by the next pull-back.
 * Legal exactly once per period, when k > 0 and k mod tau == 0; otherwise
 * OLSGD_ESTATE.                                                             */
olsgd_status olsgd_period_sync(olsgd_ctx* ctx);

/* Where the worker sum of Eq. 5 / Eq. 10-11 is formed.  In OLSGD_MODE_OVERLAP a sync step
 * writes x_{k+1} anyway, so the launches that write it also add it up over this context's
 * workers (a few rows of partial sums in the workspace) and x_{k+1} is not read a second
 * time: the weight-gradient launch of hidden layers on the tensor cores (gemm_bf16 = 1), and
 * the stand-alone update kernel on every range of a parameter row, of four workers or more,
 * that is long enough to give every multiprocessor work with one thread per 16 bytes
 * (OLSGD_FLAT rows, gemm_bf16 = 2, 3).
 * olsgd_period_sync, or olsgd_period_sync_begin in a sharded run, then finishes on the side
 * stream from those rows, and runs the worker-mean kernel only on the rest of a parameter
 * row (biases, output layer, short rows).  The one-period lag stated after Eq. 5 is
 * untouched: the anchor is written on the side stream and first read by the next sync step.
 * on == 0 moves the whole sum back to the worker-mean kernel; both ways give the same bits
 * (same summation order).  Default: on.  Legal between periods (not while olsgd_period_sync
 * is due); olsgd_anchor_fusion reports the setting, olsgd_summed_floats how many parameters
 * of a row the most recent anchor refresh took from such partial sums (0: none).          */
olsgd_status olsgd_set_anchor_fusion(olsgd_ctx* ctx, int32_t on);
int32_t olsgd_anchor_fusion(const olsgd_ctx* ctx);
int64_t olsgd_summed_floats(const olsgd_ctx* ctx);

/* The anchor refresh split in two for a worker dimension that is sharded over several
 * contexts: the only exchange of the method is the sum in Eq. 5.
 *   olsgd_period_sync_begin   legal exactly when olsgd_period_sync would be; on the side
 *                             stream, after the pull-back that closed the period, writes
 *                             the undivided sum of THIS context's worker models into
 *                             partial_sum_device (P floats rounded up to a multiple of 64,
 *                             device, 16-byte aligned; olsgd_row_floats gives the count)
 *   (caller)                  sums that buffer over all contexts, in place, ordered after the
 *                             side stream's work and before the next call: ncclAllReduce on
 *                             the side stream, or any other means
 *   olsgd_period_sync_finish  on the side stream: s = total / m_total, then Eq. 5 or Eq. 10-11
 * Both return at once; the next period's local steps overlap with all three stages, exactly
 * as with olsgd_period_sync.  OLSGD_MODE_OVERLAP only.                                   */
olsgd_status olsgd_period_sync_begin(olsgd_ctx* ctx, float* partial_sum_device);
olsgd_status olsgd_period_sync_finish(olsgd_ctx* ctx, const float* total_sum_device);
/* Floats in one padded state row (P rounded up to a multiple of 64).                    */
int64_t olsgd_row_floats(const olsgd_ctx* ctx);

/* n_iters iterations in one call: olsgd_local_step, followed by
 * olsgd_period_sync whenever a period ends.  Not for OLSGD_FLAT.
 *   loss_device  n_iters * m floats ([iteration][worker]), device; or NULL  */
olsgd_status olsgd_run(olsgd_ctx* ctx, int64_t n_iters, float* loss_device);

/* How often olsgd_run has replayed a captured CUDA graph on this context so far.  olsgd_run
 * executes its iterations as replays of one captured block of whole periods (an even number
 * of iterations); the iteration number the minibatch rule needs is then read from device
 * memory.  A run of at least three default blocks (olsgd_graph_block) launches one block
 * kernel by kernel, captures it and replays it; a run of 8 to 64 iterations on a context that
 * has already launched an ordinary and a sync step kernel by kernel is captured whole, so
 * that repeating olsgd_run(n) costs one graph launch per call.  Capturing needs main_stream
 * to be a real stream: with the legacy default stream (NULL) olsgd_run keeps launching kernel
 * by kernel and this stays 0.  The results are the same bits either way.                   */
int64_t olsgd_graph_replays(const olsgd_ctx* ctx);
/* Iterations in the default captured block of this context: whole periods, an even count, at
 * least eight.                                                                            */
int64_t olsgd_graph_block(const olsgd_ctx* ctx);

/* Process-wide switch for how the kernels of one iteration follow each other on the main
 * stream.  on != 0 (the default): they are launched with programmatic stream serialization,
 * so a kernel's blocks may become resident and set up their shared state while the kernel
 * before it is still draining; every kernel waits for its predecessors to complete before
 * its first access to global memory, so the results are the same bits.  on == 0: plain
 * stream order.  Applies to launches made after the call (a captured graph of olsgd_run
 * keeps the setting it was captured with).  Returns the previous setting.  The paper has
 * no counterpart: this is launch plumbing.                                               */
int olsgd_set_launch_overlap(int on);

/* Process-wide switch for the forward and input-gradient GEMMs of the tensor-core path.
 * on != 0: where a layer has an even number of 128-row tiles they run on CTA pairs
 * (thread-block clusters of two, one tcgen05.mma of M = 256 for both, each CTA loading half
 * of the batch operand).  on == 0 (the default: measured slightly faster on the benchmark
 * configurations): one CTA per tile.  The accumulation order of every output element is the
 * same, so the results are the same bits.  Applies to launches made after the call (a
 * captured graph keeps the setting it was captured with).  Returns the previous setting.
 * The paper has no counterpart: this is kernel plumbing.                                    */
int olsgd_set_gemm_pairs(int on);

/* How many launches of the tensor-core (tcgen05) kernels this process has made so far:
 * forward / input-gradient GEMMs and weight-gradient launches.  Lets a caller (or a test)
 * see whether a model's GEMMs ran there or on the CUDA-core kernel they fall back to.      */
int64_t olsgd_tensor_core_launches(void);

/* Copy one vector of the state to the caller.  Joins both streams (blocks
 * the host).  which: 0..m-1 worker model x^(i); -1 anchor z; -2 anchor
 * momentum v; -3 virtual sequence y = (1-alpha) mean_i x^(i) + alpha z
 * (Appendix A); -4 mean model mean_i x^(i); -5 - i local momentum u_i.
 *   dst       host or device memory
 *   n_floats  must equal P                                                   */
olsgd_status olsgd_get_params(olsgd_ctx* ctx, int32_t which, float* dst, size_t n_floats);

/* Overwrite one vector of the state (checkpoint / resume together with
 * olsgd_get_params and olsgd_set_iteration).  Joins both streams.  which: 0..m-1 worker
 * model (its bf16 copy for the tensor cores is refreshed too); -1 anchor z; -2 anchor
 * momentum v; -5 - i local momentum u_i.
 *   src       host or device memory, n_floats == P                                  */
olsgd_status olsgd_set_params(olsgd_ctx* ctx, int32_t which, const float* src, size_t n_floats);

/* Set the iteration counter k (k >= 0, k mod tau == 0: a period boundary, no anchor
 * refresh pending).  With the state vectors restored this resumes a run exactly: the
 * minibatch rule is a function of k.                                                 */
olsgd_status olsgd_set_iteration(olsgd_ctx* ctx, int64_t k);

/* Consensus distance sum_i ||x^(i) - z||^2 of the current state (the quantity the
 * convergence proof bounds, Appendix A), summed in double precision in a fixed order on
 * the device.  Joins both streams.  out_host: one double on the host.                */
olsgd_status olsgd_consensus_distance(olsgd_ctx* ctx, double* out_host);

/* The minibatch indices xi_k^(i) that iteration k uses (or used): slot j of
 * worker i is floor(w * n / 2^32) with w word (j mod 4) of the Philox4x32-10
 * block (Salmon et al., SC'11) of counter (j div 4, k, i, 1) and key
 * (seed mod 2^32, seed div 2^32).  Computed on the device; blocks the host.
 *   dst  int32 [m][batch], host or device                                   */
olsgd_status olsgd_get_indices(olsgd_ctx* ctx, int64_t k, int32_t* dst);

/* h of the epoch minibatch rule (olsgd_hparams.sampling = 1) for a partition of n samples:
 * the Feistel network permutes the 2^(2h) values of two h-bit halves, h = ceil(ceil(log2 n)
 * / 2), so 2^(2h) < 4 n and a pass of the cycle walk succeeds with probability above 1/4.
 * The device gives a slot up after 64 passes (probability below 1e-8 per draw), stores index
 * 0 for it and raises the status word: the next joining call returns OLSGD_ETIMEOUT.
 * Host only.  Returns -1 unless 1 <= n < 2^31.                                          */
int32_t olsgd_epoch_rule_half_bits(int64_t n);

/* Non-IID partition table: the two classes (of ten) each worker samples
 * from.  Class slots are concatenated seeded Fisher-Yates permutations of
 * 0..9 (permutation t, position p from 9 down to 1, swaps with
 * floor(w (p+1) / 2^32), w = word 0 of the Philox block of counter
 * (p, t, 0, 2)); worker i takes slots 2i and 2i+1.  Stand-in for the skewed
 * partitions of the paper's non-IID experiment (Section 4).  Computed on the
 * device on `stream`; blocks the host.
 *   dst  int32 [m][2], host or device                                       */
olsgd_status olsgd_class_pairs(uint64_t seed, int32_t m, int32_t* dst, void* stream);

/* The same table for callers that must not allocate.  (The paper has no
 * counterpart to this entry point; it exists for the library's users.)
 *
 * olsgd_class_pairs stages a host destination through pinned memory that it
 * allocates and frees on every call.  Some callers cannot do that: code that
 * runs between cudaStreamBeginCapture and cudaStreamEndCapture on another
 * stream of the same thread (an allocation call there invalidates the
 * capture), a process whose memory has been handed in full to a pool or to
 * another framework, or a latency-critical thread that is not allowed to take
 * the allocator's locks.  This variant calls no cudaMalloc, cudaFree,
 * cudaHostAlloc or any other allocating routine.  The kernel writes the table
 * into a fixed array that lives in the library's device image, and the result
 * is copied from there to `dst`.
 *
 *   m       at most OLSGD_NOALLOC_MAX_WORKERS; larger values are rejected with
 *           OLSGD_EINVAL and a message, nothing is launched
 *   dst     int32 [m][2], host or device
 *   stream  cudaStream_t the kernel and the copy run on; the call blocks the
 *           host until both are done
 *
 * Cost and rules of the fixed array:
 *   - every GPU on which the library is loaded holds it (128 KB) until the
 *     process exits, whether or not this entry point is ever called;
 *   - the first call on each device looks the array's device address up once
 *     (with that device current); make that first call before starting any
 *     stream capture;
 *   - all calls share the one array, which keeps what the last call wrote.
 *     Each call overwrites every entry it returns, so nothing has to be
 *     cleared, but two calls whose GPU work overlaps (different streams or
 *     threads on the same device) race on it: serialise them.                 */
#define OLSGD_NOALLOC_MAX_WORKERS 16384
olsgd_status olsgd_class_pairs_noalloc(uint64_t seed, int32_t m, int32_t* dst, void* stream);

/* Iteration counter k.                                                      */
int64_t olsgd_iteration(const olsgd_ctx* ctx);

/* Number of kernels this context has launched so far.                       */
int64_t olsgd_launch_count(const olsgd_ctx* ctx);

/* Device-time profile of the kernel classes.  When enabled, every launch is
 * bracketed by CUDA events on its own stream.  olsgd_profile_read joins both
 * streams and returns, per class c in 0..OLSGD_N_KERNEL_CLASSES-1, the launch
 * count and the summed duration in milliseconds since the last reset.       */
#define OLSGD_N_KERNEL_CLASSES 9
enum { OLSGD_KC_INDEX = 0, OLSGD_KC_GATHER = 1, OLSGD_KC_FORWARD = 2, OLSGD_KC_BACKWARD = 3,
       OLSGD_KC_UPDATE = 4, OLSGD_KC_ANCHOR = 5, OLSGD_KC_LOSS = 6, OLSGD_KC_OTHER = 7,
       OLSGD_KC_WGRAD_UPDATE = 8 /* weight-gradient GEMM with the update fused in */ };
olsgd_status olsgd_profile_enable(olsgd_ctx* ctx, int32_t on);
olsgd_status olsgd_profile_read(olsgd_ctx* ctx, int64_t* launches, double* millis, int32_t reset);
/* The same profile split by layer: entry [c * OLSGD_MAX_DIMS + l] covers the launches of class
 * c that belong to layer l (forward GEMM producing hidden layer l >= 1; OLSGD_KC_BACKWARD with
 * l >= 1: the input-gradient GEMM producing the gradient of hidden layer l, or a weight-
 * gradient GEMM that is launched by itself; OLSGD_KC_WGRAD_UPDATE: l = 0 ordinary steps, l = 1
 * sync steps; otherwise l = 0: launches that belong to no hidden layer, e.g. the output
 * layer's kernels).  Both arrays hold OLSGD_N_KERNEL_CLASSES * OLSGD_MAX_DIMS
 * entries.  Summing over l gives olsgd_profile_read.                                      */
olsgd_status olsgd_profile_read_layers(olsgd_ctx* ctx, int64_t* launches, double* millis,
                                       int32_t reset);

/* Text of the last error on this context ("" if none).  ctx may be NULL, in
 * which case the last error of a failed olsgd_init / context-free call in this
 * thread is returned.                                                       */
const char* olsgd_last_error(const olsgd_ctx* ctx);

/* Join both streams, destroy events, free host memory.  Device memory stays
 * with the caller.                                                          */
olsgd_status olsgd_destroy(olsgd_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* OLSGD_H */
