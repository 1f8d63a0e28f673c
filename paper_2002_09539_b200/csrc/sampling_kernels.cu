// Minibatch index rule and the non-IID class-pair table, on the device (Philox4x32-10 is
// in philox.cuh).
#include <cstdio>
#include <mutex>

#include "olsgd_internal.h"
#include "philox.cuh"

namespace olsgd {
namespace {

// One thread per Philox block: four consecutive slots of one worker.
__global__ void minibatch_indices_kernel(int32_t* __restrict__ idx, uint32_t k0, uint32_t k1,
                                         int m, uint64_t k_base, const long long* k_ptr,
                                         int batch, uint32_t n, uint32_t worker_offset) {
  launch_gate();
  // inside a captured graph the iteration number lives in device memory
  const uint32_t k = (uint32_t)(k_base + (k_ptr ? (uint64_t)*k_ptr : 0ull));
  const int blocks_per_worker = (batch + 3) / 4;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= m * blocks_per_worker) return;
  const int i = t / blocks_per_worker, q = t % blocks_per_worker;
  const U4 r = philox4x32_10((uint32_t)q, k, (uint32_t)i + worker_offset, kStreamMinibatch, k0, k1);
#pragma unroll
  for (int lane = 0; lane < 4; ++lane) {
    const int j = q * 4 + lane;
    if (j < batch) idx[(int64_t)i * batch + j] = (int32_t)__umulhi(r.w[lane], n);
  }
}

// One thread per permutation of the ten classes (ten slots = five workers).
__global__ void class_pairs_kernel(int32_t* __restrict__ dst, uint32_t k0, uint32_t k1, int m) {
  const int n_perm = (2 * m + 9) / 10;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n_perm) return;
  int perm[10];
#pragma unroll
  for (int c = 0; c < 10; ++c) perm[c] = c;
  for (int p = 9; p >= 1; --p) {
    const U4 r = philox4x32_10((uint32_t)p, (uint32_t)t, 0u, kStreamPartition, k0, k1);
    const int q = (int)__umulhi(r.w[0], (uint32_t)(p + 1));
    const int a = perm[p];
    perm[p] = perm[q];
    perm[q] = a;
  }
  for (int c = 0; c < 10; ++c) {
    const int slot = t * 10 + c;
    if (slot < 2 * m) dst[slot] = perm[c];
  }
}

// Epoch rule, one thread per slot: draw t = k * batch + j belongs to epoch e = t / n and takes
// sample pi(t % n); pi is a four-round balanced Feistel network on two h-bit halves whose
// round function is a Philox word, applied again while the result is >= n (cycle walking).
// The domain 2^(2h) is below 4 n, so a pass lands inside [0, n) with probability above 1/4
// and the expected number of passes is below 4; kEpochWalkLimit passes all failing has
// probability below (3/4)^64 = 1e-8 per draw of a random permutation.  Should it happen
// anyway, no out-of-range index is stored: the slot gets 0 and the status word is raised, so
// the next joining call reports OLSGD_ETIMEOUT.
constexpr int kEpochWalkLimit = 64;
__global__ void minibatch_indices_epoch_kernel(int32_t* __restrict__ idx, uint32_t k0, uint32_t k1,
                                               int m, uint64_t k_base, const long long* k_ptr,
                                               int batch, uint32_t n, int h,
                                               uint32_t worker_offset, int* status) {
  launch_gate();
  const uint64_t k = k_base + (k_ptr ? (uint64_t)*k_ptr : 0ull);
  const int t_id = blockIdx.x * blockDim.x + threadIdx.x;
  if (t_id >= m * batch) return;
  const int i = t_id / batch, j = t_id % batch;
  const uint64_t t = k * (uint64_t)batch + (uint64_t)j;
  const uint32_t e = (uint32_t)(t / n);
  uint32_t v = (uint32_t)(t % n);
  const uint32_t mask = (1u << h) - 1u;
  bool found = false;
  for (int walk = 0; walk < kEpochWalkLimit; ++walk) {
    uint32_t left = v >> h, right = v & mask;
#pragma unroll
    for (uint32_t r = 0; r < 4; ++r) {
      const U4 w = philox4x32_10(right, 4u * e + r, (uint32_t)i + worker_offset, kStreamEpoch, k0, k1);
      const uint32_t f = w.w[0] & mask;
      const uint32_t nl = right;
      right = left ^ f;
      left = nl;
    }
    v = (left << h) | right;
    if (v < n) {
      found = true;
      break;
    }
  }
  if (!found) {
    v = 0;
    if (status) atomicExch(status, (int)OLSGD_ETIMEOUT);
  }
  idx[t_id] = (int32_t)v;
}

// The device-resident iteration counter of a captured graph: *p = value, or *p += by.
__global__ void counter_kernel(long long* p, long long value, long long by, int set) {
  launch_gate();
  if (threadIdx.x == 0 && blockIdx.x == 0) *p = set ? value : *p + by;
}

__global__ void identity_indices_kernel(int32_t* __restrict__ idx, int total, int batch) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < total) idx[t] = t % batch;
}

}  // namespace

int epoch_rule_half_bits(int64_t n) {
  int bits = 1;
  while (((int64_t)1 << bits) < n) ++bits;       // ceil(log2 n), at least 1
  return (bits + 1) / 2;
}

cudaError_t launch_identity_indices(int32_t* idx, int m, int batch, cudaStream_t s) {
  const int total = m * batch, threads = 256;
  identity_indices_kernel<<<(total + threads - 1) / threads, threads, 0, s>>>(idx, total, batch);
  return cudaGetLastError();
}

cudaError_t launch_minibatch_indices(int32_t* idx, uint64_t seed, int m, int64_t k, int batch,
                                     int64_t n, int worker_offset, const int64_t* k_ptr,
                                     cudaStream_t s) {
  const int total = m * ((batch + 3) / 4);
  const int threads = 128;
  return launch_chained(minibatch_indices_kernel, dim3((total + threads - 1) / threads), dim3(threads),
                        0, s, idx, (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32), m,
                        (uint64_t)k, reinterpret_cast<const long long*>(k_ptr), batch, (uint32_t)n,
                        (uint32_t)worker_offset);
}

cudaError_t launch_minibatch_indices_epoch(int32_t* idx, uint64_t seed, int m, int64_t k, int batch,
                                           int64_t n, int worker_offset, const int64_t* k_ptr,
                                           int* status, cudaStream_t s) {
  const int h = epoch_rule_half_bits(n);
  const int total = m * batch, threads = 128;
  return launch_chained(minibatch_indices_epoch_kernel, dim3((total + threads - 1) / threads),
                        dim3(threads), 0, s, idx, (uint32_t)(seed & 0xFFFFFFFFu),
                        (uint32_t)(seed >> 32), m, (uint64_t)k,
                        reinterpret_cast<const long long*>(k_ptr), batch, (uint32_t)n, h,
                        (uint32_t)worker_offset, status);
}

cudaError_t launch_counter(int64_t* p, int64_t value, int64_t by, bool set, cudaStream_t s) {
  return launch_chained(counter_kernel, dim3(1), dim3(32), 0, s, reinterpret_cast<long long*>(p),
                        (long long)value, (long long)by, set ? 1 : 0);
}

cudaError_t launch_class_pairs(int32_t* dst, uint64_t seed, int m, cudaStream_t s) {
  const int n_perm = (2 * m + 9) / 10;
  const int threads = 64;
  class_pairs_kernel<<<(n_perm + threads - 1) / threads, threads, 0, s>>>(
      dst, (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32), m);
  return cudaGetLastError();
}

}  // namespace olsgd

// ---------------------------------------------------------------------------
// olsgd_class_pairs_noalloc: the partition table without any allocation.
//
// The staging buffer is a file-scope array in the library's device image.  In
// host code the name `g_pair_scratch` is only a handle for the runtime, not a
// device address, so it is never passed to a kernel: its address on the current
// device is looked up once per device with cudaGetSymbolAddress and that
// pointer is what the kernel and the copy receive.
namespace {

static __device__ __align__(256) int32_t g_pair_scratch[2 * OLSGD_NOALLOC_MAX_WORKERS];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
int32_t* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device (set-up on first use).
cudaError_t scratch_address(int32_t** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_pair_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = static_cast<int32_t*>(p);
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

olsgd_status noalloc_fail(olsgd_status st, const char* what, cudaError_t e) {
  char buf[256];
  if (e != cudaSuccess)
    snprintf(buf, sizeof buf, "olsgd_class_pairs_noalloc: %s: %s", what, cudaGetErrorString(e));
  else
    snprintf(buf, sizeof buf, "olsgd_class_pairs_noalloc: %s", what);
  olsgd::set_thread_error(buf);
  return st;
}

}  // namespace

extern "C" olsgd_status olsgd_class_pairs_noalloc(uint64_t seed, int32_t m, int32_t* dst,
                                                  void* stream) {
  if (m < 1) return noalloc_fail(OLSGD_EINVAL, "m must be >= 1", cudaSuccess);
  if (m > OLSGD_NOALLOC_MAX_WORKERS) {
    char buf[128];
    snprintf(buf, sizeof buf, "m = %d exceeds the fixed scratch array (at most %d workers)", m,
             OLSGD_NOALLOC_MAX_WORKERS);
    return noalloc_fail(OLSGD_EINVAL, buf, cudaSuccess);
  }
  if (!dst) return noalloc_fail(OLSGD_EINVAL, "dst is NULL", cudaSuccess);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t* scratch = nullptr;
  cudaError_t e = scratch_address(&scratch);
  if (e != cudaSuccess) return noalloc_fail(OLSGD_ECUDA, "looking up the scratch array failed", e);
  e = olsgd::launch_class_pairs(scratch, seed, m, s);
  if (e != cudaSuccess) return noalloc_fail(OLSGD_ECUDA, "kernel launch failed", e);
  e = cudaMemcpyAsync(dst, scratch, sizeof(int32_t) * 2 * (size_t)m, cudaMemcpyDefault, s);
  if (e != cudaSuccess) return noalloc_fail(OLSGD_ECUDA, "copy to dst failed", e);
  e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return noalloc_fail(OLSGD_ECUDA, "stream synchronisation failed", e);
  return OLSGD_OK;
}
