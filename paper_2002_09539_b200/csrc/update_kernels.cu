// Fused parameter update (Eq. 3 with the local Nesterov buffer, Eq. 4 on sync
// steps) and the worker-mean / anchor kernel (Eq. 5, Eq. 10-11).
//
// Both are pure streaming kernels bound by HBM bandwidth: every byte is read
// once and written once, all accesses are 128-bit and coalesced along the
// parameter dimension, and each thread keeps several independent loads in
// flight by unrolling over the worker dimension.
#include "olsgd_internal.h"
#include "update_math.cuh"

namespace olsgd {
namespace {

constexpr int kUpdateThreads = 256;
constexpr int kUnroll = 4;

__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }

__device__ __forceinline__ float4 load_g(const float* g_row, int64_t col4, int64_t P, bool vec) {
  if (vec) return ld_stream(reinterpret_cast<const float4*>(g_row) + col4);
  // unaligned rows (row stride not a multiple of 4 floats): scalar, bounds-checked
  const int64_t j = col4 * 4;
  float4 r;
  r.x = (j + 0 < P) ? __ldcs(g_row + j + 0) : 0.f;
  r.y = (j + 1 < P) ? __ldcs(g_row + j + 1) : 0.f;
  r.z = (j + 2 < P) ? __ldcs(g_row + j + 2) : 0.f;
  r.w = (j + 3 < P) ? __ldcs(g_row + j + 3) : 0.f;
  return r;
}

// One thread owns a 16-byte column strip and walks over `wpt` workers, so the
// anchor strip is read once per thread on sync steps.
// SUM (sync steps): blockIdx.y is a slice of the worker sum instead; the thread walks over
// the workers s, s + S, s + 2S, ... (S = gridDim.y), adds up the x_{k+1} it writes in that
// order, starting from zero as the worker-mean kernel does, and stores its column sums in
// row s of `part`.
template <bool MOM, bool SYNC, bool SHADOW, bool SUM>
__global__ void __launch_bounds__(kUpdateThreads)
fused_update_kernel(const float* __restrict__ x_in, float* __restrict__ x_out,
                    const float* __restrict__ g, float* __restrict__ u,
                    const float* __restrict__ z, __nv_bfloat16* __restrict__ shadow,
                    float* __restrict__ part, int64_t P, int64_t n4, int64_t ld, int64_t ldg,
                    int m, int wpt, bool gvec, float gamma, float mu, float alpha) {
  launch_gate();
  const int64_t col4 = (int64_t)blockIdx.x * kUpdateThreads + threadIdx.x;
  if (col4 >= n4) return;
  const int stride = SUM ? (int)gridDim.y : 1;
  const int i0 = SUM ? (int)blockIdx.y : (int)blockIdx.y * wpt;
  const int i1 = SUM ? m : min(m, i0 + wpt);

  float4 zz = make_float4(0.f, 0.f, 0.f, 0.f);
  if (SYNC) zz = reinterpret_cast<const float4*>(z)[col4];
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);

  for (int ib = i0; ib < i1; ib += kUnroll * stride) {
    float4 xv[kUnroll], gv[kUnroll], uv[kUnroll];
#pragma unroll
    for (int t = 0; t < kUnroll; ++t) {
      const int i = ib + t * stride;
      if (i < i1) {
        xv[t] = reinterpret_cast<const float4*>(x_in + (int64_t)i * ld)[col4];
        gv[t] = load_g(g + (int64_t)i * ldg, col4, P, gvec);
        if (MOM) uv[t] = reinterpret_cast<const float4*>(u + (int64_t)i * ld)[col4];
      }
    }
#pragma unroll
    for (int t = 0; t < kUnroll; ++t) {
      const int i = ib + t * stride;
      if (i < i1) {
        float4 x = xv[t];
        float4 uu = make_float4(0.f, 0.f, 0.f, 0.f);
        if (MOM) uu = uv[t];
        update4<MOM, SYNC>(x, uu, gv[t], zz, gamma, mu, alpha);
        if (MOM) reinterpret_cast<float4*>(u + (int64_t)i * ld)[col4] = uu;
        reinterpret_cast<float4*>(x_out + (int64_t)i * ld)[col4] = x;
        if (SHADOW) reinterpret_cast<uint2*>(shadow + (int64_t)i * ld)[col4] = pack_bf16x4(x);
        if (SUM) {
          acc.x += x.x;
          acc.y += x.y;
          acc.z += x.z;
          acc.w += x.w;
        }
      }
    }
  }
  if (SUM) __stcs(reinterpret_cast<float4*>(part + (int64_t)blockIdx.y * ld) + col4, acc);
}

constexpr int kMeanThreads = 256;

// Column sums over the worker dimension in a fixed order.  A block covers
// 256 / SLICES float4 columns; slice s adds workers s, s + S, s + 2S, ...
// sequentially (four loads in flight), the partial sums are staged in shared
// memory and slice 0 adds them in slice order.  SLICES depends on m only, so the
// result does not depend on P, on the launch shape or on timing.
// With `partial` non-null the kernel stops after the sum: it writes the undivided column
// sums of this GPU's workers there (the input of the cross-GPU all-reduce) and leaves z, v
// alone.
template <bool MOM, int SLICES>
__global__ void __launch_bounds__(kMeanThreads)
worker_mean_anchor_kernel(const float* __restrict__ x, float* __restrict__ z,
                          float* __restrict__ v, float* __restrict__ partial, int64_t n4,
                          int64_t ld, int m, float beta, float m_f) {
  constexpr int kMeanCols = kMeanThreads / SLICES;
  constexpr int kMeanSlices = SLICES;
  __shared__ float4 part[kMeanSlices][kMeanCols];
  const int64_t col4 = (int64_t)blockIdx.x * kMeanCols + threadIdx.x;
  const int slice = threadIdx.y;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  // slice 0 finishes the column: its anchor (and anchor momentum) strip is fetched together
  // with the first worker rows, not after the sum
  float4 z_old = make_float4(0.f, 0.f, 0.f, 0.f), v_old = z_old;
  if (MOM && !partial && slice == 0 && col4 < n4) {
    z_old = reinterpret_cast<const float4*>(z)[col4];
    v_old = reinterpret_cast<const float4*>(v)[col4];
  }
  if (col4 < n4) {
    for (int ib = slice; ib < m; ib += kMeanSlices * kUnroll) {
      float4 xv[kUnroll];
#pragma unroll
      for (int t = 0; t < kUnroll; ++t) {
        const int i = ib + t * kMeanSlices;
        if (i < m) xv[t] = ld_stream(reinterpret_cast<const float4*>(x + (int64_t)i * ld) + col4);
      }
#pragma unroll
      for (int t = 0; t < kUnroll; ++t) {
        const int i = ib + t * kMeanSlices;
        if (i < m) {
          acc.x += xv[t].x;
          acc.y += xv[t].y;
          acc.z += xv[t].z;
          acc.w += xv[t].w;
        }
      }
    }
  }
  part[slice][threadIdx.x] = acc;
  __syncthreads();
  if (slice != 0 || col4 >= n4) return;
  float4 s = part[0][threadIdx.x];
#pragma unroll
  for (int t = 1; t < kMeanSlices; ++t) {
    const float4 p = part[t][threadIdx.x];
    s.x += p.x;
    s.y += p.y;
    s.z += p.z;
    s.w += p.w;
  }
  if (partial) {
    reinterpret_cast<float4*>(partial)[col4] = s;
    return;
  }
  s.x /= m_f;
  s.y /= m_f;
  s.z /= m_f;
  s.w /= m_f;
  float4* z4 = reinterpret_cast<float4*>(z) + col4;
  if (MOM) {
    // Eq. 10: v <- beta v + (mean - z);  Eq. 11: z <- z + v
    float4* v4 = reinterpret_cast<float4*>(v) + col4;
    float4 zz = z_old, vv = v_old;
    vv.x = fmaf(beta, vv.x, s.x - zz.x);
    vv.y = fmaf(beta, vv.y, s.y - zz.y);
    vv.z = fmaf(beta, vv.z, s.z - zz.z);
    vv.w = fmaf(beta, vv.w, s.w - zz.w);
    zz.x += vv.x;
    zz.y += vv.y;
    zz.z += vv.z;
    zz.w += vv.w;
    *v4 = vv;
    *z4 = zz;
  } else {
    *z4 = s;  // Eq. 5
  }
}

// Blocking average of Local SGD (Eq. 2): one thread per 16-byte column strip sums the m
// worker rows in worker order (four loads in flight), then overwrites all of them.
__global__ void __launch_bounds__(kUpdateThreads)
worker_mean_broadcast_kernel(float* __restrict__ x, __nv_bfloat16* __restrict__ shadow,
                             float* __restrict__ z, int64_t n4, int64_t ld, int m, float m_f) {
  launch_gate();
  const int64_t col4 = (int64_t)blockIdx.x * kUpdateThreads + threadIdx.x;
  if (col4 >= n4) return;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int ib = 0; ib < m; ib += kUnroll) {
    float4 xv[kUnroll];
#pragma unroll
    for (int t = 0; t < kUnroll; ++t)
      if (ib + t < m) xv[t] = reinterpret_cast<const float4*>(x + (int64_t)(ib + t) * ld)[col4];
#pragma unroll
    for (int t = 0; t < kUnroll; ++t) {
      if (ib + t < m) {
        acc.x += xv[t].x;
        acc.y += xv[t].y;
        acc.z += xv[t].z;
        acc.w += xv[t].w;
      }
    }
  }
  acc.x /= m_f;
  acc.y /= m_f;
  acc.z /= m_f;
  acc.w /= m_f;
  reinterpret_cast<float4*>(z)[col4] = acc;
  const uint2 pk = pack_bf16x4(acc);
  for (int i = 0; i < m; ++i) {
    reinterpret_cast<float4*>(x + (int64_t)i * ld)[col4] = acc;
    if (shadow) reinterpret_cast<uint2*>(shadow + (int64_t)i * ld)[col4] = pk;
  }
}

// Second half of a sharded anchor refresh: `sum` holds the column sums over ALL workers
// (after the all-reduce); Eq. 5 or Eq. 10-11 with s = sum / m_total.
template <bool MOM>
__global__ void __launch_bounds__(kUpdateThreads)
anchor_from_sum_kernel(const float* __restrict__ sum, float* __restrict__ z, float* __restrict__ v,
                       int64_t n4, float beta, float m_f) {
  const int64_t col4 = (int64_t)blockIdx.x * kUpdateThreads + threadIdx.x;
  if (col4 >= n4) return;
  float4 s = reinterpret_cast<const float4*>(sum)[col4];
  s.x /= m_f;
  s.y /= m_f;
  s.z /= m_f;
  s.w /= m_f;
  float4* z4 = reinterpret_cast<float4*>(z) + col4;
  if (MOM) {
    float4* v4 = reinterpret_cast<float4*>(v) + col4;
    float4 zz = *z4, vv = *v4;
    vv.x = fmaf(beta, vv.x, s.x - zz.x);
    vv.y = fmaf(beta, vv.y, s.y - zz.y);
    vv.z = fmaf(beta, vv.z, s.z - zz.z);
    vv.w = fmaf(beta, vv.w, s.w - zz.w);
    zz.x += vv.x;
    zz.y += vv.y;
    zz.z += vv.z;
    zz.w += vv.w;
    *v4 = vv;
    *z4 = zz;
  } else {
    *z4 = s;
  }
}

// Anchor refresh from S rows of partial worker sums (row pitch ld): total in slice order,
// mean, Eq. 5 or Eq. 10-11.  The arithmetic after the total is that of
// worker_mean_anchor_kernel, so the two routes to the anchor give the same bits.
template <bool MOM>
__global__ void __launch_bounds__(kUpdateThreads)
anchor_from_slices_kernel(const float* __restrict__ part, int slices, int64_t ld,
                          float* __restrict__ z, float* __restrict__ v,
                          float* __restrict__ partial, int64_t n4, float beta, float m_f) {
  const int64_t col4 = (int64_t)blockIdx.x * kUpdateThreads + threadIdx.x;
  if (col4 >= n4) return;
  float4 zz = make_float4(0.f, 0.f, 0.f, 0.f), vv = zz;
  if (MOM && !partial) {
    zz = reinterpret_cast<const float4*>(z)[col4];
    vv = reinterpret_cast<const float4*>(v)[col4];
  }
  float4 s = __ldcs(reinterpret_cast<const float4*>(part) + col4);
  for (int t = 1; t < slices; ++t) {
    const float4 p = __ldcs(reinterpret_cast<const float4*>(part + (int64_t)t * ld) + col4);
    s.x += p.x;
    s.y += p.y;
    s.z += p.z;
    s.w += p.w;
  }
  if (partial) {
    reinterpret_cast<float4*>(partial)[col4] = s;
    return;
  }
  s.x /= m_f;
  s.y /= m_f;
  s.z /= m_f;
  s.w /= m_f;
  float4* z4 = reinterpret_cast<float4*>(z) + col4;
  if (MOM) {
    vv.x = fmaf(beta, vv.x, s.x - zz.x);
    vv.y = fmaf(beta, vv.y, s.y - zz.y);
    vv.z = fmaf(beta, vv.z, s.z - zz.z);
    vv.w = fmaf(beta, vv.w, s.w - zz.w);
    zz.x += vv.x;
    zz.y += vv.y;
    zz.z += vv.z;
    zz.w += vv.w;
    reinterpret_cast<float4*>(v)[col4] = vv;
    *z4 = zz;
  } else {
    *z4 = s;
  }
}

// Stage 1: block b adds (x_i[j] - z[j])^2 over its strided share of the m * P entries, each
// thread sequentially, then the threads in a fixed tree.  Stage 2: one thread adds the block
// partials in order.  Double precision throughout.
__global__ void __launch_bounds__(256)
consensus_partial_kernel(const float* __restrict__ x, const float* __restrict__ z,
                         double* __restrict__ partial, int64_t P, int64_t ld, int m) {
  __shared__ double sm[256];
  double acc = 0.0;
  for (int i = 0; i < m; ++i)
    for (int64_t j = (int64_t)blockIdx.x * 256 + threadIdx.x; j < P; j += (int64_t)gridDim.x * 256) {
      const double d = (double)x[(int64_t)i * ld + j] - (double)z[j];
      acc += d * d;
    }
  sm[threadIdx.x] = acc;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if ((int)threadIdx.x < s) sm[threadIdx.x] += sm[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) partial[blockIdx.x + 1] = sm[0];
}
__global__ void consensus_final_kernel(double* partial, int n) {
  double s = 0.0;
  for (int b = 0; b < n; ++b) s += partial[b + 1];
  partial[0] = s;
}

__global__ void virtual_sequence_kernel(const float* __restrict__ x, const float* __restrict__ z,
                                        float* __restrict__ dst, int64_t P, int64_t ld, int m,
                                        float alpha, float m_f) {
  const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= P) return;
  float s = 0.f;
  for (int i = 0; i < m; ++i) s += x[(int64_t)i * ld + j];
  s /= m_f;
  dst[j] = (alpha == 0.f) ? s : (1.f - alpha) * s + alpha * z[j];
}

}  // namespace

// blocks that give the update kernel a few waves over the multiprocessors
static int64_t update_target_blocks() { return (int64_t)sm_count() * 16; }

bool update_sums_workers(int64_t P, int m) {
  // The grid of a summing launch has one row of blocks per slice, so it needs a row long
  // enough to give every multiprocessor a couple of blocks; with fewer than four workers
  // the worker-mean kernel has next to nothing to re-read.  (Measured from 250k x 64 to
  // 50M x 64 parameters x workers: the iteration is 1-5 % shorter wherever this holds.)
  const int64_t n4 = (P + 3) / 4;
  const int64_t gx = (n4 + kUpdateThreads - 1) / kUpdateThreads;
  return m >= 4 && gx * worker_sum_slices(m) >= (int64_t)sm_count() * 2;
}

cudaError_t launch_fused_update(const UpdateArgs& a, cudaStream_t s) {
  const int64_t n4 = (a.P + 3) / 4;
  const int64_t gx = (n4 + kUpdateThreads - 1) / kUpdateThreads;
  // enough blocks for a few waves over the multiprocessors; the rest of the worker
  // dimension is walked inside the thread so the anchor strip is reused
  const int64_t target_blocks = update_target_blocks();
  int gy = (int)((target_blocks + gx - 1) / gx);
  if (gy < 1) gy = 1;
  if (gy > a.m) gy = a.m;
  int wpt = (a.m + gy - 1) / gy;
  gy = (a.m + wpt - 1) / wpt;
  const bool sum = a.sync && a.sum_slices > 0;
  if (sum) {
    if (a.sum_slices != worker_sum_slices(a.m) || !a.sum_part) return cudaErrorInvalidValue;
    gy = a.sum_slices;
    wpt = 0;
  }
  const bool gvec = (a.ldg % 4 == 0) && ((reinterpret_cast<uintptr_t>(a.g) & 15) == 0);
  const bool mom = a.u != nullptr && a.mu != 0.f;
  const bool shadow = a.shadow != nullptr;
  dim3 grid((unsigned)gx, (unsigned)gy), block(kUpdateThreads);
  cudaError_t err = cudaSuccess;
#define OLSGD_LAUNCH_UPD(MOM, SYNC, SH, SUM)                                                     \
  err = launch_chained(fused_update_kernel<MOM, SYNC, SH, SUM>, grid, block, 0, s, a.x_in,       \
                       a.x_out, a.g, a.u, a.z, a.shadow, a.sum_part, a.P, n4, a.ld, a.ldg, a.m,  \
                       wpt, gvec, a.gamma, a.mu, a.alpha)
#define OLSGD_LAUNCH_UPD_SH(MOM, SYNC, SUM)                                                      \
  do {                                                                                           \
    if (shadow) OLSGD_LAUNCH_UPD(MOM, SYNC, true, SUM);                                          \
    else OLSGD_LAUNCH_UPD(MOM, SYNC, false, SUM);                                                \
  } while (0)
  if (mom) {
    if (sum) OLSGD_LAUNCH_UPD_SH(true, true, true);
    else if (a.sync) OLSGD_LAUNCH_UPD_SH(true, true, false);
    else OLSGD_LAUNCH_UPD_SH(true, false, false);
  } else {
    if (sum) OLSGD_LAUNCH_UPD_SH(false, true, true);
    else if (a.sync) OLSGD_LAUNCH_UPD_SH(false, true, false);
    else OLSGD_LAUNCH_UPD_SH(false, false, false);
  }
#undef OLSGD_LAUNCH_UPD_SH
#undef OLSGD_LAUNCH_UPD
  return err;
}

template <int SLICES>
cudaError_t launch_mean(const AnchorArgs& a, cudaStream_t s) {
  const int64_t n4 = (a.P + 3) / 4;
  constexpr int cols = kMeanThreads / SLICES;
  dim3 grid((unsigned)((n4 + cols - 1) / cols)), block(cols, SLICES);
  const float m_f = (float)a.m;
  if (a.beta != 0.f)
    worker_mean_anchor_kernel<true, SLICES><<<grid, block, 0, s>>>(a.x, a.z, a.v, a.partial, n4, a.ld, a.m, a.beta, m_f);
  else
    worker_mean_anchor_kernel<false, SLICES><<<grid, block, 0, s>>>(a.x, a.z, a.v, a.partial, n4, a.ld, a.m, a.beta, m_f);
  return cudaGetLastError();
}

int worker_sum_slices(int m) {
  // Few slices: where the sync-step weight-gradient launch forms the sum, every slice costs
  // a row of partial sums that is written and read once.  At least four workers per slice
  // (every thread of the worker-mean kernel keeps four loads in flight), at most sixteen.
  return m >= 64 ? 4 : m >= 8 ? 2 : 1;
}

cudaError_t launch_worker_mean_anchor(const AnchorArgs& a, cudaStream_t s) {
  switch (worker_sum_slices(a.m)) {
    case 4: return launch_mean<4>(a, s);
    case 2: return launch_mean<2>(a, s);
    default: return launch_mean<1>(a, s);
  }
}

cudaError_t launch_worker_mean_broadcast(float* x, __nv_bfloat16* shadow, float* z, int64_t P,
                                         int64_t ld, int m, cudaStream_t s) {
  const int64_t n4 = (P + 3) / 4;
  return launch_chained(worker_mean_broadcast_kernel,
                        dim3((unsigned)((n4 + kUpdateThreads - 1) / kUpdateThreads)),
                        dim3(kUpdateThreads), 0, s, x, shadow, z, n4, ld, m, (float)m);
}

cudaError_t launch_anchor_from_sum(const float* sum, float* z, float* v, int64_t P, float beta,
                                   int m_total, cudaStream_t s) {
  const int64_t n4 = (P + 3) / 4;
  const unsigned grid = (unsigned)((n4 + kUpdateThreads - 1) / kUpdateThreads);
  if (beta != 0.f)
    anchor_from_sum_kernel<true><<<grid, kUpdateThreads, 0, s>>>(sum, z, v, n4, beta, (float)m_total);
  else
    anchor_from_sum_kernel<false><<<grid, kUpdateThreads, 0, s>>>(sum, z, v, n4, beta, (float)m_total);
  return cudaGetLastError();
}

cudaError_t launch_anchor_from_slices(const float* part, int slices, int64_t ld, float* z, float* v,
                                      int64_t P, float beta, int m, float* partial,
                                      cudaStream_t s) {
  const int64_t n4 = (P + 3) / 4;
  const unsigned grid = (unsigned)((n4 + kUpdateThreads - 1) / kUpdateThreads);
  if (beta != 0.f)
    anchor_from_slices_kernel<true><<<grid, kUpdateThreads, 0, s>>>(part, slices, ld, z, v, partial, n4, beta, (float)m);
  else
    anchor_from_slices_kernel<false><<<grid, kUpdateThreads, 0, s>>>(part, slices, ld, z, v, partial, n4, beta, (float)m);
  return cudaGetLastError();
}

cudaError_t launch_consensus_distance(const float* x, const float* z, double* scratch,
                                      int n_partials, int64_t P, int64_t ld, int m,
                                      cudaStream_t s) {
  consensus_partial_kernel<<<n_partials, 256, 0, s>>>(x, z, scratch, P, ld, m);
  consensus_final_kernel<<<1, 1, 0, s>>>(scratch, n_partials);
  return cudaGetLastError();
}

cudaError_t launch_virtual_sequence(const float* x, const float* z, float* dst, int64_t P,
                                    int64_t ld, int m, float alpha, cudaStream_t s) {
  const int threads = 256;
  virtual_sequence_kernel<<<(unsigned)((P + threads - 1) / threads), threads, 0, s>>>(
      x, z, dst, P, ld, m, alpha, (float)m);
  return cudaGetLastError();
}

}  // namespace olsgd
