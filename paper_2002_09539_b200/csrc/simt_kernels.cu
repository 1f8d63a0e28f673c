// CUDA-core kernels of the forward/backward path: minibatch gather, linear
// regression, bias gradients, bf16 casts, and a plain reference GEMM.
//
// Every reduction runs in a fixed order (no floating-point atomics), so a step
// is reproducible bit for bit from run to run.
#include "olsgd_internal.h"
#include "philox.cuh"
#include "update_math.cuh"

namespace olsgd {
namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ float bf16_round(float v) {
  return __bfloat162float(__float2bfloat16_rn(v));
}

// ------------------------------------------------------------------ casts

__global__ void cast_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst,
                                 int64_t n4) {
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n4) return;
  const float4 v = reinterpret_cast<const float4*>(src)[t];
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 pk;
  pk.x = *reinterpret_cast<uint32_t*>(&lo);
  pk.y = *reinterpret_cast<uint32_t*>(&hi);
  reinterpret_cast<uint2*>(dst)[t] = pk;
}

// ------------------------------------------------------------------ gather (S2)

constexpr int kGatherRows = 32, kGatherCols = 64;

__global__ void __launch_bounds__(256)
gather_kernel(const float* __restrict__ X, const int32_t* __restrict__ y,
              const int32_t* __restrict__ idx, float* __restrict__ xb32,
              __nv_bfloat16* __restrict__ xb16, __nv_bfloat16* __restrict__ xb16t,
              int32_t* __restrict__ yb, int batch, int64_t n, int d) {
  launch_gate();
  __shared__ __nv_bfloat16 tile[kGatherRows][kGatherCols + 2];
  __shared__ int32_t rows[kGatherRows];
  const int i = blockIdx.z;
  const int b0 = blockIdx.y * kGatherRows, j0 = blockIdx.x * kGatherCols;
  const int tx = threadIdx.x, ty = threadIdx.y;  // (64, 4)
  const int t = ty * kGatherCols + tx;
  if (t < kGatherRows) {
    const int b = b0 + t;
    const int32_t r = (b < batch) ? idx[(int64_t)i * batch + b] : 0;
    rows[t] = r;
    if (blockIdx.x == 0 && b < batch) yb[(int64_t)i * batch + b] = y[(int64_t)i * n + r];
  }
  __syncthreads();
  const int j = j0 + tx;
  for (int bl = ty; bl < kGatherRows; bl += 4) {
    const int b = b0 + bl;
    float v = 0.f;
    if (b < batch && j < d) {
      v = X[((int64_t)i * n + rows[bl]) * d + j];
      const int64_t o = ((int64_t)i * batch + b) * d + j;
      if (xb32) xb32[o] = v;
      if (xb16) xb16[o] = __float2bfloat16_rn(v);
    }
    tile[bl][tx] = __float2bfloat16_rn(v);
  }
  if (!xb16t) return;
  __syncthreads();
  for (int e = t; e < kGatherRows * kGatherCols; e += 256) {
    const int jl = e / kGatherRows, bl = e % kGatherRows;
    if (j0 + jl < d && b0 + bl < batch)
      xb16t[((int64_t)i * d + j0 + jl) * batch + b0 + bl] = tile[bl][jl];
  }
}

// Same copy for the common aligned case (d % 128 == 0, batch % 32 == 0): 128-bit
// loads of 512 contiguous bytes per row segment, 16-byte stores in both layouts.
constexpr int kGvRows = 32, kGvCols = 128;

__global__ void __launch_bounds__(256)
gather_vec_kernel(const float* __restrict__ X, const int32_t* __restrict__ y,
                  int32_t* __restrict__ idx, float* __restrict__ xb32,
                  __nv_bfloat16* __restrict__ xb16, __nv_bfloat16* __restrict__ xb16t,
                  int32_t* __restrict__ yb, int batch, int64_t n, int d, bool draw, IndexRule rule) {
  launch_gate();
  __shared__ __align__(16) __nv_bfloat16 tile[kGvRows][kGvCols + 8];
  __shared__ int32_t rows[kGvRows];
  const int i = blockIdx.z;
  const int b0 = blockIdx.y * kGvRows, j0 = blockIdx.x * kGvCols;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x < kGvRows) {
    const int64_t slot = (int64_t)i * batch + b0 + threadIdx.x;
    int32_t r;
    if (draw) {
      // S1 inside S2: the row of slot b0 + tid by the with-replacement index rule
      const uint32_t k = (uint32_t)(rule.k_base + (rule.k_ptr ? (uint64_t)*rule.k_ptr : 0ull));
      r = minibatch_index(rule.key0, rule.key1, k, (uint32_t)i + rule.worker_offset,
                          b0 + (int)threadIdx.x, (uint32_t)n);
      if (blockIdx.x == 0) idx[slot] = r;
    } else {
      r = idx[slot];
    }
    rows[threadIdx.x] = r;
    if (blockIdx.x == 0) yb[slot] = y[(int64_t)i * n + r];
  }
  __syncthreads();
#pragma unroll
  for (int t = 0; t < kGvRows / 8; ++t) {
    const int bl = warp + 8 * t;
    const float4 v = __ldcs(reinterpret_cast<const float4*>(
        X + ((int64_t)i * n + rows[bl]) * d + j0) + lane);
    const int64_t o = ((int64_t)i * batch + b0 + bl) * d + j0 + lane * 4;
    if (xb32) *reinterpret_cast<float4*>(xb32 + o) = v;
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&lo);
    pk.y = *reinterpret_cast<uint32_t*>(&hi);
    if (xb16) *reinterpret_cast<uint2*>(xb16 + o) = pk;
    *reinterpret_cast<uint2*>(&tile[bl][lane * 4]) = pk;
  }
  if (!xb16t) return;
  __syncthreads();
  // [d][B] layout: each thread writes eight consecutive batch entries of one column
#pragma unroll
  for (int pass = 0; pass < 2; ++pass) {
    const int jl = pass * 64 + (threadIdx.x >> 2), bq = threadIdx.x & 3;
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const uint16_t lo = *reinterpret_cast<const uint16_t*>(&tile[bq * 8 + 2 * e][jl]);
      const uint16_t hi = *reinterpret_cast<const uint16_t*>(&tile[bq * 8 + 2 * e + 1][jl]);
      w[e] = (uint32_t)lo | ((uint32_t)hi << 16);
    }
    *reinterpret_cast<uint4*>(xb16t + ((int64_t)i * d + j0 + jl) * batch + b0 + bq * 8) =
        make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// Minibatch rows that arrive in bf16 (host-fed steps): the [B][d] copy is the buffer itself,
// only the [d][B] copy of the weight-gradient GEMM and the label copy are made.  A block turns
// 32 rows x 64 columns; a thread loads 16 bytes of a row and stores eight consecutive batch
// entries of a column.
constexpr int kTrRows = 32, kTrCols = 64;

__global__ void __launch_bounds__(256)
transpose_bf16_kernel(const __nv_bfloat16* __restrict__ xb16, const int32_t* __restrict__ y,
                      __nv_bfloat16* __restrict__ xb16t, int32_t* __restrict__ yb, int batch, int d) {
  launch_gate();
  __shared__ __align__(16) __nv_bfloat16 tile[kTrRows][kTrCols + 8];
  const int i = blockIdx.z;
  const int b0 = blockIdx.y * kTrRows, j0 = blockIdx.x * kTrCols;
  {
    const int bl = threadIdx.x >> 3, q = threadIdx.x & 7;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (b0 + bl < batch)
      v = *reinterpret_cast<const uint4*>(xb16 + ((int64_t)i * batch + b0 + bl) * d + j0 + q * 8);
    *reinterpret_cast<uint4*>(&tile[bl][q * 8]) = v;
    if (blockIdx.x == 0 && q == 0 && b0 + bl < batch)
      yb[(int64_t)i * batch + b0 + bl] = y[(int64_t)i * batch + b0 + bl];
  }
  __syncthreads();
  const int jl = threadIdx.x >> 2, bq = threadIdx.x & 3;
  if (b0 + bq * 8 < batch) {
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const uint16_t lo = *reinterpret_cast<const uint16_t*>(&tile[bq * 8 + 2 * e][jl]);
      const uint16_t hi = *reinterpret_cast<const uint16_t*>(&tile[bq * 8 + 2 * e + 1][jl]);
      w[e] = (uint32_t)lo | ((uint32_t)hi << 16);
    }
    *reinterpret_cast<uint4*>(xb16t + ((int64_t)i * d + j0 + jl) * batch + b0 + bq * 8) =
        make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// ------------------------------------------------------------------ linear regression

__global__ void __launch_bounds__(128)
linreg_kernel(const float* __restrict__ X, const float* __restrict__ y,
              int32_t* __restrict__ idx, const float* __restrict__ x, float* __restrict__ g,
              float* __restrict__ loss, int batch, int64_t n, int d, int64_t ld,
              FusedUpdateArgs up, bool draw, IndexRule rule) {
  launch_gate();
  extern __shared__ float sm[];  // residuals [batch], then the batch's row numbers [batch]
  int32_t* rows = reinterpret_cast<int32_t*>(sm + batch);
  const int i = blockIdx.x;
  const float* w = x + (int64_t)i * ld;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32, nwarp = blockDim.x / 32;
  const float* Xi = X + (int64_t)i * n * d;
  // S1: the rows of this worker's minibatch, drawn here by the with-replacement rule (and left
  // in idx for whoever wants to see them) or taken from idx
  for (int b = threadIdx.x; b < batch; b += blockDim.x) {
    int32_t r;
    if (draw) {
      const uint32_t k = (uint32_t)(rule.k_base + (rule.k_ptr ? (uint64_t)*rule.k_ptr : 0ull));
      r = minibatch_index(rule.key0, rule.key1, k, (uint32_t)i + rule.worker_offset, b, (uint32_t)n);
      idx[(int64_t)i * batch + b] = r;
    } else {
      r = idx[(int64_t)i * batch + b];
    }
    rows[b] = r;
  }
  __syncthreads();
  for (int b = warp; b < batch; b += nwarp) {
    const int32_t r = rows[b];
    const float* row = Xi + (int64_t)r * d;
    float acc = 0.f;
    for (int j = lane; j < d; j += 32) acc = fmaf(row[j], w[j], acc);
    acc = warp_sum(acc);
    if (lane == 0) sm[b] = acc - y[(int64_t)i * n + r];
  }
  __syncthreads();
  const float inv_b = 1.0f / (float)batch;
  for (int j = threadIdx.x; j < d; j += blockDim.x) {
    float acc = 0.f;
    for (int b = 0; b < batch; ++b) acc = fmaf(sm[b], Xi[(int64_t)rows[b] * d + j], acc);
    const float gj = acc * inv_b;
    if (up.enabled) {
      // Eq. 3 / Eq. 4 for entry j of worker i, with the arithmetic of the update kernel
      const int64_t o = (int64_t)i * up.ld + j;
      const bool mom = up.u != nullptr && up.mu != 0.f;
      float xv = up.x_in[o], uv = mom ? up.u[o] : 0.f;
      update_scalar_rt(xv, uv, gj, up.sync ? up.z[j] : 0.f, up.gamma, up.mu, up.alpha, mom,
                       up.sync != 0);
      up.x_out[o] = xv;
      if (mom) up.u[o] = uv;
    } else {
      g[(int64_t)i * ld + j] = gj;
    }
  }
  if (loss && threadIdx.x == 0) {
    float s = 0.f;
    for (int b = 0; b < batch; ++b) s = fmaf(sm[b], sm[b], s);
    loss[i] = 0.5f * s * inv_b;
  }
}

// ------------------------------------------------------------------ hidden-layer bias gradient

__global__ void bias_grad_kernel(const __nv_bfloat16* __restrict__ dat, float* __restrict__ g,
                                 int64_t ld, int64_t b_off, int R, int batch) {
  launch_gate();
  const int i = blockIdx.y;
  const int r = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
  const int lane = threadIdx.x % 32;
  if (r >= R) return;
  const __nv_bfloat16* row = dat + ((int64_t)i * R + r) * batch;
  float acc = 0.f;
  for (int c = lane; c < batch; c += 32) acc += __bfloat162float(row[c]);
  acc = warp_sum(acc);
  if (lane == 0) g[(int64_t)i * ld + b_off + r] = acc;
}

// ------------------------------------------------------------------ reference GEMM

constexpr int kRefTile = 32;

__global__ void __launch_bounds__(kRefTile* kRefTile)
gemm_simt_kernel(GemmArgs a) {
  __shared__ float As[kRefTile][kRefTile + 1], Bs[kRefTile][kRefTile + 1];
  const int i = blockIdx.z;
  const int row0 = blockIdx.y * kRefTile, col0 = blockIdx.x * kRefTile;
  const int tx = threadIdx.x, ty = threadIdx.y;
  const __nv_bfloat16* A = a.A + (int64_t)i * a.a_batch;
  const __nv_bfloat16* B = a.B + (int64_t)i * a.b_batch;
  float acc = 0.f;
  for (int k0 = 0; k0 < a.K; k0 += kRefTile) {
    const int k = k0 + tx;
    As[ty][tx] = (row0 + ty < a.Ma && k < a.K)
                     ? __bfloat162float(a.a_mn_major ? A[(int64_t)k * a.lda + row0 + ty]
                                                     : A[(int64_t)(row0 + ty) * a.lda + k])
                     : 0.f;
    Bs[ty][tx] = (col0 + ty < a.Nb && k < a.K) ? __bfloat162float(B[(int64_t)(col0 + ty) * a.ldb + k]) : 0.f;
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kRefTile; ++kk) acc = fmaf(As[ty][kk], Bs[tx][kk], acc);
    __syncthreads();
  }
  const int row = row0 + ty, col = col0 + tx;
  if (row >= a.Ma || col >= a.Nb) return;
  if (a.epilogue == GEMM_EPI_STORE_F32) {
    a.out_f[(int64_t)i * a.out_batch + (int64_t)row * a.ldo + col] = acc;
    return;
  }
  float v;
  if (a.epilogue == GEMM_EPI_BIAS_RELU) {
    v = fmaxf(acc + a.bias[(int64_t)i * a.bias_batch + row], 0.f);
  } else {
    const float mk = __bfloat162float(a.mask[((int64_t)i * a.Ma + row) * a.Nb + col]);
    v = mk > 0.f ? acc : 0.f;
  }
  const __nv_bfloat16 o = __float2bfloat16_rn(v);
  if (a.out_t) a.out_t[((int64_t)i * a.Ma + row) * a.Nb + col] = o;
  if (a.out_n) a.out_n[((int64_t)i * a.Nb + col) * a.Ma + row] = o;
}

}  // namespace

cudaError_t launch_cast_bf16(const float* src, __nv_bfloat16* dst, int64_t n, cudaStream_t s) {
  const int64_t n4 = n / 4;  // callers pass padded lengths (multiples of 64)
  const int threads = 256;
  cast_bf16_kernel<<<(unsigned)((n4 + threads - 1) / threads), threads, 0, s>>>(src, dst, n4);
  return cudaGetLastError();
}

bool gather_draws_indices(int batch, int d) { return d % kGvCols == 0 && batch % kGvRows == 0; }

cudaError_t launch_gather(const float* X, const int32_t* y, int32_t* idx, float* xb32,
                          __nv_bfloat16* xb16, __nv_bfloat16* xb16t, int32_t* yb, int m, int batch,
                          int64_t n, int d, const IndexRule* rule, cudaStream_t s) {
  if (rule && !gather_draws_indices(batch, d)) return cudaErrorInvalidValue;
  if (gather_draws_indices(batch, d)) {
    dim3 grid(d / kGvCols, batch / kGvRows, m);
    return launch_chained(gather_vec_kernel, grid, dim3(256), 0, s, X, y, idx, xb32, xb16, xb16t, yb,
                          batch, n, d, rule != nullptr, rule ? *rule : IndexRule{});
  }
  dim3 grid((d + kGatherCols - 1) / kGatherCols, (batch + kGatherRows - 1) / kGatherRows, m);
  dim3 block(kGatherCols, 4);
  return launch_chained(gather_kernel, grid, block, 0, s, X, y, idx, xb32, xb16, xb16t, yb, batch, n, d);
}

cudaError_t launch_transpose_bf16(const __nv_bfloat16* xb16, const int32_t* y, __nv_bfloat16* xb16t,
                                  int32_t* yb, int m, int batch, int d, cudaStream_t s) {
  if (d % kTrCols != 0 || batch % 8 != 0) return cudaErrorInvalidValue;
  dim3 grid(d / kTrCols, (batch + kTrRows - 1) / kTrRows, m);
  return launch_chained(transpose_bf16_kernel, grid, dim3(256), 0, s, xb16, y, xb16t, yb, batch, d);
}

cudaError_t launch_linreg(const float* X, const float* y, int32_t* idx, const float* x,
                          float* g, float* loss, int m, int batch, int64_t n, int d, int64_t ld,
                          const FusedUpdateArgs* upd, const IndexRule* rule, cudaStream_t s) {
  FusedUpdateArgs up{};
  if (upd) up = *upd;
  return launch_chained(linreg_kernel, dim3(m), dim3(128),
                        (size_t)batch * (sizeof(float) + sizeof(int32_t)), s, X, y, idx, x, g, loss,
                        batch, n, d, ld, up, rule != nullptr, rule ? *rule : IndexRule{});
}

cudaError_t launch_bias_grad(const __nv_bfloat16* dat, float* g, int64_t ld, int64_t b_off, int m,
                             int R, int batch, cudaStream_t s) {
  const int warps = 8;
  dim3 grid((R + warps - 1) / warps, m), block(warps * 32);
  return launch_chained(bias_grad_kernel, grid, block, 0, s, dat, g, ld, b_off, R, batch);
}

cudaError_t launch_gemm_simt(const GemmArgs& a, cudaStream_t s) {
  dim3 grid((a.Nb + kRefTile - 1) / kRefTile, (a.Ma + kRefTile - 1) / kRefTile, a.m);
  dim3 block(kRefTile, kRefTile);
  gemm_simt_kernel<<<grid, block, 0, s>>>(a);
  return cudaGetLastError();
}

}  // namespace olsgd
