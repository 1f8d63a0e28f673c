// CUDA-core kernels of the forward/backward path: minibatch gather, linear
// regression, the (skinny) output layer with softmax cross-entropy, bias
// gradients, bf16 casts and transposes, and a plain reference GEMM.
//
// Every reduction runs in a fixed order (no floating-point atomics), so a step
// is reproducible bit for bit from run to run.
#include "olsgd_internal.h"

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

// ------------------------------------------------------------------ linear regression

__global__ void __launch_bounds__(128)
linreg_kernel(const float* __restrict__ X, const float* __restrict__ y,
              const int32_t* __restrict__ idx, const float* __restrict__ x, float* __restrict__ g,
              float* __restrict__ loss, int batch, int64_t n, int d, int64_t ld) {
  extern __shared__ float sm[];  // residuals [batch]
  const int i = blockIdx.x;
  const float* w = x + (int64_t)i * ld;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32, nwarp = blockDim.x / 32;
  const float* Xi = X + (int64_t)i * n * d;
  for (int b = warp; b < batch; b += nwarp) {
    const int32_t r = idx[(int64_t)i * batch + b];
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
    for (int b = 0; b < batch; ++b) {
      const int32_t r = idx[(int64_t)i * batch + b];
      acc = fmaf(sm[b], Xi[(int64_t)r * d + j], acc);
    }
    g[(int64_t)i * ld + j] = acc * inv_b;
  }
  if (loss && threadIdx.x == 0) {
    float s = 0.f;
    for (int b = 0; b < batch; ++b) s = fmaf(sm[b], sm[b], s);
    loss[i] = 0.5f * s * inv_b;
  }
}

// ------------------------------------------------------------------ output layer

constexpr int kHeadWarps = 8;     // rows per block
constexpr int kHeadChunk = 256;   // K elements of W staged in shared memory at a time

template <typename InT>
__device__ __forceinline__ float load_in(const InT* p);
template <>
__device__ __forceinline__ float load_in<float>(const float* p) { return *p; }
template <>
__device__ __forceinline__ float load_in<__nv_bfloat16>(const __nv_bfloat16* p) {
  return __bfloat162float(*p);
}

// One warp per batch row: logits, stable log-softmax, loss, d loss / d logits
// and, if asked, the gradient with respect to the layer's input.
template <typename InT, int CMAX>
__global__ void __launch_bounds__(kHeadWarps * 32)
head_forward_kernel(HeadArgs a) {
  __shared__ float wsm[CMAX][kHeadChunk + 1];
  __shared__ __align__(16) __nv_bfloat16 tsm[kHeadChunk][kHeadWarps];
  const int i = blockIdx.y;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int b = blockIdx.x * kHeadWarps + warp;
  const bool live = b < a.batch;
  const int K = a.K, C = a.C;
  const InT* in = (sizeof(InT) == 4 ? reinterpret_cast<const InT*>(a.in32)
                                    : reinterpret_cast<const InT*>(a.in16)) +
                  ((int64_t)i * a.batch + (live ? b : 0)) * K;
  const float* W = a.x + (int64_t)i * a.ld + a.w_off;
  const float* bias = a.x + (int64_t)i * a.ld + a.b_off;

  float acc[CMAX];
#pragma unroll
  for (int c = 0; c < CMAX; ++c) acc[c] = 0.f;

  for (int k0 = 0; k0 < K; k0 += kHeadChunk) {
    const int kc = min(kHeadChunk, K - k0);
    __syncthreads();
    for (int e = threadIdx.x; e < C * kHeadChunk; e += blockDim.x) {
      const int c = e / kHeadChunk, kk = e % kHeadChunk;
      float w = (kk < kc) ? W[(int64_t)c * K + k0 + kk] : 0.f;
      if (a.round_w_bf16) w = bf16_round(w);
      wsm[c][kk] = w;
    }
    __syncthreads();
    if (live) {
      for (int kk = lane; kk < kc; kk += 32) {
        const float xv = load_in<InT>(in + k0 + kk);
#pragma unroll
        for (int c = 0; c < CMAX; ++c)
          if (c < C) acc[c] = fmaf(xv, wsm[c][kk], acc[c]);
      }
    }
  }
  // every lane ends up with every logit
  float mx = -INFINITY;
#pragma unroll
  for (int c = 0; c < CMAX; ++c) {
    if (c < C) {
      acc[c] = warp_sum(acc[c]) + bias[c];
      mx = fmaxf(mx, acc[c]);
    }
  }
  float se = 0.f;
#pragma unroll
  for (int c = 0; c < CMAX; ++c)
    if (c < C) se += expf(acc[c] - mx);
  const float lse = mx + logf(se);
  const int label = live ? a.yb[(int64_t)i * a.batch + b] : 0;
  const float inv_b = 1.0f / (float)a.batch;
  float picked = 0.f;
#pragma unroll
  for (int c = 0; c < CMAX; ++c) {
    if (c < C) {
      if (c == label) picked = acc[c];
      acc[c] = (expf(acc[c] - lse) - (c == label ? 1.f : 0.f)) * inv_b;  // d loss / d logit
    }
  }
  if (live) {
    float* dl = a.dlogits + ((int64_t)i * a.batch + b) * C;
#pragma unroll
    for (int c = 0; c < CMAX; ++c)
      if (c < C && lane == (c & 31)) dl[c] = acc[c];
    if (lane == 0) a.rowloss[(int64_t)i * a.batch + b] = lse - picked;
  }
  if (!a.din32 && !a.din16 && !a.din16t) return;

  // gradient w.r.t. the input: din[k] = (sum_c dl[c] W[c][k]) * (in[k] > 0); the
  // operand that goes on to the tensor cores is the bf16-rounded dl
  if (a.round_w_bf16) {
#pragma unroll
    for (int c = 0; c < CMAX; ++c) acc[c] = bf16_round(acc[c]);
  }
  const int b0 = blockIdx.x * kHeadWarps;
  for (int k0 = 0; k0 < K; k0 += kHeadChunk) {
    const int kc = min(kHeadChunk, K - k0);
    __syncthreads();
    for (int e = threadIdx.x; e < C * kHeadChunk; e += blockDim.x) {
      const int c = e / kHeadChunk, kk = e % kHeadChunk;
      float w = (kk < kc) ? W[(int64_t)c * K + k0 + kk] : 0.f;
      if (a.round_w_bf16) w = bf16_round(w);
      wsm[c][kk] = w;
    }
    __syncthreads();
    for (int kk = lane; kk < kHeadChunk; kk += 32) {
      float d = 0.f;
      if (live && kk < kc) {
#pragma unroll
        for (int c = 0; c < CMAX; ++c)
          if (c < C) d = fmaf(acc[c], wsm[c][kk], d);
        if (!(load_in<InT>(in + k0 + kk) > 0.f)) d = 0.f;
        const int64_t o = ((int64_t)i * a.batch + b) * K + k0 + kk;
        if (a.din32) a.din32[o] = d;
        if (a.din16) a.din16[o] = __float2bfloat16_rn(d);
      }
      tsm[kk][warp] = __float2bfloat16_rn(d);
    }
    if (a.din16t) {
      __syncthreads();
      // [K][B] layout: eight consecutive batch entries (16 bytes) per K index
      for (int kk = threadIdx.x; kk < kc; kk += blockDim.x) {
        __nv_bfloat16* dst = a.din16t + ((int64_t)i * K + k0 + kk) * a.batch + b0;
        if (b0 + kHeadWarps <= a.batch && (a.batch % kHeadWarps) == 0) {
          *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(&tsm[kk][0]);
        } else {
          for (int r = 0; r < kHeadWarps; ++r)
            if (b0 + r < a.batch) dst[r] = tsm[kk][r];
        }
      }
    }
  }
}

constexpr int kWgradCols = 128;
constexpr int kWgradRows = 128;

template <typename InT, int CMAX>
__global__ void __launch_bounds__(kWgradCols)
head_wgrad_kernel(HeadArgs a, float* __restrict__ g, float* __restrict__ loss) {
  __shared__ float dsm[kWgradRows][CMAX + 1];
  const int i = blockIdx.y;
  const int j = blockIdx.x * kWgradCols + threadIdx.x;
  const int K = a.K, C = a.C, B = a.batch;
  const InT* in = (sizeof(InT) == 4 ? reinterpret_cast<const InT*>(a.in32)
                                    : reinterpret_cast<const InT*>(a.in16)) +
                  (int64_t)i * B * K;
  const float* dl = a.dlogits + (int64_t)i * B * C;
  float acc[CMAX];
#pragma unroll
  for (int c = 0; c < CMAX; ++c) acc[c] = 0.f;
  float bsum = 0.f;  // thread c < C of block 0 also sums the bias gradient
  for (int r0 = 0; r0 < B; r0 += kWgradRows) {
    const int rc = min(kWgradRows, B - r0);
    __syncthreads();
    for (int e = threadIdx.x; e < rc * C; e += blockDim.x) {
      float d = dl[(int64_t)r0 * C + e];
      if (a.round_w_bf16) d = bf16_round(d);
      dsm[e / C][e % C] = d;
    }
    __syncthreads();
    if (j < K) {
      for (int r = 0; r < rc; ++r) {
        const float xv = load_in<InT>(in + (int64_t)(r0 + r) * K + j);
#pragma unroll
        for (int c = 0; c < CMAX; ++c)
          if (c < C) acc[c] = fmaf(dsm[r][c], xv, acc[c]);
      }
    }
    if (blockIdx.x == 0 && threadIdx.x < C)
      for (int r = 0; r < rc; ++r) bsum += dl[(int64_t)(r0 + r) * C + threadIdx.x];
  }
  float* gi = g + (int64_t)i * a.ld;
  if (j < K) {
#pragma unroll
    for (int c = 0; c < CMAX; ++c)
      if (c < C) gi[a.w_off + (int64_t)c * K + j] = acc[c];
  }
  if (blockIdx.x == 0) {
    if (threadIdx.x < C) gi[a.b_off + threadIdx.x] = bsum;
    if (loss && threadIdx.x == kWgradCols - 1) {
      float s = 0.f;
      for (int r = 0; r < B; ++r) s += a.rowloss[(int64_t)i * B + r];
      loss[i] = s / (float)B;
    }
  }
}

// ------------------------------------------------------------------ hidden-layer bias gradient

__global__ void bias_grad_kernel(const __nv_bfloat16* __restrict__ dat, float* __restrict__ g,
                                 int64_t ld, int64_t b_off, int R, int batch) {
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

// ------------------------------------------------------------------ bf16 transpose

__global__ void transpose_bf16_kernel(const __nv_bfloat16* __restrict__ src, int64_t src_ld,
                                      int64_t src_off, __nv_bfloat16* __restrict__ dst,
                                      int64_t dst_batch, int R, int C) {
  __shared__ __nv_bfloat16 tile[32][34];
  const int i = blockIdx.z;
  const __nv_bfloat16* s = src + (int64_t)i * src_ld + src_off;
  __nv_bfloat16* d = dst + (int64_t)i * dst_batch;
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  for (int rr = threadIdx.y; rr < 32; rr += blockDim.y) {
    const int r = r0 + rr, c = c0 + threadIdx.x;
    if (r < R && c < C) tile[rr][threadIdx.x] = s[(int64_t)r * C + c];
  }
  __syncthreads();
  for (int cc = threadIdx.y; cc < 32; cc += blockDim.y) {
    const int c = c0 + cc, r = r0 + threadIdx.x;
    if (r < R && c < C) d[(int64_t)c * R + r] = tile[threadIdx.x][cc];
  }
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
    As[ty][tx] = (row0 + ty < a.Ma && k < a.K) ? __bfloat162float(A[(int64_t)(row0 + ty) * a.lda + k]) : 0.f;
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

cudaError_t launch_gather(const float* X, const int32_t* y, const int32_t* idx, float* xb32,
                          __nv_bfloat16* xb16, __nv_bfloat16* xb16t, int32_t* yb, int m, int batch,
                          int64_t n, int d, cudaStream_t s) {
  dim3 grid((d + kGatherCols - 1) / kGatherCols, (batch + kGatherRows - 1) / kGatherRows, m);
  dim3 block(kGatherCols, 4);
  gather_kernel<<<grid, block, 0, s>>>(X, y, idx, xb32, xb16, xb16t, yb, batch, n, d);
  return cudaGetLastError();
}

cudaError_t launch_linreg(const float* X, const float* y, const int32_t* idx, const float* x,
                          float* g, float* loss, int m, int batch, int64_t n, int d, int64_t ld,
                          cudaStream_t s) {
  linreg_kernel<<<m, 128, (size_t)batch * sizeof(float), s>>>(X, y, idx, x, g, loss, batch, n, d, ld);
  return cudaGetLastError();
}

cudaError_t launch_head_forward(const HeadArgs& a, cudaStream_t s) {
  dim3 grid((a.batch + kHeadWarps - 1) / kHeadWarps, a.m), block(kHeadWarps * 32);
  const bool f32 = a.in32 != nullptr;
  if (a.C <= 16) {
    if (f32) head_forward_kernel<float, 16><<<grid, block, 0, s>>>(a);
    else head_forward_kernel<__nv_bfloat16, 16><<<grid, block, 0, s>>>(a);
  } else {
    if (f32) head_forward_kernel<float, 32><<<grid, block, 0, s>>>(a);
    else head_forward_kernel<__nv_bfloat16, 32><<<grid, block, 0, s>>>(a);
  }
  return cudaGetLastError();
}

cudaError_t launch_head_wgrad(const HeadArgs& a, float* g, float* loss, cudaStream_t s) {
  dim3 grid((a.K + kWgradCols - 1) / kWgradCols, a.m), block(kWgradCols);
  const bool f32 = a.in32 != nullptr;
  if (a.C <= 16) {
    if (f32) head_wgrad_kernel<float, 16><<<grid, block, 0, s>>>(a, g, loss);
    else head_wgrad_kernel<__nv_bfloat16, 16><<<grid, block, 0, s>>>(a, g, loss);
  } else {
    if (f32) head_wgrad_kernel<float, 32><<<grid, block, 0, s>>>(a, g, loss);
    else head_wgrad_kernel<__nv_bfloat16, 32><<<grid, block, 0, s>>>(a, g, loss);
  }
  return cudaGetLastError();
}

cudaError_t launch_bias_grad(const __nv_bfloat16* dat, float* g, int64_t ld, int64_t b_off, int m,
                             int R, int batch, cudaStream_t s) {
  const int warps = 8;
  dim3 grid((R + warps - 1) / warps, m), block(warps * 32);
  bias_grad_kernel<<<grid, block, 0, s>>>(dat, g, ld, b_off, R, batch);
  return cudaGetLastError();
}

cudaError_t launch_transpose_bf16(const __nv_bfloat16* src, int64_t src_ld, int64_t src_off,
                                  __nv_bfloat16* dst, int64_t dst_batch, int m, int R, int C,
                                  cudaStream_t s) {
  dim3 grid((C + 31) / 32, (R + 31) / 32, m), block(32, 8);
  transpose_bf16_kernel<<<grid, block, 0, s>>>(src, src_ld, src_off, dst, dst_batch, R, C);
  return cudaGetLastError();
}

cudaError_t launch_gemm_simt(const GemmArgs& a, cudaStream_t s) {
  dim3 grid((a.Nb + kRefTile - 1) / kRefTile, (a.Ma + kRefTile - 1) / kRefTile, a.m);
  dim3 block(kRefTile, kRefTile);
  gemm_simt_kernel<<<grid, block, 0, s>>>(a);
  return cudaGetLastError();
}

}  // namespace olsgd
