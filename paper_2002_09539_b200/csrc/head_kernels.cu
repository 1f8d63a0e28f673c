// The output ("head") layer on CUDA cores: with ten-odd classes it is far too
// skinny for the tensor cores.  Forward, stable log-softmax, cross-entropy,
// d loss / d logits, the masked gradient with respect to the layer's input,
// and the layer's own weight and bias gradients.  All reductions have a fixed
// order; nothing uses floating-point atomics.
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

template <typename InT>
__device__ __forceinline__ float load_in(const InT* p);
template <>
__device__ __forceinline__ float load_in<float>(const float* p) { return *p; }
template <>
__device__ __forceinline__ float load_in<__nv_bfloat16>(const __nv_bfloat16* p) {
  return __bfloat162float(*p);
}

// four consecutive inputs (the row is 16-byte / 8-byte aligned when K % 4 == 0)
__device__ __forceinline__ float4 load_in4(const float* p) {
  return *reinterpret_cast<const float4*>(p);
}
__device__ __forceinline__ float4 load_in4(const __nv_bfloat16* p) {
  const uint2 w = *reinterpret_cast<const uint2*>(p);
  const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&w.x);
  const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162*>(&w.y);
  return make_float4(__low2float(lo), __high2float(lo), __low2float(hi), __high2float(hi));
}

constexpr int kHeadWarps = 8;      // batch rows per block, one warp each
constexpr int kHeadChunkMax = 1024;  // K elements of W held in shared memory at a time

// Stage W[:, k0:k0+kc] into shared memory as wsm[c][kk], row stride `ws` floats.
__device__ __forceinline__ void stage_w(float* wsm, int ws, const float* W, int C, int K, int k0,
                                        int kc, int chunk, bool round_bf16, bool vec) {
  if (vec) {
    // 128-bit loads, four in flight per thread (K % 4 == 0, so kc % 4 == 0 too)
    const int q = chunk / 4, n4 = C * q;
    for (int e0 = threadIdx.x; e0 < n4; e0 += blockDim.x * 4) {
      float4 t[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int e = e0 + u * blockDim.x;
        t[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (e < n4) {
          const int c = e / q, k4 = (e % q) * 4;
          if (k4 < kc) t[u] = *reinterpret_cast<const float4*>(W + (int64_t)c * K + k0 + k4);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int e = e0 + u * blockDim.x;
        if (e < n4) {
          const int c = e / q, k4 = (e % q) * 4;
          float4 w = t[u];
          if (round_bf16) {
            w.x = bf16_round(w.x);
            w.y = bf16_round(w.y);
            w.z = bf16_round(w.z);
            w.w = bf16_round(w.w);
          }
          *reinterpret_cast<float4*>(wsm + c * ws + k4) = w;
        }
      }
    }
    return;
  }
  for (int e = threadIdx.x; e < C * chunk; e += blockDim.x) {
    const int c = e / chunk, kk = e % chunk;
    float w = (kk < kc) ? W[(int64_t)c * K + k0 + kk] : 0.f;
    if (round_bf16) w = bf16_round(w);
    wsm[c * ws + kk] = w;
  }
}

// One warp per batch row.  Dynamic shared memory: wsm [C][chunk + 4] floats, then
// tsm [chunk][kHeadWarps] bf16 (staging of the transposed input gradient).
template <typename InT, int CMAX, bool VEC>
__global__ void __launch_bounds__(kHeadWarps * 32)
head_forward_kernel(HeadArgs a, int chunk) {
  extern __shared__ __align__(16) uint8_t head_smem[];
  const int ws = chunk + 4;
  float* wsm = reinterpret_cast<float*>(head_smem);
  __nv_bfloat16* tsm = reinterpret_cast<__nv_bfloat16*>(head_smem + (size_t)a.C * ws * sizeof(float));

  const int i = blockIdx.y;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int b0 = blockIdx.x * kHeadWarps;
  const int b = b0 + warp;
  const bool live = b < a.batch;
  const int K = a.K, C = a.C;
  const InT* in = (sizeof(InT) == 4 ? reinterpret_cast<const InT*>(a.in32)
                                    : reinterpret_cast<const InT*>(a.in16)) +
                  ((int64_t)i * a.batch + (live ? b : 0)) * K;
  const float* W = a.x + (int64_t)i * a.ld + a.w_off;
  const float* bias = a.x + (int64_t)i * a.ld + a.b_off;
  const bool single = K <= chunk;   // W fits: staged once, used by both passes

  float acc[CMAX];
#pragma unroll
  for (int c = 0; c < CMAX; ++c) acc[c] = 0.f;

  for (int k0 = 0; k0 < K; k0 += chunk) {
    const int kc = min(chunk, K - k0);
    __syncthreads();
    stage_w(wsm, ws, W, C, K, k0, kc, chunk, a.round_w_bf16, VEC);
    __syncthreads();
    if (live) {
      if (VEC) {
        float4 xs[kHeadChunkMax / 128];
#pragma unroll
        for (int it = 0; it < kHeadChunkMax / 128; ++it) {
          const int kk = lane * 4 + it * 128;
          xs[it] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (kk < kc) xs[it] = load_in4(in + k0 + kk);
        }
#pragma unroll
        for (int it = 0; it < kHeadChunkMax / 128; ++it) {
          const int kk = lane * 4 + it * 128;
          if (kk < kc) {
            const float4 xv = xs[it];
#pragma unroll
            for (int c = 0; c < CMAX; ++c) {
              if (c < C) {
                const float4 w = *reinterpret_cast<const float4*>(wsm + c * ws + kk);
                acc[c] = fmaf(xv.x, w.x, acc[c]);
                acc[c] = fmaf(xv.y, w.y, acc[c]);
                acc[c] = fmaf(xv.z, w.z, acc[c]);
                acc[c] = fmaf(xv.w, w.w, acc[c]);
              }
            }
          }
        }
      } else {
        for (int kk = lane; kk < kc; kk += 32) {
          const float xv = load_in<InT>(in + k0 + kk);
#pragma unroll
          for (int c = 0; c < CMAX; ++c)
            if (c < C) acc[c] = fmaf(xv, wsm[c * ws + kk], acc[c]);
        }
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

  // gradient w.r.t. the input: din[k] = (sum_c dl[c] W[c][k]) * (in[k] > 0); the operand
  // that goes on to the tensor cores is the bf16-rounded dl
  if (a.round_w_bf16) {
#pragma unroll
    for (int c = 0; c < CMAX; ++c) acc[c] = bf16_round(acc[c]);
  }
  for (int k0 = 0; k0 < K; k0 += chunk) {
    const int kc = min(chunk, K - k0);
    if (!single) {
      __syncthreads();
      stage_w(wsm, ws, W, C, K, k0, kc, chunk, a.round_w_bf16, VEC);
    }
    __syncthreads();   // also orders the previous chunk's reads of tsm before the writes below
    if (VEC) {
      float4 xs[kHeadChunkMax / 128];
#pragma unroll
      for (int it = 0; it < kHeadChunkMax / 128; ++it) {
        const int kk = lane * 4 + it * 128;
        xs[it] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (live && kk < kc) xs[it] = load_in4(in + k0 + kk);
      }
#pragma unroll
      for (int it = 0; it < kHeadChunkMax / 128; ++it) {
        const int kk = lane * 4 + it * 128;
        if (kk < chunk) {
          float4 d = make_float4(0.f, 0.f, 0.f, 0.f);
          if (live && kk < kc) {
#pragma unroll
            for (int c = 0; c < CMAX; ++c) {
              if (c < C) {
                const float4 w = *reinterpret_cast<const float4*>(wsm + c * ws + kk);
                d.x = fmaf(acc[c], w.x, d.x);
                d.y = fmaf(acc[c], w.y, d.y);
                d.z = fmaf(acc[c], w.z, d.z);
                d.w = fmaf(acc[c], w.w, d.w);
              }
            }
            if (!(xs[it].x > 0.f)) d.x = 0.f;
            if (!(xs[it].y > 0.f)) d.y = 0.f;
            if (!(xs[it].z > 0.f)) d.z = 0.f;
            if (!(xs[it].w > 0.f)) d.w = 0.f;
            const int64_t o = ((int64_t)i * a.batch + b) * K + k0 + kk;
            if (a.din32) *reinterpret_cast<float4*>(a.din32 + o) = d;
            if (a.din16) {
              __nv_bfloat162 lo = __floats2bfloat162_rn(d.x, d.y), hi = __floats2bfloat162_rn(d.z, d.w);
              uint2 pk;
              pk.x = *reinterpret_cast<uint32_t*>(&lo);
              pk.y = *reinterpret_cast<uint32_t*>(&hi);
              *reinterpret_cast<uint2*>(a.din16 + o) = pk;
            }
          }
          tsm[(kk + 0) * kHeadWarps + warp] = __float2bfloat16_rn(d.x);
          tsm[(kk + 1) * kHeadWarps + warp] = __float2bfloat16_rn(d.y);
          tsm[(kk + 2) * kHeadWarps + warp] = __float2bfloat16_rn(d.z);
          tsm[(kk + 3) * kHeadWarps + warp] = __float2bfloat16_rn(d.w);
        }
      }
    } else
    for (int kk = lane; kk < chunk; kk += 32) {
      float d = 0.f;
      if (live && kk < kc) {
#pragma unroll
        for (int c = 0; c < CMAX; ++c)
          if (c < C) d = fmaf(acc[c], wsm[c * ws + kk], d);
        if (!(load_in<InT>(in + k0 + kk) > 0.f)) d = 0.f;
        const int64_t o = ((int64_t)i * a.batch + b) * K + k0 + kk;
        if (a.din32) a.din32[o] = d;
        if (a.din16) a.din16[o] = __float2bfloat16_rn(d);
      }
      tsm[kk * kHeadWarps + warp] = __float2bfloat16_rn(d);
    }
    if (a.din16t) {
      __syncthreads();
      // [K][B] layout: eight consecutive batch entries (16 bytes) per K index
      for (int kk = threadIdx.x; kk < kc; kk += blockDim.x) {
        __nv_bfloat16* dst = a.din16t + ((int64_t)i * K + k0 + kk) * a.batch + b0;
        if (b0 + kHeadWarps <= a.batch && (a.batch % kHeadWarps) == 0) {
          *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(tsm + kk * kHeadWarps);
        } else {
          for (int r = 0; r < kHeadWarps; ++r)
            if (b0 + r < a.batch) dst[r] = tsm[kk * kHeadWarps + r];
        }
      }
    }
  }
}

constexpr int kWgCols = 64;    // input columns per block
constexpr int kWgSlices = 4;   // batch slices per block, combined in slice order
constexpr int kWgRows = 64;    // dlogits rows staged at a time

// dW[c][j] = sum_b dlogits[b][c] * in[b][j]: thread (col, slice) adds the rows
// b = slice, slice + 4, ... in order; slice 0 then adds the four partial sums in order.
template <typename InT, int CMAX>
__global__ void __launch_bounds__(kWgCols* kWgSlices)
head_wgrad_kernel(HeadArgs a, float* __restrict__ g, float* __restrict__ loss) {
  __shared__ float dsm[kWgRows][CMAX + 1];
  __shared__ float part[kWgSlices][CMAX][kWgCols];
  const int i = blockIdx.y;
  const int tx = threadIdx.x, ty = threadIdx.y, tid = ty * kWgCols + tx;
  const int j = blockIdx.x * kWgCols + tx;
  const int K = a.K, C = a.C, B = a.batch;
  const InT* in = (sizeof(InT) == 4 ? reinterpret_cast<const InT*>(a.in32)
                                    : reinterpret_cast<const InT*>(a.in16)) +
                  (int64_t)i * B * K;
  const float* dl = a.dlogits + (int64_t)i * B * C;
  float acc[CMAX];
#pragma unroll
  for (int c = 0; c < CMAX; ++c) acc[c] = 0.f;
  float bsum = 0.f;  // thread c < C of block 0 also sums the bias gradient over all rows
  for (int r0 = 0; r0 < B; r0 += kWgRows) {
    const int rc = min(kWgRows, B - r0);
    __syncthreads();
    for (int e = tid; e < rc * C; e += kWgCols * kWgSlices) {
      float d = dl[(int64_t)r0 * C + e];
      if (a.round_w_bf16) d = bf16_round(d);
      dsm[e / C][e % C] = d;
    }
    __syncthreads();
    if (j < K) {
      for (int rb = ty; rb < rc; rb += kWgSlices * 8) {
        float xs[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int r = rb + u * kWgSlices;
          xs[u] = (r < rc) ? load_in<InT>(in + (int64_t)(r0 + r) * K + j) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int r = rb + u * kWgSlices;
          if (r < rc) {
#pragma unroll
            for (int c = 0; c < CMAX; ++c)
              if (c < C) acc[c] = fmaf(dsm[r][c], xs[u], acc[c]);
          }
        }
      }
    }
    if (blockIdx.x == 0 && tid < C)
      for (int r = 0; r < rc; ++r) bsum += dl[(int64_t)(r0 + r) * C + tid];
  }
#pragma unroll
  for (int c = 0; c < CMAX; ++c)
    if (c < C) part[ty][c][tx] = acc[c];
  __syncthreads();
  float* gi = g + (int64_t)i * a.ld;
  // 256 threads write C rows of 64 columns: (c, tx) pairs, coalesced along tx
  for (int e = tid; e < C * kWgCols; e += kWgCols * kWgSlices) {
    const int c = e / kWgCols, col = e % kWgCols;
    const int jj = blockIdx.x * kWgCols + col;
    if (jj < K) {
      float s = part[0][c][col];
#pragma unroll
      for (int t = 1; t < kWgSlices; ++t) s += part[t][c][col];
      gi[a.w_off + (int64_t)c * K + jj] = s;
    }
  }
  if (blockIdx.x == 0) {
    if (tid < C) gi[a.b_off + tid] = bsum;
    if (loss && tid == kWgCols * kWgSlices - 1) {
      float s = 0.f;
      for (int r = 0; r < B; ++r) s += a.rowloss[(int64_t)i * B + r];
      loss[i] = s / (float)B;
    }
  }
}

template <typename InT, int CMAX>
cudaError_t launch_fwd(const HeadArgs& a, cudaStream_t s) {
  int chunk = (a.K + 127) / 128 * 128;
  if (chunk > kHeadChunkMax) chunk = kHeadChunkMax;
  const size_t smem = (size_t)a.C * (chunk + 4) * sizeof(float) +
                      (size_t)chunk * kHeadWarps * sizeof(__nv_bfloat16);
  const bool vec = a.K % 4 == 0;
  auto kern = vec ? head_forward_kernel<InT, CMAX, true> : head_forward_kernel<InT, CMAX, false>;
  static size_t configured[2] = {0, 0};
  if (smem > configured[vec]) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured[vec] = smem;
  }
  dim3 grid((a.batch + kHeadWarps - 1) / kHeadWarps, a.m), block(kHeadWarps * 32);
  kern<<<grid, block, smem, s>>>(a, chunk);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_head_forward(const HeadArgs& a, cudaStream_t s) {
  const bool f32 = a.in32 != nullptr;
  if (a.C <= 16) return f32 ? launch_fwd<float, 16>(a, s) : launch_fwd<__nv_bfloat16, 16>(a, s);
  return f32 ? launch_fwd<float, 32>(a, s) : launch_fwd<__nv_bfloat16, 32>(a, s);
}

cudaError_t launch_head_wgrad(const HeadArgs& a, float* g, float* loss, cudaStream_t s) {
  dim3 grid((a.K + kWgCols - 1) / kWgCols, a.m), block(kWgCols, kWgSlices);
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

}  // namespace olsgd
