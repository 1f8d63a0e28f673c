// The output ("head") layer on CUDA cores: with ten-odd classes it is far too
// skinny for the tensor cores.  Forward, stable log-softmax, cross-entropy,
// d loss / d logits, the masked gradient with respect to the layer's input,
// and the layer's own weight and bias gradients.  All reductions have a fixed
// order; nothing uses floating-point atomics.
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

template <typename InT>
__device__ __forceinline__ float load_in(const InT* p);
template <>
__device__ __forceinline__ float load_in<float>(const float* p) { return *p; }
template <>
__device__ __forceinline__ float load_in<__nv_bfloat16>(const __nv_bfloat16* p) {
  return __bfloat162float(*p);
}

// With the fused gather: which row of worker i's partition batch slot b holds, read from the
// index buffer or (forward kernel, a.draw) drawn on the spot by the with-replacement rule.
__device__ __forceinline__ int32_t head_slot_row(const HeadArgs& a, int i, int b) {
  if (a.draw) {
    const uint32_t k = (uint32_t)(a.rule.k_base + (a.rule.k_ptr ? (uint64_t)*a.rule.k_ptr : 0ull));
    return minibatch_index(a.rule.key0, a.rule.key1, k, (uint32_t)i + a.rule.worker_offset, b,
                           (uint32_t)a.n_rows);
  }
  return a.row_idx[(int64_t)i * a.batch + b];
}

// Row b of worker i of the layer's input, with or without the fused gather (weight-gradient
// kernels: the rows of the batch slots are in the index buffer by then).
template <typename InT>
__device__ __forceinline__ const InT* head_row(const HeadArgs& a, int i, int b) {
  if (sizeof(InT) == 4) {
    const int64_t row = a.row_idx ? (int64_t)i * a.n_rows + a.row_idx[(int64_t)i * a.batch + b]
                                  : (int64_t)i * a.batch + b;
    return reinterpret_cast<const InT*>(a.in32) + row * a.K;
  }
  return reinterpret_cast<const InT*>(a.in16) + ((int64_t)i * a.batch + b) * a.K;
}
// Forward kernels with the fused gather: thread r < R looks up (or draws, and leaves in idx_out
// for the weight-gradient kernel) the row of batch slot b0 + r once, for the whole block.
template <int R>
__device__ __forceinline__ void head_block_rows(const HeadArgs& a, int i, int b0, int rows,
                                                int32_t* slot_row) {
  if (!a.row_idx) return;
  if ((int)threadIdx.x < R) {
    const int r = threadIdx.x;
    const int32_t row = head_slot_row(a, i, b0 + (r < rows ? r : 0));
    slot_row[r] = row;
    if (a.draw && r < rows) a.idx_out[(int64_t)i * a.batch + b0 + r] = row;
  }
  __syncthreads();
}
template <typename InT>
__device__ __forceinline__ const InT* head_row_of(const HeadArgs& a, int i, int b, int32_t slot_row) {
  if (sizeof(InT) == 4) {
    const int64_t row = a.row_idx ? (int64_t)i * a.n_rows + slot_row : (int64_t)i * a.batch + b;
    return reinterpret_cast<const InT*>(a.in32) + row * a.K;
  }
  return reinterpret_cast<const InT*>(a.in16) + ((int64_t)i * a.batch + b) * a.K;
}
__device__ __forceinline__ int head_label_of(const HeadArgs& a, int i, int b, int32_t slot_row) {
  if (a.row_idx) return a.y_all[(int64_t)i * a.n_rows + slot_row];
  return a.yb[(int64_t)i * a.batch + b];
}

// four adjacent inputs of a row (16-byte fp32 or 8-byte bf16 load)
__device__ __forceinline__ float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
  const uint2 w = *reinterpret_cast<const uint2*>(p);
  const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&w.x);
  const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162*>(&w.y);
  return make_float4(__low2float(lo), __high2float(lo), __low2float(hi), __high2float(hi));
}

constexpr int kHeadThreads = 128;

// Forward, loss and input gradient of the output layer for R batch rows of one worker.
//
// Every thread owns the input columns k = tid, tid + 128, ... : it reads the R inputs and
// the C weights of a column with coalesced loads (all independent, so many are in flight)
// and keeps R x C partial logits in registers.  The partial logits of the 128 threads are
// added in a fixed order through shared memory, warp r finishes row r (stable log-softmax,
// loss, d loss / d logits), and a second sweep over the same columns forms the masked input
// gradient din[r][k] = (sum_c dl[r][c] W[c][k]) * (in[r][k] > 0), which each thread can store
// in both layouts without any transposition: R consecutive batch entries of column k are
// 2R contiguous bytes of the [K][B] copy.
template <typename InT, int CMAX, int R>
__global__ void __launch_bounds__(kHeadThreads)
head_forward_kernel(HeadArgs a) {
  launch_gate();
  extern __shared__ __align__(16) float head_smem[];
  float* red = head_smem;                                  // [R * CMAX][kHeadThreads + 1]
  float* lg = red + R * CMAX * (kHeadThreads + 1);         // [R][CMAX] logits, then dl
  const int i = blockIdx.y, b0 = blockIdx.x * R;
  const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
  const int K = a.K, C = a.C, B = a.batch;
  const float* W = a.x + (int64_t)i * a.ld + a.w_off;
  const float* bias = a.x + (int64_t)i * a.ld + a.b_off;
  const int rows = min(R, B - b0);
  __shared__ int32_t slot_row[R];
  head_block_rows<R>(a, i, b0, rows, slot_row);
  const InT* rowp[R];
#pragma unroll
  for (int r = 0; r < R; ++r) rowp[r] = head_row_of<InT>(a, i, b0 + (r < rows ? r : 0), slot_row[r]);

  float acc[R][CMAX];
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < CMAX; ++c) acc[r][c] = 0.f;

#pragma unroll 2
  for (int k = tid; k < K; k += kHeadThreads) {
    float w[CMAX], xv[R];
#pragma unroll
    for (int c = 0; c < CMAX; ++c) w[c] = (c < C) ? W[(int64_t)c * K + k] : 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) xv[r] = (r < rows) ? load_in<InT>(rowp[r] + k) : 0.f;
    if (a.round_w_bf16) {
#pragma unroll
      for (int c = 0; c < CMAX; ++c) w[c] = bf16_round(w[c]);
    }
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int c = 0; c < CMAX; ++c) acc[r][c] = fmaf(xv[r], w[c], acc[r][c]);
  }
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < CMAX; ++c) red[(r * CMAX + c) * (kHeadThreads + 1) + tid] = acc[r][c];
  __syncthreads();
  // output o = r * CMAX + c is finished by warp o % 4: each lane adds four partials in
  // order, then the lanes are combined by a fixed shuffle tree
  for (int o = warp; o < R * CMAX; o += kHeadThreads / 32) {
    const float* src = red + o * (kHeadThreads + 1);
    float sum = 0.f;
#pragma unroll
    for (int t = 0; t < kHeadThreads / 32; ++t) sum += src[lane + 32 * t];
    sum = warp_sum(sum);
    if (lane == 0) lg[o] = sum;
  }
  __syncthreads();
  // warps take the rows round-robin; lane c holds class c
  for (int r = warp; r < R; r += kHeadThreads / 32) {
    const int b = b0 + r;
    const bool live = r < rows;
    const float logit = (lane < C) ? lg[r * CMAX + lane] + bias[lane] : -INFINITY;
    float mx = logit;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    const float e = (lane < C) ? expf(logit - mx) : 0.f;
    const float lse = mx + logf(warp_sum(e));
    const int label = live ? head_label_of(a, i, b, slot_row[r]) : 0;
    const float picked = __shfl_sync(0xffffffffu, logit, label);
    float dl = 0.f;
    if (lane < C) dl = (expf(logit - lse) - (lane == label ? 1.f : 0.f)) / (float)B;
    if (live && lane < C) a.dlogits[((int64_t)i * B + b) * C + lane] = dl;
    if (live && lane == 0) a.rowloss[(int64_t)i * B + b] = lse - picked;
    // the operand of the input-gradient product is the bf16-rounded dl on the tensor-core path
    if (lane < CMAX) lg[r * CMAX + lane] = (live && lane < C) ? (a.round_w_bf16 ? bf16_round(dl) : dl) : 0.f;
  }
  if (!a.din32 && !a.din16 && !a.din16t) return;
  __syncthreads();

  float dls[R][CMAX];
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < CMAX; ++c) dls[r][c] = lg[r * CMAX + c];
  const bool vec_t = (R == 8) && (B % 8 == 0) && rows == R;
#pragma unroll 2
  for (int k = tid; k < K; k += kHeadThreads) {
    float w[CMAX], xv[R], d[R];
#pragma unroll
    for (int c = 0; c < CMAX; ++c) w[c] = (c < C) ? W[(int64_t)c * K + k] : 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) xv[r] = (r < rows) ? load_in<InT>(rowp[r] + k) : 0.f;
    if (a.round_w_bf16) {
#pragma unroll
      for (int c = 0; c < CMAX; ++c) w[c] = bf16_round(w[c]);
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float v = 0.f;
#pragma unroll
      for (int c = 0; c < CMAX; ++c) v = fmaf(dls[r][c], w[c], v);
      d[r] = (xv[r] > 0.f) ? v : 0.f;
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (r < rows) {
        const int64_t o = ((int64_t)i * B + b0 + r) * K + k;
        if (a.din32) a.din32[o] = d[r];
        if (a.din16) a.din16[o] = __float2bfloat16_rn(d[r]);
      }
    }
    if (a.din16t) {
      __nv_bfloat16* dst = a.din16t + ((int64_t)i * K + k) * B + b0;
      if (vec_t) {
        uint32_t pk[R / 2];
#pragma unroll
        for (int r = 0; r < R / 2; ++r) {
          __nv_bfloat162 p2 = __floats2bfloat162_rn(d[2 * r], d[2 * r + 1]);
          pk[r] = *reinterpret_cast<uint32_t*>(&p2);
        }
        if (R == 8) *reinterpret_cast<uint4*>(dst) = make_uint4(pk[0], pk[1], pk[2 % (R / 2)], pk[3 % (R / 2)]);
      } else {
#pragma unroll
        for (int r = 0; r < R; ++r)
          if (r < rows) dst[r] = __float2bfloat16_rn(d[r]);
      }
    }
  }
}

// The same kernel for K % 4 == 0: a thread owns FOUR adjacent input columns at a time
// (k = 4 tid, 4 tid + 512, ...), so every load is 8 or 16 bytes and one sweep needs a quarter
// of the load instructions.  Same reduction order over threads as above.
template <typename InT, int CMAX, int R>
__global__ void __launch_bounds__(kHeadThreads, (R <= 4 && CMAX <= 10) ? 4 : 2)
head_forward_vec_kernel(HeadArgs a) {
  launch_gate();
  extern __shared__ __align__(16) float head_smem[];
  float* red = head_smem;                                  // [R * CMAX][kHeadThreads + 1]
  float* lg = red + R * CMAX * (kHeadThreads + 1);         // [R][CMAX] logits, then dl
  const int i = blockIdx.y, b0 = blockIdx.x * R;
  const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
  const int K = a.K, C = a.C, B = a.batch;
  const float* W = a.x + (int64_t)i * a.ld + a.w_off;
  const float* bias = a.x + (int64_t)i * a.ld + a.b_off;
  const int rows = min(R, B - b0);
  __shared__ int32_t slot_row[R];
  head_block_rows<R>(a, i, b0, rows, slot_row);
  const InT* rowp[R];
#pragma unroll
  for (int r = 0; r < R; ++r) rowp[r] = head_row_of<InT>(a, i, b0 + (r < rows ? r : 0), slot_row[r]);

  // what the softmax step needs from global memory is fetched now, under the first sweep:
  // lane c's bias entry and the labels of the rows this warp will finish
  constexpr int kRowsPerWarp = (R + kHeadThreads / 32 - 1) / (kHeadThreads / 32);
  const float bias_c = (lane < C) ? bias[lane] : 0.f;
  int label_of[kRowsPerWarp];
#pragma unroll
  for (int j = 0; j < kRowsPerWarp; ++j) {
    const int r = warp + j * (kHeadThreads / 32);
    label_of[j] = (r < rows) ? head_label_of(a, i, b0 + r, slot_row[r]) : 0;
  }

  float acc[R][CMAX];
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < CMAX; ++c) acc[r][c] = 0.f;

  for (int k = 4 * tid; k < K; k += 4 * kHeadThreads) {
    float4 w[CMAX], xv[R];
#pragma unroll
    for (int c = 0; c < CMAX; ++c)
      w[c] = (c < C) ? load4(W + (int64_t)c * K + k) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int r = 0; r < R; ++r)
      xv[r] = (r < rows) ? load4(rowp[r] + k) : make_float4(0.f, 0.f, 0.f, 0.f);
    if (a.round_w_bf16) {
#pragma unroll
      for (int c = 0; c < CMAX; ++c) {
        w[c].x = bf16_round(w[c].x);
        w[c].y = bf16_round(w[c].y);
        w[c].z = bf16_round(w[c].z);
        w[c].w = bf16_round(w[c].w);
      }
    }
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int c = 0; c < CMAX; ++c) {
        acc[r][c] = fmaf(xv[r].x, w[c].x, acc[r][c]);
        acc[r][c] = fmaf(xv[r].y, w[c].y, acc[r][c]);
        acc[r][c] = fmaf(xv[r].z, w[c].z, acc[r][c]);
        acc[r][c] = fmaf(xv[r].w, w[c].w, acc[r][c]);
      }
  }
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < CMAX; ++c) red[(r * CMAX + c) * (kHeadThreads + 1) + tid] = acc[r][c];
  __syncthreads();
  for (int o = warp; o < R * CMAX; o += kHeadThreads / 32) {
    const float* src = red + o * (kHeadThreads + 1);
    float sum = 0.f;
#pragma unroll
    for (int t = 0; t < kHeadThreads / 32; ++t) sum += src[lane + 32 * t];
    sum = warp_sum(sum);
    if (lane == 0) lg[o] = sum;
  }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < kRowsPerWarp; ++j) {
    const int r = warp + j * (kHeadThreads / 32);
    if (r >= R) break;
    const int b = b0 + r;
    const bool live = r < rows;
    const float logit = (lane < C) ? lg[r * CMAX + lane] + bias_c : -INFINITY;
    float mx = logit;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    const float e = (lane < C) ? expf(logit - mx) : 0.f;
    const float lse = mx + logf(warp_sum(e));
    const int label = label_of[j];
    const float picked = __shfl_sync(0xffffffffu, logit, label);
    float dl = 0.f;
    if (lane < C) dl = (expf(logit - lse) - (lane == label ? 1.f : 0.f)) / (float)B;
    if (live && lane < C) a.dlogits[((int64_t)i * B + b) * C + lane] = dl;
    if (live && lane == 0) a.rowloss[(int64_t)i * B + b] = lse - picked;
    if (lane < CMAX) lg[r * CMAX + lane] = (live && lane < C) ? (a.round_w_bf16 ? bf16_round(dl) : dl) : 0.f;
  }
  if (!a.din32 && !a.din16 && !a.din16t) return;
  __syncthreads();

  // second sweep: dl is read from shared memory (a broadcast), four columns per read
  const bool vec_t = (R == 8 || R == 4) && (B % R == 0) && rows == R;
  for (int k = 4 * tid; k < K; k += 4 * kHeadThreads) {
    float4 w[CMAX], xv[R], d[R];
#pragma unroll
    for (int c = 0; c < CMAX; ++c)
      w[c] = (c < C) ? load4(W + (int64_t)c * K + k) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int r = 0; r < R; ++r)
      xv[r] = (r < rows) ? load4(rowp[r] + k) : make_float4(0.f, 0.f, 0.f, 0.f);
    if (a.round_w_bf16) {
#pragma unroll
      for (int c = 0; c < CMAX; ++c) {
        w[c].x = bf16_round(w[c].x);
        w[c].y = bf16_round(w[c].y);
        w[c].z = bf16_round(w[c].z);
        w[c].w = bf16_round(w[c].w);
      }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int c = 0; c < CMAX; ++c) {
        const float dl = lg[r * CMAX + c];
        v.x = fmaf(dl, w[c].x, v.x);
        v.y = fmaf(dl, w[c].y, v.y);
        v.z = fmaf(dl, w[c].z, v.z);
        v.w = fmaf(dl, w[c].w, v.w);
      }
      d[r].x = (xv[r].x > 0.f) ? v.x : 0.f;
      d[r].y = (xv[r].y > 0.f) ? v.y : 0.f;
      d[r].z = (xv[r].z > 0.f) ? v.z : 0.f;
      d[r].w = (xv[r].w > 0.f) ? v.w : 0.f;
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (r < rows) {
        const int64_t o = ((int64_t)i * B + b0 + r) * K + k;
        if (a.din32) *reinterpret_cast<float4*>(a.din32 + o) = d[r];
        if (a.din16) {
          const __nv_bfloat162 lo = __floats2bfloat162_rn(d[r].x, d[r].y);
          const __nv_bfloat162 hi = __floats2bfloat162_rn(d[r].z, d[r].w);
          *reinterpret_cast<uint2*>(a.din16 + o) = make_uint2(*reinterpret_cast<const uint32_t*>(&lo),
                                                              *reinterpret_cast<const uint32_t*>(&hi));
        }
      }
    }
    if (a.din16t) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        __nv_bfloat16* dst = a.din16t + ((int64_t)i * K + k + q) * B + b0;
        float dq[R];
#pragma unroll
        for (int r = 0; r < R; ++r) dq[r] = q == 0 ? d[r].x : q == 1 ? d[r].y : q == 2 ? d[r].z : d[r].w;
        if (vec_t) {
          uint32_t pk[4];
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            const __nv_bfloat162 p2 = __floats2bfloat162_rn(dq[(2 * r) % R], dq[(2 * r + 1) % R]);
            pk[r] = *reinterpret_cast<const uint32_t*>(&p2);
          }
          if (R == 8) *reinterpret_cast<uint4*>(dst) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          else *reinterpret_cast<uint2*>(dst) = make_uint2(pk[0], pk[1]);
        } else {
#pragma unroll
          for (int r = 0; r < R; ++r)
            if (r < rows) dst[r] = __float2bfloat16_rn(dq[r]);
        }
      }
    }
  }
}

// Bias gradient db[c] = sum_b dlogits[b][c] and the worker's mean loss, by one whole block
// of T threads (T a multiple of 32): with T / 32 parts, thread (c, p) adds the rows
// b = p, p + T / 32, ... of class c in order and thread c adds the partial sums in order;
// the last warp adds the per-row losses (lane l takes rows l, l + 32, ... in order, then a
// fixed shuffle tree).  `scratch` holds T floats and is free once the block has passed the
// barrier inside.
template <int T>
__device__ __forceinline__ void head_bias_and_loss(const HeadArgs& a, int i, int tid, float* scratch,
                                                   float* gi, float* loss, const FusedUpdateArgs& up) {
  const int C = a.C, B = a.batch;
  const float* dl = a.dlogits + (int64_t)i * B * C;
  __syncthreads();
  const int c = tid % 32, p = tid / 32;
  constexpr int NP = T / 32;
  if (c < C) {
    float sum = 0.f;
    for (int b = p; b < B; b += NP) sum += dl[(int64_t)b * C + c];
    scratch[p * 32 + c] = sum;
  }
  __syncthreads();
  if (tid < C) {
    float sum = scratch[tid];
#pragma unroll
    for (int q = 1; q < NP; ++q) sum += scratch[q * 32 + tid];
    if (up.enabled) {
      // Eq. 3 / Eq. 4 for bias entry tid of worker i
      const int64_t e = a.b_off + tid, o = (int64_t)i * up.ld + e;
      const bool mom = up.u != nullptr && up.mu != 0.f;
      float x = up.x_in[o], u = mom ? up.u[o] : 0.f;
      update_scalar_rt(x, u, sum, up.sync ? up.z[e] : 0.f, up.gamma, up.mu, up.alpha, mom, up.sync != 0);
      up.x_out[o] = x;
      if (mom) up.u[o] = u;
      if (up.shadow) up.shadow[o] = __float2bfloat16_rn(x);
    } else {
      gi[a.b_off + tid] = sum;
    }
  }
  if (loss && tid >= T - 32) {
    const int lane = tid % 32;
    float sum = 0.f;
    for (int b = lane; b < B; b += 32) sum += a.rowloss[(int64_t)i * B + b];
    sum = warp_sum(sum);
    if (lane == 0) loss[i] = sum / (float)B;
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
  launch_gate();
  __shared__ float dsm[kWgRows][CMAX + 1];
  __shared__ float part[kWgSlices][CMAX][kWgCols];
  const int i = blockIdx.y;
  const int tx = threadIdx.x, ty = threadIdx.y, tid = ty * kWgCols + tx;
  const int j = blockIdx.x * kWgCols + tx;
  const int K = a.K, C = a.C, B = a.batch;
  const float* dl = a.dlogits + (int64_t)i * B * C;
  float acc[CMAX];
#pragma unroll
  for (int c = 0; c < CMAX; ++c) acc[c] = 0.f;
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
          xs[u] = (r < rc) ? load_in<InT>(head_row<InT>(a, i, r0 + r) + j) : 0.f;
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
  FusedUpdateArgs none{};
  if (blockIdx.x == 0) head_bias_and_loss<kWgCols * kWgSlices>(a, i, tid, &part[0][0][0], gi, loss, none);
}

// The same product for K % 4 == 0 and at most 16 classes: a thread owns FOUR adjacent input
// columns (one 16-byte fp32 or 8-byte bf16 load per row, eight in flight) and a block of
// 16 x 8 threads covers 64 columns with eight batch slices.  Fixed order as above.
constexpr int kWvCols = 16, kWvSlices = 8, kWvRows = 128, kWvFlight = 8;


template <typename InT, int CMAX>
__global__ void __launch_bounds__(kWvCols* kWvSlices)
head_wgrad_vec_kernel(HeadArgs a, float* __restrict__ g, float* __restrict__ loss, FusedUpdateArgs up) {
  launch_gate();
  __shared__ float dsm[kWvRows][CMAX + 1];
  __shared__ __align__(16) float part[kWvSlices][CMAX][kWvCols * 4];
  const int i = blockIdx.y;
  const int tx = threadIdx.x, ty = threadIdx.y, tid = ty * kWvCols + tx;
  const int j = (blockIdx.x * kWvCols + tx) * 4;
  const int K = a.K, C = a.C, B = a.batch;
  const float* dl = a.dlogits + (int64_t)i * B * C;
  float acc[4][CMAX];
#pragma unroll
  for (int q = 0; q < 4; ++q)
#pragma unroll
    for (int c = 0; c < CMAX; ++c) acc[q][c] = 0.f;
  for (int r0 = 0; r0 < B; r0 += kWvRows) {
    const int rc = min(kWvRows, B - r0);
    __syncthreads();
    for (int e = tid; e < rc * C; e += kWvCols * kWvSlices) {
      float d = dl[(int64_t)r0 * C + e];
      if (a.round_w_bf16) d = bf16_round(d);
      dsm[e / C][e % C] = d;
    }
    __syncthreads();
    if (j < K) {
      for (int rb = ty; rb < rc; rb += kWvSlices * kWvFlight) {
        float4 xs[kWvFlight];
#pragma unroll
        for (int u = 0; u < kWvFlight; ++u) {
          const int r = rb + u * kWvSlices;
          xs[u] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (r < rc) xs[u] = load4(head_row<InT>(a, i, r0 + r) + j);
        }
#pragma unroll
        for (int u = 0; u < kWvFlight; ++u) {
          const int r = rb + u * kWvSlices;
          if (r < rc) {
#pragma unroll
            for (int c = 0; c < CMAX; ++c) {
              if (c < C) {
                const float d = dsm[r][c];
                acc[0][c] = fmaf(d, xs[u].x, acc[0][c]);
                acc[1][c] = fmaf(d, xs[u].y, acc[1][c]);
                acc[2][c] = fmaf(d, xs[u].z, acc[2][c]);
                acc[3][c] = fmaf(d, xs[u].w, acc[3][c]);
              }
            }
          }
        }
      }
    }
  }
#pragma unroll
  for (int c = 0; c < CMAX; ++c)
    if (c < C)
      *reinterpret_cast<float4*>(&part[ty][c][tx * 4]) =
          make_float4(acc[0][c], acc[1][c], acc[2][c], acc[3][c]);
  __syncthreads();
  float* gi = g + (int64_t)i * a.ld;
  for (int e = tid; e < C * kWvCols; e += kWvCols * kWvSlices) {
    const int c = e / kWvCols, col4 = e % kWvCols;
    const int jj = (blockIdx.x * kWvCols + col4) * 4;
    if (jj < K) {
      float4 s = *reinterpret_cast<const float4*>(&part[0][c][col4 * 4]);
#pragma unroll
      for (int t = 1; t < kWvSlices; ++t) {
        const float4 p = *reinterpret_cast<const float4*>(&part[t][c][col4 * 4]);
        s.x += p.x;
        s.y += p.y;
        s.z += p.z;
        s.w += p.w;
      }
      const int64_t e = a.w_off + (int64_t)c * K + jj;
      if (up.enabled) {
        // the gradient strip is consumed here: Eq. 3 (+ Nesterov) and, on sync steps, Eq. 4
        const int64_t o = (int64_t)i * up.ld + e;
        const bool mom = up.u != nullptr && up.mu != 0.f;
        float4 x = *reinterpret_cast<const float4*>(up.x_in + o);
        float4 u = mom ? *reinterpret_cast<const float4*>(up.u + o) : make_float4(0.f, 0.f, 0.f, 0.f);
        const float4 z = up.sync ? *reinterpret_cast<const float4*>(up.z + e)
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
        const bool sync = up.sync != 0;
        update_scalar_rt(x.x, u.x, s.x, z.x, up.gamma, up.mu, up.alpha, mom, sync);
        update_scalar_rt(x.y, u.y, s.y, z.y, up.gamma, up.mu, up.alpha, mom, sync);
        update_scalar_rt(x.z, u.z, s.z, z.z, up.gamma, up.mu, up.alpha, mom, sync);
        update_scalar_rt(x.w, u.w, s.w, z.w, up.gamma, up.mu, up.alpha, mom, sync);
        *reinterpret_cast<float4*>(up.x_out + o) = x;
        if (mom) *reinterpret_cast<float4*>(up.u + o) = u;
        if (up.shadow) *reinterpret_cast<uint2*>(up.shadow + o) = pack_bf16x4(x);
      } else {
        *reinterpret_cast<float4*>(gi + e) = s;
      }
    }
  }
  if (blockIdx.x == 0) head_bias_and_loss<kWvCols * kWvSlices>(a, i, tid, &part[0][0][0], gi, loss, up);
}

template <typename InT, int CMAX, int R>
cudaError_t launch_fwd(const HeadArgs& a, cudaStream_t s) {
  const size_t smem = ((size_t)R * CMAX * (kHeadThreads + 1) + (size_t)R * CMAX) * sizeof(float);
  // four columns per thread where the rows are 16-byte aligned; with 32 classes the
  // float4 weights would not fit the register file, so that case keeps one column per thread
  constexpr int VC = CMAX <= 16 ? CMAX : 1;
  const bool vec = CMAX <= 16 && a.K % 4 == 0 && a.w_off % 4 == 0 && a.ld % 4 == 0;
  auto kern = vec ? head_forward_vec_kernel<InT, VC, R> : head_forward_kernel<InT, CMAX, R>;
  static PerDeviceSmem configured[2];
  {
    const cudaError_t e = ensure_dynamic_smem(configured[vec], kern, smem);
    if (e != cudaSuccess) return e;
  }
  dim3 grid((a.batch + R - 1) / R, a.m), block(kHeadThreads);
  return launch_chained(kern, grid, block, smem, s, a);
}

template <typename InT>
cudaError_t launch_fwd_c(const HeadArgs& a, cudaStream_t s) {
  // eight batch rows per block, or four where that leaves fewer than two blocks per SM
  const bool small = (int64_t)((a.batch + 7) / 8) * a.m < 4 * (int64_t)sm_count();
  if (a.C <= 10) return small ? launch_fwd<InT, 10, 4>(a, s) : launch_fwd<InT, 10, 8>(a, s);
  if (a.C <= 16) return small ? launch_fwd<InT, 16, 4>(a, s) : launch_fwd<InT, 16, 8>(a, s);
  return launch_fwd<InT, 32, 4>(a, s);
}

}  // namespace

cudaError_t launch_head_forward(const HeadArgs& a, cudaStream_t s) {
  return a.in32 ? launch_fwd_c<float>(a, s) : launch_fwd_c<__nv_bfloat16>(a, s);
}

bool head_wgrad_can_update(const HeadArgs& a) {
  // the four-column kernel; the bias update is scalar and has no alignment rule
  return a.K % 4 == 0 && a.C <= 16 && a.w_off % 4 == 0 && a.ld % 4 == 0;
}

cudaError_t launch_head_wgrad(const HeadArgs& a, float* g, float* loss, const FusedUpdateArgs* upd,
                              cudaStream_t s) {
  const bool f32 = a.in32 != nullptr;
  cudaError_t err = cudaSuccess;
  FusedUpdateArgs up{};
  if (upd && upd->enabled) {
    if (!head_wgrad_can_update(a)) return cudaErrorInvalidValue;
    up = *upd;
  }
  if (head_wgrad_can_update(a)) {
    dim3 vgrid((a.K / 4 + kWvCols - 1) / kWvCols, a.m), vblock(kWvCols, kWvSlices);
    if (a.C <= 10) {
      if (f32) err = launch_chained(head_wgrad_vec_kernel<float, 10>, vgrid, vblock, 0, s, a, g, loss, up);
      else err = launch_chained(head_wgrad_vec_kernel<__nv_bfloat16, 10>, vgrid, vblock, 0, s, a, g, loss, up);
    } else {
      if (f32) err = launch_chained(head_wgrad_vec_kernel<float, 16>, vgrid, vblock, 0, s, a, g, loss, up);
      else err = launch_chained(head_wgrad_vec_kernel<__nv_bfloat16, 16>, vgrid, vblock, 0, s, a, g, loss, up);
    }
    return err;
  }
  dim3 grid((a.K + kWgCols - 1) / kWgCols, a.m), block(kWgCols, kWgSlices);
  if (a.C <= 16) {
    if (f32) err = launch_chained(head_wgrad_kernel<float, 16>, grid, block, 0, s, a, g, loss);
    else err = launch_chained(head_wgrad_kernel<__nv_bfloat16, 16>, grid, block, 0, s, a, g, loss);
  } else {
    if (f32) err = launch_chained(head_wgrad_kernel<float, 32>, grid, block, 0, s, a, g, loss);
    else err = launch_chained(head_wgrad_kernel<__nv_bfloat16, 32>, grid, block, 0, s, a, g, loss);
  }
  return err;
}

}  // namespace olsgd
