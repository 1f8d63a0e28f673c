// Weight-gradient GEMM of the worker-batched backward pass on the tensor cores:
//   dW[i] [Ma][Nb] = A[i] [Ma][K] * B[i] [Nb][K]^T,   K = minibatch size (64..256),
// either stored as fp32 into the stacked gradient G_k (Eq. 7) or consumed on the
// spot by the parameter update (FUSED).
//
// The contraction is short and the output large, so the kernel is bound by
// memory traffic, not by the tensor pipe.  The work is cut into units of one
// 128 x 128 tile.  A slab is a 128-row band of one worker's dW; a few CTAs share
// a slab and take its tiles round-robin, so that together they sweep adjacent
// column tiles at the same time.  A CTA's A operand (128 x K bf16) stays in
// shared memory; B tiles stream through a small TMA ring; the fp32 accumulator
// is double-buffered in tensor memory so that the MMAs of unit j+1 run under
// the epilogue of unit j.
//
// Plain variant (224 threads): warp 0 TMA loads, warp 1 MMA issue + TMEM owner,
// warps 2-5 epilogue, which moves 32 x 32 blocks from TMEM through swizzled
// shared memory to global memory with TMA stores (whole 128-byte lines).
//
// FUSED variant (352 threads, eight epilogue warps): the gradient never goes to
// memory.  Each 32 x 32 block of dW is turned, through a swizzled shared-memory
// buffer, from "one accumulator row per thread" into "one 16-byte row segment
// per thread", and the same thread then applies the parameter update to that
// segment: Eq. 3 with the local Nesterov buffer, Eq. 4 on sync steps, the new
// fp32 weights into the other half of the ping-pong pair and their bf16 copy for
// the next forward pass.  The matching tiles of x_k and of the momentum buffer
// are prefetched by TMA two blocks ahead into a per-warp ring, which is what
// keeps enough bytes in flight; results leave as whole 128-byte row segments.
// That removes the 4-byte write and the 4-byte read of G_k per parameter.
//
// One more warp in either variant adds up the rows of the resident A operand, which is the
// layer's bias gradient, in the first CTA of every slab: lane l takes the columns l, l + 32,
// ... in order and a fixed shuffle tree combines the lanes.
//
// SUM variant of the fused kernel (sync steps): besides Eq. 3 / Eq. 4 the launch forms the
// worker sums of x_{k+1} that the anchor refresh (Eq. 5, or Eq. 10-11) needs, so that no
// second pass over the m worker models is made.  A unit is then a 128 x 64 tile; a CTA stays
// on one tile POSITION and walks over the workers of one slice (slice s of S holds the
// workers s, s + S, ...: the summation order of the stand-alone worker-mean kernel), every
// epilogue thread adding its row segments of x_{k+1} in registers.  After the slice's last
// worker the partial sums go to row s of a scratch matrix [S][ld]; a small kernel on the side
// stream (launch_anchor_from_slices) later adds the S rows in slice order, divides by m and
// updates the anchor.  The launch itself only READS the anchor (the pull-back against the
// previous period's value), which keeps the one-period lag stated after Eq. 5.
//
// Every mbarrier wait is bounded (see tc_common.cuh).
#include <cstring>

#include "tc_common.cuh"
#include "update_math.cuh"

namespace olsgd {
namespace {

using namespace tc;

constexpr int kWN = 128;            // columns per tile = MMA N
constexpr int kWStages = 4;         // upper bound of the B ring (one k-block of one tile per stage)
constexpr int kMaxKB = 4;           // K <= 256

struct WgradUpd {
  const float* x_in;
  float* x_out;
  float* u;
  const float* z;
  __nv_bfloat16* shadow;
  int64_t ld, w_off;
  int64_t b_off;   // >= 0: the row-sum warp updates the layer's bias instead of storing its gradient
  float gamma, mu, alpha;
  int mom, sync;
  // SUM variant: partial worker sums of this layer's weight matrix
  float* part;         // [slices][ld]
  int slices, m;
  // SUM variant: the A operand (dA^T) in global memory, for the bias row sums
  const __nv_bfloat16* a_ptr;
  int64_t a_ld, a_batch;
};

// Where a unit lives.
struct UnitPos {
  int worker, m0, col;
  int tile;   // column tile index inside the band
  int wi;     // SUM: position of the worker inside its slice
};
// The units of one CTA.
//   plain / fused: the CTA belongs to one slab (a 128-row band of ONE worker's dW) and takes
//     the 128-column tiles first, first + chunks, ... of it.
//   SUM: the CTA belongs to one band and one slice of the workers and takes the 64-column
//     tiles first, first + chunks, ...; on each tile it visits the slice's workers in order.
struct CtaWork {
  int n_units, worker, m0, first, chunks, slice, slices, wps;
  template <bool SUM>
  __device__ __forceinline__ UnitPos at(int j) const {
    UnitPos p;
    p.m0 = m0;
    if (SUM) {
      const int t = j / wps;
      p.wi = j - t * wps;
      p.worker = slice + p.wi * slices;
      p.tile = first + t * chunks;
      p.col = p.tile * 64;
    } else {
      p.wi = 0;
      p.worker = worker;
      p.tile = first + j * chunks;
      p.col = p.tile * kWN;
    }
    return p;
  }
};
template <bool SUM>
__device__ __forceinline__ CtaWork cta_work(int cta, int n_tiles, int m_tiles, int chunks, int m,
                                            int slices) {
  CtaWork w;
  w.chunks = chunks;
  w.slices = slices;
  const int group = cta / chunks;
  w.first = cta - group * chunks;
  const int my_tiles = (n_tiles - w.first + chunks - 1) / chunks;
  if (SUM) {
    const int band = group / slices;
    w.slice = group - band * slices;
    w.m0 = band * kBM;
    w.worker = w.slice;
    w.wps = (m - w.slice + slices - 1) / slices;
    w.n_units = my_tiles * w.wps;
  } else {
    w.worker = group / m_tiles;
    w.m0 = (group - w.worker * m_tiles) * kBM;
    w.slice = 0;
    w.wps = 1;
    w.n_units = my_tiles;
  }
  return w;
}

// Update of one 32 x 32 block held as v[32] = row `lane` of the block.
//   stage    this warp's 4 KB shared buffer for the gradient block
//   xt, ut   the block's tiles of x_k and of the momentum buffer, brought into shared
//            memory by TMA with the 128-byte swizzle (row r, 16-byte chunk q at q ^ (r % 8))
//   blk_off  element offset of the block's corner inside a worker row
//   ldw      row pitch of the weight matrix (its input width)
//   zs       the block's strip of the anchor (sync steps)
//   acc      SUM: running worker sum of x_{k+1} for this thread's eight row segments
template <bool MOM, bool SYNC, bool SUM>
__device__ __forceinline__ void fused_block(const float (&v)[32], const float4 (&zs)[8], float* stage,
                                            const float* xt, const float* ut, uint32_t xu_bar,
                                            uint32_t xu_parity, volatile int* abort_flag, int lane,
                                            const WgradUpd& up, int64_t wk_off, int64_t blk_off,
                                            int ldw, float4 (&acc)[8], bool* ok) {
  const int q = lane & 7, rsub = lane >> 3;
  __syncwarp();   // the previous block's reads of the staging buffer are done
  float4* mine = reinterpret_cast<float4*>(stage + lane * 32);
#pragma unroll
  for (int c = 0; c < 8; ++c)
    mine[c ^ (lane & 7)] = make_float4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
  __syncwarp();
  *ok = mbar_wait(xu_bar, xu_parity, abort_flag);
  if (!*ok) return;
#pragma unroll
  for (int t = 0; t < 8; ++t) {
    const int row = t * 4 + rsub, slot = q ^ (row & 7);
    const int64_t off = blk_off + (int64_t)row * ldw + q * 4;
    float4 x = reinterpret_cast<const float4*>(xt + row * 32)[slot];
    float4 u = make_float4(0.f, 0.f, 0.f, 0.f);
    if (MOM) u = reinterpret_cast<const float4*>(ut + row * 32)[slot];
    const float4 g = reinterpret_cast<const float4*>(stage + row * 32)[slot];
    update4<MOM, SYNC>(x, u, g, zs[t], up.gamma, up.mu, up.alpha);
    *reinterpret_cast<float4*>(up.x_out + wk_off + off) = x;
    if (MOM) *reinterpret_cast<float4*>(up.u + wk_off + off) = u;
    *reinterpret_cast<uint2*>(up.shadow + wk_off + off) = pack_bf16x4(x);
    if (SUM) {
      acc[t].x += x.x;
      acc[t].y += x.y;
      acc[t].z += x.z;
      acc[t].w += x.w;
    }
  }
}

// SUM variant, after the last worker of a slice: this warp's 32 x 32 block of partial worker
// sums goes to row `slice` of the scratch matrix (L2 write, no reader in this launch).
__device__ __forceinline__ void store_sum_block(const float4 (&acc)[8], const WgradUpd& up,
                                                int slice, int64_t blk_off, int ldw, int lane) {
  const int q = lane & 7, rsub = lane >> 3;
  float* mine = up.part + (int64_t)slice * up.ld;
#pragma unroll
  for (int t = 0; t < 8; ++t)
    __stcg(reinterpret_cast<float4*>(mine + blk_off + (int64_t)(t * 4 + rsub) * ldw + q * 4), acc[t]);
}

struct WgradCtl {
  uint64_t a_full, a_empty;
  uint64_t b_full[kWStages];
  uint64_t b_empty[kWStages];
  uint64_t tmem_full[8];
  uint64_t tmem_empty[8];
  uint64_t xu_full[8][2];   // fused variant: per epilogue warp, x/u tile pair landed
  uint32_t tmem_base;
  int abort_flag;
};

constexpr uint32_t kXuTile = 32 * 32 * 4;        // one fp32 tile of x or u
constexpr uint32_t kXuPerWarp = 2 * 2 * kXuTile; // two buffers of (x, u)

constexpr int kFusedThreads = 352;   // TMA, MMA, eight epilogue warps, row sums
constexpr int kSumThreads = 320;     // TMA, MMA, eight epilogue warps (which also do the row sums:
                                     // ten warps leave each thread the registers the sums need)
constexpr int kPlainThreads = 224;   // TMA, MMA, four epilogue warps, row sums

// One launch covers the weight-gradient GEMMs of up to kMaxWgradLayers layers (same workers,
// same K): the CTAs of layer l are blockIdx.x in [cta_begin[l], cta_begin[l + 1]).  The layers
// do not depend on one another, and in one grid the CTAs of the next layer fill the SMs that
// the last partial wave of the previous one leaves idle.
constexpr int kMaxWgradLayers = 4;
struct WgradLayer {
  CUtensorMap map_a, map_b, map_out, map_u;
  WgradUpd up;
  float* rowsum;
  int64_t rowsum_batch;
  int n_tiles, m_tiles, chunks, ldw;
  int rows;      // Ma: the last 128-row band may reach past it (plain variant only)
  int cta_begin;
};
struct WgradBatch {
  WgradLayer layer[kMaxWgradLayers];
  int n_layers;
};

// Row sums of one 128 x K operand slab held in shared memory (128-byte swizzled k-blocks): the
// order of the bias-gradient kernel (partial l takes the columns l, l + 32, ... in order; the
// partials are combined by the tree of an xor-shuffle reduction), so both give the same bits.
// Row r of a k-block is 128 bytes whose 16-byte chunks are permuted (chunk j at j ^ (r % 8)).
__device__ __forceinline__ float slab_row_sum_smem(const uint8_t* a_smem, uint32_t block_bytes,
                                                   int num_kb, int row) {
  float part[32];
#pragma unroll
  for (int l = 0; l < 32; ++l) part[l] = 0.f;
  for (int kb = 0; kb < num_kb; ++kb) {
    const uint8_t* rowp = a_smem + kb * block_bytes + row * 128;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const uint4 q = *reinterpret_cast<const uint4*>(rowp + ((j ^ (row & 7)) << 4));
      const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        part[8 * (j & 3) + 2 * e] += __uint_as_float(w[e] << 16);
        part[8 * (j & 3) + 2 * e + 1] += __uint_as_float(w[e] & 0xffff0000u);
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1)
#pragma unroll
    for (int l = 0; l < o; ++l) part[l] += part[l + o];
  return part[0];
}
// The same sum, same order, for a row read from global memory (K contiguous bf16).
__device__ __forceinline__ float slab_row_sum_global(const __nv_bfloat16* rowp, int K) {
  float part[32];
#pragma unroll
  for (int l = 0; l < 32; ++l) part[l] = 0.f;
  for (int k0 = 0; k0 < K; k0 += 64) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const uint4 q = *reinterpret_cast<const uint4*>(rowp + k0 + j * 8);
      const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        part[8 * (j & 3) + 2 * e] += __uint_as_float(w[e] << 16);
        part[8 * (j & 3) + 2 * e + 1] += __uint_as_float(w[e] & 0xffff0000u);
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1)
#pragma unroll
    for (int l = 0; l < o; ++l) part[l] += part[l + o];
  return part[0];
}

// Eq. 3 / Eq. 4 for one bias entry, with the arithmetic of the update kernel.
__device__ __forceinline__ void update_bias_entry(const WgradUpd& up, int worker, int64_t entry,
                                                  float grad) {
  const int64_t o = (int64_t)worker * up.ld + entry;
  float x = up.x_in[o], u = up.mom ? up.u[o] : 0.f;
  update_scalar_rt(x, u, grad, up.sync ? up.z[entry] : 0.f, up.gamma, up.mu, up.alpha, up.mom != 0,
                   up.sync != 0);
  up.x_out[o] = x;
  if (up.mom) up.u[o] = u;
  up.shadow[o] = __float2bfloat16_rn(x);
}

template <bool FUSED, bool SUM>
__global__ void __launch_bounds__(FUSED ? (SUM ? kSumThreads : kFusedThreads) : kPlainThreads, 1)
wgrad_tc_kernel(const __grid_constant__ WgradBatch wb, int num_kb, int n_stages, int* status) {
  static_assert(FUSED || !SUM, "the worker sum lives in the fused epilogue");
  int layer_id = 0;
  for (int l = 1; l < wb.n_layers; ++l)
    if ((int)blockIdx.x >= wb.layer[l].cta_begin) layer_id = l;
  const WgradLayer& ly = wb.layer[layer_id];
  const CUtensorMap& map_a = ly.map_a;
  const CUtensorMap& map_b = ly.map_b;
  const CUtensorMap& map_out = ly.map_out;
  const CUtensorMap& map_u = ly.map_u;
  const int n_tiles = ly.n_tiles, m_tiles = ly.m_tiles, ldw = ly.ldw;
  const WgradUpd& up = ly.up;
  float* const rowsum = ly.rowsum;
  const int64_t rowsum_batch = ly.rowsum_batch;
  const int cta = (int)blockIdx.x - ly.cta_begin;
  constexpr int kTileN = SUM ? 64 : kWN;           // columns of one unit = MMA N
  // Accumulator buffers in tensor memory.  The fused variants have the SM to themselves and
  // take all 512 columns: the MMAs may then run several units ahead of the epilogue, and the
  // eight epilogue warps, which all have to hand a buffer back before it is reused, can
  // drift apart by as many units.  The plain variant shares the SM with a second CTA.
  constexpr int kBufs = FUSED ? 512 / kTileN : 2;
  constexpr int kBpu = SUM ? 1 : 2;                // 32-column blocks per unit and epilogue warp
  constexpr uint32_t kABlock = kBM * kBK * 2;      // one k-block of the A slab, 16 KB
  constexpr uint32_t kBBlock = kTileN * kBK * 2;   // one k-block of a B tile, 16 or 8 KB
  constexpr uint32_t kEpiBuf = 32 * 32 * 4;        // one 32 x 32 fp32 block, 4 KB

  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* a_smem = base;                                   // num_kb blocks
  uint8_t* b_smem = a_smem + num_kb * kABlock;              // n_stages blocks
  uint8_t* e_smem = b_smem + n_stages * kBBlock;            // 8 x 4 KB gradient staging
  uint8_t* xu_smem = e_smem + 8 * kEpiBuf;                  // fused: 8 warps x 2 x (x, u) tiles
  WgradCtl* ctl = reinterpret_cast<WgradCtl*>(xu_smem + (FUSED ? 8 * kXuPerWarp : 0));
  volatile int* abort_flag = &ctl->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // this CTA's units: every `chunks`-th tile of one band, so that the CTAs that share a
  // band (neighbours in the grid, running at the same time) sweep adjacent column tiles
  // together and touch each DRAM page while it is open
  const CtaWork work = cta_work<SUM>(cta, n_tiles, m_tiles, ly.chunks, up.m, up.slices);
  const int n_units = work.n_units;

  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&ctl->a_full), 1);
    mbar_init(smem_u32(&ctl->a_empty), 1);
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(smem_u32(&ctl->b_full[s]), 1);
      mbar_init(smem_u32(&ctl->b_empty[s]), 1);
    }
    for (int b = 0; b < kBufs; ++b) {
      mbar_init(smem_u32(&ctl->tmem_full[b]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[b]), FUSED ? 8 : 4);   // one arrival per epilogue warp
    }
    if (FUSED)
      for (int w = 0; w < 8; ++w)
        for (int b = 0; b < 2; ++b) mbar_init(smem_u32(&ctl->xu_full[w][b]), 1);
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(&ctl->tmem_base), kBufs * kTileN);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  // everything above touched only shared and tensor memory: it may run under the tail of
  // the kernel before this one
  launch_gate();

  constexpr int kRowsumWarp = SUM ? -1 : FUSED ? 10 : 6;
  if (warp == kRowsumWarp) {
    // ---------------- row sums of the resident A operand (the layer's bias gradient), in the
    // CTA that holds the first column tile of its slab
    const bool bias_update = FUSED && up.b_off >= 0;
    if ((rowsum || bias_update) && work.first == 0 && n_units > 0 &&
        mbar_wait(smem_u32(&ctl->a_full), 0u, abort_flag)) {
      float* dst = rowsum + (int64_t)work.worker * rowsum_batch + work.m0;
      for (int rr = 0; rr < kBM / 32; ++rr) {
        const int row = rr * 32 + lane;
        const float sum = slab_row_sum_smem(a_smem, kABlock, num_kb, row);
        if (bias_update) update_bias_entry(up, work.worker, up.b_off + work.m0 + row, sum);
        else if (work.m0 + row < ly.rows) dst[row] = sum;
      }
    }
  } else if (warp == 0 && lane == 0) {
    // ---------------- TMA producer
    const uint32_t a_full = smem_u32(&ctl->a_full);
    int issued = 0, visit = -1, cur_worker = -1;
    bool ok = true, a_pending = false;
    for (int j = 0; j < n_units && ok; ++j) {
      const UnitPos p = work.at<SUM>(j);
      if (p.worker != cur_worker) {
        // another worker's slab: it replaces the old one once the MMAs that read it retired
        ++visit;
        cur_worker = p.worker;
        ok = mbar_wait(smem_u32(&ctl->a_empty), (uint32_t)(visit & 1) ^ 1u, abort_flag);
        if (!ok) break;
        mbar_expect_tx(a_full, num_kb * kABlock);
        for (int kb = 0; kb < num_kb; ++kb)
          tma_load_3d(smem_u32(a_smem + kb * kABlock), &map_a, a_full, kb * kBK, p.m0, p.worker);
        a_pending = true;
      }
      for (int kb = 0; kb < num_kb; ++kb) {
        const int t = j * num_kb + kb, s = t % n_stages;
        const uint32_t ph = (t / n_stages) & 1;
        ok = mbar_wait(smem_u32(&ctl->b_empty[s]), ph ^ 1, abort_flag);
        if (!ok) break;
        const uint32_t full = smem_u32(&ctl->b_full[s]);
        mbar_expect_tx(full, kBBlock);
        tma_load_3d(smem_u32(b_smem + s * kBBlock), &map_b, full, kb * kBK, p.col, p.worker);
        issued = t + 1;
      }
    }
    if (*abort_flag) {
      // drain: wait (bounded) for the copies this thread still has in flight
      if (a_pending)
        for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(a_full, (uint32_t)(visit & 1)); ++it) {
        }
      for (int t = max(0, issued - n_stages); t < issued; ++t) {
        const uint32_t full = smem_u32(&ctl->b_full[t % n_stages]);
        const uint32_t ph = (t / n_stages) & 1;
        for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(full, ph); ++it) {
        }
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------- MMA issuer
    constexpr uint32_t idesc = instr_desc_bf16(kTileN);
    bool ok = true;
    int visit = -1, cur_worker = -1;
    for (int j = 0; j < n_units && ok; ++j) {
      const UnitPos p = work.at<SUM>(j);
      if (p.worker != cur_worker) {
        ++visit;
        cur_worker = p.worker;
        ok = mbar_wait(smem_u32(&ctl->a_full), (uint32_t)(visit & 1), abort_flag);
        if (!ok) break;
      }
      const int buf = j % kBufs, use = j / kBufs;
      ok = mbar_wait(smem_u32(&ctl->tmem_empty[buf]), (use & 1) ^ 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + (uint32_t)(buf * kTileN);
      for (int kb = 0; kb < num_kb; ++kb) {
        const int t = j * num_kb + kb, s = t % n_stages;
        const uint32_t ph = (t / n_stages) & 1;
        ok = mbar_wait(smem_u32(&ctl->b_full[s]), ph, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint64_t a_desc = smem_desc_k_sw128(smem_u32(a_smem + kb * kABlock));
        const uint64_t b_desc = smem_desc_k_sw128(smem_u32(b_smem + s * kBBlock));
#pragma unroll
        for (int k = 0; k < kBK / kUmmaK; ++k)
          umma_bf16(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                    (kb > 0 || k > 0) ? 1u : 0u);
        umma_commit(smem_u32(&ctl->b_empty[s]));
      }
      if (!ok) break;
      umma_commit(smem_u32(&ctl->tmem_full[buf]));
      // last unit on this worker's slab: the A buffer is free once these MMAs retire
      if (j + 1 < n_units && work.at<SUM>(j + 1).worker != p.worker) umma_commit(smem_u32(&ctl->a_empty));
    }
  } else if (FUSED && warp >= 2) {
    // ---------------- epilogue with the parameter update fused in: eight warps, two per
    // TMEM lane group.  Plain fused variant: a warp takes alternate 32-column blocks of every
    // 128-column unit (two per unit); SUM variant: its one block of every 64-column unit.
    // map_out covers x_k and map_u the momentum buffer; each warp prefetches the tiles of its
    // next two blocks with TMA while it works on the current one.
    const int ew = warp - 2, lane_group = warp & 3, half = ew >> 2;
    float* stage = reinterpret_cast<float*>(e_smem + ew * kEpiBuf);
    uint8_t* xu = xu_smem + ew * kXuPerWarp;
    const int n_blocks = n_units * kBpu;
    if (SUM && up.b_off >= 0 && work.first == 0 && n_units > 0) {
      // The bias gradient (row sums of dA^T) and its update, in the CTA that holds the first
      // column tile of its band.  The A slab changes with every unit in this variant, so the
      // rows are read from global memory: the 256 epilogue threads share the 128 rows of the
      // slice's workers among themselves before their first accumulator is ready.
      const int tid = ew * 32 + lane;
      for (int e = tid; e < work.wps * kBM; e += 8 * 32) {
        const int wi = e / kBM, row = e - wi * kBM, worker = work.slice + wi * work.slices;
        const __nv_bfloat16* rowp = up.a_ptr + (int64_t)worker * up.a_batch +
                                    (int64_t)(work.m0 + row) * up.a_ld;
        update_bias_entry(up, worker, up.b_off + work.m0 + row, slab_row_sum_global(rowp, num_kb * kBK));
      }
    }
    // block n of this warp: unit n / kBpu, column block `half` (+ 2 for the unit's second block)
    auto block_col = [&](int n) { return (half + 2 * (n % kBpu)) * 32; };
    int issued = 0;
    auto issue = [&](int n) {
      const UnitPos p = work.at<SUM>(n / kBpu);
      const int b = n & 1, col = p.col + block_col(n), row = p.m0 + lane_group * 32;
      const uint32_t bar = smem_u32(&ctl->xu_full[ew][b]);
      mbar_expect_tx(bar, up.mom ? 2 * kXuTile : kXuTile);
      tma_load_3d(smem_u32(xu + b * 2 * kXuTile), &map_out, bar, col, row, p.worker);
      if (up.mom) tma_load_3d(smem_u32(xu + b * 2 * kXuTile + kXuTile), &map_u, bar, col, row, p.worker);
      issued = n + 1;
    };
    if (lane == 0) {
      if (n_blocks > 0) issue(0);
      if (n_blocks > 1) issue(1);
    }
    // The anchor strip of a block comes straight from global memory into registers.  The
    // anchor is shared by all workers, whose CTAs reach the same strip at different times
    // while a gigabyte of read-once x and u tiles passes through L2: the loads ask L2 to
    // evict the anchor's lines last.  Plain fused variant: the strip of the next block is
    // fetched one block ahead, its latency hidden behind the update of the block before.
    // SUM variant: a CTA stays on one tile position for all workers of its slice, so the strip
    // is fetched once per position, ahead of the waits that precede its first use.
    float4 zs[8], zn[8], acc[8];   // zn: plain fused variant only; acc: SUM variant only
#pragma unroll
    for (int t = 0; t < 8; ++t) zs[t] = zn[t] = acc[t] = make_float4(0.f, 0.f, 0.f, 0.f);
    auto load_z = [&](int nn, float4 (&dst)[8]) {
      const UnitPos pz = work.at<SUM>(nn / kBpu);
      const float* zp = up.z + up.w_off + (int64_t)(pz.m0 + lane_group * 32 + (lane >> 3)) * ldw +
                        pz.col + block_col(nn) + (lane & 7) * 4;
#pragma unroll
      for (int t = 0; t < 8; ++t) dst[t] = ld_global_keep_l2(zp + (int64_t)(t * 4) * ldw);
    };
    if (!SUM && up.sync && n_blocks > 0) load_z(0, zs);
    bool ok = true;
    int n = 0;
    for (; n < n_blocks && ok; ++n) {
      const int j = n / kBpu, buf = j % kBufs, use = j / kBufs, b = n & 1;
      const UnitPos p = work.at<SUM>(j);
      if (SUM) {
        if (p.wi == 0) {
          load_z(n, zs);
#pragma unroll
          for (int t = 0; t < 8; ++t) acc[t] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
      } else if (up.sync && n + 1 < n_blocks) {
        load_z(n + 1, zn);
      }
      if (n % kBpu == 0) {
        ok = mbar_wait(smem_u32(&ctl->tmem_full[buf]), use & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
      }
      float v[32];
      tmem_ld32(tmem_base + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)(buf * kTileN + block_col(n)), v);
      const int64_t wk_off = (int64_t)p.worker * up.ld;
      const int64_t blk_off = up.w_off + (int64_t)(p.m0 + lane_group * 32) * ldw + p.col + block_col(n);
      const float* xt = reinterpret_cast<const float*>(xu + b * 2 * kXuTile);
      const float* ut = xt + kXuTile / 4;
      const uint32_t bar = smem_u32(&ctl->xu_full[ew][b]);
      const uint32_t par = (uint32_t)(n >> 1) & 1u;
      if (up.mom) {
        if (SUM || up.sync) fused_block<true, true, SUM>(v, zs, stage, xt, ut, bar, par, abort_flag, lane, up, wk_off, blk_off, ldw, acc, &ok);
        else fused_block<true, false, false>(v, zs, stage, xt, ut, bar, par, abort_flag, lane, up, wk_off, blk_off, ldw, acc, &ok);
      } else {
        if (SUM || up.sync) fused_block<false, true, SUM>(v, zs, stage, xt, ut, bar, par, abort_flag, lane, up, wk_off, blk_off, ldw, acc, &ok);
        else fused_block<false, false, false>(v, zs, stage, xt, ut, bar, par, abort_flag, lane, up, wk_off, blk_off, ldw, acc, &ok);
      }
      if (!ok) break;
      if (!SUM) {
#pragma unroll
        for (int t = 0; t < 8; ++t) zs[t] = zn[t];
      }
      __syncwarp();   // every lane has read this buffer's tiles: it may be refilled
      if (lane == 0 && n + 2 < n_blocks) issue(n + 2);
      if (n % kBpu == kBpu - 1) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[buf]));
      }
      // the slice's last worker on this position: hand in the block's partial sums
      if (SUM && p.wi == work.wps - 1) store_sum_block(acc, up, work.slice, blk_off, ldw, lane);
    }
    if (lane == 0 && n < issued) {
      // gave up early: wait (bounded) for the tiles that are still on their way
      for (int t = n; t < issued; ++t) {
        const uint32_t bar = smem_u32(&ctl->xu_full[ew][t & 1]);
        for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar, (uint32_t)(t >> 1) & 1u); ++it) {
        }
      }
    }
  } else if (warp >= 2) {
    // ---------------- epilogue: fp32 store
    const int lane_group = warp & 3;
    uint8_t* my_buf = e_smem + (warp - 2) * 2 * kEpiBuf;
    int store_count = 0;
    bool ok = true;
    for (int j = 0; j < n_units && ok; ++j) {
      const int buf = j % kBufs, use = j / kBufs;
      ok = mbar_wait(smem_u32(&ctl->tmem_full[buf]), use & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const UnitPos p = work.at<SUM>(j);
#pragma unroll 1
      for (int c = 0; c < kWN / 32; ++c) {
        float v[32];
        tmem_ld32(tmem_base + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)(buf * kWN + c * 32), v);
        uint8_t* stage = my_buf + (store_count & 1) * kEpiBuf;
        // the TMA store issued two blocks ago must have finished reading this buffer
        if (lane == 0) bulk_wait_read<1>();
        __syncwarp();
        // row = lane; 16-byte chunk q of the row goes to slot q ^ (lane % 8) (128-byte swizzle)
        float4* row = reinterpret_cast<float4*>(stage + lane * 128);
#pragma unroll
        for (int q = 0; q < 8; ++q)
          row[q ^ (lane & 7)] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          // a box that reaches past the matrix is clipped by the copy; one that lies outside
          // it altogether is not issued
          if (p.col + c * 32 < ldw && p.m0 + lane_group * 32 < ly.rows)
            tma_store_3d(&map_out, smem_u32(stage), p.col + c * 32, p.m0 + lane_group * 32, p.worker);
          bulk_commit();
        }
        ++store_count;
      }
      // this warp has read its share of the accumulator buffer
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[buf]));
    }
    if (lane == 0) bulk_wait<0>();
    __syncwarp();
  }

  // ---------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    if (lane == 0 && *abort_flag) {
      // bounded grace period for MMAs that were issued but whose commit nobody waited for
      const uint64_t t0 = global_ns();
      while (global_ns() - t0 < 1000000ull) {
      }
    }
    __syncwarp();
    tmem_dealloc(tmem_base, kBufs * kTileN);
  }
  if (threadIdx.x == 0 && *abort_flag && status) atomicExch(status, (int)OLSGD_ETIMEOUT);
}

}  // namespace

bool wgrad_tc_supported(const GemmArgs& a) {
  auto al16 = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; };
  if (a.epilogue != GEMM_EPI_STORE_F32) return false;
  if (a.Ma < 1 || a.Nb < 1 || a.K % kBK != 0 || a.K < kBK || a.K > kMaxKB * kBK) return false;
  if (a.lda % 8 || a.ldb % 8 || a.a_batch % 8 || a.b_batch % 8) return false;
  if (!al16(a.A) || !al16(a.B)) return false;
  if ((int64_t)((a.Ma + kBM - 1) / kBM) * a.m * ((a.Nb + kWN - 1) / kWN) > 0x7FFFFFFF) return false;
  if (a.upd.enabled) {
    const FusedUpdateArgs& u = a.upd;
    // the fused epilogue writes whole tiles with plain stores: no partial bands or tiles
    // (the variant that stores the gradient clips them: rows and columns past the matrix
    // are loaded as zeros and its TMA stores drop what lies outside)
    if (a.Ma % kBM != 0 || a.Nb % kWN != 0) return false;
    if (a.K > 2 * kBK) return false;   // the x/u tile ring needs the shared memory
    if (!al16(u.x_in) || !al16(u.x_out) || !al16(u.shadow) || (u.u && !al16(u.u)) ||
        (u.sync && !al16(u.z)))
      return false;
    if (u.ld % 8 || u.w_off % 8) return false;
  } else if (!al16(a.out_f) || a.ldo % 4 || a.out_batch % 4) {
    return false;
  }
  return true;
}

cudaError_t launch_wgrad_tc_batch(const GemmArgs* args, int n, cudaStream_t s) {
  if (n < 1 || n > kMaxWgradLayers) return cudaErrorInvalidValue;
  const bool fused = args[0].upd.enabled != 0;
  // the sync-step variant that also forms the worker sum and refreshes the anchor
  const bool sum = fused && args[0].upd.sum_slices > 0;
  const int num_kb = args[0].K / kBK;
  const int tile_n = sum ? 64 : kWN;
  WgradBatch wb;
  memset(&wb, 0, sizeof wb);
  wb.n_layers = n;
  int ctas = 0;
  for (int l = 0; l < n; ++l) {
    const GemmArgs& a = args[l];
    if (!wgrad_tc_supported(a) || (a.upd.enabled != 0) != fused || a.K != args[0].K ||
        a.m != args[0].m || a.status != args[0].status ||
        (fused && (a.upd.sum_slices > 0) != sum))
      return cudaErrorInvalidValue;
    if (sum && (!a.upd.sync || !a.upd.sum_part)) return cudaErrorInvalidValue;
    WgradLayer& ly = wb.layer[l];
    if (!make_map(&ly.map_a, a.A, a.K, a.Ma, a.m, a.lda, a.a_batch, kBM)) return cudaErrorInvalidValue;
    if (!make_map(&ly.map_b, a.B, a.K, a.Nb, a.m, a.ldb, a.b_batch, tile_n)) return cudaErrorInvalidValue;
    ly.map_u = ly.map_a;
    if (fused) {
      // map_out covers x_k, map_u the momentum buffer: [m][Ma][Nb] fp32 views of the weight matrix
      if (!make_map_f32(&ly.map_out, a.upd.x_in + a.upd.w_off, a.Nb, a.Ma, a.m, a.Nb, a.upd.ld, 32))
        return cudaErrorInvalidValue;
      if (a.upd.u && a.upd.mu != 0.f &&
          !make_map_f32(&ly.map_u, a.upd.u + a.upd.w_off, a.Nb, a.Ma, a.m, a.Nb, a.upd.ld, 32))
        return cudaErrorInvalidValue;
    } else if (!make_map_f32(&ly.map_out, a.out_f, a.Nb, a.Ma, a.m, a.ldo, a.out_batch, 32)) {
      return cudaErrorInvalidValue;
    }
    ly.n_tiles = (a.Nb + tile_n - 1) / tile_n;
    ly.m_tiles = (a.Ma + kBM - 1) / kBM;
    ly.ldw = a.Nb;
    ly.rows = a.Ma;
    ly.rowsum = a.rowsum_out;
    ly.rowsum_batch = a.rowsum_batch;
    ly.cta_begin = ctas;
    int64_t mine;
    if (sum) {
      // a CTA walks over the workers of one slice on each of its tile positions: about eight
      // units (128 x 64 tiles) per CTA
      const int slices = a.upd.sum_slices;
      const int wps = (a.m + slices - 1) / slices;
      int tiles_per_cta = (8 + wps / 2) / wps;
      if (tiles_per_cta < 1) tiles_per_cta = 1;
      ly.chunks = (ly.n_tiles + tiles_per_cta - 1) / tiles_per_cta;
      mine = (int64_t)ly.m_tiles * slices * ly.chunks;
    } else {
      // `chunks` CTAs share a slab and take its column tiles round-robin: about three tiles per
      // CTA.  Measured on 16 workers x (1024 x 3072) and x (1024 x 1024), and on 64 workers x
      // (512 x 3072): with fewer CTAs per slab the joint sweep over adjacent column tiles gets
      // narrower and the last partial wave of CTAs weighs more; with one or two tiles per CTA its
      // set-up (A slab, barriers, tensor memory) is no longer amortised.
      ly.chunks = ly.n_tiles / 3;
      if (ly.chunks < 1) ly.chunks = 1;
      mine = (int64_t)ly.m_tiles * a.m * ly.chunks;
    }
    if (mine + ctas > 0x7FFFFFFF) return cudaErrorInvalidValue;
    ctas += (int)mine;
    WgradUpd& up = ly.up;
    up.b_off = -1;
    up.m = a.m;
    up.slices = 1;
    if (fused) {
      up.x_in = a.upd.x_in;
      up.x_out = a.upd.x_out;
      up.u = a.upd.u;
      up.z = a.upd.z;
      up.shadow = a.upd.shadow;
      up.ld = a.upd.ld;
      up.w_off = a.upd.w_off;
      up.gamma = a.upd.gamma;
      up.mu = a.upd.mu;
      up.alpha = a.upd.alpha;
      up.mom = (a.upd.u != nullptr && a.upd.mu != 0.f) ? 1 : 0;
      up.sync = a.upd.sync;
      up.b_off = a.upd.b_off;
    }
    if (sum) {
      up.part = a.upd.sum_part;
      up.slices = a.upd.sum_slices;
      up.a_ptr = a.A;
      up.a_ld = a.lda;
      up.a_batch = a.a_batch;
    }
  }
  // shared memory: the fused variant fills an SM by itself (x/u tile rings); the plain one
  // takes as many B stages as still let two CTAs share an SM's 227 KB
  const size_t b_block = (size_t)tile_n * kBK * 2;
  const size_t fixed = (size_t)num_kb * kBM * kBK * 2 + 8 * 32 * 32 * 4 + sizeof(WgradCtl) + 1024;
  const size_t per_cta = (227 * 1024) / 2 - 1024;
  int n_stages = fixed < per_cta ? (int)((per_cta - fixed) / b_block) : 0;
  if (n_stages > kWStages) n_stages = kWStages;
  if (n_stages < 2 || fused) n_stages = 2;
  if (sum) n_stages = 4;   // 8 KB blocks: the same 32 KB ring
  const size_t smem = fixed + (size_t)n_stages * b_block + (fused ? 8 * kXuPerWarp : 0);
  static PerDeviceSmem configured[3];
  {
    const cudaError_t e = sum     ? ensure_dynamic_smem(configured[2], wgrad_tc_kernel<true, true>, smem)
                          : fused ? ensure_dynamic_smem(configured[1], wgrad_tc_kernel<true, false>, smem)
                                  : ensure_dynamic_smem(configured[0], wgrad_tc_kernel<false, false>, smem);
    if (e != cudaSuccess) return e;
  }
  g_tc_launches += 1;
  if (sum)
    return launch_chained(wgrad_tc_kernel<true, true>, dim3(ctas), dim3(kSumThreads), smem, s, wb,
                          num_kb, n_stages, args[0].status);
  if (fused)
    return launch_chained(wgrad_tc_kernel<true, false>, dim3(ctas), dim3(kFusedThreads), smem, s, wb,
                          num_kb, n_stages, args[0].status);
  return launch_chained(wgrad_tc_kernel<false, false>, dim3(ctas), dim3(kPlainThreads), smem, s, wb,
                        num_kb, n_stages, args[0].status);
}

cudaError_t launch_wgrad_tc(const GemmArgs& a, cudaStream_t s) { return launch_wgrad_tc_batch(&a, 1, s); }

int wgrad_tc_batch_limit() { return kMaxWgradLayers; }

}  // namespace olsgd
