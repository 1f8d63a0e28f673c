// Worker-batched bf16 GEMM on the fifth-generation tensor cores (sm_100a):
//   D[i] = A[i] * B[i]^T,  A [Ma][K] and B [Nb][K] both K-major, fp32 accumulate.
//
// One CTA computes one 128 x BN tile of one worker's D.  Operand tiles of 64 K
// elements (128 bytes per row) are brought in by TMA with the 128-byte swizzle
// into a ring of shared-memory stages; one elected thread issues tcgen05.mma
// (M = 128, N = BN, K = 16 per instruction) with the accumulator in tensor
// memory; eight warps read the accumulator back with tcgen05.ld and run the
// epilogue (bias + ReLU, ReLU mask, or fp32 store).
//
// Warp roles (320 threads): warp 0 TMA producer, warp 1 MMA issuer and owner
// of the tensor-memory allocation, warps 2-9 epilogue (warp w reads the 32
// TMEM lanes of group w % 4; warps 2-5 take the left half of the tile's
// columns, warps 6-9 the right half: the epilogue is the serial tail of a
// CTA with one tile, and two warps per lane group halve it).
//
// Every wait on an mbarrier is bounded.  A wait that runs out raises a flag in
// shared memory that all roles poll, records OLSGD_ETIMEOUT in the status word
// the host reads, and the CTA drains its own copies, frees its tensor memory
// and returns.
#include "tc_common.cuh"

namespace olsgd {
namespace {

using namespace tc;

struct EpiArgs {
  int a_early;   // A was complete before the kernel ahead of this one started (see GemmArgs)
  int once;      // A is read once: its TMA loads carry an evict-first policy
  int epilogue;
  int Ma, Nb;
  int full;      // no partial tiles in this launch
  const float* bias;
  int64_t bias_batch;
  const __nv_bfloat16* mask;
  __nv_bfloat16* out_t;
  __nv_bfloat16* out_n;
  float* out_f;
  int64_t ldo, out_batch;
  int* status;
};

struct SharedCtl {
  uint64_t full[8];
  uint64_t empty[8];
  uint64_t tmem_full;
  uint32_t tmem_base;
  int abort_flag;
};

// The epilogue of one 128 x BN accumulator tile, run by the eight warps 2-9 of a CTA: TMEM lane
// r <-> row m0 + r, column j <-> col n0 + j.  What it needs besides the accumulator is
// fetched while the main loop runs: the row's bias, or the first 32 columns of its ReLU mask
// (the next 32 are fetched while the current ones are applied).
// FULL: every tile of the launch lies inside the matrix (Ma a multiple of 128, Nb of BN), so
// the row and column tests are compiled out.
template <int BN, bool FULL>
__device__ __forceinline__ void gemm_epilogue(const EpiArgs& ea, uint32_t tmem_base, uint32_t tmem_full_bar,
                                              volatile int* abort_flag, int warp, int lane, int m0,
                                              int n0, int worker) {
  // eight warps, two per TMEM lane group (a warp reads the lanes of group warp % 4): the
  // first four take the left half of the tile's 32-column blocks, the others the right half
  const int lane_group = warp & 3, half = (warp - 2) >> 2;
  constexpr int kBlocksPerWarp = BN / 64;
  const int c_begin = half * kBlocksPerWarp, c_end = c_begin + kBlocksPerWarp;
  const int row = m0 + lane_group * 32 + lane;
  // the last tile of a band may reach past row Ma - 1: those rows were loaded as zeros and
  // are neither looked up nor stored
  const bool live = FULL || row < ea.Ma;
  const int64_t wk = worker;
  float bias = 0.f;
  if (ea.epilogue == GEMM_EPI_BIAS_RELU && live) bias = ea.bias[wk * ea.bias_batch + row];
  uint4 mk[4], mk_next[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) mk[q] = mk_next[q] = make_uint4(0u, 0u, 0u, 0u);
  const uint4* mask_row = nullptr;
  // likewise the last column tile may reach past column Nb - 1 (Nb is a multiple of 8, the
  // width of one 16-byte piece of a row): pieces past it are neither looked up nor stored
  if (ea.epilogue == GEMM_EPI_RELU_MASK && live) {
    mask_row = reinterpret_cast<const uint4*>(ea.mask + (wk * ea.Ma + row) * ea.Nb + n0);
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (FULL || n0 + c_begin * 32 + 8 * q < ea.Nb) mk[q] = mask_row[c_begin * 4 + q];
  }
  if (mbar_wait(tmem_full_bar, 0, abort_flag) && !*abort_flag) {
    tc_fence_after();
#pragma unroll 1
    for (int c = c_begin; c < c_end; ++c) {
      if (mask_row && c + 1 < c_end) {
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (FULL || n0 + (c + 1) * 32 + 8 * q < ea.Nb) mk_next[q] = mask_row[(c + 1) * 4 + q];
      }
      float v[32];
      if (!FULL) __syncwarp();
      tmem_ld32(tmem_base + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)(c * 32), v);
      // (the load above is collective: every lane takes part in it, and meets the others
      // again at the end of the iteration)
      const int col0 = n0 + c * 32;
      const int ncols = FULL ? 32 : ea.Nb - col0;   // columns of this block inside the matrix (>= 32: all)
      if (live && ncols > 0) {
        if (ea.epilogue == GEMM_EPI_STORE_F32) {
          float4* dst = reinterpret_cast<float4*>(ea.out_f + wk * ea.out_batch +
                                                    (int64_t)row * ea.ldo + col0);
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (4 * j < ncols) dst[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
        } else {
          const int64_t t_off = (wk * ea.Ma + row) * ea.Nb + col0;
          if (ea.epilogue == GEMM_EPI_BIAS_RELU) {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j] + bias, 0.f);
          } else {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const uint4 w = mk[q];
              const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                // a bf16 is positive iff its sign bit is clear and it is not zero
                const uint32_t lo = ws[e] & 0xFFFFu, hi = ws[e] >> 16;
                if (!(lo != 0 && lo < 0x8000u)) v[q * 8 + e * 2] = 0.f;
                if (!(hi != 0 && hi < 0x8000u)) v[q * 8 + e * 2 + 1] = 0.f;
              }
              mk[q] = mk_next[q];
            }
          }
          uint32_t pk[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            __nv_bfloat162 b2 = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
            pk[j] = *reinterpret_cast<uint32_t*>(&b2);
          }
          if (ea.out_t) {
            uint4* dst = reinterpret_cast<uint4*>(ea.out_t + t_off);
#pragma unroll
            for (int q = 0; q < 4; ++q)
              if (8 * q < ncols) dst[q] = make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
          }
          if (ea.out_n) {
            // [Nb][Ma]: for a fixed column the 32 lanes of the warp write 32 consecutive rows
            __nv_bfloat16* dst = ea.out_n + (wk * ea.Nb + col0) * ea.Ma + row;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const uint32_t w = pk[j >> 1];
              const uint16_t h = (j & 1) ? (uint16_t)(w >> 16) : (uint16_t)(w & 0xFFFFu);
              if (j < ncols) *reinterpret_cast<uint16_t*>(dst + (int64_t)j * ea.Ma) = h;
            }
          }
        }
      }
      if (!FULL) __syncwarp();
    }
  }
}

template <int BN, int STAGES>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               int num_kb, int a_mn, EpiArgs ea) {
  constexpr uint32_t kABytes = kBM * kBK * 2;
  constexpr uint32_t kBBytes = BN * kBK * 2;
  constexpr uint32_t kStageBytes = kABytes + kBBytes;
  constexpr uint32_t kTmemCols = BN < 32 ? 32 : BN;  // power of two for BN in {64,128,256}

  extern __shared__ uint8_t smem_raw[];
  // operand tiles need 1024-byte alignment for the 128-byte swizzle
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                              ~static_cast<uintptr_t>(1023));
  SharedCtl* ctl = reinterpret_cast<SharedCtl*>(tiles + STAGES * kStageBytes);
  volatile int* abort_flag = &ctl->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * BN, m0 = blockIdx.y * kBM, worker = blockIdx.z;

  if (threadIdx.x == 0) {
    prefetch_tensormap(&map_a);
    prefetch_tensormap(&map_b);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    mbar_init(smem_u32(&ctl->tmem_full), 1);
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  auto load_a = [&](int kb, uint32_t a_dst, uint32_t full) {
    if (a_mn) {
      // A is stored [K][Ma]: two boxes of 64 (Ma) x 64 (K rows)
      tma_load_3d(a_dst, &map_a, full, m0, kb * kBK, worker);
      tma_load_3d(a_dst + kABytes / 2, &map_a, full, m0 + 64, kb * kBK, worker);
    } else if (ea.once) {
      tma_load_3d_once(a_dst, &map_a, full, kb * kBK, m0, worker);
    } else {
      tma_load_3d(a_dst, &map_a, full, kb * kBK, m0, worker);
    }
  };
  // Everything above touched only shared and tensor memory: it may run under the tail of
  // the kernel before this one.  So may the first loads of an A operand (weights) that the
  // kernel before this one does not write: the ring's first stages are filled with A while
  // that kernel drains, and only the B operand (its output) waits for the gate.
  const int n_early = ea.a_early ? (num_kb < STAGES ? num_kb : STAGES) : 0;
  if (warp == 0 && lane == 0) {
    for (int kb = 0; kb < n_early; ++kb) {
      const uint32_t full = smem_u32(&ctl->full[kb]);
      mbar_expect_tx(full, kStageBytes);
      load_a(kb, smem_u32(tiles + kb * kStageBytes), full);
    }
  }
  launch_gate();

  if (warp == 0 && lane == 0) {
    // ---------------- TMA producer
    int issued = n_early;
    for (int kb = 0; kb < num_kb; ++kb) {
      const int s = kb % STAGES;
      const uint32_t ph = (kb / STAGES) & 1;
      const uint32_t full = smem_u32(&ctl->full[s]);
      const uint32_t a_dst = smem_u32(tiles + s * kStageBytes);
      if (kb >= n_early) {
        if (!mbar_wait(smem_u32(&ctl->empty[s]), ph ^ 1, abort_flag)) break;
        mbar_expect_tx(full, kStageBytes);
        load_a(kb, a_dst, full);
      }
      tma_load_3d(a_dst + kABytes, &map_b, full, kb * kBK, n0, worker);
      if (kb + 1 > issued) issued = kb + 1;
    }
    if (*abort_flag) {
      // drain: wait (bounded) for the copies this thread still has in flight
      for (int kb = max(0, issued - STAGES); kb < issued; ++kb) {
        const uint32_t full = smem_u32(&ctl->full[kb % STAGES]);
        const uint32_t ph = (kb / STAGES) & 1;
        for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(full, ph); ++it) {
          if ((it & 1023u) == 1023u && global_ns() == 0) break;  // keeps the loop observable
        }
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------- MMA issuer
    const uint32_t idesc = instr_desc_bf16(BN) | (a_mn ? (1u << 15) : 0u);
    bool ok = true;
    for (int kb = 0; kb < num_kb && ok; ++kb) {
      const int s = kb % STAGES;
      const uint32_t ph = (kb / STAGES) & 1;
      ok = mbar_wait(smem_u32(&ctl->full[s]), ph, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const uint32_t a_addr = smem_u32(tiles + s * kStageBytes);
      const uint64_t a_desc = a_mn ? smem_desc_mn_sw128(a_addr) : smem_desc_k_sw128(a_addr);
      // one MMA consumes 16 K elements: 32 bytes along a K-major row, or 16 K rows of
      // 128 bytes (2048 bytes) of an MN-major tile; in 16-byte descriptor units
      const uint64_t a_step = a_mn ? 128u : 2u;
      const uint64_t b_desc = smem_desc_k_sw128(a_addr + kABytes);
#pragma unroll
      for (int k = 0; k < kBK / kUmmaK; ++k) {
        // 16 K elements = 32 bytes = 2 units of the descriptor's start address
        umma_bf16(tmem_base, a_desc + a_step * (uint64_t)k, b_desc + (uint64_t)(2 * k), idesc,
                  (kb > 0 || k > 0) ? 1u : 0u);
      }
      umma_commit(smem_u32(&ctl->empty[s]));  // stage reusable once these MMAs retire
    }
    umma_commit(smem_u32(&ctl->tmem_full));   // accumulator complete
  } else if (warp >= 2) {
    if (ea.full) gemm_epilogue<BN, true>(ea, tmem_base, smem_u32(&ctl->tmem_full), abort_flag, warp, lane, m0, n0, worker);
    else gemm_epilogue<BN, false>(ea, tmem_base, smem_u32(&ctl->tmem_full), abort_flag, warp, lane, m0, n0, worker);
  }

  // ---------------- teardown: every role arrives here, all waits above are bounded
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    if (lane == 0 && *abort_flag) {
      // let the MMAs that were issued retire before the tensor memory is released
      for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(smem_u32(&ctl->tmem_full), 0); ++it) {
      }
    }
    __syncwarp();
    tmem_dealloc(tmem_base, kTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag && ea.status) atomicExch(ea.status, (int)OLSGD_ETIMEOUT);
}

// The same GEMM on CTA pairs: the two CTAs of a cluster take two adjacent 128-row tiles of
// one worker's D and issue ONE tcgen05.mma.cta_group::2 of M = 256 per 16 K elements.  Each
// CTA still loads its own 128 rows of A, but only HALF of the B tile (the batch operand, which
// every tile of a worker needs): the operand bytes per SM and k-block drop from 16 + BN / 8 KB
// to 16 + BN / 16 KB, and delivery of operands into the SM is what bounds this kernel.
// Every CTA fetches what it holds with its own TMA loads (no multicast); the loads of both
// CTAs are counted on the full-barrier of the pair's leader (even rank), which alone issues
// the MMAs; its commits arrive on the empty- and accumulator-barriers of both CTAs.
template <int BN, int STAGES>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                    int num_kb, int a_mn, EpiArgs ea) {
  constexpr uint32_t kABytes = kBM * kBK * 2;
  constexpr uint32_t kBBytes = (BN / 2) * kBK * 2;         // this CTA's half of the B tile
  constexpr uint32_t kStageBytes = kABytes + kBBytes;
  constexpr uint32_t kTmemCols = BN < 32 ? 32 : BN;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                              ~static_cast<uintptr_t>(1023));
  SharedCtl* ctl = reinterpret_cast<SharedCtl*>(tiles + STAGES * kStageBytes);
  volatile int* abort_flag = &ctl->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // the pair lies along the grid's x dimension, which counts the 128-row tiles here
  const int m0 = blockIdx.x * kBM, n0 = blockIdx.y * BN, worker = blockIdx.z;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;

  if (threadIdx.x == 0) {
    prefetch_tensormap(&map_a);
    prefetch_tensormap(&map_b);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    mbar_init(smem_u32(&ctl->tmem_full), 1);
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // the same warp of both CTAs allocates the pair's tensor memory
  if (warp == 1) tmem_alloc_pair(smem_u32(&ctl->tmem_base), kTmemCols);
  tc_fence_before();
  __syncthreads();
  // the peer's barriers are signalled from here: they must be initialised first
  cluster_barrier();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  auto load_a = [&](int kb, uint32_t a_dst, uint32_t bar) {
    if (a_mn) {
      tma_load_3d_pair(a_dst, &map_a, bar, m0, kb * kBK, worker);
      tma_load_3d_pair(a_dst + kABytes / 2, &map_a, bar, m0 + 64, kb * kBK, worker);
    } else {
      tma_load_3d_pair(a_dst, &map_a, bar, kb * kBK, m0, worker);
    }
  };
  // weights that the kernel ahead of this one does not write are requested before the gate
  // (see gemm_tc_kernel); the leader announces both CTAs' bytes of a stage
  const int n_early = ea.a_early ? (num_kb < STAGES ? num_kb : STAGES) : 0;
  if (warp == 0 && lane == 0) {
    for (int kb = 0; kb < n_early; ++kb) {
      if (leader) mbar_expect_tx(smem_u32(&ctl->full[kb]), 2 * kStageBytes);
      load_a(kb, smem_u32(tiles + kb * kStageBytes), pair_leader_addr(smem_u32(&ctl->full[kb])));
    }
  }
  launch_gate();

  if (warp == 0 && lane == 0) {
    // ---------------- TMA producer (both CTAs)
    for (int kb = 0; kb < num_kb; ++kb) {
      const int s = kb % STAGES;
      const uint32_t ph = (kb / STAGES) & 1;
      const uint32_t full = smem_u32(&ctl->full[s]);
      const uint32_t a_dst = smem_u32(tiles + s * kStageBytes);
      if (kb >= n_early) {
        if (!mbar_wait(smem_u32(&ctl->empty[s]), ph ^ 1, abort_flag)) break;
        if (leader) mbar_expect_tx(full, 2 * kStageBytes);
        load_a(kb, a_dst, pair_leader_addr(full));
      }
      tma_load_3d_pair(a_dst + kABytes, &map_b, pair_leader_addr(full), kb * kBK,
                       n0 + (int)rank * (BN / 2), worker);
    }
    // a CTA that gave up leaves its copies to the bounded grace period below
  } else if (warp == 1 && lane == 0 && leader) {
    // ---------------- MMA issuer (leader only)
    const uint32_t idesc = instr_desc_bf16_pair(BN) | (a_mn ? (1u << 15) : 0u);
    bool ok = true;
    for (int kb = 0; kb < num_kb && ok; ++kb) {
      const int s = kb % STAGES;
      const uint32_t ph = (kb / STAGES) & 1;
      ok = mbar_wait(smem_u32(&ctl->full[s]), ph, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const uint32_t a_addr = smem_u32(tiles + s * kStageBytes);
      const uint64_t a_desc = a_mn ? smem_desc_mn_sw128(a_addr) : smem_desc_k_sw128(a_addr);
      const uint64_t a_step = a_mn ? 128u : 2u;
      const uint64_t b_desc = smem_desc_k_sw128(a_addr + kABytes);
#pragma unroll
      for (int k = 0; k < kBK / kUmmaK; ++k)
        umma_bf16_pair(tmem_base, a_desc + a_step * (uint64_t)k, b_desc + (uint64_t)(2 * k), idesc,
                       (kb > 0 || k > 0) ? 1u : 0u);
      umma_commit_pair(smem_u32(&ctl->empty[s]));   // the stage is free in both CTAs
    }
    umma_commit_pair(smem_u32(&ctl->tmem_full));    // both accumulators are complete
  } else if (warp >= 2) {
    if (ea.full) gemm_epilogue<BN, true>(ea, tmem_base, smem_u32(&ctl->tmem_full), abort_flag, warp, lane, m0, n0, worker);
    else gemm_epilogue<BN, false>(ea, tmem_base, smem_u32(&ctl->tmem_full), abort_flag, warp, lane, m0, n0, worker);
  }

  // ---------------- teardown: every role of both CTAs arrives here, all waits are bounded
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) {
    // bounded grace period for copies and MMAs that may still be in flight in the pair
    const uint64_t t0 = global_ns();
    while (global_ns() - t0 < 1000000ull) {
    }
  }
  // neither CTA's shared or tensor memory may go while the other can still reach it
  cluster_barrier();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag && ea.status) atomicExch(ea.status, (int)OLSGD_ETIMEOUT);
}

// ------------------------------------------------------------------ host side

// The column-tile width for Nb columns (a multiple of 8): the widest that divides Nb, else 64
// with a partial last tile.
int pick_bn(int Nb) {
  if (Nb % 8 != 0 || Nb < 8) return 0;
  if (Nb % 256 == 0) return 256;
  if (Nb % 128 == 0) return 128;
  return 64;
}

template <int BN, int STAGES>
cudaError_t launch_one(const GemmArgs& a, const CUtensorMap& ma, const CUtensorMap& mb,
                       cudaStream_t s) {
  constexpr size_t smem = (size_t)STAGES * (kBM * kBK * 2 + BN * kBK * 2) + sizeof(SharedCtl) + 1024;
  static PerDeviceSmem configured;
  auto kern = gemm_tc_kernel<BN, STAGES>;
  {
    const cudaError_t e = ensure_dynamic_smem(configured, kern, smem);
    if (e != cudaSuccess) return e;
  }
  EpiArgs ea;
  ea.epilogue = a.epilogue;
  ea.once = a.a_read_once;
  ea.a_early = a.a_ready_early;
  ea.Ma = a.Ma;
  ea.Nb = a.Nb;
  ea.full = (a.Ma % kBM == 0 && a.Nb % BN == 0) ? 1 : 0;
  ea.bias = a.bias;
  ea.bias_batch = a.bias_batch;
  ea.mask = a.mask;
  ea.out_t = a.out_t;
  ea.out_n = a.out_n;
  ea.out_f = a.out_f;
  ea.ldo = a.ldo;
  ea.out_batch = a.out_batch;
  ea.status = a.status;
  dim3 grid((a.Nb + BN - 1) / BN, (a.Ma + kBM - 1) / kBM, a.m);
  g_tc_launches += 1;
  return launch_chained(kern, grid, dim3(kThreads), smem, s, ma, mb, (a.K + kBK - 1) / kBK,
                        a.a_mn_major ? 1 : 0, ea);
}

template <int BN, int STAGES>
cudaError_t launch_pair(const GemmArgs& a, const CUtensorMap& ma, const CUtensorMap& mb, cudaStream_t s) {
  constexpr size_t smem = (size_t)STAGES * (kBM * kBK * 2 + (BN / 2) * kBK * 2) + sizeof(SharedCtl) + 1024;
  static PerDeviceSmem configured;
  auto kern = gemm_tc_pair_kernel<BN, STAGES>;
  {
    const cudaError_t e = ensure_dynamic_smem(configured, kern, smem);
    if (e != cudaSuccess) return e;
  }
  EpiArgs ea;
  ea.epilogue = a.epilogue;
  ea.once = a.a_read_once;
  ea.a_early = a.a_ready_early;
  ea.Ma = a.Ma;
  ea.Nb = a.Nb;
  ea.full = (a.Ma % kBM == 0 && a.Nb % BN == 0) ? 1 : 0;
  ea.bias = a.bias;
  ea.bias_batch = a.bias_batch;
  ea.mask = a.mask;
  ea.out_t = a.out_t;
  ea.out_n = a.out_n;
  ea.out_f = a.out_f;
  ea.ldo = a.ldo;
  ea.out_batch = a.out_batch;
  ea.status = a.status;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(a.Ma / kBM, a.Nb / BN, a.m);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;   // pairs of adjacent 128-row tiles
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (g_launch_overlap && !g_launch_plain) ? 2 : 1;
  g_tc_launches += 1;
  return cudaLaunchKernelEx(&cfg, kern, ma, mb, a.K / kBK, a.a_mn_major ? 1 : 0, ea);
}

// Self-test of the bounded wait: one thread waits on an mbarrier that nothing ever
// arrives on, gives up after `limit_ns` and reports OLSGD_ETIMEOUT exactly as the GEMM
// kernels do.  The context stays usable.
__global__ void wait_selftest_kernel(int* status, uint64_t limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const bool ok = mbar_wait_ns(smem_u32(&bar), 0, &abort_flag, limit_ns);
    if (!ok && status) atomicExch(status, (int)OLSGD_ETIMEOUT);
  }
}

}  // namespace

bool gemm_tc_supported(const GemmArgs& a) {
  auto al16 = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; };
  // Ma, Nb and K need not fill their last 128-row tile, column tile or 64-wide k-block: TMA
  // delivers zeros for what lies outside the operands, and the epilogue skips the rows past
  // Ma and the 16-byte pieces past Nb.  What remains are the alignment rules of the tensor
  // maps (16-byte row pitches) and Nb % 8 == 0.
  if (a.Ma < 1 || a.K < 1 || pick_bn(a.Nb) == 0) return false;
  if (a.lda % 8 || a.ldb % 8 || a.a_batch % 8 || a.b_batch % 8) return false;
  if (!al16(a.A) || !al16(a.B)) return false;
  if (a.epilogue == GEMM_EPI_STORE_F32) {
    if (!al16(a.out_f) || a.ldo % 4 || a.out_batch % 4) return false;
  } else {
    if ((a.out_t && !al16(a.out_t)) || a.Nb % 8) return false;
    if (a.epilogue == GEMM_EPI_RELU_MASK && !al16(a.mask)) return false;
  }
  return true;
}

cudaError_t launch_gemm_tc(const GemmArgs& a, cudaStream_t s) {
  if (!gemm_tc_supported(a)) return cudaErrorInvalidValue;
  const int bn = pick_bn(a.Nb);
  CUtensorMap ma, mb;
  if (a.a_mn_major) {
    // A stored [K][Ma] (Ma contiguous): 64-element boxes along Ma, 64 rows along K
    if (!make_map(&ma, a.A, a.Ma, a.K, a.m, a.lda, a.a_batch, 64)) return cudaErrorInvalidValue;
  } else if (!make_map(&ma, a.A, a.K, a.Ma, a.m, a.lda, a.a_batch, kBM)) {
    return cudaErrorInvalidValue;
  }
  // long K and an even number of 128-row tiles: CTA pairs, each CTA loading half of the B tile
  const bool pairs = g_gemm_pairs && a.K % kBK == 0 && a.K / kBK > 2 && a.Ma % (2 * kBM) == 0 &&
                     a.Nb % bn == 0 && (bn == 128 || bn == 64);
  if (pairs) {
    if (!make_map(&mb, a.B, a.K, a.Nb, a.m, a.ldb, a.b_batch, bn / 2)) return cudaErrorInvalidValue;
    return bn == 128 ? launch_pair<128, 8>(a, ma, mb, s) : launch_pair<64, 8>(a, ma, mb, s);
  }
  if (!make_map(&mb, a.B, a.K, a.Nb, a.m, a.ldb, a.b_batch, bn)) return cudaErrorInvalidValue;
  // short K (weight gradients, K = batch): few stages so several CTAs share an SM
  const bool short_k = (a.K + kBK - 1) / kBK <= 2;
  switch (bn) {
    case 256: return short_k ? launch_one<256, 2>(a, ma, mb, s) : launch_one<256, 4>(a, ma, mb, s);
    case 128: return short_k ? launch_one<128, 2>(a, ma, mb, s) : launch_one<128, 6>(a, ma, mb, s);
    default: {
      // more tiles than SMs: four stages (96 KB) so that two CTAs share an SM and the
      // whole grid is resident in one wave
      const int64_t ctas = (int64_t)((a.Nb + 63) / 64) * ((a.Ma + kBM - 1) / kBM) * a.m;
      if (short_k) return launch_one<64, 2>(a, ma, mb, s);
      return ctas > sm_count() ? launch_one<64, 4>(a, ma, mb, s) : launch_one<64, 8>(a, ma, mb, s);
    }
  }
}

cudaError_t launch_wait_selftest(int* status, uint64_t limit_ns, cudaStream_t s) {
  wait_selftest_kernel<<<1, 32, 0, s>>>(status, limit_ns);
  return cudaGetLastError();
}

}  // namespace olsgd
