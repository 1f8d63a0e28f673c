// Weight-gradient GEMM of the worker-batched backward pass on the tensor cores:
//   dW[i] [Ma][Nb] = A[i] [Ma][K] * B[i] [Nb][K]^T,   K = minibatch size (64..256),
// fp32 result written straight into the stacked gradient G_k (Eq. 7).
//
// The contraction is short and the output large, so the kernel is bound by the
// fp32 store.  One CTA owns a 128-row slab of one worker's dW and walks over a
// range of 128-column tiles: its A slab (128 x K bf16) is loaded once and stays
// in shared memory, B tiles stream through a small TMA ring, and the fp32
// accumulator is double-buffered in tensor memory so that the MMAs of tile j+1
// run under the epilogue of tile j.  The epilogue moves 32 x 32 blocks from
// TMEM through swizzled shared memory to global memory with TMA stores, which
// writes whole 128-byte lines.
//
// Warp roles (192 threads): warp 0 TMA loads, warp 1 MMA issue + TMEM owner,
// warps 2-5 epilogue.  Every mbarrier wait is bounded (see tc_common.cuh).
#include "tc_common.cuh"

namespace olsgd {
namespace {

using namespace tc;

constexpr int kWN = 128;            // columns per tile = MMA N
constexpr int kWStages = 4;         // upper bound of the B ring (one k-block of one tile per stage)
constexpr int kMaxKB = 4;           // K <= 256

struct WgradCtl {
  uint64_t a_full;
  uint64_t b_full[kWStages];
  uint64_t b_empty[kWStages];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

__global__ void __launch_bounds__(kThreads, 1)
wgrad_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                const __grid_constant__ CUtensorMap map_out, int num_kb, int n_stages,
                int tiles_per_cta, int* status) {
  constexpr uint32_t kABlock = kBM * kBK * 2;   // one k-block of the A slab, 16 KB
  constexpr uint32_t kBBlock = kWN * kBK * 2;   // one k-block of a B tile, 16 KB
  constexpr uint32_t kEpiBuf = 32 * 32 * 4;     // one 32 x 32 fp32 block, 4 KB

  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* a_smem = base;                                   // num_kb blocks
  uint8_t* b_smem = a_smem + num_kb * kABlock;              // n_stages blocks
  uint8_t* e_smem = b_smem + n_stages * kBBlock;            // 4 warps x 2 buffers
  WgradCtl* ctl = reinterpret_cast<WgradCtl*>(e_smem + 8 * kEpiBuf);
  volatile int* abort_flag = &ctl->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.y * kBM, worker = blockIdx.z;
  const int tile0 = blockIdx.x * tiles_per_cta;

  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&ctl->a_full), 1);
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(smem_u32(&ctl->b_full[s]), 1);
      mbar_init(smem_u32(&ctl->b_empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&ctl->tmem_full[b]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[b]), 4);   // one arrival per epilogue warp
    }
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(&ctl->tmem_base), 2 * kWN);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;

  if (warp == 0 && lane == 0) {
    // ---------------- TMA producer
    const uint32_t a_full = smem_u32(&ctl->a_full);
    mbar_expect_tx(a_full, num_kb * kABlock);
    for (int kb = 0; kb < num_kb; ++kb)
      tma_load_3d(smem_u32(a_smem + kb * kABlock), &map_a, a_full, kb * kBK, m0, worker);
    int issued = 0;
    bool ok = true;
    for (int j = 0; j < tiles_per_cta && ok; ++j) {
      for (int kb = 0; kb < num_kb; ++kb) {
        const int t = j * num_kb + kb, s = t % n_stages;
        const uint32_t ph = (t / n_stages) & 1;
        ok = mbar_wait(smem_u32(&ctl->b_empty[s]), ph ^ 1, abort_flag);
        if (!ok) break;
        const uint32_t full = smem_u32(&ctl->b_full[s]);
        mbar_expect_tx(full, kBBlock);
        tma_load_3d(smem_u32(b_smem + s * kBBlock), &map_b, full, kb * kBK, (tile0 + j) * kWN, worker);
        issued = t + 1;
      }
    }
    if (*abort_flag) {
      for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(a_full, 0); ++it) {
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
    constexpr uint32_t idesc = instr_desc_bf16(kWN);
    bool ok = mbar_wait(smem_u32(&ctl->a_full), 0, abort_flag);
    for (int j = 0; j < tiles_per_cta && ok; ++j) {
      const int buf = j & 1, use = j >> 1;
      ok = mbar_wait(smem_u32(&ctl->tmem_empty[buf]), (use & 1) ^ 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + (uint32_t)(buf * kWN);
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
      if (ok) umma_commit(smem_u32(&ctl->tmem_full[buf]));
    }
  } else if (warp >= 2) {
    // ---------------- epilogue
    const int lane_group = warp & 3;
    uint8_t* my_buf = e_smem + (warp - 2) * 2 * kEpiBuf;
    int store_count = 0;
    bool ok = true;
    for (int j = 0; j < tiles_per_cta && ok; ++j) {
      const int buf = j & 1, use = j >> 1;
      ok = mbar_wait(smem_u32(&ctl->tmem_full[buf]), use & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const int col_tile = (tile0 + j) * kWN;
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
          tma_store_3d(&map_out, smem_u32(stage), col_tile + c * 32, m0 + lane_group * 32, worker);
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
    tmem_dealloc(tmem_base, 2 * kWN);
  }
  if (threadIdx.x == 0 && *abort_flag && status) atomicExch(status, (int)OLSGD_ETIMEOUT);
}

}  // namespace

bool wgrad_tc_supported(const GemmArgs& a) {
  auto al16 = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; };
  if (a.epilogue != GEMM_EPI_STORE_F32) return false;
  if (a.Ma % kBM != 0 || a.Nb % kWN != 0 || a.K % kBK != 0 || a.K < kBK || a.K > kMaxKB * kBK)
    return false;
  if (a.lda % 8 || a.ldb % 8 || a.a_batch % 8 || a.b_batch % 8) return false;
  if (!al16(a.A) || !al16(a.B) || !al16(a.out_f) || a.ldo % 4 || a.out_batch % 4) return false;
  return true;
}

cudaError_t launch_wgrad_tc(const GemmArgs& a, cudaStream_t s) {
  if (!wgrad_tc_supported(a)) return cudaErrorInvalidValue;
  CUtensorMap ma, mb, mo;
  if (!make_map(&ma, a.A, a.K, a.Ma, a.m, a.lda, a.a_batch, kBM)) return cudaErrorInvalidValue;
  if (!make_map(&mb, a.B, a.K, a.Nb, a.m, a.ldb, a.b_batch, kWN)) return cudaErrorInvalidValue;
  if (!make_map_f32(&mo, a.out_f, a.Nb, a.Ma, a.m, a.ldo, a.out_batch, 32)) return cudaErrorInvalidValue;
  const int num_kb = a.K / kBK;
  const int n_tiles = a.Nb / kWN;
  // about two CTAs per SM in one wave: split the tile range of a slab over `chunks` CTAs
  const int slabs = (a.Ma / kBM) * a.m;
  int chunks = (2 * 148) / slabs;
  if (chunks < 1) chunks = 1;
  if (chunks > n_tiles) chunks = n_tiles;
  while (n_tiles % chunks) --chunks;
  // as many B stages as still let two CTAs share an SM's 227 KB of shared memory
  const size_t fixed = (size_t)num_kb * kBM * kBK * 2 + 8 * 32 * 32 * 4 + sizeof(WgradCtl) + 1024;
  const size_t per_cta = (227 * 1024) / 2 - 1024;
  int n_stages = fixed < per_cta ? (int)((per_cta - fixed) / (kWN * kBK * 2)) : 0;
  if (n_stages > kWStages) n_stages = kWStages;
  if (n_stages < 2) n_stages = 2;
  const size_t smem = fixed + (size_t)n_stages * kWN * kBK * 2;
  static size_t configured = 0;
  if (smem > configured) {
    cudaError_t e = cudaFuncSetAttribute(wgrad_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  dim3 grid(chunks, a.Ma / kBM, a.m);
  wgrad_tc_kernel<<<grid, kThreads, smem, s>>>(ma, mb, mo, num_kb, n_stages, n_tiles / chunks,
                                               a.status);
  return cudaGetLastError();
}

}  // namespace olsgd
