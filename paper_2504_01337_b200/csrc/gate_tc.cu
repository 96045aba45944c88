// Gate logits (Eq. 1) for bf16 hidden states on the tensor cores: L = X Wg^T and z = X wsg.
//
// The product is HBM-bound (X is read once, E <= 64 output columns), so the kernel is a streaming
// one: a CTA owns 128-token tiles, TMA brings [128 x 64] blocks of X and the matching [64 x 64]
// block of Wg (rows >= E are zero-filled by the tensor map) and [16 x 64] block of wsg (row 0 is
// the vector, rows 1..15 zero fill) through an 8-stage ring, one thread issues one tcgen05 MMA per
// 16 k-elements (N = 64 for the routed gate, N = 80 when the shared-expert gate's block rides along) into tensor
// memory, and four warps write the fp32 accumulators out.  Waits are bounded like in the grouped
// GEMM kernel.
#include "gemm.h"
#include "tc_common.cuh"

namespace c2r {

constexpr int GT_STAGES = 8;
constexpr int GT_X_BYTES = BM * BK * 2;    // 16 KB
constexpr int GT_W_BYTES = 64 * BK * 2;    //  8 KB
constexpr int GT_S_BYTES = 16 * BK * 2;    //  2 KB
constexpr int GT_STAGE_BYTES = GT_X_BYTES + GT_W_BYTES + GT_S_BYTES;
constexpr int GT_THREADS = 192;
constexpr int GT_TMEM_COLS = 256;          // two accumulators of 128 columns (64 logits | 16 shared gate | unused)

__global__ void __launch_bounds__(GT_THREADS, 1)
gate_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
               const __grid_constant__ CUtensorMap map_s, float* __restrict__ L, float* __restrict__ z, int N, int d,
               int E, int has_shared, int32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  __shared__ uint64_t bars[2 * GT_STAGES + 4];
  __shared__ uint32_t tmem_slot;
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[GT_STAGES]);
  const uint32_t tfull0 = smem_u32(&bars[2 * GT_STAGES]), tempty0 = smem_u32(&bars[2 * GT_STAGES + 2]);
  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < GT_STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull0 + 8 * b, 1); mbar_init(tempty0 + 8 * b, 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                 "r"(GT_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  volatile int* abort_flag = &s_abort;

  const int tiles = (N + BM - 1) / BM;
  const int kblocks = (d + BK - 1) / BK;
  const int n_mma = (E + 15) / 16 * 16;  // MMA-N of the routed gate
  const uint32_t tx_bytes = GT_X_BYTES + GT_W_BYTES + (has_shared ? GT_S_BYTES : 0);

  if (warp == 0) {
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x) {
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(empty0 + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t fb = full0 + 8 * stage;
          const uint32_t sx = smem_base + stage * GT_STAGE_BYTES;
          mbar_expect_tx(fb, tx_bytes);
          tma_load_2d(sx, &map_x, fb, kb * BK, t * BM);
          tma_load_2d(sx + GT_X_BYTES, &map_w, fb, kb * BK, 0);
          if (has_shared) tma_load_2d(sx + GT_X_BYTES + GT_W_BYTES, &map_s, fb, kb * BK, 0);
          if (++stage == GT_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) { *abort_flag = 1; if (status) atomicOr(status, C2R_STATUS_WAIT_TIMEOUT); }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
      // with a shared gate, its [16 x 64] block follows the [64 x 64] block of Wg in shared memory (same 128-byte
      // swizzle rows), so one MMA of N = 80 covers both: accumulator columns 0..63 logits, 64 the shared gate
      const uint32_t idesc_w = instr_desc(has_shared ? 80 : n_mma, false, false);
      bool ok = true;
      for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x) {
        if (!mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * 128;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(full0 + 8 * stage, phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sx = smem_base + stage * GT_STAGE_BYTES;
          const uint32_t sw = sx + GT_X_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t da = smem_desc(sx + k * 32, 16, 1024);
            const uint32_t accum = (kb > 0 || k > 0) ? 1u : 0u;
            tc_mma(d_tmem, da, smem_desc(sw + k * 32, 16, 1024), idesc_w, accum);
          }
          tc_commit(empty0 + 8 * stage);
          if (++stage == GT_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(tfull0 + 8 * acc);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) { *abort_flag = 1; if (status) atomicOr(status, C2R_STATUS_WAIT_TIMEOUT); }
    }
  } else {
    const int q = warp & 3;
    uint32_t acc = 0, acc_phase = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x) {
      if (!mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + acc * 128 + ((uint32_t)(32 * q) << 16);
      const long long tok = (long long)t * BM + 32 * q + lane;
      for (int c = 0; c < n_mma; c += 16) {
        uint32_t r[16];
        tc_ld16(taddr + c, r);
        tc_ld_wait();
        if (tok < N) {
          float* o = L + tok * E + c;
          if ((E & 3) == 0) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
              if (c + 4 * i < E)
                reinterpret_cast<float4*>(o)[i] = make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]),
                                                              __uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i)
              if (c + i < E) o[i] = __uint_as_float(r[i]);
          }
        }
      }
      if (has_shared) {
        uint32_t r[16];
        tc_ld16(taddr + 64, r);
        tc_ld_wait();
        if (tok < N) z[tok] = __uint_as_float(r[0]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (!ok && lane == 0) { *abort_flag = 1; if (status) atomicOr(status, C2R_STATUS_WAIT_TIMEOUT); }
  }

  // after a wait gave up, let TMA loads still in flight land before the CTA (and its shared memory) goes away
  __syncthreads();
  if (*abort_flag)
    for (int i = 0; i < 128; ++i) __nanosleep(2000);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(GT_TMEM_COLS) : "memory");
  }
}

bool gate_tc_supported(const c2r_config* cfg) {
  return cfg->dtype == C2R_BF16 && cfg->E <= 64 && cfg->d % 8 == 0 && cfg->N > 0 && get_encode() != nullptr;
}

int gate_tc_launch(const c2r_config* cfg, const void* X, const void* Wg, const void* wsg, float* L, float* z,
                   int32_t* status, cudaStream_t s) {
  CUtensorMap mx, mw, ms;
  int rc = make_map(&mx, X, cfg->d, cfg->N, 0, BK, BM);
  if (rc) return rc;
  rc = make_map(&mw, Wg, cfg->d, cfg->E, 0, BK, 64);
  if (rc) return rc;
  rc = make_map(&ms, wsg ? wsg : Wg, cfg->d, 1, 0, BK, 16);
  if (rc) return rc;
  constexpr int smem = GT_STAGES * GT_STAGE_BYTES + 1024;
  constexpr int MAX_DEV = 64;
  static int sms_of_device[MAX_DEV] = {};  // SM count, also "the kernel's shared-memory limit is set on this device"
  int dev = 0;
  C2R_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= MAX_DEV) return C2R_ERR_UNSUPPORTED_SHAPE;
  int sms = __atomic_load_n(&sms_of_device[dev], __ATOMIC_ACQUIRE);
  if (sms == 0) {
    C2R_CUDA(cudaFuncSetAttribute(gate_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    C2R_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    __atomic_store_n(&sms_of_device[dev], sms, __ATOMIC_RELEASE);
  }
  const int tiles = (cfg->N + BM - 1) / BM;
  const int grid = tiles < sms ? tiles : sms;
  gate_tc_kernel<<<grid, GT_THREADS, smem, s>>>(mx, mw, ms, L, z, cfg->N, cfg->d, cfg->E, wsg != nullptr, status);
  C2R_LAUNCH_CHECK();
  return C2R_OK;
}

}  // namespace c2r
