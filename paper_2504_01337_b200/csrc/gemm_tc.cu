// Grouped bf16 expert GEMMs on the 5th-generation tensor cores (sm_100a): tcgen05.mma with the
// accumulator in tensor memory, operands staged in shared memory by TMA (128-byte swizzle), a
// persistent warp-specialised CTA per SM and a per-expert tile schedule built on the device from
// the routing counts (no host synchronisation between routing and the GEMMs).
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer (owns the TMEM
// allocation), warps 2..5 = epilogue (TMEM -> registers -> global, fused SwiGLU forms).
// Pipelines: smem stages (full/empty mbarriers) between producer and MMA; two TMEM accumulators
// (tmem_full/tmem_empty) between MMA and epilogue, so the epilogue of tile i overlaps the MMAs of
// tile i+1.  Every wait is bounded: on expiry the kernel raises C2R_STATUS_WAIT_TIMEOUT in the
// status word, all roles leave their loops, TMEM is released and the kernel returns.
#include "gemm.h"
#include "tc_common.cuh"

namespace c2r {

constexpr int STAGES = 4;
constexpr int A_STAGE_BYTES = BM * BK * 2;        // 16 KB
constexpr int B_STAGE_BYTES_MAX = 256 * BK * 2;   // 32 KB
constexpr int TC_THREADS = 192;
constexpr int TMEM_COLS = 512;

struct TcParams {
  int mode;        // TC_ROWS / TC_WGRAD
  int epi;         // TC_EPI_*
  int n_experts;
  int R;           // rows of the row-indexed operands
  int Mout, Nout;  // TC_WGRAD: per-expert output [Mout, Nout]; TC_ROWS: Nout = output columns (H columns for the SwiGLU forms)
  int K;           // TC_ROWS: contraction length
  int n_tiles;     // tiles along N
  int m_tiles;     // TC_WGRAD: tiles along M per expert
  int I;           // expert intermediate size (column packing of AB)
  int accumulate;
  long long ldc;   // row pitch of C (elements)
  long long sC;    // TC_WGRAD: per-expert stride of C (elements)
  const int32_t* counts;
  const int32_t* offsets;
  void* C;         // main output
  const void* AB;  // TC_EPI_SWIGLU_BWD: saved (A, B)
  void* H;         // TC_EPI_SWIGLU_FWD: H output
  int32_t* status;
};

struct TileInfo {
  int expert;   // group
  int m0;       // first output row (TC_ROWS: global row; TC_WGRAD: row inside the expert's output)
  int jn;       // tile index along N
  int kblocks;  // BK-blocks of the contraction
  int krow0;    // TC_WGRAD: first contraction row
};

// Decode linear tile id `t` for this problem.  Returns false when t is past the last tile.
__device__ __forceinline__ bool decode_tile(const TcParams& p, const int* s_off, const int* s_cnt, int total_rows_tiles,
                                            long long t, TileInfo& ti) {
  if (p.mode == TC_ROWS) {
    const long long total = (long long)total_rows_tiles * p.n_tiles;
    if (t >= total) return false;
    const int mt = (int)(t / p.n_tiles);
    ti.jn = (int)(t % p.n_tiles);
    ti.m0 = mt * BM;
    ti.kblocks = (p.K + BK - 1) / BK;
    ti.krow0 = 0;
    ti.expert = -1;
    for (int e = 0; e < p.n_experts; ++e) {
      const int lo = s_off[e], hi = lo + (s_cnt[e] + BM - 1) / BM * BM;
      if (ti.m0 >= lo && ti.m0 < hi) { ti.expert = e; break; }
    }
    return true;
  }
  const int per = p.m_tiles * p.n_tiles;
  const long long total = (long long)p.n_experts * per;
  if (t >= total) return false;
  ti.expert = (int)(t / per);
  const int r = (int)(t % per);
  ti.m0 = (r / p.n_tiles) * BM;
  ti.jn = r % p.n_tiles;
  ti.kblocks = (s_cnt[ti.expert] + BK - 1) / BK;
  ti.krow0 = s_off[ti.expert];
  return true;
}

// Width of MMA-N for N-tile jn and the first B-row / output column it covers.
template <int BN>
__device__ __forceinline__ void n_geometry(const TcParams& p, int jn, int& n_mma, int& w) {
  if (p.epi == TC_EPI_SWIGLU_FWD) {
    w = min(128, p.I - 128 * jn);
    n_mma = 2 * w;
  } else {
    w = min(BN, p.Nout - BN * jn);
    n_mma = w;
  }
}

__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void store_bf16x16(__nv_bfloat16* dst, const float* v) {
  uint4 a = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
  uint4 b = make_uint4(pack_bf16x2(v[8], v[9]), pack_bf16x2(v[10], v[11]), pack_bf16x2(v[12], v[13]),
                       pack_bf16x2(v[14], v[15]));
  reinterpret_cast<uint4*>(dst)[0] = a;
  reinterpret_cast<uint4*>(dst)[1] = b;
}
__device__ __forceinline__ void load_bf16x16(const __nv_bfloat16* src, float* v) {
  const uint4 a = reinterpret_cast<const uint4*>(src)[0];
  const uint4 b = reinterpret_cast<const uint4*>(src)[1];
  const uint32_t u[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    v[2 * i] = __uint_as_float(u[i] << 16);
    v[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
  }
}

// A_MN / B_MN: operand is MN-major in global memory (the contraction index is the row index).
template <bool A_MN, bool B_MN, int BN>
__global__ void __launch_bounds__(TC_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  constexpr int B_STAGE_BYTES = BN * BK * 2;
  // 1024-byte aligned operand stages (required by the 128-byte swizzle)
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t a_base = smem_base;
  const uint32_t b_base = smem_base + STAGES * A_STAGE_BYTES;
  __shared__ uint64_t bars[2 * STAGES + 4];
  __shared__ uint32_t tmem_slot;
  __shared__ int s_off[65];
  __shared__ int s_cnt[64];
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[STAGES]);
  const uint32_t tfull0 = smem_u32(&bars[2 * STAGES]), tempty0 = smem_u32(&bars[2 * STAGES + 2]);

  for (int i = threadIdx.x; i <= p.n_experts; i += blockDim.x) s_off[i] = p.offsets[i];
  for (int i = threadIdx.x; i < p.n_experts; i += blockDim.x) s_cnt[i] = p.counts[i];
  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull0 + 8 * b, 1); mbar_init(tempty0 + 8 * b, 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  volatile int* abort_flag = &s_abort;

  int rows_tiles = 0;
  if (p.mode == TC_ROWS) {
    int end = s_off[p.n_experts];
    if (end > p.R) end = p.R;
    rows_tiles = (end + BM - 1) / BM;
  }

  if (warp == 0) {
    // ------------------------------- TMA producer ------------------------------------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (long long t = blockIdx.x; ok; t += gridDim.x) {
        TileInfo ti;
        if (!decode_tile(p, s_off, s_cnt, rows_tiles, t, ti)) break;
        int n_mma, w;
        n_geometry<BN>(p, ti.jn, n_mma, w);
        const int brow0 = (p.epi == TC_EPI_SWIGLU_FWD) ? 256 * ti.jn : BN * ti.jn;
        for (int kb = 0; kb < ti.kblocks; ++kb) {
          if (!mbar_wait(empty0 + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t fb = full0 + 8 * stage;
          mbar_expect_tx(fb, A_STAGE_BYTES + B_STAGE_BYTES);
          const uint32_t sa = a_base + stage * A_STAGE_BYTES;
          const uint32_t sb = b_base + stage * B_STAGE_BYTES;
          if (!A_MN) {
            tma_load_2d(sa, &map_a, fb, kb * BK, ti.m0);  // [128 rows][64 k]
          } else {
            const int kr = ti.krow0 + kb * BK;
#pragma unroll
            for (int h = 0; h < BM / 64; ++h) tma_load_2d(sa + h * 8192, &map_a, fb, ti.m0 + 64 * h, kr);  // [64 k][64 m]
          }
          if (!B_MN) {
            tma_load_3d(sb, &map_b, fb, kb * BK, brow0, ti.expert);  // [BN rows][64 k] of expert's weights
          } else if (p.mode == TC_ROWS) {
#pragma unroll
            for (int h = 0; h < BN / 64; ++h)
              tma_load_3d(sb + h * 8192, &map_b, fb, brow0 + 64 * h, kb * BK, ti.expert);  // [64 k][64 n]
          } else {
            const int kr = ti.krow0 + kb * BK;
#pragma unroll
            for (int h = 0; h < BN / 64; ++h) tma_load_2d(sb + h * 8192, &map_b, fb, brow0 + 64 * h, kr);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) { *abort_flag = 1; if (p.status) atomicOr(p.status, C2R_STATUS_WAIT_TIMEOUT); }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer --------------------------------------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      uint32_t acc = 0, acc_phase = 0;
      bool ok = true;
      for (long long t = blockIdx.x; ok; t += gridDim.x) {
        TileInfo ti;
        if (!decode_tile(p, s_off, s_cnt, rows_tiles, t, ti)) break;
        if (ti.kblocks == 0) continue;  // empty contraction: the epilogue writes zeros on its own
        int n_mma, w;
        n_geometry<BN>(p, ti.jn, n_mma, w);
        const uint32_t idesc = instr_desc(n_mma, A_MN, B_MN);
        if (!mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * 256;
        for (int kb = 0; kb < ti.kblocks; ++kb) {
          if (!mbar_wait(full0 + 8 * stage, phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = a_base + stage * A_STAGE_BYTES;
          const uint32_t sb = b_base + stage * B_STAGE_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // K-major: 16 k-elements = 32 bytes inside the swizzle row; 8-row groups 1024 bytes apart.
            // MN-major: 64-element MN groups 8192 bytes apart, 8-k groups 1024 bytes apart, 16 k = 2048 bytes.
            const uint64_t da = A_MN ? smem_desc(sa + k * 2048, 8192, 1024) : smem_desc(sa + k * 32, 16, 1024);
            const uint64_t db = B_MN ? smem_desc(sb + k * 2048, 8192, 1024) : smem_desc(sb + k * 32, 16, 1024);
            tc_mma(d_tmem, da, db, idesc, (kb > 0 || k > 0) ? 1u : 0u);
          }
          tc_commit(empty0 + 8 * stage);  // frees the stage once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(tfull0 + 8 * acc);  // accumulator complete
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) { *abort_flag = 1; if (p.status) atomicOr(p.status, C2R_STATUS_WAIT_TIMEOUT); }
    }
  } else {
    // ------------------------------- epilogue ----------------------------------------------
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    uint32_t acc = 0, acc_phase = 0;
    bool ok = true;
    for (long long t = blockIdx.x; ok; t += gridDim.x) {
      TileInfo ti;
      if (!decode_tile(p, s_off, s_cnt, rows_tiles, t, ti)) break;
      int n_mma, w;
      n_geometry<BN>(p, ti.jn, n_mma, w);
      const bool have_acc = ti.kblocks > 0;
      const int row_in_tile = 32 * q + lane;
      const uint32_t taddr_row = tmem_base + acc * 256 + ((uint32_t)(32 * q) << 16);
      const int mrow = ti.m0 + row_in_tile;
      const bool row_ok = (p.mode == TC_ROWS) ? (mrow < p.R) : (mrow < p.Mout);
      if (p.epi == TC_EPI_SWIGLU_BWD) {
        // The saved (A, B) do not depend on the accumulator: four 16-column chunks of both are
        // requested at once (and the first batch before the accumulator is awaited), so a tile
        // pays two global-memory round trips instead of one per chunk.
        const __nv_bfloat16* ab = (const __nv_bfloat16*)p.AB + (long long)mrow * 2 * p.I + 256 * ti.jn;
        __nv_bfloat16* dab = (__nv_bfloat16*)p.C + (long long)mrow * 2 * p.I + 256 * ti.jn;
        bool waited = !have_acc;
        for (int c0 = 0; c0 < w; c0 += 64) {
          uint4 qa[4][2], qb[4][2];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int c = c0 + 16 * j;
            if (row_ok && c < w) {
              qa[j][0] = reinterpret_cast<const uint4*>(ab + c)[0];
              qa[j][1] = reinterpret_cast<const uint4*>(ab + c)[1];
              qb[j][0] = reinterpret_cast<const uint4*>(ab + w + c)[0];
              qb[j][1] = reinterpret_cast<const uint4*>(ab + w + c)[1];
            } else {
              qa[j][0] = qa[j][1] = qb[j][0] = qb[j][1] = make_uint4(0, 0, 0, 0);
            }
          }
          if (!waited) {
            if (!mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            waited = true;
          }
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int c = c0 + 16 * j;
            if (c >= w) break;  // warp-uniform
            uint32_t r0[16];
            float v0[16];
            if (have_acc) {
              tc_ld16(taddr_row + c, r0);
              tc_ld_wait();
#pragma unroll
              for (int i = 0; i < 16; ++i) v0[i] = __uint_as_float(r0[i]);
            } else {
#pragma unroll
              for (int i = 0; i < 16; ++i) v0[i] = 0.f;
            }
            if (!row_ok) continue;
            const uint32_t ua[8] = {qa[j][0].x, qa[j][0].y, qa[j][0].z, qa[j][0].w, qa[j][1].x, qa[j][1].y, qa[j][1].z, qa[j][1].w};
            const uint32_t ub[8] = {qb[j][0].x, qb[j][0].y, qb[j][0].z, qb[j][0].w, qb[j][1].x, qb[j][1].y, qb[j][1].z, qb[j][1].w};
            float da[16], db[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float a = __uint_as_float((i & 1) ? (ua[i >> 1] & 0xFFFF0000u) : (ua[i >> 1] << 16));
              const float b = __uint_as_float((i & 1) ? (ub[i >> 1] & 0xFFFF0000u) : (ub[i >> 1] << 16));
              const float s = 1.0f / (1.0f + __expf(-a));
              da[i] = v0[i] * b * (s * (1.0f + a * (1.0f - s)));
              db[i] = v0[i] * (a * s);
            }
            store_bf16x16(dab + c, da);
            store_bf16x16(dab + w + c, db);
          }
        }
        if (!ok) break;
        if (have_acc) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
          if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        continue;
      }
      if (have_acc) {
        if (!mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag)) { ok = false; break; }
        tc_fence_after();
      }
      for (int c = 0; c < w; c += 16) {
        uint32_t r0[16], r1[16];
        float v0[16], v1[16];
        if (have_acc) {
          tc_ld16(taddr_row + c, r0);
          if (p.epi == TC_EPI_SWIGLU_FWD) tc_ld16(taddr_row + w + c, r1);
          tc_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) { v0[i] = __uint_as_float(r0[i]); v1[i] = __uint_as_float(r1[i]); }
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) { v0[i] = 0.f; v1[i] = 0.f; }
        }
        if (!row_ok) continue;
        if (p.epi == TC_EPI_SWIGLU_FWD) {
          const int pg = 256 * ti.jn + c, pu = pg + w;
          __nv_bfloat16* ab = (__nv_bfloat16*)p.C + (long long)mrow * 2 * p.I;
          store_bf16x16(ab + pg, v0);
          store_bf16x16(ab + pu, v1);
          float h[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) h[i] = v0[i] / (1.0f + __expf(-v0[i])) * v1[i];
          store_bf16x16((__nv_bfloat16*)p.H + (long long)mrow * p.I + 128 * ti.jn + c, h);
        } else if (p.epi == TC_EPI_F32) {
          float* o = (float*)p.C + (long long)mrow * p.ldc + BN * ti.jn + c;
#pragma unroll
          for (int i = 0; i < 4; ++i)
            reinterpret_cast<float4*>(o)[i] = make_float4(v0[4 * i], v0[4 * i + 1], v0[4 * i + 2], v0[4 * i + 3]);
        } else {  // TC_EPI_WGRAD_BF16
          __nv_bfloat16* o = (__nv_bfloat16*)p.C + (long long)ti.expert * p.sC + (long long)mrow * p.ldc + BN * ti.jn + c;
          if (p.accumulate) {
            float old[16];
            load_bf16x16(o, old);
#pragma unroll
            for (int i = 0; i < 16; ++i) v0[i] += old[i];
          }
          store_bf16x16(o, v0);
        }
      }
      if (have_acc) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
    if (!ok && lane == 0) { *abort_flag = 1; if (p.status) atomicOr(p.status, C2R_STATUS_WAIT_TIMEOUT); }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
template <bool A_MN, bool B_MN, int BN>
static int launch(const CUtensorMap& ma, const CUtensorMap& mb, const TcParams& p, cudaStream_t s) {
  constexpr int smem = STAGES * (A_STAGE_BYTES + BN * BK * 2) + 1024;
  static bool configured = false;
  if (!configured) {
    C2R_CUDA(cudaFuncSetAttribute(tc_gemm_kernel<A_MN, B_MN, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    configured = true;
  }
  tc_gemm_kernel<A_MN, B_MN, BN><<<sm_count(), TC_THREADS, smem, s>>>(ma, mb, p);
  C2R_LAUNCH_CHECK();
  return C2R_OK;
}

bool tc_supported(const c2r_config* cfg, int nE, int I, int64_t R) {
  // TMA needs 16-byte row pitches; MMA-N needs multiples of 16; with several experts every
  // segment must start on an M-tile boundary so that no tile straddles two experts.
  return cfg->dtype == C2R_BF16 && cfg->d % 16 == 0 && I % 16 == 0 && R < (1ll << 31) &&
         (nE == 1 || cfg->row_align % BM == 0) && get_encode() != nullptr;
}

int tc_swiglu_fwd(const c2r_config* cfg, int nE, int I, int64_t R, const void* Xp, const int32_t* counts,
                  const int32_t* offsets, const void* W13p, const void* W2, void* AB, void* H, void* Yp,
                  int32_t* status, cudaStream_t s) {
  const int d = cfg->d;
  CUtensorMap ma, mb;
  TcParams p{};
  p.mode = TC_ROWS; p.n_experts = nE; p.R = (int)R; p.I = I; p.counts = counts; p.offsets = offsets; p.status = status;
  // (A | B) = Xp W13p^T with the SwiGLU epilogue: AB packed + H
  int rc = make_map(&ma, Xp, d, R, 0, BK, BM);
  if (rc) return rc;
  rc = make_map(&mb, W13p, d, 2 * I, nE, BK, 256);
  if (rc) return rc;
  p.epi = TC_EPI_SWIGLU_FWD; p.K = d; p.Nout = I; p.n_tiles = (I + 127) / 128; p.C = AB; p.H = H;
  rc = launch<false, false, 256>(ma, mb, p, s);
  if (rc) return rc;
  // Yp = H W2^T (fp32)
  rc = make_map(&ma, H, I, R, 0, BK, BM);
  if (rc) return rc;
  rc = make_map(&mb, W2, I, d, nE, BK, 256);
  if (rc) return rc;
  p.epi = TC_EPI_F32; p.K = I; p.Nout = d; p.n_tiles = (d + 255) / 256; p.C = Yp; p.ldc = d; p.H = nullptr;
  return launch<false, false, 256>(ma, mb, p, s);
}

int tc_swiglu_bwd(const c2r_config* cfg, int nE, int I, int64_t R, const void* Xp, const int32_t* counts,
                  const int32_t* offsets, const void* W13p, const void* W2, const void* AB, const void* H,
                  const void* dYp, void* dAB, void* dXp, void* dW13p, void* dW2, int accumulate, int32_t* status,
                  cudaStream_t s) {
  const int d = cfg->d;
  CUtensorMap ma, mb;
  TcParams p{};
  p.n_experts = nE; p.R = (int)R; p.I = I; p.counts = counts; p.offsets = offsets; p.status = status;
  // dH = dYp W2 -> (dA | dB) packed
  p.mode = TC_ROWS;
  int rc = make_map(&ma, dYp, d, R, 0, BK, BM);
  if (rc) return rc;
  rc = make_map(&mb, W2, I, d, nE, 64, 64);  // W2_e is [d (k)][I (n)]: MN-major B
  if (rc) return rc;
  p.epi = TC_EPI_SWIGLU_BWD; p.K = d; p.Nout = I; p.n_tiles = (I + 127) / 128; p.C = dAB; p.AB = AB;
  rc = launch<false, true, 128>(ma, mb, p, s);
  if (rc) return rc;
  // dXp = dAB W13p (fp32)
  rc = make_map(&ma, dAB, 2 * I, R, 0, BK, BM);
  if (rc) return rc;
  rc = make_map(&mb, W13p, d, 2 * I, nE, 64, 64);  // W13p_e is [2I (k)][d (n)]: MN-major B
  if (rc) return rc;
  p.epi = TC_EPI_F32; p.K = 2 * I; p.Nout = d; p.n_tiles = (d + 255) / 256; p.C = dXp; p.ldc = d; p.AB = nullptr;
  rc = launch<false, true, 256>(ma, mb, p, s);
  if (rc) return rc;
  // dW2_e = dYp_e^T H_e  [d, I]
  p.mode = TC_WGRAD; p.epi = TC_EPI_WGRAD_BF16; p.accumulate = accumulate;
  rc = make_map(&ma, dYp, d, R, 0, 64, 64);
  if (rc) return rc;
  rc = make_map(&mb, H, I, R, 0, 64, 64);
  if (rc) return rc;
  p.Mout = d; p.Nout = I; p.m_tiles = (d + BM - 1) / BM; p.n_tiles = (I + 255) / 256;
  p.C = dW2; p.ldc = I; p.sC = (long long)d * I;
  rc = launch<true, true, 256>(ma, mb, p, s);
  if (rc) return rc;
  // dW13p_e = dAB_e^T Xp_e  [2I, d]
  rc = make_map(&ma, dAB, 2 * I, R, 0, 64, 64);
  if (rc) return rc;
  rc = make_map(&mb, Xp, d, R, 0, 64, 64);
  if (rc) return rc;
  p.Mout = 2 * I; p.Nout = d; p.m_tiles = (2 * I + BM - 1) / BM; p.n_tiles = (d + 255) / 256;
  p.C = dW13p; p.ldc = d; p.sC = (long long)2 * I * d;
  return launch<true, true, 256>(ma, mb, p, s);
}

}  // namespace c2r
