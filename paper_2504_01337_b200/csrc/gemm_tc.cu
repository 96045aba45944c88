// Grouped bf16 expert GEMMs on the 5th-generation tensor cores (sm_100a).
//
// Two CTAs of a cluster (a CTA pair on neighbouring SMs) compute one 256 x 256 output tile with
// tcgen05.mma.cta_group::2: each CTA stages 128 rows of A and half of B's rows in its own shared
// memory (TMA, 128-byte swizzle, no multicast), so every SM reads 32 KB of operands per 64
// k-elements instead of the 48 KB a single-CTA 128 x 256 tile needs, and each CTA keeps the
// accumulator rows of its own 128 A rows in its tensor memory.  The kernel is persistent (one
// pair per two SMs) and walks a per-expert tile schedule decoded on the device from the routing
// counts, so no host synchronisation separates routing from the GEMMs.
//
// Warp roles (320 threads per CTA): warp 0 = TMA producer (both CTAs, each for its own halves),
// warp 1 = MMA issuer (even CTA only; owns the TMEM allocation in both), warps 2..9 = epilogue
// (TMEM -> registers -> a per-warp staging tile in shared memory -> global, row-contiguously; fused
// SwiGLU forms; two warps per TMEM lane quarter).
// Pipelines: 5 shared-memory stages (full barrier in the even CTA counts both CTAs' bytes; the
// MMA's commit frees the stage in both CTAs) and two TMEM accumulators of 256 columns, so the
// epilogue of tile i overlaps the MMAs of tile i+1.  Every wait is bounded: on expiry the kernel
// raises C2R_STATUS_WAIT_TIMEOUT in the status word, the roles leave their loops, both CTAs meet
// at the cluster barrier, TMEM is released and the kernel returns.
#include "gemm.h"
#include "tc_common.cuh"

namespace c2r {

constexpr int STAGES = 5;
constexpr int HALF_BYTES = 128 * BK * 2;          // one CTA's share of either operand per stage: 16 KB
constexpr int STAGE_BYTES = 2 * HALF_BYTES;       // A half + B half
constexpr int TC_THREADS = 320;
constexpr int EPI_WARPS = 8;
constexpr int TMEM_COLS = 512;
constexpr int STG_BYTES = 32 * 128;                // a warp's staging tile: 32 rows x 128 bytes
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_WARPS * 2 * STG_BYTES + 1024;
constexpr int TILE_M = 256;                       // rows of a pair tile (128 per CTA)
constexpr int TILE_N = 256;                       // widest MMA-N

struct TcParams {
  int mode;        // TC_ROWS / TC_WGRAD
  int epi;         // TC_EPI_*
  int n_experts;
  int R;           // rows of the row-indexed operands
  int Mout, Nout;  // TC_WGRAD: per-expert output [Mout, Nout]; TC_ROWS: Nout = output columns (H columns for the SwiGLU forms)
  int K;           // TC_ROWS: contraction length
  int n_tiles;     // tiles along N
  int m_tiles;     // TC_WGRAD: pair tiles along M per expert
  int I;           // expert intermediate size (column packing of AB)
  int accumulate;
  long long ldc;   // row pitch of C (elements)
  long long sC;    // TC_WGRAD: per-expert stride of C (elements)
  const int32_t* counts;
  const int32_t* offsets;
  void* C;         // main output
  const void* AB;  // TC_EPI_SWIGLU_BWD: the two local derivatives the forward pass saved
  void* H;         // TC_EPI_SWIGLU_FWD: H output; TC_EPI_SWIGLU_BWD: the forward's H (read for the row dots), may be NULL
  int32_t* status;
  // per-row scale of H (SwiGLU forms): H = s_r silu(A) B, s_r = row_scale[r] (kind 1) or sigmoid(row_scale[r]) (kind 2)
  const float* row_scale;
  int scale_kind;
  float* qpart;    // TC_EPI_SWIGLU_BWD: [2 * n_tiles][R] partial row dots <dH_r, H_r>, or NULL
  float* token_acc;  // TC_EPI_F32: add row r into token_acc[slot_of_row[r] / slots_per_token, :] instead of storing it
  // row-gathering variants: the operand's rows are token rows of X picked through slot_of_row
  const int32_t* slot_of_row;  // [R], -1 = padding (reads zeros)
  int slots_per_token;         // K of the routing
  int n_tokens;                // rows of X
};

struct TileInfo {
  int expert;   // group
  int m0;       // first output row of the pair tile (TC_ROWS: global row; TC_WGRAD: row inside the expert's output)
  int m_end;    // rows at or beyond it are not this tile's to write (end of the expert's 128-aligned segment / Mout)
  int jn;       // tile index along N
  int kblocks;  // BK-blocks of the contraction
  int krow0;    // TC_WGRAD: first contraction row
};

// Decode linear tile id `t`.  s_pt[e] = number of pair tiles of the experts before e (TC_ROWS).
// Returns false when t is past the last tile.  e_hint: the expert of the tile this role decoded last (a role walks
// its tiles in increasing order, so the search for the expert resumes there instead of starting at expert 0).
__device__ __forceinline__ bool decode_tile(const TcParams& p, const int* s_off, const int* s_cnt, const int* s_pt,
                                            long long t, TileInfo& ti, int& e_hint) {
  if (p.mode == TC_ROWS) {
    const long long total = (long long)s_pt[p.n_experts] * p.n_tiles;
    if (t >= total) return false;
    const int mp = (int)(t / p.n_tiles);
    ti.jn = (int)(t % p.n_tiles);
    int e = (e_hint < p.n_experts && s_pt[e_hint] <= mp) ? e_hint : 0;
    while (e + 1 < p.n_experts && s_pt[e + 1] <= mp) ++e;
    e_hint = e;
    ti.expert = e;
    ti.m0 = s_off[e] + TILE_M * (mp - s_pt[e]);
    ti.m_end = min(p.R, s_off[e] + (s_cnt[e] + BM - 1) / BM * BM);
    ti.kblocks = (p.K + BK - 1) / BK;
    ti.krow0 = 0;
    return true;
  }
  const int per = p.m_tiles * p.n_tiles;
  const long long total = (long long)p.n_experts * per;
  if (t >= total) return false;
  ti.expert = (int)(t / per);
  const int r = (int)(t % per);
  ti.m0 = (r / p.n_tiles) * TILE_M;
  ti.m_end = p.Mout;
  ti.jn = r % p.n_tiles;
  ti.kblocks = (s_cnt[ti.expert] + BK - 1) / BK;
  ti.krow0 = s_off[ti.expert];
  return true;
}

// MMA-N of N-tile jn, the first B row (= n index of accumulator column 0) it covers, and the
// number of output columns w the epilogue walks (SwiGLU forward: w gate + w up columns).
__device__ __forceinline__ void n_geometry(const TcParams& p, int jn, int& n_mma, int& w, int& brow0) {
  if (p.epi == TC_EPI_SWIGLU_FWD) {
    w = min(128, p.I - 128 * jn);
    n_mma = 2 * w;
    brow0 = 256 * jn;
  } else {
    w = min(TILE_N, p.Nout - TILE_N * jn);
    n_mma = w;
    brow0 = TILE_N * jn;
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
__device__ __forceinline__ void unpack_bf16x16(const uint4& a, const uint4& b, float* v) {
  const uint32_t u[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    v[2 * i] = __uint_as_float(u[i] << 16);
    v[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ void load_bf16x16(const __nv_bfloat16* src, float* v) {
  unpack_bf16x16(reinterpret_cast<const uint4*>(src)[0], reinterpret_cast<const uint4*>(src)[1], v);
}

__device__ __forceinline__ uint4 pack_bf16x8(const float* v) {
  return make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
}

// ---- warp-private staging tiles ---------------------------------------------------------------
// 32 rows x 128 bytes.  The 16-byte chunks of a row are permuted by (chunk ^ (row & 7)), which
// keeps both access patterns free of bank conflicts: "row per lane" (what a TMEM load gives a
// thread) and "row contiguous" (8 lanes cover the 128 bytes of one row, 4 rows per instruction:
// the coalesced shape for global memory).
__device__ __forceinline__ uint32_t stg_addr(uint32_t buf, int row, int chunk) {
  return buf + row * 128 + ((chunk ^ (row & 7)) << 4);
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
  return v;
}
// Staging tile -> global rows [0, rows_valid) x bytes [0, valid_bytes) starting at g (row pitch in bytes).
__device__ __forceinline__ void stage_to_global(uint32_t buf, uint8_t* g, long long pitch, int rows_valid, int valid_bytes,
                                                int lane) {
  const int chunk = lane & 7, sub = lane >> 3;
  if (16 * chunk >= valid_bytes) return;
#pragma unroll
  for (int it = 0; it < 8; ++it) {
    const int row = 4 * it + sub;
    if (row < rows_valid) *reinterpret_cast<uint4*>(g + row * pitch + 16 * chunk) = lds128(stg_addr(buf, row, chunk));
  }
}
// Staging tile (fp32) -> added into rows of an fp32 array starting at g (row pitch in bytes): the row of the tile
// held by lane l goes to row tok_mine of lane l; a negative token skips the row.  Vector reductions of 16 bytes,
// 4 rows x 128 bytes per instruction.  Every lane of the warp must call.
__device__ __forceinline__ void stage_red_to_rows(uint32_t buf, uint8_t* g, long long pitch, int tok_mine, int valid_bytes,
                                                  int lane) {
  const int chunk = lane & 7, sub = lane >> 3;
#pragma unroll
  for (int it = 0; it < 8; ++it) {
    const int row = 4 * it + sub;
    const int tok = __shfl_sync(0xffffffffu, tok_mine, row);
    if (tok >= 0 && 16 * chunk < valid_bytes) {
      const uint4 v = lds128(stg_addr(buf, row, chunk));
      asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(g + (long long)tok * pitch + 16 * chunk),
                   "f"(__uint_as_float(v.x)), "f"(__uint_as_float(v.y)), "f"(__uint_as_float(v.z)), "f"(__uint_as_float(v.w))
                   : "memory");
    }
  }
}
// Global rows [0, rows_valid) x bytes [0, valid_bytes) -> staging tile, asynchronously (16-byte cp.async per lane and
// row, no registers involved); zeros elsewhere.  Complete after async_copies_wait() + __syncwarp().
__device__ __forceinline__ void global_rows_to_stage_async(uint32_t buf, const uint8_t* g, long long pitch, int rows_valid,
                                                           int valid_bytes, int lane) {
  const int chunk = lane & 7, sub = lane >> 3;
#pragma unroll
  for (int it = 0; it < 8; ++it) {
    const int row = 4 * it + sub;
    const bool live = row < rows_valid && 16 * chunk < valid_bytes;
    const uint8_t* src = live ? g + row * pitch + 16 * chunk : g;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(stg_addr(buf, row, chunk)), "l"(src),
                 "r"(live ? 16 : 0)
                 : "memory");
  }
}
__device__ __forceinline__ void async_copies_wait() {
  asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}
// Global rows [0, rows_valid) x bytes [0, valid_bytes) -> registers in the row-contiguous shape
// (v[it] = chunk (lane & 7) of row 4*it + (lane >> 3)); zeros elsewhere.
__device__ __forceinline__ void global_rows_load(uint4 (&v)[8], const uint8_t* g, long long pitch, int rows_valid,
                                                 int valid_bytes, int lane) {
  const int chunk = lane & 7, sub = lane >> 3;
#pragma unroll
  for (int it = 0; it < 8; ++it) {
    const int row = 4 * it + sub;
    v[it] = (row < rows_valid && 16 * chunk < valid_bytes)
                ? *reinterpret_cast<const uint4*>(g + row * pitch + 16 * chunk)
                : make_uint4(0, 0, 0, 0);
  }
}
__device__ __forceinline__ void stage_rows_store(uint32_t buf, const uint4 (&v)[8], int lane) {
  const int chunk = lane & 7, sub = lane >> 3;
#pragma unroll
  for (int it = 0; it < 8; ++it) sts128(stg_addr(buf, 4 * it + sub, chunk), v[it]);
}

// Token rows behind four consecutive rows r..r+3 of the permuted layout (r a multiple of 4): slot / K, and an
// out-of-range row (-> zero fill) for padding or rows past the layout.
__device__ __forceinline__ int4 gather_rows(const TcParams& p, int r) {
  int4 s = make_int4(-1, -1, -1, -1);
  if (r >= 0 && r + 3 < p.R) s = *reinterpret_cast<const int4*>(p.slot_of_row + r);
  const int K = p.slots_per_token, oob = p.n_tokens;
  return make_int4(s.x < 0 ? oob : s.x / K, s.y < 0 ? oob : s.y / K, s.z < 0 ? oob : s.z / K, s.w < 0 ? oob : s.w / K);
}

// Scale of row r (see TcParams::row_scale); rows that do not exist get 0.
__device__ __forceinline__ float row_scale_of(const TcParams& p, long long r, bool valid) {
  if (p.scale_kind == 0 || p.row_scale == nullptr) return 1.f;
  if (!valid) return 0.f;
  const float v = p.row_scale[r];
  return p.scale_kind == 2 ? 1.0f / (1.0f + expf(-v)) : v;
}

// A_MN / B_MN: operand is MN-major in global memory (the contraction index is the row index).
// GATHER: 0 = both operands are plain arrays; 1 = A's rows (TC_ROWS, K-major) are token rows gathered from X;
// 2 = B's contraction rows (TC_WGRAD, MN-major) are token rows gathered from X.  map_a / map_b is then the
// one-row-box map of X, and the permuted copy of X is never needed.
// EPI: the epilogue (TC_EPI_*), a template parameter so that every form gets its own register allocation.
template <bool A_MN, bool B_MN, int GATHER, int EPI>
__global__ void __launch_bounds__(TC_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte aligned operand stages (required by the 128-byte swizzle); same offsets in both CTAs
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  __shared__ uint64_t bars[2 * STAGES + 4];
  __shared__ uint32_t tmem_slot;
  __shared__ int s_off[65];
  __shared__ int s_cnt[64];
  __shared__ int s_pt[65];
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = the CTA that issues the MMAs
  const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[STAGES]);
  const uint32_t tfull0 = smem_u32(&bars[2 * STAGES]), tempty0 = smem_u32(&bars[2 * STAGES + 2]);

  for (int i = threadIdx.x; i <= p.n_experts; i += blockDim.x) s_off[i] = p.offsets[i];
  for (int i = threadIdx.x; i < p.n_experts; i += blockDim.x) s_cnt[i] = p.counts[i];
  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull0 + 8 * b, 1); mbar_init(tempty0 + 8 * b, 2 * EPI_WARPS); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = 0;
    for (int e = 0; e < p.n_experts; ++e) {
      s_pt[e] = run;
      const int rows = min(s_cnt[e], max(p.R - s_off[e], 0));
      run += (rows + TILE_M - 1) / TILE_M;
    }
    s_pt[p.n_experts] = run;
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers are initialised before anything can arrive on them
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  volatile int* abort_flag = &s_abort;
  const long long pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (warp == 0) {
    // ------------------------------- TMA producer (each CTA loads its own halves) ----------
    if constexpr (GATHER == 0) {
      // plain operands: one thread waits for a free stage and issues the 2 to 4 tiled loads of a k-block
      if (lane == 0) {
        const uint32_t full_mma0 = map_to_cta(full0, 0);  // completion bytes are counted where the MMAs are issued
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        int e_hint = 0;
        for (long long t = pair_id; ok; t += n_pairs) {
          TileInfo ti;
          if (!decode_tile(p, s_off, s_cnt, s_pt, t, ti, e_hint)) break;
          int n_mma, w, brow0;
          n_geometry(p, ti.jn, n_mma, w, brow0);
          int a0 = ti.m0 + BM * (int)rank;                     // this CTA's A rows (or output-row range for MN-major A)
          const int b0 = brow0 + (n_mma >> 1) * (int)rank;     // this CTA's B rows
          // The odd CTA's half of an expert's last tile may lie past the expert's segment: its rows would be another
          // expert's, computed and thrown away.  Loading from beyond the array instead makes TMA fill zeros without
          // touching memory: no operand traffic for that half, and a tensor core that multiplies zeros draws less power.
          if (!A_MN && p.mode == TC_ROWS && a0 >= ti.m_end) a0 = p.R;
          for (int kb = 0; kb < ti.kblocks; ++kb) {
            if (!mbar_wait(empty0 + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
            if (rank == 0) mbar_expect_tx(full0 + 8 * stage, 2 * STAGE_BYTES);
            const uint32_t fb = full_mma0 + 8 * stage;
            const uint32_t sa = smem_base + stage * STAGE_BYTES;
            const uint32_t sb = sa + HALF_BYTES;
            if (!A_MN) {
              tma_pair_load_2d(sa, &map_a, fb, kb * BK, a0);  // [128 rows][64 k]
            } else {
              const int kr = ti.krow0 + kb * BK;
              tma_pair_load_2d(sa, &map_a, fb, a0, kr);  // [64 k][64 m] twice
              tma_pair_load_2d(sa + 8192, &map_a, fb, a0 + 64, kr);
            }
            if (!B_MN) {
              tma_pair_load_3d(sb, &map_b, fb, kb * BK, b0, ti.expert);  // [128 n][64 k] of the expert's weights
            } else if (p.mode == TC_ROWS) {
              tma_pair_load_3d(sb, &map_b, fb, b0, kb * BK, ti.expert);  // [64 k][64 n] twice
              tma_pair_load_3d(sb + 8192, &map_b, fb, b0 + 64, kb * BK, ti.expert);
            } else {
              const int kr = ti.krow0 + kb * BK;
              tma_pair_load_2d(sb, &map_b, fb, b0, kr);
              tma_pair_load_2d(sb + 8192, &map_b, fb, b0 + 64, kr);
            }
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
          }
        }
        if (!ok) { *abort_flag = 1; if (p.status) atomicOr(p.status, C2R_STATUS_WAIT_TIMEOUT); }
      }
    } else {
      // a gathered operand: lane 0 waits and issues the tiled loads of the other operand, all 32 lanes fetch four
      // token rows each
      {
        const uint32_t full_mma0 = map_to_cta(full0, 0);  // completion bytes are counted where the MMAs are issued
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        int e_hint = 0;
        for (long long t = pair_id; ok; t += n_pairs) {
          TileInfo ti;
          if (!decode_tile(p, s_off, s_cnt, s_pt, t, ti, e_hint)) break;
          int n_mma, w, brow0;
          n_geometry(p, ti.jn, n_mma, w, brow0);
          const int a0 = ti.m0 + BM * (int)rank;               // this CTA's A rows (or output-row range for MN-major A)
          const int b0 = brow0 + (n_mma >> 1) * (int)rank;     // this CTA's B rows
          int4 rows = make_int4(0, 0, 0, 0);
          if (GATHER == 1) rows = gather_rows(p, a0 + 4 * lane);                       // the same rows for every k-block
          if (GATHER == 2) rows = gather_rows(p, ti.krow0 + 4 * (lane & 15));          // k-block 0; refreshed below
          for (int kb = 0; kb < ti.kblocks; ++kb) {
            int4 next_rows = rows;
            if (GATHER == 2 && kb + 1 < ti.kblocks) next_rows = gather_rows(p, ti.krow0 + (kb + 1) * BK + 4 * (lane & 15));
            if (lane == 0) ok = mbar_wait(empty0 + 8 * stage, phase ^ 1u, abort_flag);
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            if (!ok) break;
            if (lane == 0 && rank == 0) mbar_expect_tx(full0 + 8 * stage, 2 * STAGE_BYTES);
            const uint32_t fb = full_mma0 + 8 * stage;
            const uint32_t sa = smem_base + stage * STAGE_BYTES;
            const uint32_t sb = sa + HALF_BYTES;
            if (GATHER == 1) {
              tma_pair_gather4(sa + 512 * lane, &map_a, fb, kb * BK, rows.x, rows.y, rows.z, rows.w);  // [128 rows][64 k]
            } else if (lane == 0) {
              if (!A_MN) {
                tma_pair_load_2d(sa, &map_a, fb, kb * BK, a0);  // [128 rows][64 k]
              } else {
                const int kr = ti.krow0 + kb * BK;
                tma_pair_load_2d(sa, &map_a, fb, a0, kr);  // [64 k][64 m] twice
                tma_pair_load_2d(sa + 8192, &map_a, fb, a0 + 64, kr);
              }
            }
            if (GATHER == 2) {
              // [64 k][64 n] twice: lanes 0..15 fill the first box, lanes 16..31 the second (64 columns further)
              const int h = lane >> 4;
              tma_pair_gather4(sb + 8192 * h + 512 * (lane & 15), &map_b, fb, b0 + 64 * h, rows.x, rows.y, rows.z, rows.w);
            } else if (lane == 0) {
              if (!B_MN) {
                tma_pair_load_3d(sb, &map_b, fb, kb * BK, b0, ti.expert);  // [128 n][64 k] of the expert's weights
              } else if (p.mode == TC_ROWS) {
                tma_pair_load_3d(sb, &map_b, fb, b0, kb * BK, ti.expert);  // [64 k][64 n] twice
                tma_pair_load_3d(sb + 8192, &map_b, fb, b0 + 64, kb * BK, ti.expert);
              } else {
                const int kr = ti.krow0 + kb * BK;
                tma_pair_load_2d(sb, &map_b, fb, b0, kr);
                tma_pair_load_2d(sb + 8192, &map_b, fb, b0 + 64, kr);
              }
            }
            rows = next_rows;
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
          }
        }
        if (!ok && lane == 0) { *abort_flag = 1; if (p.status) atomicOr(p.status, C2R_STATUS_WAIT_TIMEOUT); }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer (even CTA of the pair) ----------------------
    if (lane == 0 && rank == 0) {
      uint32_t stage = 0, phase = 0;
      uint32_t acc = 0, acc_phase = 0;
      bool ok = true;
      int e_hint = 0;
        for (long long t = pair_id; ok; t += n_pairs) {
        TileInfo ti;
        if (!decode_tile(p, s_off, s_cnt, s_pt, t, ti, e_hint)) break;
        if (ti.kblocks == 0) continue;  // empty contraction: the epilogue writes zeros on its own
        int n_mma, w, brow0;
        n_geometry(p, ti.jn, n_mma, w, brow0);
        const uint32_t idesc = instr_desc_pair(n_mma, A_MN, B_MN);
        if (!mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * TILE_N;
        for (int kb = 0; kb < ti.kblocks; ++kb) {
          if (!mbar_wait(full0 + 8 * stage, phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_base + stage * STAGE_BYTES;
          const uint32_t sb = sa + HALF_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // K-major: 16 k-elements = 32 bytes inside the swizzle row; 8-row groups 1024 bytes apart.
            // MN-major: 64-element MN groups 8192 bytes apart, 8-k groups 1024 bytes apart, 16 k = 2048 bytes.
            const uint64_t da = A_MN ? smem_desc(sa + k * 2048, 8192, 1024) : smem_desc(sa + k * 32, 16, 1024);
            const uint64_t db = B_MN ? smem_desc(sb + k * 2048, 8192, 1024) : smem_desc(sb + k * 32, 16, 1024);
            tc_pair_mma(d_tmem, da, db, idesc, (kb > 0 || k > 0) ? 1u : 0u);
          }
          tc_pair_commit(empty0 + 8 * stage);  // frees the stage in both CTAs once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_pair_commit(tfull0 + 8 * acc);  // accumulator complete, in both CTAs
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) { *abort_flag = 1; if (p.status) atomicOr(p.status, C2R_STATUS_WAIT_TIMEOUT); }
    }
  } else {
    // ------------------------------- epilogue (8 warps) -------------------------------------
    // TMEM hands every thread one accumulator row, which is the worst shape for global memory (32
    // rows per access).  Each warp therefore passes its 32 x 128-byte pieces through a private
    // staging tile in shared memory and moves them to / from global memory row-contiguously.
    const int q = warp & 3;            // TMEM lane quarter this warp may read
    const int hsel = (warp - 2) >> 2;  // which of the two warps of that quarter: takes every other column group
    const uint32_t buf0 = smem_base + STAGES * STAGE_BYTES + (warp - 2) * (2 * STG_BYTES), buf1 = buf0 + STG_BYTES;
    const uint32_t tempty_mma0 = map_to_cta(tempty0, 0);
    uint32_t acc = 0, acc_phase = 0;
    bool ok = true;
    int e_hint = 0;
        for (long long t = pair_id; ok; t += n_pairs) {
      TileInfo ti;
      if (!decode_tile(p, s_off, s_cnt, s_pt, t, ti, e_hint)) break;
      int n_mma, w, brow0;
      n_geometry(p, ti.jn, n_mma, w, brow0);
      const bool have_acc = ti.kblocks > 0;
      const uint32_t taddr_row = tmem_base + acc * TILE_N + ((uint32_t)(32 * q) << 16);
      const int row0 = ti.m0 + BM * (int)rank + 32 * q;  // first of this warp's 32 rows
      const int rows_valid = max(0, min(32, ti.m_end - row0));
      const long long mrow = row0 + lane;
      bool waited = !have_acc;
      const float sc = row_scale_of(p, mrow, lane < rows_valid);  // requested before the accumulator is awaited
      int tok_mine = -1;  // fused combine: the token this lane's row belongs to
      if (EPI == TC_EPI_F32 && p.token_acc != nullptr && lane < rows_valid) {
        const int sl = p.slot_of_row[mrow];
        tok_mine = sl >= 0 ? sl / p.slots_per_token : -1;
      }
      if constexpr (EPI == TC_EPI_SWIGLU_BWD) {
        // dA = s_r dH (dH/dA), dB = s_r dH (dH/dB) on groups of 64 H columns, s_r the row's scale; the forward pass
        // saved both local derivatives.  With qpart, also the row dot <dH_r, H_r> over this warp's columns (H as the
        // forward stored it, scale included): the gradient w.r.t. the scale times the scale.  None of the loads
        // depends on the accumulator, so the first group's are issued before it is awaited.
        const int n_groups = (w + 63) >> 6;
        const bool want_q = p.qpart != nullptr;
        float qacc = 0.f;
        for (int g = hsel; g < n_groups; g += 2) {
          const int hc0 = TILE_N * ti.jn + 64 * g;  // first H column of the group; a group never leaves its
          const int blk = hc0 >> 7;                 // 128-channel block of the packed (A | B) layout
          const int col_a = 256 * blk + (hc0 & 127);
          const int col_b = col_a + min(128, p.I - 128 * blk);
          const int vbytes = 2 * min(64, w - 64 * g);
          const long long pitch = 4ll * p.I;  // bytes per row of AB / dAB
          const uint8_t* gsrc = (const uint8_t*)p.AB + row0 * pitch;
          uint8_t* go = (uint8_t*)p.C + row0 * pitch;
          // The two saved derivatives travel global -> staging tile asynchronously; the H piece (row dots) is read
          // straight into registers, every lane its own row.  All of it is in flight at once.
          global_rows_to_stage_async(buf0, gsrc + 2 * col_a, pitch, rows_valid, vbytes, lane);
          global_rows_to_stage_async(buf1, gsrc + 2 * col_b, pitch, rows_valid, vbytes, lane);
          uint4 hrow[8];
          if (want_q) {
            const uint8_t* hp = (const uint8_t*)p.H + mrow * (2ll * p.I) + 2 * hc0;
#pragma unroll
            for (int c = 0; c < 8; ++c)
              hrow[c] = (lane < rows_valid && 16 * c < vbytes) ? *reinterpret_cast<const uint4*>(hp + 16 * c) : make_uint4(0, 0, 0, 0);
          }
          async_copies_wait();
          __syncwarp();
          if (!waited) {
            if (!mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            waited = true;
          }
#pragma unroll
          for (int pc = 0; pc < 4; ++pc) {
            if (32 * pc >= vbytes) break;  // warp-uniform
            uint32_t r0[16];
            float v0[16], ga[16], gb[16], da[16], db[16];
            if (have_acc) {
              tc_ld16(taddr_row + 64 * g + 16 * pc, r0);
              tc_ld_wait();
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) v0[i] = have_acc ? __uint_as_float(r0[i]) : 0.f;
            if (want_q) {
              float hv[16];
              unpack_bf16x16(hrow[2 * pc], hrow[2 * pc + 1], hv);
#pragma unroll
              for (int i = 0; i < 16; ++i) qacc = fmaf(v0[i], hv[i], qacc);
            }
            const uint32_t sa0 = stg_addr(buf0, lane, 2 * pc), sa1 = stg_addr(buf0, lane, 2 * pc + 1);
            const uint32_t sb0 = stg_addr(buf1, lane, 2 * pc), sb1 = stg_addr(buf1, lane, 2 * pc + 1);
            unpack_bf16x16(lds128(sa0), lds128(sa1), ga);
            unpack_bf16x16(lds128(sb0), lds128(sb1), gb);
#pragma unroll
            for (int i = 0; i < 16; ++i) { const float v = sc * v0[i]; da[i] = v * ga[i]; db[i] = v * gb[i]; }
            sts128(sa0, pack_bf16x8(da)); sts128(sa1, pack_bf16x8(da + 8));
            sts128(sb0, pack_bf16x8(db)); sts128(sb1, pack_bf16x8(db + 8));
          }
          __syncwarp();
          stage_to_global(buf0, go + 2 * col_a, pitch, rows_valid, vbytes, lane);
          stage_to_global(buf1, go + 2 * col_b, pitch, rows_valid, vbytes, lane);
          __syncwarp();
        }
        if (!ok) break;
        // one partial per (row, N tile, warp of the lane quarter); a warp without a group writes its zero
        if (want_q && lane < rows_valid) p.qpart[(long long)(2 * ti.jn + hsel) * p.R + mrow] = qacc;
      }
      if (!waited) {
        if (!mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag)) { ok = false; break; }
        tc_fence_after();
      }
      if constexpr (EPI == TC_EPI_SWIGLU_FWD) {
        // accumulator columns [0,w) = gate (A), [w,2w) = up (B): H = silu(A) * B, and for the backward pass
        // its local derivatives dH/dA = B silu'(A) (gate columns of the packed buffer) and dH/dB = silu(A) (up columns)
        const int n_groups = (w + 63) >> 6;
        for (int g = hsel; g < n_groups; g += 2) {
          const int c = 64 * g;
          const int vbytes = 2 * min(64, w - c);
          const bool keep = p.C != nullptr;  // false: inference, only H is produced
          uint4 up[8];
#pragma unroll
          for (int pc = 0; pc < 4; ++pc) {
            if (32 * pc >= vbytes) break;
            uint32_t r0[16], r1[16];
            float ga[16], gb[16], h[16];
            if (have_acc) {
              tc_ld16(taddr_row + c + 16 * pc, r0);
              tc_ld16(taddr_row + w + c + 16 * pc, r1);
              tc_ld_wait();
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float a = have_acc ? __uint_as_float(r0[i]) : 0.f;
              const float b = have_acc ? __uint_as_float(r1[i]) : 0.f;
              const float sg = sigmoid_fast(a);
              const float as = a * sg;             // silu(a)
              h[i] = sc * (as * b);
              ga[i] = b * (sg + as - as * sg);     // b silu'(a), silu'(a) = s (1 + a (1 - s))
              gb[i] = as;
            }
            sts128(stg_addr(buf1, lane, 2 * pc), pack_bf16x8(h)); sts128(stg_addr(buf1, lane, 2 * pc + 1), pack_bf16x8(h + 8));
            if (keep) {
              sts128(stg_addr(buf0, lane, 2 * pc), pack_bf16x8(ga)); sts128(stg_addr(buf0, lane, 2 * pc + 1), pack_bf16x8(ga + 8));
              up[2 * pc] = pack_bf16x8(gb); up[2 * pc + 1] = pack_bf16x8(gb + 8);
            }
          }
          __syncwarp();
          uint8_t* gab = (uint8_t*)p.C + row0 * (4ll * p.I) + 2 * (256 * ti.jn + c);
          if (keep) stage_to_global(buf0, gab, 4ll * p.I, rows_valid, vbytes, lane);
          stage_to_global(buf1, (uint8_t*)p.H + row0 * (2ll * p.I) + 2 * (128 * ti.jn + c), 2ll * p.I, rows_valid, vbytes, lane);
          __syncwarp();
          if (keep) {
#pragma unroll
            for (int pc = 0; pc < 4; ++pc) {
              if (32 * pc >= vbytes) break;
              sts128(stg_addr(buf0, lane, 2 * pc), up[2 * pc]); sts128(stg_addr(buf0, lane, 2 * pc + 1), up[2 * pc + 1]);
            }
            __syncwarp();
            stage_to_global(buf0, gab + 2 * w, 4ll * p.I, rows_valid, vbytes, lane);
            __syncwarp();
          }
        }
      } else if constexpr (EPI == TC_EPI_F32) {
        const int n_groups = (w + 31) >> 5;  // 32 fp32 columns = 128 bytes
        for (int g = hsel; g < n_groups; g += 2) {
          const int c = 32 * g;
          const int vbytes = 4 * min(32, w - c);
          const uint32_t buf = (g & 2) ? buf1 : buf0;  // alternate tiles: the next group's writes need not wait
#pragma unroll
          for (int pc = 0; pc < 2; ++pc) {
            if (64 * pc >= vbytes) break;
            uint32_t r0[16];
            if (have_acc) {
              tc_ld16(taddr_row + c + 16 * pc, r0);
              tc_ld_wait();
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
              sts128(stg_addr(buf, lane, 4 * pc + i),
                     have_acc ? make_uint4(r0[4 * i], r0[4 * i + 1], r0[4 * i + 2], r0[4 * i + 3]) : make_uint4(0, 0, 0, 0));
          }
          __syncwarp();
          if (p.token_acc != nullptr)
            stage_red_to_rows(buf, (uint8_t*)p.token_acc + 4ll * (TILE_N * ti.jn + c), 4 * p.ldc, tok_mine, vbytes, lane);
          else
            stage_to_global(buf, (uint8_t*)p.C + row0 * (4 * p.ldc) + 4ll * (TILE_N * ti.jn + c), 4 * p.ldc, rows_valid, vbytes,
                            lane);
        }
        __syncwarp();
      } else if constexpr (EPI == TC_EPI_WGRAD_BF16) {
        const int n_groups = (w + 63) >> 6;
        for (int g = hsel; g < n_groups; g += 2) {
          const int c = 64 * g;
          const int vbytes = 2 * min(64, w - c);
          __nv_bfloat16* orow = (__nv_bfloat16*)p.C + (long long)ti.expert * p.sC + mrow * p.ldc + TILE_N * ti.jn + c;
          const uint32_t buf = (g & 2) ? buf1 : buf0;
#pragma unroll
          for (int pc = 0; pc < 4; ++pc) {
            if (32 * pc >= vbytes) break;
            uint32_t r0[16];
            float v0[16];
            if (have_acc) {
              tc_ld16(taddr_row + c + 16 * pc, r0);
              tc_ld_wait();
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) v0[i] = have_acc ? __uint_as_float(r0[i]) : 0.f;
            if (p.accumulate) {  // read-modify-write in fp32 straight on the thread's own row
              if (lane < rows_valid) {
                float old[16];
                load_bf16x16(orow + 16 * pc, old);
#pragma unroll
                for (int i = 0; i < 16; ++i) v0[i] += old[i];
                store_bf16x16(orow + 16 * pc, v0);
              }
            } else {
              sts128(stg_addr(buf, lane, 2 * pc), pack_bf16x8(v0));
              sts128(stg_addr(buf, lane, 2 * pc + 1), pack_bf16x8(v0 + 8));
            }
          }
          if (!p.accumulate) {
            __syncwarp();
            stage_to_global(buf, (uint8_t*)((__nv_bfloat16*)p.C + (long long)ti.expert * p.sC + (long long)row0 * p.ldc +
                                            TILE_N * ti.jn + c),
                            2 * p.ldc, rows_valid, vbytes, lane);
          }
        }
        __syncwarp();
      } else if constexpr (EPI == TC_EPI_T_F32) {
        // transposed fp32 store out[group][column][row]: a warp's 32 rows are contiguous in memory
        float* obase = (float*)p.C + (long long)ti.expert * p.sC + mrow;
        for (int ci = hsel; ci < (w >> 4); ci += 2) {
          uint32_t r0[16];
          if (have_acc) {
            tc_ld16(taddr_row + 16 * ci, r0);
            tc_ld_wait();
          }
          if (lane < rows_valid) {
#pragma unroll
            for (int i = 0; i < 16; ++i)
              obase[(long long)(TILE_N * ti.jn + 16 * ci + i) * p.ldc] = have_acc ? __uint_as_float(r0[i]) : 0.f;
          }
        }
      }
      if (have_acc) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(tempty_mma0 + 8 * acc);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
    if (!ok && lane == 0) { *abort_flag = 1; if (p.status) atomicOr(p.status, C2R_STATUS_WAIT_TIMEOUT); }
  }

  // After a wait gave up, TMA loads nobody will wait for may still be in flight towards this CTA's shared memory:
  // give them time to land (they complete within microseconds) before the CTA can exit.  The peer is held at the
  // cluster barrier meanwhile, so its shared memory outlives its own stragglers too.
  __syncthreads();
  if (*abort_flag)
    for (int i = 0; i < 128; ++i) __nanosleep(2000);
  // Both CTAs are done with each other's shared and tensor memory before either leaves.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
template <bool A_MN, bool B_MN, int EPI, int GATHER = 0>
static int launch(const CUtensorMap& ma, const CUtensorMap& mb, const TcParams& p, cudaStream_t s) {
  constexpr int smem = SMEM_BYTES;
  constexpr int MAX_DEV = 64;
  static int grid_of_device[MAX_DEV] = {};  // CTAs of the persistent grid (2 per co-resident pair), per device
  int dev = 0;
  C2R_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= MAX_DEV) return C2R_ERR_UNSUPPORTED_SHAPE;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.blockDim = dim3(TC_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int grid = __atomic_load_n(&grid_of_device[dev], __ATOMIC_ACQUIRE);
  if (grid == 0) {
    C2R_CUDA(cudaFuncSetAttribute(tc_gemm_kernel<A_MN, B_MN, GATHER, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    int sms = 0, pairs = 0;
    C2R_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    cfg.gridDim = dim3(sms / 2 * 2);
    C2R_CUDA(cudaOccupancyMaxActiveClusters(&pairs, tc_gemm_kernel<A_MN, B_MN, GATHER, EPI>, &cfg));
    if (pairs < 1) return C2R_ERR_UNSUPPORTED_SHAPE;
    grid = 2 * (pairs < sms / 2 ? pairs : sms / 2);
    __atomic_store_n(&grid_of_device[dev], grid, __ATOMIC_RELEASE);
  }
  cfg.gridDim = dim3(grid);
  C2R_CUDA(cudaLaunchKernelEx(&cfg, tc_gemm_kernel<A_MN, B_MN, GATHER, EPI>, ma, mb, p));
  C2R_LAUNCH_CHECK();
  return C2R_OK;
}

bool tc_supported(const c2r_config* cfg, int nE, int I, int64_t R) {
  // TMA needs 16-byte row pitches; MMA-N needs multiples of 16; with several experts every
  // segment must start on a 128-row boundary so that no CTA's rows straddle two experts.
  return cfg->dtype == C2R_BF16 && cfg->d % 16 == 0 && I % 16 == 0 && R < (1ll << 31) &&
         (nE == 1 || cfg->row_align % BM == 0) && get_encode() != nullptr;
}

int swiglu_qparts(const c2r_config* cfg, int nE, int I, int64_t R) {
  return tc_supported(cfg, nE, I, R) ? 2 * ((I + TILE_N - 1) / TILE_N) : (I + 63) / 64;
}

int tc_swiglu_fwd(const c2r_config* cfg, const SwigluCall& a, cudaStream_t s) {
  const int d = cfg->d, I = a.I, nE = a.nE;
  const int64_t R = a.R;
  CUtensorMap ma, mb;
  TcParams p{};
  p.mode = TC_ROWS; p.n_experts = nE; p.R = (int)R; p.I = I; p.counts = a.counts; p.offsets = a.offsets; p.status = a.status;
  // (A | B) = Xp W13p^T with the SwiGLU epilogue: AB packed + H
  const bool gather = a.X != nullptr && a.slot_of_row != nullptr;  // rows of X picked inside the GEMM, no permuted copy
  int rc = gather ? make_map(&ma, a.X, d, cfg->N, 0, BK, 1) : make_map(&ma, a.Xp, d, R, 0, BK, BM);
  if (rc) return rc;
  rc = make_map(&mb, a.W13p, d, 2 * I, nE, BK, 128);
  if (rc) return rc;
  p.epi = TC_EPI_SWIGLU_FWD; p.K = d; p.Nout = I; p.n_tiles = (I + 127) / 128; p.C = a.AB; p.H = a.H;
  p.row_scale = a.row_scale; p.scale_kind = a.row_scale ? a.scale_kind : 0;
  p.slot_of_row = a.slot_of_row; p.slots_per_token = cfg->K; p.n_tokens = cfg->N;
  rc = gather ? launch<false, false, TC_EPI_SWIGLU_FWD, 1>(ma, mb, p, s) : launch<false, false, TC_EPI_SWIGLU_FWD>(ma, mb, p, s);
  if (rc) return rc;
  // Yp = H W2^T (fp32)
  rc = make_map(&ma, a.H, I, R, 0, BK, BM);
  if (rc) return rc;
  rc = make_map(&mb, a.W2, I, d, nE, BK, 128);
  if (rc) return rc;
  p.epi = TC_EPI_F32; p.K = I; p.Nout = d; p.n_tiles = (d + TILE_N - 1) / TILE_N; p.C = a.Yp; p.ldc = d; p.H = nullptr;
  p.row_scale = nullptr; p.scale_kind = 0;
  p.token_acc = a.token_acc; p.slot_of_row = a.slot_of_row;  // fused combine: rows are added into their tokens
  return launch<false, false, TC_EPI_F32>(ma, mb, p, s);
}

int tc_swiglu_bwd(const c2r_config* cfg, const SwigluCall& a, cudaStream_t s) {
  const int d = cfg->d, I = a.I, nE = a.nE;
  const int64_t R = a.R;
  CUtensorMap ma, mb;
  TcParams p{};
  p.n_experts = nE; p.R = (int)R; p.I = I; p.counts = a.counts; p.offsets = a.offsets; p.status = a.status;
  // dH = dYp W2 -> (dA | dB) packed
  p.mode = TC_ROWS;
  int rc = make_map(&ma, a.dYp, d, R, 0, BK, BM);
  if (rc) return rc;
  rc = make_map(&mb, a.W2, I, d, nE, 64, 64);  // W2_e is [d (k)][I (n)]: MN-major B
  if (rc) return rc;
  p.epi = TC_EPI_SWIGLU_BWD; p.K = d; p.Nout = I; p.n_tiles = (I + TILE_N - 1) / TILE_N; p.C = a.dAB; p.AB = a.AB;
  p.row_scale = a.row_scale; p.scale_kind = a.row_scale ? a.scale_kind : 0; p.qpart = a.qpart; p.H = a.H;
  rc = launch<false, true, TC_EPI_SWIGLU_BWD>(ma, mb, p, s);
  if (rc) return rc;
  p.row_scale = nullptr; p.scale_kind = 0; p.qpart = nullptr; p.H = nullptr;
  // dXp = dAB W13p (fp32)
  rc = make_map(&ma, a.dAB, 2 * I, R, 0, BK, BM);
  if (rc) return rc;
  rc = make_map(&mb, a.W13p, d, 2 * I, nE, 64, 64);  // W13p_e is [2I (k)][d (n)]: MN-major B
  if (rc) return rc;
  p.epi = TC_EPI_F32; p.K = 2 * I; p.Nout = d; p.n_tiles = (d + TILE_N - 1) / TILE_N; p.C = a.dXp; p.ldc = d; p.AB = nullptr;
  p.token_acc = a.token_acc; p.slot_of_row = a.slot_of_row; p.slots_per_token = cfg->K;
  rc = launch<false, true, TC_EPI_F32>(ma, mb, p, s);
  if (rc) return rc;
  p.token_acc = nullptr;
  // dW2_e = dYp_e^T H_e  [d, I]
  p.mode = TC_WGRAD; p.epi = TC_EPI_WGRAD_BF16; p.accumulate = a.accumulate;
  rc = make_map(&ma, a.dYp, d, R, 0, 64, 64);
  if (rc) return rc;
  rc = make_map(&mb, a.H, I, R, 0, 64, 64);
  if (rc) return rc;
  p.Mout = d; p.Nout = I; p.m_tiles = (d + TILE_M - 1) / TILE_M; p.n_tiles = (I + TILE_N - 1) / TILE_N;
  p.C = a.dW2; p.ldc = I; p.sC = (long long)d * I;
  rc = launch<true, true, TC_EPI_WGRAD_BF16>(ma, mb, p, s);
  if (rc) return rc;
  // dW13p_e = dAB_e^T Xp_e  [2I, d]
  rc = make_map(&ma, a.dAB, 2 * I, R, 0, 64, 64);
  if (rc) return rc;
  const bool gather = a.X != nullptr && a.slot_of_row != nullptr;
  rc = gather ? make_map(&mb, a.X, d, cfg->N, 0, 64, 1) : make_map(&mb, a.Xp, d, R, 0, 64, 64);
  if (rc) return rc;
  p.Mout = 2 * I; p.Nout = d; p.m_tiles = (2 * I + TILE_M - 1) / TILE_M; p.n_tiles = (d + TILE_N - 1) / TILE_N;
  p.C = a.dW13p; p.ldc = d; p.sC = (long long)2 * I * d;
  p.slot_of_row = a.slot_of_row; p.slots_per_token = cfg->K; p.n_tokens = cfg->N;
  return gather ? launch<true, true, TC_EPI_WGRAD_BF16, 2>(ma, mb, p, s) : launch<true, true, TC_EPI_WGRAD_BF16>(ma, mb, p, s);
}

int tc_gate_wgrad(const c2r_config* cfg, const void* X, const void* dLd, float* partial, int n_splits,
                  const int32_t* split_counts, const int32_t* split_offsets, int32_t* status, cudaStream_t s) {
  const int d = cfg->d;
  CUtensorMap ma, mb;
  TcParams p{};
  p.mode = TC_WGRAD; p.epi = TC_EPI_T_F32; p.n_experts = n_splits; p.R = cfg->N; p.I = 0;
  p.counts = split_counts; p.offsets = split_offsets; p.status = status;
  // out^T[d, 64] = X^T dLd per split: A = X as [k = token][m = d], B = dLd as [k = token][n = 64], both MN-major
  int rc = make_map(&ma, X, d, cfg->N, 0, 64, 64);
  if (rc) return rc;
  rc = make_map(&mb, dLd, 64, cfg->N, 0, 64, 64);
  if (rc) return rc;
  p.Mout = d; p.Nout = 64; p.m_tiles = (d + TILE_M - 1) / TILE_M; p.n_tiles = 1;
  p.C = partial; p.ldc = d; p.sC = 64ll * d;
  return launch<true, true, TC_EPI_T_F32>(ma, mb, p, s);
}

}  // namespace c2r
