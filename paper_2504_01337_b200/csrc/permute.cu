// Dispatch on one device: atomic-free histogram / prefix-scan / stable rank over experts, the
// 16-byte vectorised row gather, the weighted combine and their backward twins.
#include "c2r_common.cuh"
#include "gemm.h"

namespace c2r {

// Blocking of the counting sort: a block owns perm_tokens_per_block(K) consecutive tokens, i.e. at most 512
// consecutive slots, a whole number of 32-slot groups.  One warp per group.
constexpr int PERM_THREADS = 512;
constexpr int PERM_GROUPS = PERM_THREADS / 32;  // 32-slot groups a block can own

__device__ __forceinline__ uint32_t lanemask_lt() {
  uint32_t m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}

// Expert key of slot s (clamped into [0,E); -1 = the slot takes no part: past the end, or a key of -1 when
// skip_negative is set, which the de-duplicated dispatch uses).
__device__ __forceinline__ int slot_key(const int32_t* __restrict__ idx, long long s, long long NK, int E, int skip_negative,
                                        int& flags) {
  if (s >= NK) return -1;
  int e = idx[s];
  if (e < 0 || e >= E) {
    if (skip_negative && e == -1) return -1;
    flags |= C2R_STATUS_BAD_INDEX;
    e = min(max(e, 0), E - 1);
  }
  return e;
}

// Per-group, per-expert counts of this block's slots: inside a 32-slot group, lanes with equal expert form a
// peer set (match.any) whose lowest lane records the set size -- no atomics, and the order of slots is kept.
// grp_cnt must be zero on entry.  Returns this thread's key.
__device__ __forceinline__ int group_count(const int32_t* __restrict__ idx, long long NK, int E, int slots_per_block,
                                           int (*grp_cnt)[64], int& flags, int skip_negative) {
  const int lane = threadIdx.x & 31, g = threadIdx.x >> 5;
  int e = -1;
  if (32 * g < slots_per_block)
    e = slot_key(idx, (long long)blockIdx.x * slots_per_block + threadIdx.x, NK, E, skip_negative, flags);
  const uint32_t peers = __match_any_sync(0xffffffffu, e);
  if (e >= 0 && lane == __ffs(peers) - 1) grp_cnt[g][e] = __popc(peers);
  return e;
}

// Layout position -> expert from expert_rank (NULL = identity).  A table that is not a permutation of
// [0,E) (an entry out of range, a duplicate, hence a hole) is replaced by the identity order and reported.
// All threads of the block must call; needs E <= 64 <= blockDim.x.  Ends with a barrier.
__device__ __forceinline__ void layout_order(const int32_t* __restrict__ expert_rank, int E, int* s_by_rank, int* s_bad) {
  if (threadIdx.x < 64) s_by_rank[threadIdx.x] = -1;
  if (threadIdx.x == 0) *s_bad = 0;
  __syncthreads();
  if ((int)threadIdx.x < E) {
    const int r = expert_rank ? expert_rank[threadIdx.x] : (int)threadIdx.x;
    if (r < 0 || r >= E) *s_bad = 1;
    else s_by_rank[r] = threadIdx.x;  // duplicates: one writer wins and some other position stays -1
  }
  __syncthreads();
  if ((int)threadIdx.x < E && s_by_rank[threadIdx.x] < 0) *s_bad = 1;
  __syncthreads();
  if (*s_bad && (int)threadIdx.x < E) s_by_rank[threadIdx.x] = threadIdx.x;
  __syncthreads();
}

__global__ void __launch_bounds__(PERM_THREADS) perm_hist_kernel(const int32_t* __restrict__ idx, long long NK, int E,
                                                                 int slots_per_block, int32_t* __restrict__ block_counts,
                                                                 int32_t* __restrict__ status, int skip_negative) {
  __shared__ int grp_cnt[PERM_GROUPS][64];
  for (int i = threadIdx.x; i < PERM_GROUPS * 64; i += blockDim.x) (&grp_cnt[0][0])[i] = 0;
  __syncthreads();
  int flags = 0;
  group_count(idx, NK, E, slots_per_block, grp_cnt, flags, skip_negative);
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    int s = 0;
#pragma unroll
    for (int g = 0; g < PERM_GROUPS; ++g) s += grp_cnt[g][e];
    block_counts[(size_t)blockIdx.x * E + e] = s;
  }
  if (status != nullptr && flags) atomicOr(status, flags);
}

// One block: per expert an exclusive scan of the block counts over blocks (a warp per expert,
// 32 blocks per shuffle scan), then the segment offsets in layout (rank) order with alignment.
__global__ void __launch_bounds__(1024) perm_scan_kernel(int32_t* __restrict__ block_counts, int n_blocks, int E,
                                                         const int32_t* __restrict__ expert_rank, int row_align,
                                                         int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
                                                         int32_t* __restrict__ status) {
  __shared__ int s_counts[64];
  __shared__ int s_by_rank[64];
  __shared__ int s_bad;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int e = warp; e < E; e += 32) {
    int running = 0;
    for (int b0 = 0; b0 < n_blocks; b0 += 32) {
      const int b = b0 + lane;
      const int v = (b < n_blocks) ? block_counts[(size_t)b * E + e] : 0;
      int incl = v;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        int o = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += o;
      }
      if (b < n_blocks) block_counts[(size_t)b * E + e] = running + incl - v;
      running += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) s_counts[e] = running;
  }
  layout_order(expert_rank, E, s_by_rank, &s_bad);
  if (threadIdx.x == 0) {
    int cursor = 0;
    for (int r = 0; r < E; ++r) {
      const int e = s_by_rank[r];
      offsets[e] = cursor;
      cursor += (s_counts[e] + row_align - 1) / row_align * row_align;
    }
    offsets[E] = cursor;
    if (s_bad && status != nullptr) atomicOr(status, C2R_STATUS_BAD_INDEX);
  }
  if (threadIdx.x < E) counts[threadIdx.x] = s_counts[threadIdx.x];
}

// Stable rank of a block's slots once grp_cnt holds the per-group counts and s_start[e] the row at which the
// block's first slot of expert e lands: rows of earlier groups of the block, then lower lanes of the group.
// w (optional): w_row[row] = w[slot], the routing weight of the slot that owns the row.
__device__ __forceinline__ void rank_and_write(int e, long long NK, int E, int slots_per_block, int (*grp_cnt)[64],
                                               const int* s_start, int32_t* __restrict__ row_of_slot,
                                               int32_t* __restrict__ slot_of_row, const float* __restrict__ w,
                                               float* __restrict__ w_row) {
  for (int x = threadIdx.x; x < E; x += blockDim.x) {
    int run = s_start[x];
#pragma unroll
    for (int g = 0; g < PERM_GROUPS; ++g) {
      const int c = grp_cnt[g][x];
      grp_cnt[g][x] = run;
      run += c;
    }
  }
  __syncthreads();
  const int g = threadIdx.x >> 5;
  const uint32_t peers = __match_any_sync(0xffffffffu, e);
  if (e >= 0) {
    const long long s = (long long)blockIdx.x * slots_per_block + threadIdx.x;
    const int row = grp_cnt[g][e] + __popc(peers & lanemask_lt());
    row_of_slot[s] = row;
    slot_of_row[row] = (int32_t)s;
    if (w_row != nullptr) w_row[row] = w[s];
  }
}

__global__ void __launch_bounds__(PERM_THREADS) perm_rank_kernel(const int32_t* __restrict__ idx, long long NK, int E,
                                                                 int slots_per_block,
                                                                 const int32_t* __restrict__ block_base,
                                                                 const int32_t* __restrict__ offsets,
                                                                 int32_t* __restrict__ row_of_slot,
                                                                 int32_t* __restrict__ slot_of_row, int skip_negative,
                                                                 const float* __restrict__ w, float* __restrict__ w_row) {
  __shared__ int grp_cnt[PERM_GROUPS][64];
  __shared__ int s_start[64];
  for (int i = threadIdx.x; i < PERM_GROUPS * 64; i += blockDim.x) (&grp_cnt[0][0])[i] = 0;
  for (int e = threadIdx.x; e < E; e += blockDim.x) s_start[e] = offsets[e] + block_base[(size_t)blockIdx.x * E + e];
  __syncthreads();
  int flags = 0;
  const int e = group_count(idx, NK, E, slots_per_block, grp_cnt, flags, skip_negative);
  __syncthreads();
  rank_and_write(e, NK, E, slots_per_block, grp_cnt, s_start, row_of_slot, slot_of_row, w, w_row);
}

// The scan folded into the rank pass (for batches of at most PERM_FUSED_MAX_BLOCKS blocks): every block
// adds up the histogram rows of the blocks before it and of all blocks (E columns, coalesced), derives the
// aligned segment offsets itself, and block 0 publishes counts and offsets.  The blocks also mark the rows
// that hold no slot (the padding that closes every aligned segment and the rows past the layout's end, up
// to R) with -1 in slot_of_row and 0 in w_row, so the call needs no memset: two launches fewer and one
// dependent round trip fewer than memset -> hist -> scan -> rank.
constexpr int PERM_FUSED_MAX_BLOCKS = 1024;
__global__ void __launch_bounds__(PERM_THREADS) perm_rank_fused_kernel(const int32_t* __restrict__ idx, long long NK, int E,
                                                                       int slots_per_block,
                                                                       const int32_t* __restrict__ block_counts,
                                                                       int n_blocks,
                                                                       const int32_t* __restrict__ expert_rank,
                                                                       int row_align, long long R,
                                                                       int32_t* __restrict__ counts,
                                                                       int32_t* __restrict__ offsets,
                                                                       int32_t* __restrict__ row_of_slot,
                                                                       int32_t* __restrict__ slot_of_row,
                                                                       const float* __restrict__ w,
                                                                       float* __restrict__ w_row,
                                                                       int32_t* __restrict__ status) {
  constexpr int PARTS = PERM_THREADS / 64;
  __shared__ int grp_cnt[PERM_GROUPS][64];
  __shared__ int s_start[64], s_total[64], s_by_rank[64], s_off[65];
  __shared__ int s_part[2][PARTS][64];  // partial sums: [before | total][share of the blocks][expert]
  __shared__ int s_bad;
  for (int i = threadIdx.x; i < PERM_GROUPS * 64; i += blockDim.x) (&grp_cnt[0][0])[i] = 0;
  {
    const int e = threadIdx.x & 63, part = threadIdx.x >> 6;
    int before = 0, total = 0;
    if (e < E) {
#pragma unroll 8
      for (int b = part; b < n_blocks; b += PARTS) {
        const int v = block_counts[(size_t)b * E + e];
        total += v;
        before += (b < (int)blockIdx.x) ? v : 0;
      }
    }
    s_part[0][part][e] = before;
    s_part[1][part][e] = total;
  }
  layout_order(expert_rank, E, s_by_rank, &s_bad);  // (its barriers also publish s_part and the zeroed grp_cnt)
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    int before = 0, total = 0;
#pragma unroll
    for (int q = 0; q < PARTS; ++q) { before += s_part[0][q][e]; total += s_part[1][q][e]; }
    s_start[e] = before;
    s_total[e] = total;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int cursor = 0;
    for (int r = 0; r < E; ++r) {
      const int e = s_by_rank[r];
      s_off[e] = cursor;
      cursor += (s_total[e] + row_align - 1) / row_align * row_align;
    }
    s_off[E] = cursor;
    if (blockIdx.x == 0 && s_bad && status != nullptr) atomicOr(status, C2R_STATUS_BAD_INDEX);
  }
  int flags = 0;
  const int e_mine = group_count(idx, NK, E, slots_per_block, grp_cnt, flags, 0);
  __syncthreads();
  if (blockIdx.x == 0) {
    for (int e = threadIdx.x; e <= E; e += blockDim.x) {
      offsets[e] = s_off[e];
      if (e < E) counts[e] = s_total[e];
    }
  }
  // rows without a slot: expert x's padding is written by block x mod gridDim.x, the tail by the last block
  for (int x = blockIdx.x; x < E; x += gridDim.x) {
    const int r0 = s_off[x] + s_total[x], r1 = s_off[x] + (s_total[x] + row_align - 1) / row_align * row_align;
    for (int r = r0 + threadIdx.x; r < r1; r += blockDim.x) {
      slot_of_row[r] = -1;
      if (w_row != nullptr) w_row[r] = 0.f;
    }
  }
  if (blockIdx.x == gridDim.x - 1) {
    for (long long r = s_off[E] + threadIdx.x; r < R; r += blockDim.x) {
      slot_of_row[r] = -1;
      if (w_row != nullptr) w_row[r] = 0.f;
    }
  }
  for (int e = threadIdx.x; e < E; e += blockDim.x) s_start[e] += s_off[e];
  __syncthreads();
  rank_and_write(e_mine, NK, E, slots_per_block, grp_cnt, s_start, row_of_slot, slot_of_row, w, w_row);
}

// Row gather, one warp per token: the token's row is read once and written to its K rows.  Blocks past the
// token blocks zero the padding rows that close each expert's aligned segment (block j: expert j).
template <typename T>
__global__ void __launch_bounds__(256) permute_rows_kernel(const T* __restrict__ X,
                                                           const int32_t* __restrict__ row_of_slot, T* __restrict__ Xp,
                                                           int N, int d, int K, const int32_t* __restrict__ counts,
                                                           const int32_t* __restrict__ offsets, int token_blocks,
                                                           int row_align) {
  using V = Vec16<T>;
  const int lane = threadIdx.x & 31;
  if ((int)blockIdx.x >= token_blocks) {
    const int e = blockIdx.x - token_blocks;
    const int n = counts[e];
    const int r0 = offsets[e] + n, r1 = offsets[e] + (n + row_align - 1) / row_align * row_align;
    V zero;
    float zf[V::N] = {};
    zero.from_float(zf);
    for (int r = r0 + (threadIdx.x >> 5); r < r1; r += blockDim.x >> 5)
      for (int c = lane; c < d / V::N; c += 32) zero.store(Xp + (size_t)r * d + (size_t)c * V::N);
    return;
  }
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (t >= N) return;  // warp-uniform
  const int my_row = (lane < K) ? row_of_slot[(size_t)t * K + lane] : 0;
  int rows[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) rows[k] = __shfl_sync(0xffffffffu, my_row, k);
  const int chunks = d / V::N;
  const T* src = X + (size_t)t * d;
  for (int c0 = lane; c0 < chunks; c0 += 32 * 4) {
    V v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (c0 + 32 * u < chunks) v[u].load(src + (size_t)(c0 + 32 * u) * V::N);
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      if (k >= K) break;
      T* dst = Xp + (size_t)rows[k] * d;
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (c0 + 32 * u < chunks) v[u].store(dst + (size_t)(c0 + 32 * u) * V::N);
    }
  }
}

// Zero the padding rows (slot_of_row < 0) of a permuted buffer; one warp per row.
template <typename T>
__global__ void __launch_bounds__(256) zero_pad_rows_kernel(const int32_t* __restrict__ slot_of_row, T* __restrict__ Xp,
                                                            long long R, int d) {
  using V = Vec16<T>;
  const int lane = threadIdx.x & 31;
  const int chunks = d / V::N;
  V zero;
  float zf[V::N] = {};
  zero.from_float(zf);
  for (long long r = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); r < R;
       r += (long long)gridDim.x * (blockDim.x >> 5)) {
    if (slot_of_row[r] >= 0) continue;
    T* dst = Xp + (size_t)r * d;
    for (int c = lane; c < chunks; c += 32) zero.store(dst + (size_t)c * V::N);
  }
}

// Loads V::N consecutive elements of type S starting at p as floats (S = float or the storage type).
template <typename T, typename S>
__device__ __forceinline__ void load_as_float(const S* p, float* f) {
  constexpr int NV = Vec16<T>::N;
  if constexpr (sizeof(S) == 4) {
#pragma unroll
    for (int q = 0; q < NV / 4; ++q) {
      const float4 v = *reinterpret_cast<const float4*>(p + 4 * q);
      f[4 * q] = v.x; f[4 * q + 1] = v.y; f[4 * q + 2] = v.z; f[4 * q + 3] = v.w;
    }
  } else {
    Vec16<S> v;
    v.load(p);
    v.to_float(f);
  }
}

// out[t,:] = sum_k coef[t,k] * src[rows[t*K+k],:]            (coef == NULL -> 1)
//          + ecoef(t) * extra[t,:]                           (ecoef = sigmoid(z[t]) if z else 1)
//          + sum_k dl[t,k] * Wg[idx[t,k],:] + dz[t] * wsg[:] (gate terms, optional)
//          + out[t,:] if accumulate.
// src == NULL: no such term (the producer already added its rows into extra).  src / extra are the fp32 partial results of the expert GEMMs; out has the storage type.
// One warp per token, fp32 accumulation in k order.  Serves the combine and the gradient un-permute.
template <typename T>
__global__ void __launch_bounds__(256) gather_sum_kernel(const float* __restrict__ src, const int32_t* __restrict__ rows_g,
                                                         const float* __restrict__ coef, const float* __restrict__ extra,
                                                         const float* __restrict__ z, const int32_t* __restrict__ idx,
                                                         const float* __restrict__ dl, const T* __restrict__ Wg,
                                                         const float* __restrict__ dz, const T* __restrict__ wsg,
                                                         T* __restrict__ out, int accumulate, int N, int d, int K) {
  using V = Vec16<T>;
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (t >= N) return;  // warp-uniform
  int my_row = 0, my_idx = 0;
  float my_coef = 1.f, my_dl = 0.f;
  if (lane < K) {
    my_row = rows_g[(size_t)t * K + lane];
    if (coef) my_coef = coef[(size_t)t * K + lane];
    if (dl) { my_dl = dl[(size_t)t * K + lane]; my_idx = idx[(size_t)t * K + lane]; }
  }
  int rows[8], eidx[8];
  float cf[8], gl[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    rows[k] = __shfl_sync(0xffffffffu, my_row, k);
    eidx[k] = __shfl_sync(0xffffffffu, my_idx, k);
    cf[k] = __shfl_sync(0xffffffffu, my_coef, k);
    gl[k] = __shfl_sync(0xffffffffu, my_dl, k);
  }
  const float ecoef = (extra && z) ? 1.0f / (1.0f + expf(-z[t])) : 1.0f;
  const float dzt = (dz && wsg) ? dz[t] : 0.f;
  const int chunks = d / V::N;
  for (int c = lane; c < chunks; c += 32) {
    const size_t col = (size_t)c * V::N;
    float acc[V::N];
#pragma unroll
    for (int j = 0; j < V::N; ++j) acc[j] = 0.f;
    if (src != nullptr) {
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (k >= K) break;
        float f[V::N];
        load_as_float<T, float>(src + (size_t)rows[k] * d + col, f);
#pragma unroll
        for (int j = 0; j < V::N; ++j) acc[j] = fmaf(cf[k], f[j], acc[j]);
      }
    }
    if (extra) {
      float f[V::N];
      load_as_float<T, float>(extra + (size_t)t * d + col, f);
#pragma unroll
      for (int j = 0; j < V::N; ++j) acc[j] = fmaf(ecoef, f[j], acc[j]);
    }
    if (dl) {
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (k >= K) break;
        float f[V::N];
        load_as_float<T, T>(Wg + (size_t)eidx[k] * d + col, f);
#pragma unroll
        for (int j = 0; j < V::N; ++j) acc[j] = fmaf(gl[k], f[j], acc[j]);
      }
    }
    if (dz && wsg) {
      float f[V::N];
      load_as_float<T, T>(wsg + col, f);
#pragma unroll
      for (int j = 0; j < V::N; ++j) acc[j] = fmaf(dzt, f[j], acc[j]);
    }
    T* o = out + (size_t)t * d + col;
    if (accumulate) {
      float f[V::N];
      load_as_float<T, T>(o, f);
#pragma unroll
      for (int j = 0; j < V::N; ++j) acc[j] += f[j];
    }
    V r;
    r.from_float(acc);
    r.store(o);
  }
}

// Backward of the combine, one warp per token.  Yp / Ys are the fp32 partials; dYp / dYs feed the
// backward GEMMs and have the storage type.
template <typename T>
__global__ void __launch_bounds__(256) combine_bwd_kernel(const T* __restrict__ dY, const float* __restrict__ Yp,
                                                          const float* __restrict__ w,
                                                          const int32_t* __restrict__ rows_g,
                                                          const float* __restrict__ Ys, const float* __restrict__ z,
                                                          T* __restrict__ dYp, float* __restrict__ dw,
                                                          T* __restrict__ dYs, float* __restrict__ dz, int N, int d,
                                                          int K) {
  using V = Vec16<T>;
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (t >= N) return;  // warp-uniform
  int my_row = 0;
  float my_w = 0.f;
  if (lane < K) { my_row = rows_g[(size_t)t * K + lane]; my_w = w[(size_t)t * K + lane]; }
  int rows[8];
  float wk[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    rows[k] = __shfl_sync(0xffffffffu, my_row, k);
    wk[k] = __shfl_sync(0xffffffffu, my_w, k);
  }
  const float g = Ys ? 1.0f / (1.0f + expf(-z[t])) : 0.f;
  float dot[9];
#pragma unroll
  for (int k = 0; k < 9; ++k) dot[k] = 0.f;
  const int chunks = d / V::N;
  for (int c = lane; c < chunks; c += 32) {
    const size_t col = (size_t)c * V::N;
    float gf[V::N];
    load_as_float<T, T>(dY + (size_t)t * d + col, gf);
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      if (k >= K) break;
      float yf[V::N], of[V::N];
      load_as_float<T, float>(Yp + (size_t)rows[k] * d + col, yf);
#pragma unroll
      for (int j = 0; j < V::N; ++j) { dot[k] = fmaf(gf[j], yf[j], dot[k]); of[j] = wk[k] * gf[j]; }
      V ov;
      ov.from_float(of);
      ov.store(dYp + (size_t)rows[k] * d + col);
    }
    if (Ys) {
      float sf[V::N], of[V::N];
      load_as_float<T, float>(Ys + (size_t)t * d + col, sf);
#pragma unroll
      for (int j = 0; j < V::N; ++j) { dot[8] = fmaf(gf[j], sf[j], dot[8]); of[j] = g * gf[j]; }
      V ov;
      ov.from_float(of);
      ov.store(dYs + (size_t)t * d + col);
    }
  }
#pragma unroll
  for (int k = 0; k < 9; ++k) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) dot[k] += __shfl_xor_sync(0xffffffffu, dot[k], off);
  }
  if (lane == 0) {
#pragma unroll
    for (int k = 0; k < 8; ++k)
      if (k < K) dw[(size_t)t * K + k] = dot[k];
    if (Ys) dz[t] = dot[8] * g * (1.0f - g);
  }
}

// dWg[e, cols] = sum over expert e's rows r of dl[slot_of_row[r]] * Xp[r, cols].
// grid (d / (32*VEC), E); 8 warps split the rows, partial sums merged in warp order.
template <typename T>
__global__ void __launch_bounds__(256) gate_wgrad_kernel(const T* __restrict__ Xp, const int32_t* __restrict__ counts,
                                                         const int32_t* __restrict__ offsets,
                                                         const int32_t* __restrict__ slot_of_row,
                                                         const float* __restrict__ dl, float* __restrict__ dWg, int d,
                                                         int accumulate) {
  using V = Vec16<T>;
  __shared__ float part[8][32 * V::N];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int e = blockIdx.y;
  const int col = (blockIdx.x * 32 + lane) * V::N;
  const int r0 = offsets[e], r1 = r0 + counts[e];
  float acc[V::N];
#pragma unroll
  for (int j = 0; j < V::N; ++j) acc[j] = 0.f;
  if (col < d) {
    for (int r = r0 + w; r < r1; r += 8) {
      const float g = dl[slot_of_row[r]];
      V v;
      v.load(Xp + (size_t)r * d + col);
      float f[V::N];
      v.to_float(f);
#pragma unroll
      for (int j = 0; j < V::N; ++j) acc[j] = fmaf(g, f[j], acc[j]);
    }
  }
#pragma unroll
  for (int j = 0; j < V::N; ++j) part[w][lane * V::N + j] = acc[j];
  __syncthreads();
  for (int i = threadIdx.x; i < 32 * V::N; i += blockDim.x) {
    float s = 0.f;
#pragma unroll
    for (int ww = 0; ww < 8; ++ww) s += part[ww][i];
    const int c = blockIdx.x * 32 * V::N + i;
    if (c < d) dWg[(size_t)e * d + c] = s + (accumulate ? dWg[(size_t)e * d + c] : 0.f);
  }
}

// Partial column sums  ws[split, cols] = sum_{t in split} dz[t] * X[t, cols];  second kernel adds the splits in order.
constexpr int GWS_SPLITS = 64;
template <typename T>
__global__ void __launch_bounds__(256) shared_gate_wgrad_kernel(const T* __restrict__ X, const float* __restrict__ dz,
                                                                float* __restrict__ ws, int N, int d) {
  using V = Vec16<T>;
  __shared__ float part[8][32 * V::N];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int col = (blockIdx.x * 32 + lane) * V::N;
  const int per = (N + GWS_SPLITS - 1) / GWS_SPLITS;
  const int t0 = blockIdx.y * per, t1 = min(N, t0 + per);
  float acc[V::N];
#pragma unroll
  for (int j = 0; j < V::N; ++j) acc[j] = 0.f;
  if (col < d) {
    for (int t = t0 + w; t < t1; t += 8) {
      const float g = dz[t];
      V v;
      v.load(X + (size_t)t * d + col);
      float f[V::N];
      v.to_float(f);
#pragma unroll
      for (int j = 0; j < V::N; ++j) acc[j] = fmaf(g, f[j], acc[j]);
    }
  }
#pragma unroll
  for (int j = 0; j < V::N; ++j) part[w][lane * V::N + j] = acc[j];
  __syncthreads();
  for (int i = threadIdx.x; i < 32 * V::N; i += blockDim.x) {
    float s = 0.f;
#pragma unroll
    for (int ww = 0; ww < 8; ++ww) s += part[ww][i];
    const int c = blockIdx.x * 32 * V::N + i;
    if (c < d) ws[(size_t)blockIdx.y * d + c] = s;
  }
}

__global__ void sum_splits_kernel(const float* __restrict__ ws, float* __restrict__ out, int d, int accumulate) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= d) return;
  float s = 0.f;
  for (int i = 0; i < GWS_SPLITS; ++i) s += ws[(size_t)i * d + c];
  out[c] = s + (accumulate ? out[c] : 0.f);
}

inline int perm_blocks(const c2r_config* cfg) {
  const int tb = perm_tokens_per_block(cfg->K);
  return (cfg->N + tb - 1) / tb;
}

size_t permute_ws_bytes(const c2r_config* cfg) {
  return sizeof(int32_t) * (size_t)(perm_blocks(cfg) > 0 ? perm_blocks(cfg) : 1) * cfg->E;
}
// ---- gate weight gradient as a tensor-core GEMM (bf16) -----------------------------------------
// dWg = dL^T X with dL dense [N,64] bf16: column e holds dl of the slot routed to expert e, column E
// the shared-gate gradient dz, everything else zero.  The token range is cut into splits that run
// as the "groups" of the grouped GEMM; their fp32 partial results are added in split order.
constexpr int GW_COLS = 64;

struct GateWgradPlan {
  int splits, per;                     // tokens per split (a multiple of 64)
  size_t off_partial, off_counts, bytes;
};
static GateWgradPlan gate_wgrad_plan(const c2r_config* cfg) {
  GateWgradPlan g;
  const int m_tiles = (cfg->d + 255) / 256;
  int splits = 64 / (m_tiles > 0 ? m_tiles : 1);
  if (splits < 1) splits = 1;
  int per = (cfg->N + splits - 1) / splits;
  per = (per + 63) / 64 * 64;
  if (per < 64) per = 64;
  splits = cfg->N > 0 ? (cfg->N + per - 1) / per : 1;
  g.splits = splits; g.per = per;
  size_t o = ((size_t)(cfg->N > 0 ? cfg->N : 1) * GW_COLS * 2 + 255) / 256 * 256;
  g.off_partial = o;
  o += ((size_t)splits * GW_COLS * cfg->d * sizeof(float) + 255) / 256 * 256;
  g.off_counts = o;
  o += 256 * ((2 * (size_t)splits + 1) * sizeof(int32_t) / 256 + 1);
  g.bytes = o;
  return g;
}

// one block per expert: scatter the slot gradients of the expert's rows into its column of dL
__global__ void __launch_bounds__(256) gate_dl_scatter_kernel(const int32_t* __restrict__ counts,
                                                              const int32_t* __restrict__ offsets,
                                                              const int32_t* __restrict__ slot_of_row,
                                                              const float* __restrict__ dl,
                                                              __nv_bfloat16* __restrict__ dLd, int K) {
  const int e = blockIdx.x;
  const int r0 = offsets[e], n = counts[e];
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const int sl = slot_of_row[r0 + i];
    if (sl >= 0) dLd[(size_t)(sl / K) * GW_COLS + e] = __float2bfloat16_rn(dl[sl]);
  }
}
// The whole dense row of a token in one pass (needs idx): a warp per token, lane l owns columns 2l and 2l+1, so
// the row leaves as one 128-byte store and neither a memset nor the per-expert scatter is needed.  Block 0 also
// writes the split table.
__global__ void __launch_bounds__(256) gate_dl_dense_kernel(const int32_t* __restrict__ idx, const float* __restrict__ dl,
                                                            const float* __restrict__ dz, __nv_bfloat16* __restrict__ dLd,
                                                            int N, int E, int K, int per, int splits,
                                                            int32_t* __restrict__ split_counts,
                                                            int32_t* __restrict__ split_offsets) {
  if (blockIdx.x == 0 && (int)threadIdx.x <= splits) {
    const int lo = min(N, (int)threadIdx.x * per);
    split_offsets[threadIdx.x] = lo;
    if ((int)threadIdx.x < splits) split_counts[threadIdx.x] = min(N, lo + per) - lo;
  }
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (t >= N) return;  // warp-uniform
  float v0 = 0.f, v1 = 0.f;
  for (int k = 0; k < K; ++k) {
    const int e = min(max(idx[(size_t)t * K + k], 0), E - 1);
    const float g = dl[(size_t)t * K + k];
    if ((e >> 1) == lane) { if (e & 1) v1 = g; else v0 = g; }
  }
  if (dz != nullptr && (E >> 1) == lane) { if (E & 1) v1 = dz[t]; else v0 = dz[t]; }
  reinterpret_cast<__nv_bfloat162*>(dLd + (size_t)t * GW_COLS)[lane] = __floats2bfloat162_rn(v0, v1);
}
// shared-gate column and the split table
__global__ void __launch_bounds__(256) gate_dz_kernel(const float* __restrict__ dz, __nv_bfloat16* __restrict__ dLd, int N,
                                                      int E, int per, int splits, int32_t* __restrict__ split_counts,
                                                      int32_t* __restrict__ split_offsets) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (dz != nullptr && t < N) dLd[(size_t)t * GW_COLS + E] = __float2bfloat16_rn(dz[t]);
  if (blockIdx.x == 0 && threadIdx.x <= splits) {
    const int lo = min(N, threadIdx.x * per);
    split_offsets[threadIdx.x] = lo;
    if (threadIdx.x < splits) split_counts[threadIdx.x] = min(N, lo + per) - lo;
  }
}
__global__ void __launch_bounds__(256) gate_wgrad_reduce_kernel(const float* __restrict__ partial, int splits, int E, int d,
                                                                float* __restrict__ dWg, float* __restrict__ dwsg,
                                                                int accumulate) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  const int e = blockIdx.y;  // 0..E: row E is the shared gate
  if (c >= d) return;
  float acc = 0.f;
  for (int sp = 0; sp < splits; ++sp) acc += partial[((size_t)sp * GW_COLS + e) * d + c];
  if (e < E) dWg[(size_t)e * d + c] = acc + (accumulate ? dWg[(size_t)e * d + c] : 0.f);
  else if (dwsg != nullptr) dwsg[c] = acc + (accumulate ? dwsg[c] : 0.f);
}

size_t gate_bwd_ws_bytes(const c2r_config* cfg) {
  const size_t simt = sizeof(float) * (size_t)GWS_SPLITS * cfg->d;
  const size_t tc = cfg->dtype == C2R_BF16 ? gate_wgrad_plan(cfg).bytes : 0;
  return simt > tc ? simt : tc;
}

// have_hist: block_counts already holds the per-block expert counts of idx in this blocking (the routing
// kernel wrote them), so the histogram launch is skipped.  w / w_row (both or neither): see rank_and_write.
template <typename T>
int permute_impl(const c2r_config* cfg, const int32_t* idx, const int32_t* expert_rank, const T* X, int32_t* counts,
                 int32_t* offsets, int32_t* row_of_slot, int32_t* slot_of_row, T* Xp, int32_t* status, void* ws,
                 cudaStream_t s, bool have_hist, const float* w, float* w_row) {
  const long long NK = (long long)cfg->N * cfg->K;
  const long long R = permuted_rows(cfg);
  const int nb = perm_blocks(cfg);
  const int spb = perm_tokens_per_block(cfg->K) * cfg->K;
  int32_t* block_counts = (int32_t*)ws;
  if (w == nullptr) w_row = nullptr;
  if (nb > 0 && !have_hist) {
    perm_hist_kernel<<<nb, PERM_THREADS, 0, s>>>(idx, NK, cfg->E, spb, block_counts, status, 0);
    C2R_LAUNCH_CHECK();
  }
  if (nb > 0 && nb <= PERM_FUSED_MAX_BLOCKS) {
    perm_rank_fused_kernel<<<nb, PERM_THREADS, 0, s>>>(idx, NK, cfg->E, spb, block_counts, nb, expert_rank, cfg->row_align,
                                                       R, counts, offsets, row_of_slot, slot_of_row, w, w_row, status);
    C2R_LAUNCH_CHECK();
  } else {
    C2R_CUDA(cudaMemsetAsync(slot_of_row, 0xFF, sizeof(int32_t) * R, s));
    if (w_row != nullptr) C2R_CUDA(cudaMemsetAsync(w_row, 0, sizeof(float) * R, s));
    perm_scan_kernel<<<1, 1024, 0, s>>>(block_counts, nb, cfg->E, expert_rank, cfg->row_align, counts, offsets, status);
    C2R_LAUNCH_CHECK();
    if (nb > 0) {
      perm_rank_kernel<<<nb, PERM_THREADS, 0, s>>>(idx, NK, cfg->E, spb, block_counts, offsets, row_of_slot, slot_of_row, 0,
                                                   w, w_row);
      C2R_LAUNCH_CHECK();
    }
  }
  if (X != nullptr) {
    // the gather, plus one block per expert that zeroes the padding rows closing its aligned segment
    const int token_blocks = (cfg->N + 7) / 8;
    const int pad_blocks = cfg->row_align > 1 ? cfg->E : 0;
    if (token_blocks + pad_blocks > 0) {
      permute_rows_kernel<T><<<token_blocks + pad_blocks, 256, 0, s>>>(X, row_of_slot, Xp, cfg->N, cfg->d, cfg->K, counts,
                                                                    offsets, token_blocks, cfg->row_align);
      C2R_LAUNCH_CHECK();
    }
  }
  return C2R_OK;
}

}  // namespace c2r

using namespace c2r;

int c2r::permute_call(const c2r_config* cfg, const int32_t* idx, const int32_t* expert_rank, const void* X, int32_t* counts,
                      int32_t* offsets, int32_t* row_of_slot, int32_t* slot_of_row, void* Xp, int32_t* status, void* ws,
                      size_t ws_bytes, void* stream, bool have_hist, const float* w, float* w_row) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(idx && counts && offsets && row_of_slot && slot_of_row, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(!X || Xp, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(!w_row || w, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(ws && ws_bytes >= permute_ws_bytes(cfg), C2R_ERR_WORKSPACE);
  if (cfg->dtype == C2R_BF16)
    return permute_impl<__nv_bfloat16>(cfg, idx, expert_rank, (const __nv_bfloat16*)X, counts, offsets, row_of_slot,
                                       slot_of_row, (__nv_bfloat16*)Xp, status, ws, as_stream(stream), have_hist, w, w_row);
  return permute_impl<float>(cfg, idx, expert_rank, (const float*)X, counts, offsets, row_of_slot, slot_of_row,
                             (float*)Xp, status, ws, as_stream(stream), have_hist, w, w_row);
}

extern "C" int c2r_permute(const c2r_config* cfg, const int32_t* idx, const int32_t* expert_rank, const void* X,
                           const float* w, int32_t* counts, int32_t* offsets, int32_t* row_of_slot, int32_t* slot_of_row,
                           void* Xp, float* w_row, int32_t* status, void* ws, size_t ws_bytes, int ws_has_histogram,
                           void* stream) {
  return permute_call(cfg, idx, expert_rank, X, counts, offsets, row_of_slot, slot_of_row, Xp, status, ws, ws_bytes, stream,
                      ws_has_histogram != 0 && cfg && cfg->N > 0, w, w_row);
}

extern "C" int c2r_permute_rows(const c2r_config* cfg, const void* X, const int32_t* row_of_slot, const int32_t* counts,
                                const int32_t* offsets, void* Xp, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(X && row_of_slot && counts && offsets && Xp, C2R_ERR_INVALID_ARG);
  const int token_blocks = (cfg->N + 7) / 8;
  const int pad_blocks = cfg->row_align > 1 ? cfg->E : 0;
  if (token_blocks + pad_blocks == 0) return C2R_OK;
  cudaStream_t s = as_stream(stream);
  if (cfg->dtype == C2R_BF16)
    permute_rows_kernel<__nv_bfloat16><<<token_blocks + pad_blocks, 256, 0, s>>>(
        (const __nv_bfloat16*)X, row_of_slot, (__nv_bfloat16*)Xp, cfg->N, cfg->d, cfg->K, counts, offsets, token_blocks,
        cfg->row_align);
  else
    permute_rows_kernel<float><<<token_blocks + pad_blocks, 256, 0, s>>>((const float*)X, row_of_slot, (float*)Xp, cfg->N,
                                                                         cfg->d, cfg->K, counts, offsets, token_blocks,
                                                                         cfg->row_align);
  C2R_LAUNCH_CHECK();
  return C2R_OK;
}

template <typename T>
static int gather_sum_launch(const c2r_config* cfg, const void* src, const int32_t* rows, const float* coef,
                             const void* extra, const float* z, const int32_t* idx, const float* dl, const void* Wg,
                             const float* dz, const void* wsg, void* out, int accumulate, cudaStream_t s) {
  if (cfg->N == 0) return C2R_OK;
  gather_sum_kernel<T><<<(cfg->N + 7) / 8, 256, 0, s>>>((const float*)src, rows, coef, (const float*)extra, z, idx, dl,
                                                        (const T*)Wg, dz, (const T*)wsg, (T*)out, accumulate, cfg->N,
                                                        cfg->d, cfg->K);
  C2R_LAUNCH_CHECK();
  return C2R_OK;
}

extern "C" int c2r_combine(const c2r_config* cfg, const void* Yp, const float* w, const int32_t* row_of_slot,
                           const void* Ys, const float* z, void* Y, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE((Yp || Ys) && row_of_slot && Y, C2R_ERR_INVALID_ARG);
  if (cfg->dtype == C2R_BF16)
    return gather_sum_launch<__nv_bfloat16>(cfg, Yp, row_of_slot, w, Ys, z, nullptr, nullptr, nullptr, nullptr,
                                            nullptr, Y, 0, as_stream(stream));
  return gather_sum_launch<float>(cfg, Yp, row_of_slot, w, Ys, z, nullptr, nullptr, nullptr, nullptr, nullptr, Y, 0,
                                  as_stream(stream));
}

extern "C" int c2r_unpermute_grad(const c2r_config* cfg, const void* dXp, const int32_t* row_of_slot, const void* dXs,
                                  const int32_t* idx, const float* dl, const void* Wg, const float* dz,
                                  const void* wsg, void* dX, int accumulate, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE((dXp || dXs) && row_of_slot && dX, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(!dl || (idx && Wg), C2R_ERR_INVALID_ARG);
  C2R_REQUIRE((dz == nullptr) == (wsg == nullptr), C2R_ERR_INVALID_ARG);
  if (cfg->dtype == C2R_BF16)
    return gather_sum_launch<__nv_bfloat16>(cfg, dXp, row_of_slot, nullptr, dXs, nullptr, idx, dl, Wg, dz, wsg, dX,
                                            accumulate, as_stream(stream));
  return gather_sum_launch<float>(cfg, dXp, row_of_slot, nullptr, dXs, nullptr, idx, dl, Wg, dz, wsg, dX, accumulate,
                                  as_stream(stream));
}

template <typename T>
static int combine_bwd_launch(const c2r_config* cfg, const void* dY, const void* Yp, const float* w,
                              const int32_t* rows, const int32_t* slot_of_row, const void* Ys, const float* z,
                              void* dYp, float* dw, void* dYs, float* dz, cudaStream_t s) {
  const long long R = permuted_rows(cfg);
  if (cfg->N > 0) {
    combine_bwd_kernel<T><<<(cfg->N + 7) / 8, 256, 0, s>>>((const T*)dY, (const float*)Yp, w, rows, (const float*)Ys, z,
                                                           (T*)dYp, dw, (T*)dYs, dz, cfg->N, cfg->d, cfg->K);
    C2R_LAUNCH_CHECK();
  }
  if (R > (long long)cfg->N * cfg->K) {
    int blocks = (int)((R + 7) / 8);
    if (blocks > 1184) blocks = 1184;
    zero_pad_rows_kernel<T><<<blocks, 256, 0, s>>>(slot_of_row, (T*)dYp, R, cfg->d);
    C2R_LAUNCH_CHECK();
  }
  return C2R_OK;
}

extern "C" int c2r_combine_bwd(const c2r_config* cfg, const void* dY, const void* Yp, const float* w,
                               const int32_t* row_of_slot, const int32_t* slot_of_row, const void* Ys, const float* z,
                               void* dYp, float* dw, void* dYs, float* dz, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(dY && Yp && w && row_of_slot && slot_of_row && dYp && dw, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(!Ys || (z && dYs && dz), C2R_ERR_INVALID_ARG);
  if (cfg->dtype == C2R_BF16)
    return combine_bwd_launch<__nv_bfloat16>(cfg, dY, Yp, w, row_of_slot, slot_of_row, Ys, z, dYp, dw, dYs, dz,
                                             as_stream(stream));
  return combine_bwd_launch<float>(cfg, dY, Yp, w, row_of_slot, slot_of_row, Ys, z, dYp, dw, dYs, dz,
                                   as_stream(stream));
}

template <typename T>
static int gate_bwd_launch(const c2r_config* cfg, const void* X, const void* Xp, const int32_t* counts,
                           const int32_t* offsets, const int32_t* slot_of_row, const int32_t* idx, const float* dl,
                           const float* dz, float* dWg, float* dwsg, int accumulate, void* ws, cudaStream_t s) {
  using V = Vec16<T>;
  if (sizeof(T) == 2 && X != nullptr && ws != nullptr && cfg->N > 0 && cfg->d % 16 == 0 && cfg->E < GW_COLS &&
      ((uintptr_t)X & 15u) == 0 && tc_supported(cfg, 1, 16, cfg->N)) {
    const GateWgradPlan g = gate_wgrad_plan(cfg);
    __nv_bfloat16* dLd = (__nv_bfloat16*)ws;
    float* partial = (float*)((char*)ws + g.off_partial);
    int32_t* sc = (int32_t*)((char*)ws + g.off_counts);
    int32_t* so = sc + g.splits;
    if (idx != nullptr) {
      gate_dl_dense_kernel<<<(cfg->N + 7) / 8, 256, 0, s>>>(idx, dl, dz, dLd, cfg->N, cfg->E, cfg->K, g.per, g.splits, sc, so);
      C2R_LAUNCH_CHECK();
    } else {
      C2R_CUDA(cudaMemsetAsync(dLd, 0, (size_t)cfg->N * GW_COLS * 2, s));
      gate_dl_scatter_kernel<<<cfg->E, 256, 0, s>>>(counts, offsets, slot_of_row, dl, dLd, cfg->K);
      C2R_LAUNCH_CHECK();
      gate_dz_kernel<<<(cfg->N + 255) / 256, 256, 0, s>>>(dz, dLd, cfg->N, cfg->E, g.per, g.splits, sc, so);
      C2R_LAUNCH_CHECK();
    }
    int rc = tc_gate_wgrad(cfg, X, dLd, partial, g.splits, sc, so, nullptr, s);
    if (rc) return rc;
    gate_wgrad_reduce_kernel<<<dim3((cfg->d + 255) / 256, cfg->E + 1), 256, 0, s>>>(partial, g.splits, cfg->E, cfg->d,
                                                                                   dWg, dz ? dwsg : nullptr, accumulate);
    C2R_LAUNCH_CHECK();
    return C2R_OK;
  }
  C2R_REQUIRE(Xp != nullptr, C2R_ERR_INVALID_ARG);  // the row-serial form walks the permuted rows
  const int colblocks = (cfg->d + 32 * V::N - 1) / (32 * V::N);
  gate_wgrad_kernel<T><<<dim3(colblocks, cfg->E), 256, 0, s>>>((const T*)Xp, counts, offsets, slot_of_row, dl, dWg,
                                                               cfg->d, accumulate);
  C2R_LAUNCH_CHECK();
  if (dz) {
    shared_gate_wgrad_kernel<T><<<dim3(colblocks, GWS_SPLITS), 256, 0, s>>>((const T*)X, dz, (float*)ws, cfg->N, cfg->d);
    C2R_LAUNCH_CHECK();
    sum_splits_kernel<<<(cfg->d + 255) / 256, 256, 0, s>>>((const float*)ws, dwsg, cfg->d, accumulate);
    C2R_LAUNCH_CHECK();
  }
  return C2R_OK;
}

extern "C" int c2r_gate_bwd(const c2r_config* cfg, const void* X, const void* Xp, const int32_t* counts,
                            const int32_t* offsets, const int32_t* slot_of_row, const int32_t* idx, const float* dl,
                            const float* dz, float* dWg, float* dwsg, int accumulate, void* ws, size_t ws_bytes,
                            void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(counts && offsets && slot_of_row && dl && dWg, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(!dz || (X && dwsg), C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(!dz || (ws && ws_bytes >= gate_bwd_ws_bytes(cfg)), C2R_ERR_WORKSPACE);
  if (ws && ws_bytes < gate_bwd_ws_bytes(cfg)) ws = nullptr;  // too small for the tensor-core form: row-serial kernel
  if (cfg->dtype == C2R_BF16)
    return gate_bwd_launch<__nv_bfloat16>(cfg, X, Xp, counts, offsets, slot_of_row, idx, dl, dz, dWg, dwsg, accumulate, ws,
                                          as_stream(stream));
  return gate_bwd_launch<float>(cfg, X, Xp, counts, offsets, slot_of_row, idx, dl, dz, dWg, dwsg, accumulate, ws,
                                as_stream(stream));
}

// ---------------------------------------------------------------------------------------------
// c2r_permute_static: the same dispatch with its scratch in this library's own device image.
// ---------------------------------------------------------------------------------------------
namespace c2r {

constexpr size_t PERM_STATIC_INTS = C2R_PERMUTE_STATIC_SCRATCH_BYTES / sizeof(int32_t);

// Per-block expert counts of c2r_permute_static.  One copy lives on every GPU that loads the
// library, from load until the process exits.  Nothing in it has to start at zero: each call
// writes every entry it later reads (the histogram kernel stores all E counts of every block it
// launches), so the leftovers of the previous call are never observed.
static __device__ __align__(256) int32_t g_perm_static_scratch[PERM_STATIC_INTS];

// Device address of the array above on the current device.  In host code the array's name only
// stands for the symbol; the address a kernel can use has to be asked for, per device.
static int perm_static_scratch(int32_t** out) {
  constexpr int MAX_DEV = 64;
  static int32_t* cache[MAX_DEV] = {};
  int dev = 0;
  C2R_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= MAX_DEV) return C2R_ERR_UNSUPPORTED_SHAPE;
  int32_t* p = __atomic_load_n(&cache[dev], __ATOMIC_ACQUIRE);
  if (p == nullptr) {
    void* addr = nullptr;
    C2R_CUDA(cudaGetSymbolAddress(&addr, g_perm_static_scratch));
    p = static_cast<int32_t*>(addr);
    __atomic_store_n(&cache[dev], p, __ATOMIC_RELEASE);  // racing first calls store the same value
  }
  *out = p;
  return C2R_OK;
}

}  // namespace c2r

extern "C" int c2r_permute_static(const c2r_config* cfg, const int32_t* idx, const int32_t* expert_rank, const void* X,
                                  int32_t* counts, int32_t* offsets, int32_t* row_of_slot, int32_t* slot_of_row,
                                  void* Xp, int32_t* status, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(idx && counts && offsets && row_of_slot && slot_of_row, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(!X || Xp, C2R_ERR_INVALID_ARG);
  // the scratch holds one int32 per (block of the sort, expert)
  if (permute_ws_bytes(cfg) > C2R_PERMUTE_STATIC_SCRATCH_BYTES) return C2R_ERR_STATIC_SCRATCH;
  int32_t* scratch = nullptr;
  rc = perm_static_scratch(&scratch);
  if (rc) return rc;
  if (cfg->dtype == C2R_BF16)
    return permute_impl<__nv_bfloat16>(cfg, idx, expert_rank, (const __nv_bfloat16*)X, counts, offsets, row_of_slot,
                                       slot_of_row, (__nv_bfloat16*)Xp, status, scratch, as_stream(stream), false, nullptr,
                                       nullptr);
  return permute_impl<float>(cfg, idx, expert_rank, (const float*)X, counts, offsets, row_of_slot, slot_of_row,
                             (float*)Xp, status, scratch, as_stream(stream), false, nullptr, nullptr);
}

// ---------------------------------------------------------------------------------------------
// Zero-redundancy dispatch (Sec. 3.4) in two stages: one copy of a token per partition that hosts
// any of its experts (what an all-to-all would carry), then replication inside the partition into
// the per-expert layout.
// ---------------------------------------------------------------------------------------------
namespace c2r {

// key[t,k] = partition of slot (t,k) if no earlier slot of the token maps to that partition, else -1.
__global__ void __launch_bounds__(256) dedup_keys_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ part,
                                                         int32_t* __restrict__ key, int N, int E, int K, int P) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= N) return;
  int q[8];
  for (int k = 0; k < K; ++k) {
    const int e = min(max(idx[(size_t)t * K + k], 0), E - 1);
    q[k] = min(max(part[e], 0), P - 1);
    bool first = true;
    for (int j = 0; j < k; ++j) first = first && (q[j] != q[k]);
    key[(size_t)t * K + k] = first ? q[k] : -1;
  }
}

// Slots that are not the first of their (token, partition) read the row of the one that is.
__global__ void __launch_bounds__(256) dedup_fill_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ part,
                                                         const int32_t* __restrict__ key,
                                                         int32_t* __restrict__ recv_row_of_slot, int N, int E, int K, int P) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= N) return;
  for (int k = 1; k < K; ++k) {
    if (key[(size_t)t * K + k] >= 0) continue;
    const int q = min(max(part[min(max(idx[(size_t)t * K + k], 0), E - 1)], 0), P - 1);
    for (int j = 0; j < k; ++j)
      if (key[(size_t)t * K + j] == q) { recv_row_of_slot[(size_t)t * K + k] = recv_row_of_slot[(size_t)t * K + j]; break; }
  }
}

__global__ void __launch_bounds__(256) dedup_tokens_kernel(const int32_t* __restrict__ slot_of_recv_row,
                                                           int32_t* __restrict__ token_of_recv_row, long long cap, int K) {
  const long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= cap) return;
  const int s = slot_of_recv_row[r];
  token_of_recv_row[r] = s >= 0 ? s / K : -1;
}

// Stage 1, one warp per token: the token's row is read once and written to the receive row of every
// partition that needs it.
template <typename T>
__global__ void __launch_bounds__(256) dedup_send_kernel(const T* __restrict__ X, const int32_t* __restrict__ key,
                                                         const int32_t* __restrict__ recv_row_of_slot, T* __restrict__ Xr,
                                                         int N, int d, int K) {
  using V = Vec16<T>;
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (t >= N) return;  // warp-uniform
  int my_row = -1;
  if (lane < K && key[(size_t)t * K + lane] >= 0) my_row = recv_row_of_slot[(size_t)t * K + lane];
  int rows[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) rows[k] = __shfl_sync(0xffffffffu, my_row, k);
  const int chunks = d / V::N;
  const T* src = X + (size_t)t * d;
  for (int c = lane; c < chunks; c += 32) {
    V v;
    v.load(src + (size_t)c * V::N);
#pragma unroll
    for (int k = 0; k < 8; ++k)
      if (k < K && rows[k] >= 0) v.store(Xr + (size_t)rows[k] * d + (size_t)c * V::N);
  }
}

// Stage 2, one warp per row of the per-expert layout: Xp[r] = Xr[recv_row_of_slot[slot_of_row[r]]], padding rows zero.
template <typename T>
__global__ void __launch_bounds__(256) dedup_replicate_kernel(const T* __restrict__ Xr, const int32_t* __restrict__ slot_of_row,
                                                              const int32_t* __restrict__ recv_row_of_slot,
                                                              T* __restrict__ Xp, long long R, int d) {
  using V = Vec16<T>;
  const int lane = threadIdx.x & 31;
  const long long r = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= R) return;  // warp-uniform
  const int s = slot_of_row[r];
  const int chunks = d / V::N;
  T* dst = Xp + (size_t)r * d;
  if (s < 0) {
    V zero;
    float zf[V::N] = {};
    zero.from_float(zf);
    for (int c = lane; c < chunks; c += 32) zero.store(dst + (size_t)c * V::N);
    return;
  }
  const T* src = Xr + (size_t)recv_row_of_slot[s] * d;
  for (int c = lane; c < chunks; c += 32) {
    V v;
    v.load(src + (size_t)c * V::N);
    v.store(dst + (size_t)c * V::N);
  }
}

static size_t align256_(size_t x) { return (x + 255) / 256 * 256; }

size_t dispatch_dedup_ws_bytes(const c2r_config* cfg) {
  const size_t nk = (size_t)cfg->N * cfg->K;
  return align256_(permute_ws_bytes(cfg)) + 2 * align256_(sizeof(int32_t) * (nk > 0 ? nk : 1));
}

template <typename T>
static int dispatch_dedup_impl(const c2r_config* cfg, const int32_t* idx, const int32_t* part, const int32_t* expert_rank,
                               const T* X, int32_t* counts, int32_t* offsets, int32_t* row_of_slot, int32_t* slot_of_row,
                               int32_t* recv_counts, int32_t* recv_offsets, int32_t* recv_row_of_slot,
                               int32_t* token_of_recv_row, T* Xr, T* Xp, int32_t* status, void* ws, cudaStream_t s) {
  const int N = cfg->N, K = cfg->K, E = cfg->E, P = cfg->P;
  const long long NK = (long long)N * K;
  const long long R = permuted_rows(cfg);
  const long long cap = (long long)N * (K < P ? K : P);  // rows the receive side can need
  // the per-expert layout itself (counts, offsets, both row maps) is the plain dispatch's
  int rc = permute_impl<T>(cfg, idx, expert_rank, nullptr, counts, offsets, row_of_slot, slot_of_row, nullptr, status, ws, s,
                           false, nullptr, nullptr);
  if (rc) return rc;
  int32_t* block_counts = (int32_t*)ws;  // free again: the calls above are ordered on the stream
  int32_t* key = (int32_t*)((char*)ws + align256_(permute_ws_bytes(cfg)));
  int32_t* slot_of_recv_row = (int32_t*)((char*)key + align256_(sizeof(int32_t) * (NK > 0 ? NK : 1)));
  const int nb = perm_blocks(cfg);
  const int spb = perm_tokens_per_block(K) * K;
  if (N > 0) {
    dedup_keys_kernel<<<(N + 255) / 256, 256, 0, s>>>(idx, part, key, N, E, K, P);
    C2R_LAUNCH_CHECK();
    C2R_CUDA(cudaMemsetAsync(slot_of_recv_row, 0xFF, sizeof(int32_t) * NK, s));
    perm_hist_kernel<<<nb, PERM_THREADS, 0, s>>>(key, NK, P, spb, block_counts, status, 1);
    C2R_LAUNCH_CHECK();
  }
  perm_scan_kernel<<<1, 1024, 0, s>>>(block_counts, nb, P, nullptr, 1, recv_counts, recv_offsets, nullptr);
  C2R_LAUNCH_CHECK();
  if (N > 0) {
    perm_rank_kernel<<<nb, PERM_THREADS, 0, s>>>(key, NK, P, spb, block_counts, recv_offsets, recv_row_of_slot,
                                                 slot_of_recv_row, 1, nullptr, nullptr);
    C2R_LAUNCH_CHECK();
    dedup_fill_kernel<<<(N + 255) / 256, 256, 0, s>>>(idx, part, key, recv_row_of_slot, N, E, K, P);
    C2R_LAUNCH_CHECK();
    dedup_tokens_kernel<<<(int)((cap + 255) / 256), 256, 0, s>>>(slot_of_recv_row, token_of_recv_row, cap, K);
    C2R_LAUNCH_CHECK();
    if (X != nullptr) {
      dedup_send_kernel<T><<<(N + 7) / 8, 256, 0, s>>>(X, key, recv_row_of_slot, Xr, N, cfg->d, K);
      C2R_LAUNCH_CHECK();
    }
  }
  if (X != nullptr && R > 0) {
    dedup_replicate_kernel<T><<<(int)((R + 7) / 8), 256, 0, s>>>(Xr, slot_of_row, recv_row_of_slot, Xp, R, cfg->d);
    C2R_LAUNCH_CHECK();
  }
  return C2R_OK;
}

}  // namespace c2r

extern "C" int c2r_dispatch_dedup(const c2r_config* cfg, const int32_t* idx, const int32_t* part,
                                  const int32_t* expert_rank, const void* X, int32_t* counts, int32_t* offsets,
                                  int32_t* row_of_slot, int32_t* slot_of_row, int32_t* recv_counts,
                                  int32_t* recv_offsets, int32_t* recv_row_of_slot, int32_t* token_of_recv_row,
                                  void* Xr, void* Xp, int32_t* status, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(idx && part && counts && offsets && row_of_slot && slot_of_row, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(recv_counts && recv_offsets && recv_row_of_slot && token_of_recv_row, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(cfg->P >= 1 && cfg->P <= cfg->E, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(!X || (Xr && Xp), C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(ws && ws_bytes >= dispatch_dedup_ws_bytes(cfg), C2R_ERR_WORKSPACE);
  if (cfg->dtype == C2R_BF16)
    return dispatch_dedup_impl<__nv_bfloat16>(cfg, idx, part, expert_rank, (const __nv_bfloat16*)X, counts, offsets,
                                              row_of_slot, slot_of_row, recv_counts, recv_offsets, recv_row_of_slot,
                                              token_of_recv_row, (__nv_bfloat16*)Xr, (__nv_bfloat16*)Xp, status, ws,
                                              as_stream(stream));
  return dispatch_dedup_impl<float>(cfg, idx, part, expert_rank, (const float*)X, counts, offsets, row_of_slot, slot_of_row,
                                    recv_counts, recv_offsets, recv_row_of_slot, token_of_recv_row, (float*)Xr, (float*)Xp,
                                    status, ws, as_stream(stream));
}
