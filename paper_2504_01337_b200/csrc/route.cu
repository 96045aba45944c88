// Gate logits, C2R / Top-K routing, collaboration matrix, Top-T sets and dispatch volume.
// Integer outputs are exact and independent of scheduling (integer atomics only where the
// result does not depend on their order).
#include "c2r_common.cuh"
#include "gemm.h"

namespace c2r {

thread_local int g_last_cuda_error = 0;
unsigned long long g_launch_count = 0;

// ---------------------------------------------------------------------------------------------
// Gate logits (Eq. 1): L = X Wg^T, z = X wsg.  CUDA-core kernel: a block owns TM tokens and all
// E (+1) gate columns, streams d in chunks through shared memory; X is read from HBM once.
// ---------------------------------------------------------------------------------------------
constexpr int GL_TM = 32;   // tokens per block
constexpr int GL_DK = 64;   // d-chunk
constexpr int GL_COLS = 64; // gate columns held (E routed + optional shared gate)

template <typename T>
__global__ void __launch_bounds__(256) gate_logits_kernel(const T* __restrict__ X, const T* __restrict__ Wg,
                                                          const T* __restrict__ wsg, float* __restrict__ L,
                                                          float* __restrict__ z, int N, int d, int E) {
  __shared__ float sx[GL_TM][GL_DK + 1];
  __shared__ float sw[GL_COLS][GL_DK + 1];
  const int tid = threadIdx.x;
  const int t0 = blockIdx.x * GL_TM;
  const int cols = E + (wsg != nullptr ? 1 : 0);
  const int tx = tid & 15;  // column group: columns tx, tx+16, tx+32, tx+48
  const int ty = tid >> 4;  // token group: tokens ty, ty+16
  float acc[2][4] = {};
  for (int k0 = 0; k0 < d; k0 += GL_DK) {
    for (int i = tid; i < GL_TM * GL_DK; i += 256) {
      int r = i / GL_DK, c = i % GL_DK;
      int t = t0 + r;
      sx[r][c] = (t < N && k0 + c < d) ? to_f32(X[(size_t)t * d + k0 + c]) : 0.f;
    }
    for (int i = tid; i < GL_COLS * GL_DK; i += 256) {
      int r = i / GL_DK, c = i % GL_DK;
      float v = 0.f;
      if (k0 + c < d) {
        if (r < E) v = to_f32(Wg[(size_t)r * d + k0 + c]);
        else if (r == E && wsg != nullptr) v = to_f32(wsg[k0 + c]);
      }
      sw[r][c] = v;
    }
    __syncthreads();
#pragma unroll 8
    for (int k = 0; k < GL_DK; ++k) {
      float xa = sx[ty][k], xb = sx[ty + 16][k];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float wv = sw[tx + 16 * j][k];
        acc[0][j] = fmaf(xa, wv, acc[0][j]);
        acc[1][j] = fmaf(xb, wv, acc[1][j]);
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    int t = t0 + ty + 16 * i;
    if (t >= N) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int c = tx + 16 * j;
      if (c < E) L[(size_t)t * E + c] = acc[i][j];
      else if (c == E && c < cols) z[t] = acc[i][j];
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Routing (Sec. 3.3 step 2).  One warp per token; lane l holds logits l and l+32.  K rounds of a
// shuffle arg-max under the total order (value desc, index asc); after round 0 the candidate set
// is intersected with the top-1 expert's collaborator mask.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ bool better(float va, int ia, float vb, int ib) {
  return (va > vb) || (va == vb && ia < ib);
}

constexpr int ROUTE_WARPS = 32;

// A block owns tokens_per_block consecutive tokens (the blocking of the dispatch's counting sort), a warp
// every ROUTE_WARPS-th of them.  block_counts (optional): [blocks][E] experts' slot counts of the block's
// tokens -- the histogram the dispatch starts from, so it need not read idx again to build it.  A token's
// K experts are distinct, hence lanes 0..K-1 bump different counters of the warp's private row: no atomics.
__global__ void __launch_bounds__(ROUTE_WARPS * 32) route_kernel(const float* __restrict__ L, const uint64_t* __restrict__ mask,
                                                                 int32_t* __restrict__ idx, float* __restrict__ w,
                                                                 float* __restrict__ p, int32_t* __restrict__ status, int N,
                                                                 int E, int K, int renorm, int tokens_per_block,
                                                                 int32_t* __restrict__ block_counts) {
  __shared__ int warp_cnt[ROUTE_WARPS][64];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (block_counts != nullptr) {
    for (int i = threadIdx.x; i < ROUTE_WARPS * 64; i += blockDim.x) (&warp_cnt[0][0])[i] = 0;
    __syncthreads();
  }
  const float NEG_INF = -INFINITY;
  const int t_end = min(N, (int)(blockIdx.x + 1) * tokens_per_block);
  int flags = 0;
  int t = blockIdx.x * tokens_per_block + warp;
  float n0 = NEG_INF, n1 = NEG_INF;  // the next token's logits, requested one token ahead
  if (t < t_end) {
    if (lane < E) n0 = L[(size_t)t * E + lane];
    if (lane + 32 < E) n1 = L[(size_t)t * E + lane + 32];
  }
  for (; t < t_end; t += ROUTE_WARPS) {
    float v0 = n0, v1 = n1;
    if (t + ROUTE_WARPS < t_end) {
      if (lane < E) n0 = L[(size_t)(t + ROUTE_WARPS) * E + lane];
      if (lane + 32 < E) n1 = L[(size_t)(t + ROUTE_WARPS) * E + lane + 32];
    }
    if (v0 != v0) { v0 = NEG_INF; flags |= C2R_STATUS_NAN_LOGIT; }
    if (v1 != v1) { v1 = NEG_INF; flags |= C2R_STATUS_NAN_LOGIT; }
    uint64_t avail = (E == 64) ? ~0ull : ((1ull << E) - 1ull);
    const uint64_t valid = avail;
    uint64_t chosen = 0;
    float my_sel = NEG_INF;  // lane k keeps the logit picked in round k
    int my_idx = 0;
    for (int k = 0; k < K; ++k) {
      const bool ok0 = (avail >> lane) & 1ull;
      const bool ok1 = (avail >> (lane + 32)) & 1ull;
      float bv;
      int bi;
      if (ok0 && (!ok1 || v0 >= v1)) { bv = v0; bi = lane; }
      else if (ok1) { bv = v1; bi = lane + 32; }
      else { bv = NEG_INF; bi = 1 << 20; }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        float ov = __shfl_xor_sync(0xffffffffu, bv, off);
        int oi = __shfl_xor_sync(0xffffffffu, bi, off);
        if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
      }
      if (bi >= E) {  // candidate set exhausted: fall back to the lowest unselected expert
        flags |= C2R_STATUS_SET_TOO_SMALL;
        bi = __ffsll((long long)(valid & ~chosen)) - 1;
        bv = NEG_INF;
      }
      chosen |= 1ull << bi;
      avail &= ~(1ull << bi);
      if (k == 0 && mask != nullptr) avail &= mask[bi];
      if (lane == k) { my_sel = bv; my_idx = bi; }
    }
    // Eq. 1 weights.  The round-0 logit is the row maximum, so it is the softmax shift for both forms.
    const float top = __shfl_sync(0xffffffffu, my_sel, 0);
    float denom;
    if (renorm) {
      float ek = (lane < K) ? expf(my_sel - top) : 0.f;
      denom = ek;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) denom += __shfl_xor_sync(0xffffffffu, denom, off);
      if (lane < K) w[(size_t)t * K + lane] = ek / denom;
    }
    if (!renorm || p != nullptr) {
      float e0 = (lane < E) ? expf(v0 - top) : 0.f;
      float e1 = (lane + 32 < E) ? expf(v1 - top) : 0.f;
      float s = e0 + e1;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
      if (p != nullptr) {
        if (lane < E) p[(size_t)t * E + lane] = e0 / s;
        if (lane + 32 < E) p[(size_t)t * E + lane + 32] = e1 / s;
      }
      if (!renorm && lane < K) w[(size_t)t * K + lane] = expf(my_sel - top) / s;
    }
    if (lane < K) {
      idx[(size_t)t * K + lane] = my_idx;
      if (block_counts != nullptr) warp_cnt[warp][my_idx] += 1;
    }
  }
  if (block_counts != nullptr) {
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
      int s = 0;
#pragma unroll
      for (int x = 0; x < ROUTE_WARPS; ++x) s += warp_cnt[x][e];
      block_counts[(size_t)blockIdx.x * E + e] = s;
    }
  }
  if (status != nullptr) {
    flags = __reduce_or_sync(0xffffffffu, flags);
    if (flags && lane == 0) atomicOr(status, flags);
  }
}

__global__ void route_bwd_kernel(const float* __restrict__ w, const float* __restrict__ dw, float* __restrict__ dl,
                                 int N, int K) {
  int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= N) return;
  float s = 0.f;
  for (int k = 0; k < K; ++k) s = fmaf(w[(size_t)t * K + k], dw[(size_t)t * K + k], s);
  for (int k = 0; k < K; ++k) dl[(size_t)t * K + k] = w[(size_t)t * K + k] * (dw[(size_t)t * K + k] - s);
}

// Backward of the Eq. 1 weights when the experts applied them themselves (row-scaled SwiGLU): the backward
// GEMM left, per permuted row, partial dots whose sum is q = s_r <dH_r, H_r / s_r> = w dL/dw.  With
// S = sum_j q_j:  dl_k = w_k (dw_k - sum_j w_j dw_j) = q_k - w_k S  -- no division by a weight that may be 0.
// dw (optional, informational) = q_k / w_k where w_k > 0.  Shared expert: q_s = g dL/dg, dz = q_s (1 - g).
// Partials are added in index order.
constexpr int RBS_TOKENS = 64;  // tokens per block; one thread per slot
__global__ void __launch_bounds__(RBS_TOKENS * 8) route_bwd_scaled_kernel(const float* __restrict__ w,
                                                                          const int32_t* __restrict__ row_of_slot,
                                                                          const float* __restrict__ qpart, int nq,
                                                                          long long R, const float* __restrict__ z,
                                                                          const float* __restrict__ qspart, int nqs,
                                                                          float* __restrict__ dw, float* __restrict__ dl,
                                                                          float* __restrict__ dz, int N, int K) {
  __shared__ float s_q[RBS_TOKENS * 8];
  const int lt = threadIdx.x / K, k = threadIdx.x - lt * K;  // token of the block, slot of the token
  const int t = blockIdx.x * RBS_TOKENS + lt;
  float q = 0.f;
  if (t < N) {
    const long long row = row_of_slot[(size_t)t * K + k];
    for (int j = 0; j < nq; ++j) q += qpart[(long long)j * R + row];
  }
  s_q[threadIdx.x] = q;
  __syncthreads();
  if (t >= N) return;
  float S = 0.f;
  for (int j = 0; j < K; ++j) S += s_q[lt * K + j];  // slot order
  const float wk = w[(size_t)t * K + k];
  dl[(size_t)t * K + k] = q - wk * S;
  if (dw != nullptr) dw[(size_t)t * K + k] = wk > 0.f ? q / wk : 0.f;
  if (dz != nullptr && k == 0) {
    float acc = 0.f;
    for (int j = 0; j < nqs; ++j) acc += qspart[(long long)j * N + t];
    const float g = 1.0f / (1.0f + expf(-z[t]));
    dz[t] = acc * (1.0f - g);
  }
}

// ---------------------------------------------------------------------------------------------
// Collaboration matrix (Eq. 2): per-block table in shared memory, merged with integer adds.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) collab_count_kernel(const int32_t* __restrict__ idx, long long n_tokens,
                                                           int32_t* __restrict__ C, int E, int K) {
  extern __shared__ int32_t tab[];
  for (int i = threadIdx.x; i < E * E; i += blockDim.x) tab[i] = 0;
  __syncthreads();
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < n_tokens;
       t += (long long)gridDim.x * blockDim.x) {
    int sel[8];
    for (int k = 0; k < K; ++k) {
      int e = idx[t * K + k];
      sel[k] = min(max(e, 0), E - 1);
    }
    for (int a = 0; a < K; ++a)
      for (int b = 0; b < K; ++b) atomicAdd(&tab[sel[a] * E + sel[b]], 1);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < E * E; i += blockDim.x)
    if (tab[i]) atomicAdd(&C[i], tab[i]);
}

// Top-T sets (Eq. 4): one warp per row; T rounds of arg-max under (count desc, index asc), self excluded.
__global__ void collab_sets_kernel(const int32_t* __restrict__ C, int32_t* __restrict__ I_T,
                                   uint64_t* __restrict__ mask, int E, int T) {
  const int lane = threadIdx.x & 31;
  const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (i >= E) return;
  long long c0 = (lane < E && lane != i) ? (long long)C[i * E + lane] : -1;
  long long c1 = (lane + 32 < E && lane + 32 != i) ? (long long)C[i * E + lane + 32] : -1;
  // negative counts cannot occur; -1 marks "not a candidate"
  uint64_t m = 0;
  for (int r = 0; r < T; ++r) {
    long long bv;
    int bi;
    const bool ok0 = c0 >= 0 && !((m >> lane) & 1ull);
    const bool ok1 = c1 >= 0 && !((m >> (lane + 32)) & 1ull);
    if (ok0 && (!ok1 || c0 >= c1)) { bv = c0; bi = lane; }
    else if (ok1) { bv = c1; bi = lane + 32; }
    else { bv = -1; bi = 1 << 20; }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      long long ov = __shfl_xor_sync(0xffffffffu, bv, off);
      int oi = __shfl_xor_sync(0xffffffffu, bi, off);
      if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    m |= 1ull << bi;
    if (lane == 0) I_T[i * T + r] = bi;
  }
  if (lane == 0) mask[i] = m;
}

// Collaboration degree (Eq. 3): P_i = - sum_{j != i} p_ij ln p_ij with p_ij = c_ij / sum_{j != i} c_ij
// (a row without co-activations gives 0; 0 ln 0 = 0).  One block; a warp per row, lanes over the
// columns, and a fixed-order sum over rows for the layer mean.
__global__ void __launch_bounds__(1024) collab_degree_kernel(const int32_t* __restrict__ C, float* __restrict__ degree,
                                                             float* __restrict__ mean, int E) {
  __shared__ float s_deg[64];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int i = warp; i < E; i += 32) {
    float c0 = (lane < E && lane != i) ? (float)max(C[i * E + lane], 0) : 0.f;
    float c1 = (lane + 32 < E && lane + 32 != i) ? (float)max(C[i * E + lane + 32], 0) : 0.f;
    float tot = c0 + c1;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, off);
    float h = 0.f;
    if (tot > 0.f) {
      const float p0 = c0 / tot, p1 = c1 / tot;
      if (p0 > 0.f) h -= p0 * logf(p0);
      if (p1 > 0.f) h -= p1 * logf(p1);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) h += __shfl_xor_sync(0xffffffffu, h, off);
    if (lane == 0) { s_deg[i] = h; degree[i] = h; }
  }
  __syncthreads();
  if (threadIdx.x == 0 && mean != nullptr) {
    float m = 0.f;
    for (int i = 0; i < E; ++i) m += s_deg[i];
    *mean = m / (float)E;
  }
}

// ---------------------------------------------------------------------------------------------
// Dispatch volume (Sec. 3.4 / 4.1): distinct (token, partition) pairs vs (token, expert) pairs.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) dispatch_volume_kernel(const int32_t* __restrict__ idx,
                                                              const int32_t* __restrict__ part,
                                                              unsigned long long* __restrict__ totals,
                                                              unsigned long long* __restrict__ send_naive,
                                                              unsigned long long* __restrict__ send_dedup, int N,
                                                              int E, int K, int P) {
  extern __shared__ uint32_t sm[];
  uint32_t* s_naive = sm;           // [P*P]
  uint32_t* s_dedup = sm + P * P;   // [P*P]
  uint32_t* s_part = sm + 2 * P * P;  // [E]
  for (int i = threadIdx.x; i < 2 * P * P; i += blockDim.x) sm[i] = 0;
  for (int i = threadIdx.x; i < E; i += blockDim.x) s_part[i] = (uint32_t)min(max(part[i], 0), P - 1);
  __syncthreads();
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < N; t += (long long)gridDim.x * blockDim.x) {
    const int home = (int)((t * P) / N);
    uint64_t seen = 0;
    for (int k = 0; k < K; ++k) {
      int e = min(max(idx[t * K + k], 0), E - 1);
      int q = s_part[e];
      atomicAdd(&s_naive[home * P + q], 1u);
      if (!((seen >> q) & 1ull)) {
        seen |= 1ull << q;
        atomicAdd(&s_dedup[home * P + q], 1u);
      }
    }
  }
  __syncthreads();
  unsigned long long tn = 0, td = 0, tnx = 0, tdx = 0;
  for (int i = threadIdx.x; i < P * P; i += blockDim.x) {
    uint32_t a = s_naive[i], b = s_dedup[i];
    if (a) atomicAdd(&send_naive[i], (unsigned long long)a);
    if (b) atomicAdd(&send_dedup[i], (unsigned long long)b);
    tn += a; td += b;
    if (i / P != i % P) { tnx += a; tdx += b; }
  }
  if (tn) atomicAdd(&totals[0], tn);
  if (td) atomicAdd(&totals[1], td);
  if (tnx) atomicAdd(&totals[2], tnx);
  if (tdx) atomicAdd(&totals[3], tdx);
}

}  // namespace c2r

using namespace c2r;

extern "C" int c2r_last_cuda_error(void) { return g_last_cuda_error; }

extern "C" uint64_t c2r_launch_count(void) { return __atomic_load_n(&g_launch_count, __ATOMIC_RELAXED); }

int c2r::gate_logits_impl(const c2r_config* cfg, const void* X, const void* Wg, const void* wsg, float* L, float* z,
                          int32_t* status, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(X && Wg && L, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(!wsg || z, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(cfg->E + (wsg ? 1 : 0) <= GL_COLS, C2R_ERR_UNSUPPORTED_SHAPE);
  if (cfg->N == 0) return C2R_OK;
  const bool aligned = (((uintptr_t)X | (uintptr_t)Wg | (uintptr_t)wsg | (uintptr_t)L) & 15u) == 0;
  if (aligned && gate_tc_supported(cfg)) return gate_tc_launch(cfg, X, Wg, wsg, L, z, status, as_stream(stream));
  dim3 grid((cfg->N + GL_TM - 1) / GL_TM);
  if (cfg->dtype == C2R_BF16)
    gate_logits_kernel<__nv_bfloat16><<<grid, 256, 0, as_stream(stream)>>>(
        (const __nv_bfloat16*)X, (const __nv_bfloat16*)Wg, (const __nv_bfloat16*)wsg, L, z, cfg->N, cfg->d, cfg->E);
  else
    gate_logits_kernel<float><<<grid, 256, 0, as_stream(stream)>>>((const float*)X, (const float*)Wg,
                                                                   (const float*)wsg, L, z, cfg->N, cfg->d, cfg->E);
  C2R_LAUNCH_CHECK();
  return C2R_OK;
}

extern "C" int c2r_gate_logits(const c2r_config* cfg, const void* X, const void* Wg, const void* wsg, float* L,
                               float* z, void* stream) {
  return gate_logits_impl(cfg, X, Wg, wsg, L, z, nullptr, stream);
}

int c2r::route_impl(const c2r_config* cfg, const float* L, const uint64_t* mask, int32_t* idx, float* w, float* p,
                    int32_t* status, int32_t* block_counts, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(L && idx && w, C2R_ERR_INVALID_ARG);
  if (mask) C2R_REQUIRE(cfg->T >= cfg->K - 1 && cfg->T <= cfg->E - 1, C2R_ERR_INVALID_ARG);
  if (cfg->N == 0) return C2R_OK;
  const int tpb = perm_tokens_per_block(cfg->K);
  route_kernel<<<(cfg->N + tpb - 1) / tpb, ROUTE_WARPS * 32, 0, as_stream(stream)>>>(L, mask, idx, w, p, status, cfg->N, cfg->E,
                                                                                   cfg->K, cfg->renorm, tpb, block_counts);
  C2R_LAUNCH_CHECK();
  return C2R_OK;
}

extern "C" int c2r_route(const c2r_config* cfg, const float* L, const uint64_t* mask, int32_t* idx, float* w, float* p,
                         int32_t* status, void* permute_ws, void* stream) {
  return route_impl(cfg, L, mask, idx, w, p, status, (int32_t*)permute_ws, stream);
}

extern "C" int c2r_route_bwd_scaled(const c2r_config* cfg, const float* w, const int32_t* row_of_slot, const float* qpart,
                                    int nq, const float* z, const float* qspart, int nqs, float* dw, float* dl, float* dz,
                                    void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(w && row_of_slot && qpart && dl && nq >= 0, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(!dz || (z && qspart && nqs >= 0), C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(cfg->renorm == 1, C2R_ERR_UNSUPPORTED_SHAPE);
  if (cfg->N == 0) return C2R_OK;
  route_bwd_scaled_kernel<<<(cfg->N + RBS_TOKENS - 1) / RBS_TOKENS, RBS_TOKENS * cfg->K, 0, as_stream(stream)>>>(w, row_of_slot, qpart, nq, permuted_rows(cfg),
                                                                              z, qspart, nqs, dw, dl, dz, cfg->N, cfg->K);
  C2R_LAUNCH_CHECK();
  return C2R_OK;
}

extern "C" int c2r_route_bwd(const c2r_config* cfg, const float* w, const float* dw, float* dl, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(w && dw && dl, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(cfg->renorm == 1, C2R_ERR_UNSUPPORTED_SHAPE);
  if (cfg->N == 0) return C2R_OK;
  route_bwd_kernel<<<(cfg->N + 255) / 256, 256, 0, as_stream(stream)>>>(w, dw, dl, cfg->N, cfg->K);
  C2R_LAUNCH_CHECK();
  return C2R_OK;
}

extern "C" int c2r_collab_count(const c2r_config* cfg, const int32_t* idx, int64_t n_tokens, int32_t* C,
                                int accumulate, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(idx && C && n_tokens >= 0, C2R_ERR_INVALID_ARG);
  const int E = cfg->E;
  if (!accumulate) C2R_CUDA(cudaMemsetAsync(C, 0, sizeof(int32_t) * E * E, as_stream(stream)));
  if (n_tokens == 0) return C2R_OK;
  int blocks = (int)((n_tokens + 255) / 256);
  if (blocks > 296) blocks = 296;
  collab_count_kernel<<<blocks, 256, sizeof(int32_t) * E * E, as_stream(stream)>>>(idx, (long long)n_tokens, C, E,
                                                                                 cfg->K);
  C2R_LAUNCH_CHECK();
  return C2R_OK;
}

extern "C" int c2r_collab_sets(const c2r_config* cfg, const int32_t* C, int32_t* I_T, uint64_t* mask, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(C && I_T && mask, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(cfg->T >= 0 && cfg->T <= cfg->E - 1, C2R_ERR_INVALID_ARG);
  const int warps = 4;
  collab_sets_kernel<<<(cfg->E + warps - 1) / warps, warps * 32, 0, as_stream(stream)>>>(C, I_T, mask, cfg->E, cfg->T);
  C2R_LAUNCH_CHECK();
  return C2R_OK;
}

extern "C" int c2r_collab_degree(const c2r_config* cfg, const int32_t* C, float* degree, float* mean, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(C && degree, C2R_ERR_INVALID_ARG);
  collab_degree_kernel<<<1, 1024, 0, as_stream(stream)>>>(C, degree, mean, cfg->E);
  C2R_LAUNCH_CHECK();
  return C2R_OK;
}

extern "C" int c2r_dispatch_volume(const c2r_config* cfg, const int32_t* idx, const int32_t* part, uint64_t* totals,
                                   uint64_t* send_naive, uint64_t* send_dedup, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(idx && part && totals && send_naive && send_dedup, C2R_ERR_INVALID_ARG);
  const int P = cfg->P;
  C2R_REQUIRE(P >= 1 && P <= cfg->E, C2R_ERR_INVALID_ARG);
  cudaStream_t s = as_stream(stream);
  if (send_naive == totals + 4 && send_dedup == send_naive + P * P) {  // one buffer (the layer drivers' layout)
    C2R_CUDA(cudaMemsetAsync(totals, 0, sizeof(uint64_t) * (4 + 2 * P * P), s));
  } else {
    C2R_CUDA(cudaMemsetAsync(totals, 0, 4 * sizeof(uint64_t), s));
    C2R_CUDA(cudaMemsetAsync(send_naive, 0, sizeof(uint64_t) * P * P, s));
    C2R_CUDA(cudaMemsetAsync(send_dedup, 0, sizeof(uint64_t) * P * P, s));
  }
  if (cfg->N == 0) return C2R_OK;
  int blocks = (cfg->N + 255) / 256;
  if (blocks > 296) blocks = 296;
  size_t smem = sizeof(uint32_t) * (2 * P * P + cfg->E);
  dispatch_volume_kernel<<<blocks, 256, smem, s>>>(idx, part, (unsigned long long*)totals,
                                                   (unsigned long long*)send_naive, (unsigned long long*)send_dedup,
                                                   cfg->N, cfg->E, cfg->K, P);
  C2R_LAUNCH_CHECK();
  return C2R_OK;
}
