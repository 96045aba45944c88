// CUDA-core grouped GEMMs for the expert MLPs: the fp32 path (exact-arithmetic configurations)
// and any bf16 shape the tensor-core kernels do not cover.  Also the W1/W3 packing helpers.
#include "c2r_common.cuh"
#include "gemm.h"

namespace c2r {

__host__ __device__ inline int pack_col(int i, int I) {
  const int j = i >> 7;
  return (j << 8) + (i - (j << 7));
}
__host__ __device__ inline int pack_width(int i, int I) {
  const int j = i >> 7;
  const int rem = I - (j << 7);
  return rem < 128 ? rem : 128;
}

// rows of W1 / W3  <->  rows of W13p
template <typename T>
__global__ void pack_kernel(const T* __restrict__ W1, const T* __restrict__ W3, T* __restrict__ W13p, int I, int d,
                            int unpack, T* __restrict__ W1o, T* __restrict__ W3o) {
  using V = Vec16<T>;
  const int e = blockIdx.y;
  const int i = blockIdx.x;
  const int pg = pack_col(i, I), pu = pg + pack_width(i, I);
  const size_t src = ((size_t)e * I + i) * d;
  const size_t dg = ((size_t)e * 2 * I + pg) * d, du = ((size_t)e * 2 * I + pu) * d;
  for (int c = threadIdx.x * V::N; c < d; c += blockDim.x * V::N) {
    V a, b;
    if (!unpack) {
      a.load(W1 + src + c);
      b.load(W3 + src + c);
      a.store(W13p + dg + c);
      b.store(W13p + du + c);
    } else {
      a.load(W13p + dg + c);
      b.load(W13p + du + c);
      a.store(W1o + src + c);
      b.store(W3o + src + c);
    }
  }
}

constexpr int ST = 64;  // tile M = N
constexpr int SK = 16;  // tile K

// C_g(m,n) = sum_k A_g(m,k) B_g(n,k) with arbitrary strides; see SimtGemm for the two modes.
template <typename T, typename TC>
__global__ void __launch_bounds__(256) simt_gemm_kernel(SimtGemm g) {
  __shared__ float sa[SK][ST + 4];
  __shared__ float sb[SK][ST + 4];
  __shared__ float sb2[SK][ST + 4];  // up-projection tile of the fused SwiGLU forward
  __shared__ float sred[ST][17];     // per-row partial dots of the SwiGLU backward, one column per thread column
  const bool dual = g.epi == SIMT_EPI_SWIGLU_FWD;
  const int grp = blockIdx.z;
  int M, Kd;
  long long a_off, b_off, c_off;
  const int cnt = g.counts[grp], r0 = g.offsets[grp];
  if (g.mode == SIMT_ROWS) {
    M = cnt; Kd = g.Kdim;
    a_off = (long long)r0 * g.sam; b_off = (long long)grp * g.sB; c_off = (long long)r0 * g.ldc;
  } else {
    M = g.Mdim; Kd = cnt;
    a_off = (long long)r0 * g.sak; b_off = (long long)r0 * g.sbk; c_off = (long long)grp * g.sC;
  }
  const int m0 = blockIdx.y * ST, n0 = blockIdx.x * ST;
  if (m0 >= M || n0 >= g.Ndim) return;
  const T* A = (const T*)g.A + a_off;
  const T* B = (const T*)g.B + b_off;
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  float acc[4][4] = {};
  float acc2[4][4] = {};
  for (int k0 = 0; k0 < Kd; k0 += SK) {
    for (int i = tid; i < ST * SK; i += 256) {
      int m, k;
      if (g.sak == 1) { k = i % SK; m = i / SK; } else { m = i % ST; k = i / ST; }
      float v = 0.f;
      if (m0 + m < M && k0 + k < Kd) v = to_f32(A[(long long)(m0 + m) * g.sam + (long long)(k0 + k) * g.sak]);
      sa[k][m] = v;
    }
    for (int i = tid; i < ST * SK; i += 256) {
      int n, k;
      if (g.sbk == 1) { k = i % SK; n = i / SK; } else { n = i % ST; k = i / ST; }
      float v = 0.f, v2 = 0.f;
      if (n0 + n < g.Ndim && k0 + k < Kd) {
        if (!dual) {
          v = to_f32(B[(long long)(n0 + n) * g.sbn + (long long)(k0 + k) * g.sbk]);
        } else {  // column n of H pairs packed rows pg (gate) and pu (up) of W13p
          const int pg = pack_col(n0 + n, g.I), pu = pg + pack_width(n0 + n, g.I);
          v = to_f32(B[(long long)pg * g.sbn + (long long)(k0 + k) * g.sbk]);
          v2 = to_f32(B[(long long)pu * g.sbn + (long long)(k0 + k) * g.sbk]);
        }
      }
      sb[k][n] = v;
      if (dual) sb2[k][n] = v2;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < SK; ++k) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { av[i] = sa[k][ty * 4 + i]; bv[i] = sb[k][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
      if (dual) {
#pragma unroll
        for (int i = 0; i < 4; ++i) bv[i] = sb2[k][tx * 4 + i];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc2[i][j] = fmaf(av[i], bv[j], acc2[i][j]);
      }
    }
    __syncthreads();
  }
  TC* C = (TC*)g.C + c_off;
  const bool want_q = g.epi == SIMT_EPI_SWIGLU_BWD && g.qpart != nullptr;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    float qrow = 0.f;
    if (want_q) sred[ty * 4 + i][tx] = 0.f;
    if (m >= M) continue;
    float sc = 1.f;  // per-row scale of H (SwiGLU forms)
    if (g.scale_kind != 0 && g.row_scale != nullptr) {
      const float v = g.row_scale[r0 + m];
      sc = g.scale_kind == 2 ? 1.0f / (1.0f + expf(-v)) : v;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= g.Ndim) continue;
      float v = acc[i][j];
      if (g.epi == SIMT_EPI_STORE && g.token_acc != nullptr) {
        // fused combine: the row is added into its token's accumulator (fp32 atomics, order not fixed)
        const int sl = g.slot_of_row[r0 + m];
        if (sl >= 0) atomicAdd(g.token_acc + (long long)(sl / g.slots_per_token) * g.ldc + n, v);
      } else if (g.epi == SIMT_EPI_STORE) {
        TC* o = C + (long long)m * g.ldc + n;
        if (g.accumulate) v += to_f32(*o);
        *o = from_f32<TC>(v);
      } else if (g.epi == SIMT_EPI_SWIGLU_FWD) {
        // v = A[r,n], acc2 = B[r,n]: H = silu(A) * B; the backward pass needs only the two local
        // derivatives dH/dA = B silu'(A) and dH/dB = silu(A), which are what is kept (packed columns)
        const int pg = pack_col(n, g.I), pu = pg + pack_width(n, g.I);
        const float b = acc2[i][j];
        const float sg = 1.0f / (1.0f + expf(-v));
        const float as = v * sg;
        if (g.C != nullptr) {  // inference: nothing is kept for a backward pass
          T* sv = (T*)g.C + (long long)(r0 + m) * 2 * g.I;
          sv[pg] = from_f32<T>(b * (sg + as - as * sg));
          sv[pu] = from_f32<T>(as);
        }
        ((T*)g.aux_out)[(long long)(r0 + m) * g.I + n] = from_f32<T>(sc * (as * b));
      } else {  // SIMT_EPI_SWIGLU_BWD: v = dH[r, n]; dA = dH * (dH/dA), dB = dH * (dH/dB) at the packed columns
        const int pg = pack_col(n, g.I), pu = pg + pack_width(n, g.I);
        const T* sv = (const T*)g.aux + (long long)(r0 + m) * 2 * g.I;
        T* dab = (T*)g.C + (long long)(r0 + m) * 2 * g.I;
        dab[pg] = from_f32<T>(sc * v * to_f32(sv[pg]));
        dab[pu] = from_f32<T>(sc * v * to_f32(sv[pu]));
        if (want_q) qrow = fmaf(v, to_f32(((const T*)g.aux2)[(long long)(r0 + m) * g.I + n]), qrow);
      }
    }
    if (want_q) sred[ty * 4 + i][tx] = qrow;
  }
  if (want_q) {  // (uniform across the block) row dots <dH_r, H_r> over this block's 64 columns, in column order
    __syncthreads();
    if (tid < ST && m0 + tid < M) {
      float q = 0.f;
#pragma unroll
      for (int x = 0; x < 16; ++x) q += sred[tid][x];
      g.qpart[(long long)blockIdx.x * g.R + r0 + m0 + tid] = q;
    }
  }
}

template <typename T, typename TC = T>
int simt_launch(const SimtGemm& g, int n_groups, int max_m, cudaStream_t s) {
  if (n_groups == 0 || max_m == 0 || g.Ndim == 0) return C2R_OK;
  dim3 grid((g.Ndim + ST - 1) / ST, (max_m + ST - 1) / ST, n_groups);
  simt_gemm_kernel<T, TC><<<grid, 256, 0, s>>>(g);
  C2R_LAUNCH_CHECK();
  return C2R_OK;
}

template <typename T>
int simt_swiglu_fwd(const c2r_config* cfg, const SwigluCall& a, cudaStream_t s) {
  const int d = cfg->d, I = a.I;
  const int max_m = (int)a.R;
  SimtGemm g{};
  g.counts = a.counts; g.offsets = a.offsets; g.mode = SIMT_ROWS; g.I = I; g.R = a.R;
  // A = Xp W1^T, B = Xp W3^T in one pass over Xp; epilogue stores H = s silu(A) * B and the two local derivatives
  g.epi = SIMT_EPI_SWIGLU_FWD; g.aux_out = a.H;
  g.row_scale = a.row_scale; g.scale_kind = a.row_scale ? a.scale_kind : 0;
  g.A = a.Xp; g.sam = d; g.sak = 1; g.B = a.W13p; g.sbn = d; g.sbk = 1; g.sB = (long long)2 * I * d;
  g.C = a.AB; g.ldc = 2 * I; g.Ndim = I; g.Kdim = d;
  int rc = simt_launch<T>(g, a.nE, max_m, s);
  if (rc) return rc;
  g.epi = SIMT_EPI_STORE; g.aux_out = nullptr; g.row_scale = nullptr; g.scale_kind = 0;
  // Yp = H W2^T  (fp32 partial result)
  g.A = a.H; g.sam = I; g.sak = 1; g.B = a.W2; g.sbn = I; g.sbk = 1; g.sB = (long long)d * I;
  g.C = a.Yp; g.ldc = d; g.Ndim = d; g.Kdim = I;
  g.token_acc = a.token_acc; g.slot_of_row = a.slot_of_row; g.slots_per_token = cfg->K;
  return simt_launch<T, float>(g, a.nE, max_m, s);
}

template <typename T>
int simt_swiglu_bwd(const c2r_config* cfg, const SwigluCall& a, cudaStream_t s) {
  const int d = cfg->d, I = a.I, nE = a.nE;
  const int max_m = (int)a.R;
  SimtGemm g{};
  g.counts = a.counts; g.offsets = a.offsets; g.I = I; g.R = a.R;
  // dH = dYp W2  (epilogue turns it into dA, dB at the packed columns, and the row dots with H)
  g.mode = SIMT_ROWS; g.epi = SIMT_EPI_SWIGLU_BWD; g.aux = a.AB; g.aux2 = a.H; g.qpart = a.qpart;
  g.row_scale = a.row_scale; g.scale_kind = a.row_scale ? a.scale_kind : 0;
  g.A = a.dYp; g.sam = d; g.sak = 1; g.B = a.W2; g.sbn = 1; g.sbk = I; g.sB = (long long)d * I;
  g.C = a.dAB; g.ldc = 2 * I; g.Ndim = I; g.Kdim = d;
  int rc = simt_launch<T>(g, nE, max_m, s);
  if (rc) return rc;
  // dXp = dAB W13p  (fp32 partial result)
  g.epi = SIMT_EPI_STORE; g.aux = nullptr; g.aux2 = nullptr; g.qpart = nullptr; g.row_scale = nullptr; g.scale_kind = 0;
  g.A = a.dAB; g.sam = 2 * I; g.sak = 1; g.B = a.W13p; g.sbn = 1; g.sbk = d; g.sB = (long long)2 * I * d;
  g.C = a.dXp; g.ldc = d; g.Ndim = d; g.Kdim = 2 * I;
  g.token_acc = a.token_acc; g.slot_of_row = a.slot_of_row; g.slots_per_token = cfg->K;
  rc = simt_launch<T, float>(g, nE, max_m, s);
  if (rc) return rc;
  g.token_acc = nullptr;
  // dW2_e = dYp_e^T H_e   [d, I]
  g.mode = SIMT_WGRAD; g.accumulate = a.accumulate;
  g.A = a.dYp; g.sam = 1; g.sak = d; g.B = a.H; g.sbn = 1; g.sbk = I;
  g.C = a.dW2; g.ldc = I; g.sC = (long long)d * I; g.Mdim = d; g.Ndim = I;
  rc = simt_launch<T>(g, nE, d, s);
  if (rc) return rc;
  // dW13p_e = dAB_e^T Xp_e   [2I, d]
  g.A = a.dAB; g.sam = 1; g.sak = 2 * I; g.B = a.Xp; g.sbn = 1; g.sbk = d;
  g.C = a.dW13p; g.ldc = d; g.sC = (long long)2 * I * d; g.Mdim = 2 * I; g.Ndim = d;
  return simt_launch<T>(g, nE, 2 * I, s);
}

template int simt_swiglu_fwd<float>(const c2r_config*, const SwigluCall&, cudaStream_t);
template int simt_swiglu_fwd<__nv_bfloat16>(const c2r_config*, const SwigluCall&, cudaStream_t);
template int simt_swiglu_bwd<float>(const c2r_config*, const SwigluCall&, cudaStream_t);
template int simt_swiglu_bwd<__nv_bfloat16>(const c2r_config*, const SwigluCall&, cudaStream_t);

}  // namespace c2r

using namespace c2r;

static int pack_common(const c2r_config* cfg, int nE, int I, const void* W1, const void* W3, void* W13p, int unpack,
                       void* W1o, void* W3o, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(nE >= 0 && I > 0 && I % 16 == 0, C2R_ERR_UNSUPPORTED_SHAPE);
  if (nE == 0) return C2R_OK;
  dim3 grid(I, nE);
  if (cfg->dtype == C2R_BF16)
    pack_kernel<__nv_bfloat16><<<grid, 128, 0, as_stream(stream)>>>((const __nv_bfloat16*)W1, (const __nv_bfloat16*)W3,
                                                                    (__nv_bfloat16*)W13p, I, cfg->d, unpack,
                                                                    (__nv_bfloat16*)W1o, (__nv_bfloat16*)W3o);
  else
    pack_kernel<float><<<grid, 128, 0, as_stream(stream)>>>((const float*)W1, (const float*)W3, (float*)W13p, I, cfg->d,
                                                            unpack, (float*)W1o, (float*)W3o);
  C2R_LAUNCH_CHECK();
  return C2R_OK;
}

extern "C" int c2r_pack_weights(const c2r_config* cfg, int n_experts, int I, const void* W1, const void* W3,
                                void* W13p, void* stream) {
  C2R_REQUIRE(W1 && W3 && W13p, C2R_ERR_INVALID_ARG);
  return pack_common(cfg, n_experts, I, W1, W3, W13p, 0, nullptr, nullptr, stream);
}

extern "C" int c2r_unpack_weights(const c2r_config* cfg, int n_experts, int I, const void* W13p, void* W1, void* W3,
                                  void* stream) {
  C2R_REQUIRE(W1 && W3 && W13p, C2R_ERR_INVALID_ARG);
  return pack_common(cfg, n_experts, I, nullptr, nullptr, (void*)W13p, 1, W1, W3, stream);
}
