// Internal interface between the API layer and the expert-GEMM implementations.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "c2r.h"

namespace c2r {

enum { SIMT_ROWS = 0, SIMT_WGRAD = 1 };
enum { SIMT_EPI_STORE = 0, SIMT_EPI_SWIGLU_BWD = 1, SIMT_EPI_SWIGLU_FWD = 2 };

// C_g(m,n) = sum_k A(m,k) B(n,k), one problem per group (expert) g with element strides
//   A(m,k) = A[a_off + m*sam + k*sak],  B(n,k) = B[b_off + n*sbn + k*sbk].
// SIMT_ROWS : M = counts[g] rows starting at offsets[g] (row stride sam / ldc), K = Kdim,
//             B of group g starts at g*sB, C rows are the same rows.
// SIMT_WGRAD: the contraction runs over the group's rows (stride sak / sbk), M = Mdim, N = Ndim,
//             C of group g starts at g*sC.
struct SimtGemm {
  const void* A;
  const void* B;
  void* C;
  const void* aux;
  void* aux_out;
  const int32_t* counts;
  const int32_t* offsets;
  long long sam, sak, sbn, sbk, sB, sC, ldc;
  int mode, epi, Mdim, Ndim, Kdim, I, accumulate;
};

template <typename T>
int simt_swiglu_fwd(const c2r_config* cfg, int nE, int I, int64_t R, const void* Xp, const int32_t* counts,
                    const int32_t* offsets, const void* W13p, const void* W2, void* AB, void* H, void* Yp,
                    cudaStream_t s);
template <typename T>
int simt_swiglu_bwd(const c2r_config* cfg, int nE, int I, int64_t R, const void* Xp, const int32_t* counts,
                    const int32_t* offsets, const void* W13p, const void* W2, const void* AB, const void* H,
                    const void* dYp, void* dAB, void* dXp, void* dW13p, void* dW2, int accumulate, cudaStream_t s);

// Tensor-core (tcgen05) path, bf16 only.
enum { TC_ROWS = 0, TC_WGRAD = 1 };
enum { TC_EPI_SWIGLU_FWD = 0, TC_EPI_F32 = 1, TC_EPI_SWIGLU_BWD = 2, TC_EPI_WGRAD_BF16 = 3, TC_EPI_T_F32 = 4 };
bool tc_supported(const c2r_config* cfg, int nE, int I, int64_t R);
// X / slot_of_row (both or neither): the rows of the permuted operand are fetched from X inside the kernels
// (TMA row gather) and Xp is not read.
int tc_swiglu_fwd(const c2r_config* cfg, int nE, int I, int64_t R, const void* Xp, const int32_t* counts,
                  const int32_t* offsets, const void* W13p, const void* W2, void* AB, void* H, void* Yp,
                  int32_t* status, cudaStream_t s, const void* X = nullptr, const int32_t* slot_of_row = nullptr);
int tc_swiglu_bwd(const c2r_config* cfg, int nE, int I, int64_t R, const void* Xp, const int32_t* counts,
                  const int32_t* offsets, const void* W13p, const void* W2, const void* AB, const void* H,
                  const void* dYp, void* dAB, void* dXp, void* dW13p, void* dW2, int accumulate, int32_t* status,
                  cudaStream_t s, const void* X = nullptr, const int32_t* slot_of_row = nullptr);

// Gate logits on the tensor cores (bf16 only).
bool gate_tc_supported(const c2r_config* cfg);
int gate_tc_launch(const c2r_config* cfg, const void* X, const void* Wg, const void* wsg, float* L, float* z,
                   int32_t* status, cudaStream_t s);
// c2r_gate_logits with a status word for the bounded waits of the tensor-core kernel.
int gate_logits_impl(const c2r_config* cfg, const void* X, const void* Wg, const void* wsg, float* L, float* z,
                     int32_t* status, void* stream);

// Gate weight gradient on the tensor cores: partial[s][c][:] = sum over the tokens of split s of dLd[t,c] X[t,:],
// dLd [N,64] bf16 the dense gradient w.r.t. the logits (column E: shared gate), splits given by device arrays.
int tc_gate_wgrad(const c2r_config* cfg, const void* X, const void* dLd, float* partial, int n_splits,
                  const int32_t* split_counts, const int32_t* split_offsets, int32_t* status, cudaStream_t s);

size_t permute_ws_bytes(const c2r_config* cfg);
size_t gate_bwd_ws_bytes(const c2r_config* cfg);
size_t dispatch_dedup_ws_bytes(const c2r_config* cfg);

}  // namespace c2r
