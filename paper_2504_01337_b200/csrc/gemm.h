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
  const void* aux2;        // SIMT_EPI_SWIGLU_BWD: the forward's H (for the row dots), or NULL
  const float* row_scale;  // SwiGLU forms: per-row scale of H, see SwigluCall
  int scale_kind;
  float* qpart;            // SIMT_EPI_SWIGLU_BWD: [ceil(I / 64)][R] partial row dots, or NULL
  long long R;
  float* token_acc;        // SIMT_EPI_STORE: add row r into token_acc[slot_of_row[r] / slots_per_token] instead of storing
  const int32_t* slot_of_row;
  int slots_per_token;
  const int32_t* counts;
  const int32_t* offsets;
  long long sam, sak, sbn, sbk, sB, sC, ldc;
  int mode, epi, Mdim, Ndim, Kdim, I, accumulate;
};

// One grouped SwiGLU evaluation (forward or backward); members a direction does not use stay NULL.
// Per-row scale: H = s_r silu(A) B with s_r = 1 (kind C2R_SCALE_NONE), row_scale[r] (C2R_SCALE_ROW) or
// sigmoid(row_scale[r]) (C2R_SCALE_SIGMOID).
struct SwigluCall {
  int nE, I;
  int64_t R;
  const void* Xp;
  const int32_t* counts;
  const int32_t* offsets;
  const void* W13p;
  const void* W2;
  const float* row_scale;
  int scale_kind;
  void* AB;   // forward: out (NULL = keep nothing for a backward pass); backward: in
  void* H;    // forward: out; backward: in
  void* Yp;   // forward: out, float
  const void* dYp;
  void* dAB;
  void* dXp;
  void* dW13p;
  void* dW2;
  float* qpart;  // backward: [swiglu_qparts][R] partial row dots <dH_r, H_r>, or NULL
  int accumulate;
  int32_t* status;
  // gather-fused dispatch (X with slot_of_row): rows of the permuted operand are fetched from X inside the kernels
  const void* X;
  const int32_t* slot_of_row;
  // fused combine (token_acc with slot_of_row): the [R,d] float result is added into token_acc[slot_of_row[r] / K]
  float* token_acc;
};

template <typename T>
int simt_swiglu_fwd(const c2r_config* cfg, const SwigluCall& a, cudaStream_t s);
template <typename T>
int simt_swiglu_bwd(const c2r_config* cfg, const SwigluCall& a, cudaStream_t s);

// Tensor-core (tcgen05) path, bf16 only.
enum { TC_ROWS = 0, TC_WGRAD = 1 };
enum { TC_EPI_SWIGLU_FWD = 0, TC_EPI_F32 = 1, TC_EPI_SWIGLU_BWD = 2, TC_EPI_WGRAD_BF16 = 3, TC_EPI_T_F32 = 4 };
bool tc_supported(const c2r_config* cfg, int nE, int I, int64_t R);
int tc_swiglu_fwd(const c2r_config* cfg, const SwigluCall& a, cudaStream_t s);
int tc_swiglu_bwd(const c2r_config* cfg, const SwigluCall& a, cudaStream_t s);
// Rows of the partial-dot buffer the backward call writes for this shape (depends on which kernel serves it).
int swiglu_qparts(const c2r_config* cfg, int nE, int I, int64_t R);

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

// c2r_route that can also leave the dispatch's per-block expert histogram in block_counts (may be NULL).
int route_impl(const c2r_config* cfg, const float* L, const uint64_t* mask, int32_t* idx, float* w, float* p,
               int32_t* status, int32_t* block_counts, void* stream);
// c2r_permute with its options: have_hist = block_counts (the workspace) already holds the histogram route_impl
// wrote; w / w_row: also write the routing weight of every permuted row.
int permute_call(const c2r_config* cfg, const int32_t* idx, const int32_t* expert_rank, const void* X, int32_t* counts,
                 int32_t* offsets, int32_t* row_of_slot, int32_t* slot_of_row, void* Xp, int32_t* status, void* ws,
                 size_t ws_bytes, void* stream, bool have_hist, const float* w, float* w_row);

size_t permute_ws_bytes(const c2r_config* cfg);
size_t layer_ws_bytes(const c2r_config* cfg);
size_t gate_bwd_ws_bytes(const c2r_config* cfg);
size_t dispatch_dedup_ws_bytes(const c2r_config* cfg);

}  // namespace c2r
