// Host-side entry points that carry no kernel of their own: sizes, expert placement, the
// expert-MLP dispatch and the whole-layer drivers.
#include <vector>

#include "c2r_common.cuh"
#include "gemm.h"

using namespace c2r;

extern "C" int64_t c2r_permuted_rows(const c2r_config* cfg) {
  if (check_config(cfg) != C2R_OK) return -1;
  return permuted_rows(cfg);
}

static size_t align256(size_t x) { return (x + 255) / 256 * 256; }

extern "C" size_t c2r_workspace_bytes(const c2r_config* cfg, int which) {
  if (check_config(cfg) != C2R_OK) return 0;
  switch (which) {
    case C2R_WS_PERMUTE: return align256(permute_ws_bytes(cfg));
    case C2R_WS_GATE_BWD: return align256(gate_bwd_ws_bytes(cfg));
    case C2R_WS_LAYER: return align256(permute_ws_bytes(cfg)) + align256(gate_bwd_ws_bytes(cfg));
    case C2R_WS_DISPATCH_DEDUP: return align256(dispatch_dedup_ws_bytes(cfg));
    default: return 0;
  }
}

extern "C" int c2r_place_experts(const c2r_config* cfg, const int32_t* C, int mode, int32_t* part, int32_t* rank) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(part && rank, C2R_ERR_INVALID_ARG);
  const int E = cfg->E, P = cfg->P;
  C2R_REQUIRE(P >= 1 && P <= E, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(mode == 0 || mode == 1, C2R_ERR_INVALID_ARG);
  if (mode == 1) {
    for (int e = 0; e < E; ++e) part[e] = (int32_t)(((int64_t)e * P) / E);
  } else {
    C2R_REQUIRE(C, C2R_ERR_INVALID_ARG);
    for (int e = 0; e < E; ++e) part[e] = -1;
    for (int p = 0; p < P; ++p) {
      const int size = E / P + (p < E % P ? 1 : 0);
      std::vector<int64_t> affinity(E, 0);  // co-activation with the current members of partition p
      int members = 0;
      while (members < size) {
        int best = -1;
        int64_t best_v = -1;
        for (int e = 0; e < E; ++e) {
          if (part[e] >= 0) continue;
          const int64_t v = (members == 0) ? (int64_t)C[e * E + e] : affinity[e];
          if (v > best_v) { best_v = v; best = e; }  // strict '>' keeps the lower id on ties
        }
        if (best < 0) break;
        part[best] = p;
        ++members;
        for (int e = 0; e < E; ++e) affinity[e] += C[e * E + best];
      }
    }
  }
  int pos = 0;
  for (int p = 0; p < P; ++p)
    for (int e = 0; e < E; ++e)
      if (part[e] == p) rank[e] = pos++;
  return C2R_OK;
}

static int check_gemm_args(const c2r_config* cfg, int nE, int I, int64_t R) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(nE >= 1 && nE <= 64 && R >= 0 && R < (1ll << 31), C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(I > 0 && I % 16 == 0, C2R_ERR_UNSUPPORTED_SHAPE);
  return C2R_OK;
}

extern "C" int c2r_grouped_swiglu_fwd(const c2r_config* cfg, int n_experts, int I, int64_t R, const void* Xp,
                                      const int32_t* counts, const int32_t* offsets, const void* W13p, const void* W2,
                                      void* AB, void* H, void* Yp, int32_t* status, void* stream) {
  int rc = check_gemm_args(cfg, n_experts, I, R);
  if (rc) return rc;
  C2R_REQUIRE(Xp && counts && offsets && W13p && W2 && H && Yp, C2R_ERR_INVALID_ARG);
  if (R == 0) return C2R_OK;
  cudaStream_t s = as_stream(stream);
  if (cfg->dtype == C2R_F32) {
    return simt_swiglu_fwd<float>(cfg, n_experts, I, R, Xp, counts, offsets, W13p, W2, AB, H, Yp, s);
  }
  if (tc_supported(cfg, n_experts, I, R))
    return tc_swiglu_fwd(cfg, n_experts, I, R, Xp, counts, offsets, W13p, W2, AB, H, Yp, status, s);
  return simt_swiglu_fwd<__nv_bfloat16>(cfg, n_experts, I, R, Xp, counts, offsets, W13p, W2, AB, H, Yp, s);
}

extern "C" int c2r_grouped_swiglu_bwd(const c2r_config* cfg, int n_experts, int I, int64_t R, const void* Xp,
                                      const int32_t* counts, const int32_t* offsets, const void* W13p, const void* W2,
                                      const void* AB, const void* H, const void* dYp, void* dAB, void* dXp,
                                      void* dW13p, void* dW2, int accumulate, int32_t* status, void* stream) {
  int rc = check_gemm_args(cfg, n_experts, I, R);
  if (rc) return rc;
  C2R_REQUIRE(Xp && counts && offsets && W13p && W2 && AB && H && dYp && dAB && dXp && dW13p && dW2,
              C2R_ERR_INVALID_ARG);
  cudaStream_t s = as_stream(stream);
  if (cfg->dtype == C2R_F32)
    return simt_swiglu_bwd<float>(cfg, n_experts, I, R, Xp, counts, offsets, W13p, W2, AB, H, dYp, dAB, dXp, dW13p,
                                  dW2, accumulate, s);
  if (tc_supported(cfg, n_experts, I, R))
    return tc_swiglu_bwd(cfg, n_experts, I, R, Xp, counts, offsets, W13p, W2, AB, H, dYp, dAB, dXp, dW13p, dW2,
                         accumulate, status, s);
  return simt_swiglu_bwd<__nv_bfloat16>(cfg, n_experts, I, R, Xp, counts, offsets, W13p, W2, AB, H, dYp, dAB, dXp,
                                        dW13p, dW2, accumulate, s);
}

extern "C" int c2r_grouped_swiglu_fwd_gather(const c2r_config* cfg, int n_experts, int I, int64_t R, const void* X,
                                             const int32_t* slot_of_row, const int32_t* counts, const int32_t* offsets,
                                             const void* W13p, const void* W2, void* AB, void* H, void* Yp,
                                             int32_t* status, void* stream) {
  int rc = check_gemm_args(cfg, n_experts, I, R);
  if (rc) return rc;
  C2R_REQUIRE(X && slot_of_row && counts && offsets && W13p && W2 && H && Yp, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(tc_supported(cfg, n_experts, I, R) && (((uintptr_t)X) & 15u) == 0, C2R_ERR_UNSUPPORTED_SHAPE);
  if (R == 0) return C2R_OK;
  return tc_swiglu_fwd(cfg, n_experts, I, R, nullptr, counts, offsets, W13p, W2, AB, H, Yp, status, as_stream(stream), X,
                       slot_of_row);
}

extern "C" int c2r_grouped_swiglu_bwd_gather(const c2r_config* cfg, int n_experts, int I, int64_t R, const void* X,
                                             const int32_t* slot_of_row, const int32_t* counts, const int32_t* offsets,
                                             const void* W13p, const void* W2, const void* AB, const void* H,
                                             const void* dYp, void* dAB, void* dXp, void* dW13p, void* dW2,
                                             int accumulate, int32_t* status, void* stream) {
  int rc = check_gemm_args(cfg, n_experts, I, R);
  if (rc) return rc;
  C2R_REQUIRE(X && slot_of_row && counts && offsets && W13p && W2 && AB && H && dYp && dAB && dXp && dW13p && dW2,
              C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(tc_supported(cfg, n_experts, I, R) && (((uintptr_t)X) & 15u) == 0, C2R_ERR_UNSUPPORTED_SHAPE);
  return tc_swiglu_bwd(cfg, n_experts, I, R, nullptr, counts, offsets, W13p, W2, AB, H, dYp, dAB, dXp, dW13p, dW2, accumulate,
                       status, as_stream(stream), X, slot_of_row);
}

// ---------------------------------------------------------------------------------------------
// Whole-layer drivers: the calls above chained on one stream, no host synchronisation.
// ---------------------------------------------------------------------------------------------
#define C2R_TRY(expr)         \
  do {                        \
    int _rc = (expr);         \
    if (_rc) return _rc;      \
  } while (0)

// The gather-fused dispatch is used when asked for and the routed experts run on the tensor-core path.
static bool gather_fused(const c2r_config* cfg, const void* X) {
  return (cfg->flags & C2R_FLAG_GATHER_FUSED) != 0 && X != nullptr && (((uintptr_t)X) & 15u) == 0 &&
         cfg->E < 64 && tc_supported(cfg, cfg->E, cfg->I, permuted_rows(cfg));
}

extern "C" int c2r_layer_fwd(const c2r_config* cfg, const c2r_layer_buffers* b, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(b, C2R_ERR_INVALID_ARG);
  const bool shared = cfg->I_s > 0;
  C2R_REQUIRE(b->ws && b->ws_bytes >= c2r_workspace_bytes(cfg, C2R_WS_LAYER), C2R_ERR_WORKSPACE);
  if (shared)
    C2R_REQUIRE(b->wsg && b->z && b->Ws13p && b->Ws2 && b->Hs && b->Ys && b->s_counts && b->s_offsets,
                C2R_ERR_INVALID_ARG);
  const int64_t R = permuted_rows(cfg);
  C2R_TRY(gate_logits_impl(cfg, b->X, b->Wg, shared ? b->wsg : nullptr, b->L, b->z, b->status, stream));
  C2R_TRY(c2r_route(cfg, b->L, b->mask, b->idx, b->w, nullptr, b->status, stream));
  const bool fused = gather_fused(cfg, b->X);
  C2R_TRY(c2r_permute(cfg, b->idx, b->expert_rank, fused ? nullptr : b->X, b->counts, b->offsets, b->row_of_slot,
                      b->slot_of_row, b->Xp, b->status, b->ws, b->ws_bytes, stream));
  if (fused)
    C2R_TRY(c2r_grouped_swiglu_fwd_gather(cfg, cfg->E, cfg->I, R, b->X, b->slot_of_row, b->counts, b->offsets, b->W13p,
                                          b->W2, b->AB, b->H, b->Yp, b->status, stream));
  else
    C2R_TRY(c2r_grouped_swiglu_fwd(cfg, cfg->E, cfg->I, R, b->Xp, b->counts, b->offsets, b->W13p, b->W2, b->AB, b->H,
                                   b->Yp, b->status, stream));
  if (shared)
    C2R_TRY(c2r_grouped_swiglu_fwd(cfg, 1, cfg->I_s, cfg->N, b->X, b->s_counts, b->s_offsets, b->Ws13p, b->Ws2, b->ABs,
                                   b->Hs, b->Ys, b->status, stream));
  C2R_TRY(c2r_combine(cfg, b->Yp, b->w, b->row_of_slot, shared ? b->Ys : nullptr, shared ? b->z : nullptr, b->Y,
                      stream));
  if (b->part && b->volume) {
    const int P = cfg->P;
    C2R_TRY(c2r_dispatch_volume(cfg, b->idx, b->part, b->volume, b->volume + 4, b->volume + 4 + P * P, stream));
  }
  return C2R_OK;
}

extern "C" int c2r_layer_bwd(const c2r_config* cfg, const c2r_layer_buffers* b, int accumulate, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(b, C2R_ERR_INVALID_ARG);
  const bool shared = cfg->I_s > 0;
  C2R_REQUIRE(b->ws && b->ws_bytes >= c2r_workspace_bytes(cfg, C2R_WS_LAYER), C2R_ERR_WORKSPACE);
  C2R_REQUIRE(b->dY && b->dYp && b->dAB && b->dXp && b->dw && b->dl && b->dW13p && b->dW2 && b->dWg && b->dX,
              C2R_ERR_INVALID_ARG);
  if (shared)
    C2R_REQUIRE(b->dYs && b->dABs && b->dXs && b->dz && b->dWs13p && b->dWs2 && b->dwsg, C2R_ERR_INVALID_ARG);
  const int64_t R = permuted_rows(cfg);
  char* ws_gate = (char*)b->ws + align256(permute_ws_bytes(cfg));
  C2R_TRY(c2r_combine_bwd(cfg, b->dY, b->Yp, b->w, b->row_of_slot, b->slot_of_row, shared ? b->Ys : nullptr,
                          shared ? b->z : nullptr, b->dYp, b->dw, shared ? b->dYs : nullptr,
                          shared ? b->dz : nullptr, stream));
  if (gather_fused(cfg, b->X))
    C2R_TRY(c2r_grouped_swiglu_bwd_gather(cfg, cfg->E, cfg->I, R, b->X, b->slot_of_row, b->counts, b->offsets, b->W13p,
                                          b->W2, b->AB, b->H, b->dYp, b->dAB, b->dXp, b->dW13p, b->dW2, accumulate,
                                          b->status, stream));
  else
    C2R_TRY(c2r_grouped_swiglu_bwd(cfg, cfg->E, cfg->I, R, b->Xp, b->counts, b->offsets, b->W13p, b->W2, b->AB, b->H,
                                   b->dYp, b->dAB, b->dXp, b->dW13p, b->dW2, accumulate, b->status, stream));
  if (shared)
    C2R_TRY(c2r_grouped_swiglu_bwd(cfg, 1, cfg->I_s, cfg->N, b->X, b->s_counts, b->s_offsets, b->Ws13p, b->Ws2, b->ABs,
                                   b->Hs, b->dYs, b->dABs, b->dXs, b->dWs13p, b->dWs2, accumulate, b->status, stream));
  C2R_TRY(c2r_route_bwd(cfg, b->w, b->dw, b->dl, stream));
  C2R_TRY(c2r_gate_bwd(cfg, b->X, b->Xp, b->counts, b->offsets, b->slot_of_row, b->dl, shared ? b->dz : nullptr,
                       b->dWg, shared ? b->dwsg : nullptr, ws_gate, align256(gate_bwd_ws_bytes(cfg)), stream));
  C2R_TRY(c2r_unpermute_grad(cfg, b->dXp, b->row_of_slot, shared ? b->dXs : nullptr, b->idx, b->dl, b->Wg,
                             shared ? b->dz : nullptr, shared ? b->wsg : nullptr, b->dX, 0, stream));
  return C2R_OK;
}

extern "C" int c2r_train_step(const c2r_config* cfg, const c2r_layer_buffers* b, void* stream) {
  C2R_REQUIRE(b && b->C && b->I_T && b->mask_next, C2R_ERR_INVALID_ARG);
  C2R_TRY(c2r_layer_fwd(cfg, b, stream));
  C2R_TRY(c2r_layer_bwd(cfg, b, 0, stream));
  C2R_TRY(c2r_collab_count(cfg, b->idx, cfg->N, b->C, 0, stream));
  C2R_TRY(c2r_collab_sets(cfg, b->C, b->I_T, b->mask_next, stream));
  return C2R_OK;
}
