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
    case C2R_WS_LAYER: return layer_ws_bytes(cfg);
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

// Validates the options and copies them into the call.
static int apply_opts(const c2r_config* cfg, const c2r_expert_opts* o, SwigluCall& a, bool backward) {
  if (o == nullptr) return C2R_OK;
  C2R_REQUIRE(o->scale_kind == C2R_SCALE_NONE || o->scale_kind == C2R_SCALE_ROW || o->scale_kind == C2R_SCALE_SIGMOID,
              C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(o->scale_kind == C2R_SCALE_NONE || o->row_scale != nullptr, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE((!o->X && !o->token_acc) || o->slot_of_row, C2R_ERR_INVALID_ARG);
  C2R_REQUIRE(backward || !o->qpart, C2R_ERR_INVALID_ARG);
  a.row_scale = o->row_scale; a.scale_kind = o->scale_kind;
  a.X = o->X; a.slot_of_row = o->slot_of_row; a.token_acc = o->token_acc; a.qpart = o->qpart;
  if (a.X != nullptr)  // the row gather exists on the tensor-core path only
    C2R_REQUIRE(tc_supported(cfg, a.nE, a.I, a.R) && (((uintptr_t)a.X) & 15u) == 0, C2R_ERR_UNSUPPORTED_SHAPE);
  if (a.token_acc != nullptr) C2R_REQUIRE((((uintptr_t)a.token_acc) & 15u) == 0, C2R_ERR_INVALID_ARG);
  return C2R_OK;
}

static int swiglu_fwd_dispatch(const c2r_config* cfg, const SwigluCall& a, cudaStream_t s) {
  if (a.R == 0) return C2R_OK;
  if (cfg->dtype == C2R_F32) return simt_swiglu_fwd<float>(cfg, a, s);
  if (tc_supported(cfg, a.nE, a.I, a.R)) return tc_swiglu_fwd(cfg, a, s);
  return simt_swiglu_fwd<__nv_bfloat16>(cfg, a, s);
}

static int swiglu_bwd_dispatch(const c2r_config* cfg, const SwigluCall& a, cudaStream_t s) {
  if (a.R == 0) return C2R_OK;
  if (cfg->dtype == C2R_F32) return simt_swiglu_bwd<float>(cfg, a, s);
  if (tc_supported(cfg, a.nE, a.I, a.R)) return tc_swiglu_bwd(cfg, a, s);
  return simt_swiglu_bwd<__nv_bfloat16>(cfg, a, s);
}

extern "C" int c2r_swiglu_qparts(const c2r_config* cfg, int n_experts, int I, int64_t R) {
  if (check_gemm_args(cfg, n_experts, I, R) != C2R_OK) return -1;
  return swiglu_qparts(cfg, n_experts, I, R);
}

extern "C" int c2r_grouped_swiglu_fwd(const c2r_config* cfg, int n_experts, int I, int64_t R, const void* Xp,
                                      const int32_t* counts, const int32_t* offsets, const void* W13p, const void* W2,
                                      void* AB, void* H, void* Yp, const c2r_expert_opts* opts, int32_t* status,
                                      void* stream) {
  int rc = check_gemm_args(cfg, n_experts, I, R);
  if (rc) return rc;
  SwigluCall a{};
  a.nE = n_experts; a.I = I; a.R = R; a.Xp = Xp; a.counts = counts; a.offsets = offsets; a.W13p = W13p; a.W2 = W2;
  a.AB = AB; a.H = H; a.Yp = Yp; a.status = status;
  if ((rc = apply_opts(cfg, opts, a, false))) return rc;
  C2R_REQUIRE((Xp || a.X) && counts && offsets && W13p && W2 && H && (Yp || a.token_acc), C2R_ERR_INVALID_ARG);
  return swiglu_fwd_dispatch(cfg, a, as_stream(stream));
}

extern "C" int c2r_grouped_swiglu_bwd(const c2r_config* cfg, int n_experts, int I, int64_t R, const void* Xp,
                                      const int32_t* counts, const int32_t* offsets, const void* W13p, const void* W2,
                                      const void* AB, const void* H, const void* dYp, void* dAB, void* dXp,
                                      void* dW13p, void* dW2, int accumulate, const c2r_expert_opts* opts,
                                      int32_t* status, void* stream) {
  int rc = check_gemm_args(cfg, n_experts, I, R);
  if (rc) return rc;
  SwigluCall a{};
  a.nE = n_experts; a.I = I; a.R = R; a.Xp = Xp; a.counts = counts; a.offsets = offsets; a.W13p = W13p; a.W2 = W2;
  a.AB = const_cast<void*>(AB); a.H = const_cast<void*>(H); a.dYp = dYp; a.dAB = dAB; a.dXp = dXp; a.dW13p = dW13p;
  a.dW2 = dW2; a.accumulate = accumulate; a.status = status;
  if ((rc = apply_opts(cfg, opts, a, true))) return rc;
  C2R_REQUIRE((Xp || a.X) && counts && offsets && W13p && W2 && AB && H && dYp && dAB && (dXp || a.token_acc) && dW13p &&
                  dW2,
              C2R_ERR_INVALID_ARG);
  return swiglu_bwd_dispatch(cfg, a, as_stream(stream));
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

// Layout of the C2R_WS_LAYER workspace.
struct LayerWs {
  char* permute;    // per-block expert counts of the dispatch
  char* gate_bwd;   // scratch of c2r_gate_bwd
  float* qpart;     // [nq][R] partial row dots of the routed experts' backward
  float* qspart;    // [nqs][N] the same for the shared expert
  int nq, nqs;
  size_t bytes;
};
static LayerWs layer_ws(const c2r_config* cfg, void* base) {
  LayerWs w;
  const int64_t R = permuted_rows(cfg);
  w.nq = swiglu_qparts(cfg, cfg->E, cfg->I > 0 ? cfg->I : 16, R);
  w.nqs = cfg->I_s > 0 ? swiglu_qparts(cfg, 1, cfg->I_s, cfg->N) : 0;
  size_t o = 0;
  w.permute = (char*)base + o; o += align256(permute_ws_bytes(cfg));
  w.gate_bwd = (char*)base + o; o += align256(gate_bwd_ws_bytes(cfg));
  w.qpart = (float*)((char*)base + o); o += align256(sizeof(float) * (size_t)w.nq * (size_t)R);
  w.qspart = (float*)((char*)base + o); o += align256(sizeof(float) * (size_t)w.nqs * (size_t)cfg->N);
  w.bytes = o;
  return w;
}
size_t c2r::layer_ws_bytes(const c2r_config* cfg) { return layer_ws(cfg, nullptr).bytes; }

// The shared expert depends on nothing the routing chain produces.  With a second stream (and two events) in the
// buffers its GEMMs are enqueued there, between fork() and join(); without, everything stays on the one stream.
struct SideStream {
  cudaStream_t main, side;
  cudaEvent_t fork_ev, join_ev;
  bool on;
  SideStream(const c2r_layer_buffers* b, void* stream, bool wanted)
      : main(as_stream(stream)), side((cudaStream_t)b->stream2), fork_ev((cudaEvent_t)b->ev_fork),
        join_ev((cudaEvent_t)b->ev_join), on(wanted && b->stream2 && b->ev_fork && b->ev_join) {}
  void* work() const { return on ? (void*)side : (void*)main; }
  int fork() const {
    if (!on) return C2R_OK;
    C2R_CUDA(cudaEventRecord(fork_ev, main));
    C2R_CUDA(cudaStreamWaitEvent(side, fork_ev, 0));
    return C2R_OK;
  }
  int join() const {
    if (!on) return C2R_OK;
    C2R_CUDA(cudaEventRecord(join_ev, side));
    C2R_CUDA(cudaStreamWaitEvent(main, join_ev, 0));
    return C2R_OK;
  }
};

// The fused combine needs the fp32 per-token accumulators.
static bool fused_combine(const c2r_config* cfg) { return (cfg->flags & C2R_FLAG_FUSED_COMBINE) != 0; }

extern "C" int c2r_layer_fwd(const c2r_config* cfg, const c2r_layer_buffers* b, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  C2R_REQUIRE(b, C2R_ERR_INVALID_ARG);
  const bool shared = cfg->I_s > 0;
  const bool fcomb = fused_combine(cfg);
  C2R_REQUIRE(b->ws && b->ws_bytes >= c2r_workspace_bytes(cfg, C2R_WS_LAYER), C2R_ERR_WORKSPACE);
  C2R_REQUIRE(b->w_row && (fcomb ? b->Yacc != nullptr : b->Yp != nullptr), C2R_ERR_INVALID_ARG);
  if (shared)
    C2R_REQUIRE(b->wsg && b->z && b->Ws13p && b->Ws2 && b->Hs && (fcomb || b->Ys) && b->s_counts && b->s_offsets,
                C2R_ERR_INVALID_ARG);
  const int64_t R = permuted_rows(cfg);
  const LayerWs ws = layer_ws(cfg, b->ws);
  const SideStream ss(b, stream, shared);
  C2R_TRY(gate_logits_impl(cfg, b->X, b->Wg, shared ? b->wsg : nullptr, b->L, b->z, b->status, stream));
  if (shared) {
    // shared expert, its sigmoid gate applied to H inside the GEMM: Ys = sigmoid(z) * Shared(x).  With the fused
    // combine its output initialises the per-token accumulator the routed experts then add to.
    c2r_expert_opts o{};
    o.row_scale = b->z; o.scale_kind = C2R_SCALE_SIGMOID;
    C2R_TRY(ss.fork());
    C2R_TRY(c2r_grouped_swiglu_fwd(cfg, 1, cfg->I_s, cfg->N, b->X, b->s_counts, b->s_offsets, b->Ws13p, b->Ws2, b->ABs,
                                   b->Hs, fcomb ? (void*)b->Yacc : b->Ys, &o, b->status, ss.work()));
  } else if (fcomb) {
    C2R_CUDA(cudaMemsetAsync(b->Yacc, 0, sizeof(float) * (size_t)cfg->N * cfg->d, as_stream(stream)));
  }
  // routing leaves the dispatch's per-block histogram in the workspace; the dispatch also spreads the weights
  C2R_TRY(route_impl(cfg, b->L, b->mask, b->idx, b->w, nullptr, b->status, (int32_t*)ws.permute, stream));
  const bool gfused = gather_fused(cfg, b->X);
  C2R_TRY(permute_call(cfg, b->idx, b->expert_rank, gfused ? nullptr : b->X, b->counts, b->offsets, b->row_of_slot,
                       b->slot_of_row, b->Xp, b->status, ws.permute, align256(permute_ws_bytes(cfg)), stream, cfg->N > 0,
                       b->w, b->w_row));
  // routed experts with the Eq. 1 weight of each row applied to H: Yp = w * Expert(x)
  c2r_expert_opts o{};
  o.row_scale = b->w_row; o.scale_kind = C2R_SCALE_ROW;
  if (gfused) { o.X = b->X; o.slot_of_row = b->slot_of_row; }
  if (fcomb) {
    o.token_acc = b->Yacc; o.slot_of_row = b->slot_of_row;
    C2R_TRY(ss.join());  // the accumulator holds the shared expert's term before the routed rows are added
  }
  C2R_TRY(c2r_grouped_swiglu_fwd(cfg, cfg->E, cfg->I, R, gfused ? nullptr : b->Xp, b->counts, b->offsets, b->W13p, b->W2,
                                 b->AB, b->H, fcomb ? nullptr : b->Yp, &o, b->status, stream));
  if (!fcomb) C2R_TRY(ss.join());
  // the weights are already inside Yp and Ys: a plain sum over the token's K rows plus the shared term
  // (fused combine: the sum is complete, what is left is the conversion to the storage type)
  C2R_TRY(c2r_combine(cfg, fcomb ? nullptr : b->Yp, nullptr, b->row_of_slot,
                      fcomb ? (void*)b->Yacc : (shared ? b->Ys : nullptr), nullptr, b->Y, stream));
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
  const bool fcomb = fused_combine(cfg);
  C2R_REQUIRE(b->ws && b->ws_bytes >= c2r_workspace_bytes(cfg, C2R_WS_LAYER), C2R_ERR_WORKSPACE);
  C2R_REQUIRE(b->dY && b->dYp && b->dAB && (fcomb ? b->dXacc != nullptr : b->dXp != nullptr) && b->dl && b->dW13p &&
                  b->dW2 && b->dWg && b->dX && b->w_row,
              C2R_ERR_INVALID_ARG);
  if (shared) C2R_REQUIRE(b->dABs && (fcomb || b->dXs) && b->dz && b->dWs13p && b->dWs2 && b->dwsg, C2R_ERR_INVALID_ARG);
  const int64_t R = permuted_rows(cfg);
  const LayerWs ws = layer_ws(cfg, b->ws);
  const SideStream ss(b, stream, shared);
  if (shared) {
    // the shared expert reads dY as it is; its gate enters through the row scale
    c2r_expert_opts o{};
    o.row_scale = b->z; o.scale_kind = C2R_SCALE_SIGMOID; o.qpart = ws.qspart;
    C2R_TRY(ss.fork());
    C2R_TRY(c2r_grouped_swiglu_bwd(cfg, 1, cfg->I_s, cfg->N, b->X, b->s_counts, b->s_offsets, b->Ws13p, b->Ws2, b->ABs,
                                   b->Hs, b->dY, b->dABs, fcomb ? (void*)b->dXacc : b->dXs, b->dWs13p, b->dWs2, accumulate,
                                   &o, b->status, ss.work()));
  } else if (fcomb) {
    C2R_CUDA(cudaMemsetAsync(b->dXacc, 0, sizeof(float) * (size_t)cfg->N * cfg->d, as_stream(stream)));
  }
  // transpose of the combine's gather: every permuted row receives its token's dY unchanged
  C2R_TRY(c2r_permute_rows(cfg, b->dY, b->row_of_slot, b->counts, b->offsets, b->dYp, stream));
  const bool gfused = gather_fused(cfg, b->X);
  c2r_expert_opts o{};
  o.row_scale = b->w_row; o.scale_kind = C2R_SCALE_ROW; o.qpart = ws.qpart;
  if (gfused) { o.X = b->X; o.slot_of_row = b->slot_of_row; }
  if (fcomb) {
    o.token_acc = b->dXacc; o.slot_of_row = b->slot_of_row;
    C2R_TRY(ss.join());  // the shared expert's dX term is in the accumulator before the routed rows are added
  }
  C2R_TRY(c2r_grouped_swiglu_bwd(cfg, cfg->E, cfg->I, R, gfused ? nullptr : b->Xp, b->counts, b->offsets, b->W13p, b->W2,
                                 b->AB, b->H, b->dYp, b->dAB, fcomb ? nullptr : b->dXp, b->dW13p, b->dW2, accumulate, &o,
                                 b->status, stream));
  if (!fcomb) C2R_TRY(ss.join());
  C2R_TRY(c2r_route_bwd_scaled(cfg, b->w, b->row_of_slot, ws.qpart, ws.nq, shared ? b->z : nullptr, ws.qspart, ws.nqs, b->dw,
                               b->dl, shared ? b->dz : nullptr, stream));
  C2R_TRY(c2r_gate_bwd(cfg, b->X, b->Xp, b->counts, b->offsets, b->slot_of_row, b->idx, b->dl, shared ? b->dz : nullptr,
                       b->dWg, shared ? b->dwsg : nullptr, accumulate, ws.gate_bwd, align256(gate_bwd_ws_bytes(cfg)),
                       stream));
  C2R_TRY(c2r_unpermute_grad(cfg, fcomb ? nullptr : b->dXp, b->row_of_slot,
                             fcomb ? (void*)b->dXacc : (shared ? b->dXs : nullptr), b->idx, b->dl, b->Wg,
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
