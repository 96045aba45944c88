/*
 * c2r.h -- C ABI of the B200 (sm_100a) hot path of collaboration-constrained routing (C2R)
 * for Mixture-of-Experts layers (arXiv 2504.01337).
 *
 * Conventions, valid for every call unless its comment says otherwise
 *   - Pointers are DEVICE pointers; the few host pointers are named *_host.
 *   - The caller owns every buffer.  The library allocates no device memory, keeps no pointer
 *     after the enqueued kernels finish, never synchronises the stream and never traps.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = default stream).
 *   - Return value: C2R_OK or a negative c2r_error.  Argument and shape checks run on the host
 *     before anything is enqueued; after C2R_ERR_CUDA, c2r_last_cuda_error() gives the
 *     cudaError_t of the failed runtime call.
 *   - Matrices are row-major and dense.  "T" below is the storage type selected by
 *     cfg->dtype: float (C2R_F32) or bfloat16 (C2R_BF16).  Accumulation is always fp32.
 *     The per-(token, expert) partial results that are summed over k afterwards (Yp, Ys, dXp,
 *     dXs) are always float, so that the only rounding to T on the output path is the final one.
 *   - Notation follows the paper: N tokens, d hidden size, E routed experts, I expert
 *     intermediate size, K experts per token, T collaborator-set size, P logical partitions.
 *   - Shape limits: 1 <= K <= 8, K-1 <= T <= E-1, E <= 64 (E <= 63 with a shared expert),
 *     d % 8 == 0, I % 16 == 0, 1 <= P <= E, N*K < 2^30.
 */
#ifndef C2R_H_
#define C2R_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum c2r_error {
  C2R_OK = 0,
  C2R_ERR_INVALID_ARG = -1,       /* NULL where a buffer is required, or a value out of range */
  C2R_ERR_UNSUPPORTED_SHAPE = -2, /* a documented shape limit is violated */
  C2R_ERR_WORKSPACE = -3,         /* workspace missing or smaller than c2r_workspace_bytes() */
  C2R_ERR_CUDA = -4,              /* a CUDA runtime / driver call failed */
  C2R_ERR_STATIC_SCRATCH = -5     /* c2r_permute_static: the batch needs more than the built-in scratch */
} c2r_error;

enum { C2R_F32 = 0, C2R_BF16 = 1 };

/* status bits OR-ed into the optional device status word of c2r_route / c2r_permute */
enum {
  C2R_STATUS_NAN_LOGIT = 1,     /* a NaN logit was ordered as -inf */
  C2R_STATUS_SET_TOO_SMALL = 2, /* a collaborator mask offered fewer than K-1 experts */
  C2R_STATUS_BAD_INDEX = 4,     /* an expert index outside [0,E) was clamped */
  C2R_STATUS_WAIT_TIMEOUT = 8   /* a bounded wait inside a kernel gave up */
};

typedef struct c2r_config {
  int32_t N;         /* tokens in the batch */
  int32_t d;         /* hidden size */
  int32_t E;         /* routed experts */
  int32_t I;         /* intermediate size of a routed expert */
  int32_t K;         /* experts per token */
  int32_t T;         /* collaborator-set size, |Top-T(E_i)| (Eq. 4) */
  int32_t P;         /* logical expert partitions (expert-parallel degree that is modelled) */
  int32_t I_s;       /* intermediate size of the always-on shared expert, 0 = none */
  int32_t dtype;     /* C2R_F32 or C2R_BF16 */
  int32_t row_align; /* every expert's segment of the permuted layout starts at a multiple of this
                        (>= 1; the tensor-core GEMMs of the bf16 path need a multiple of 128) */
  int32_t renorm;    /* 1: weights = softmax over the K kept logits (Eq. 1); 0: full-softmax probabilities */
  int32_t flags;     /* OR of C2R_FLAG_* */
} c2r_config;

/* c2r_config.flags */
enum {
  C2R_FLAG_GATHER_FUSED = 1,  /* layer drivers (bf16 tensor-core path): the expert GEMMs fetch token rows straight
                                 from X through slot_of_row (TMA row gather); Xp is neither written nor read */
  C2R_FLAG_FUSED_COMBINE = 2  /* layer drivers: the down-projection and the dXp GEMM add their rows straight into
                                 per-token fp32 accumulators (Yacc, dXacc) instead of storing Yp / dXp for a gather
                                 pass; order of the fp32 adds not fixed (see c2r_expert_opts.token_acc) */
};

enum { C2R_WS_PERMUTE = 0, C2R_WS_GATE_BWD = 1, C2R_WS_LAYER = 2, C2R_WS_DISPATCH_DEDUP = 3 };

/* Per-row scale s_r the grouped SwiGLU calls can apply to H = s_r silu(A) B (and undo in their backward):
 * none, s_r = row_scale[r] (the Eq. 1 weight of the row's slot), or s_r = sigmoid(row_scale[r]) (the
 * shared expert's gate from its logit). */
enum { C2R_SCALE_NONE = 0, C2R_SCALE_ROW = 1, C2R_SCALE_SIGMOID = 2 };

/* Bytes of scratch the named call needs for this configuration (host function). */
size_t c2r_workspace_bytes(const c2r_config* cfg, int which);

/* Rows the permuted buffers (Xp, Yp, ...) must hold: N*K plus worst-case alignment padding. */
int64_t c2r_permuted_rows(const c2r_config* cfg);

/* cudaError_t of the last failed CUDA call made by this library on the calling thread. */
int c2r_last_cuda_error(void);

/* Number of kernels this library has launched in this process (all threads, all streams). */
uint64_t c2r_launch_count(void);

/* Sec. 3.1, Eq. 1 (argument of Top-K): L[t,e] = <X[t,:], Wg[e,:]>.
 * X [N,d] T; Wg [E,d] T; wsg [d] T or NULL (gate vector of the shared expert);
 * out: L [N,E] float; z [N] float = <X[t,:], wsg> (required iff wsg != NULL). */
int c2r_gate_logits(const c2r_config* cfg, const void* X, const void* Wg, const void* wsg,
                    float* L, float* z, void* stream);

/* Sec. 3.3 step 2 (C2R) and Eq. 1 (conventional Top-K when mask == NULL).
 * The top-1 expert i* is the arg-max of L[t,:]; the other K-1 experts are the best-scoring
 * j with bit j of mask[i*] set.  Order everywhere: (logit descending, index ascending);
 * NaN orders as -inf.  Selection is made on the raw fp32 logits.
 * L [N,E] float; mask [E] uint64 or NULL;
 * out: idx [N,K] int32 (column 0 = top-1, then selection order); w [N,K] float (Eq. 1 weights);
 *      p [N,E] float full-row softmax or NULL; status: one int32 (OR of C2R_STATUS_*) or NULL;
 *      permute_ws (optional, C2R_WS_PERMUTE bytes): receives the per-block expert histogram of idx that
 *      c2r_permute starts from; hand the same buffer to c2r_permute with ws_has_histogram = 1 and it skips
 *      its own histogram pass. */
int c2r_route(const c2r_config* cfg, const float* L, const uint64_t* mask, int32_t* idx, float* w,
              float* p, int32_t* status, void* permute_ws, void* stream);

/* Sec. 3.2, Eq. 2: C[i,j] = number of tokens whose selected set contains both i and j.
 * idx [n_tokens,K] int32; C [E,E] int32.  accumulate != 0 adds to C (profiling over several
 * batches), otherwise C is overwritten. */
int c2r_collab_count(const c2r_config* cfg, const int32_t* idx, int64_t n_tokens, int32_t* C,
                     int accumulate, void* stream);

/* Sec. 3.3 step 1, Eq. 4: I_T[i,:] = the cfg->T experts j != i with the largest C[i,j]
 * (ties: lower j); mask[i] has exactly those bits set.  C [E,E] int32; I_T [E,T] int32; mask [E] uint64. */
int c2r_collab_sets(const c2r_config* cfg, const int32_t* C, int32_t* I_T, uint64_t* mask, void* stream);

/* Sec. 3.2, Eq. 3 (collaboration degree): degree[i] = - sum_{j != i} p_ij ln p_ij with
 * p_ij = C[i,j] / sum_{j != i} C[i,j] (the normaliser runs over the same j != i as the sum; natural
 * logarithm; 0 ln 0 = 0; a row without co-activations gives 0).  Lower = more specialised collaboration.
 * C [E,E] int32; out: degree [E] float; mean (one float, may be NULL) = the layer's average over experts. */
int c2r_collab_degree(const c2r_config* cfg, const int32_t* C, float* degree, float* mean, void* stream);

/* Sec. 3.4: placement of the experts on devices by collaboration.  HOST function, host arrays.
 * mode 0 (greedy): partition p holds floor(E/P) + (p < E mod P) experts; it is seeded with the
 * unassigned expert of largest C[e,e] and grown by the unassigned expert with the largest summed
 * co-activation with its members (ties: lower id).  mode 1: part[e] = floor(e*P/E).
 * out: part_host [E]; rank_host [E] = position of expert e in the partition-major,
 * id-ascending layout order. */
int c2r_place_experts(const c2r_config* cfg, const int32_t* C_host, int mode, int32_t* part_host,
                      int32_t* rank_host);

/* The "dispatch" of Sec. 3.1 on one device: stable counting sort of the slots s = t*K+k by
 * expert_rank[idx[s]] (NULL = identity), then the row gather.
 * out: counts [E] int32; offsets [E+1] int32 (start row of expert e, a multiple of row_align;
 * offsets[E] = end of the layout); row_of_slot [N*K] int32; slot_of_row [c2r_permuted_rows] int32
 * (-1 = padding); Xp [c2r_permuted_rows, d] T with Xp[r,:] = X[slot_of_row[r]/K,:]; the padding rows that
 * close an expert's aligned segment are zero, rows at or beyond offsets[E] are not written.
 * X == NULL builds the index only.  w [N,K] float (optional) with w_row [c2r_permuted_rows] float (optional):
 * w_row[r] = w[slot_of_row[r]], 0 on rows without a slot -- the per-row scale of the expert calls below.
 * Atomic-free and deterministic.  An expert_rank that is not a permutation of [0,E) is replaced by the
 * identity order and reported as C2R_STATUS_BAD_INDEX.  ws: C2R_WS_PERMUTE bytes; ws_has_histogram != 0: c2r_route
 * already left the histogram of this very idx there.  status as in c2r_route. */
int c2r_permute(const c2r_config* cfg, const int32_t* idx, const int32_t* expert_rank, const void* X, const float* w,
                int32_t* counts, int32_t* offsets, int32_t* row_of_slot, int32_t* slot_of_row, void* Xp, float* w_row,
                int32_t* status, void* ws, size_t ws_bytes, int ws_has_histogram, void* stream);

/* The row gather of c2r_permute alone, for another [N,d] tensor and an index already built (the backward
 * pass spreads dY this way: every permuted row receives its token's row unchanged).
 * Xp[row_of_slot[t*K+k],:] = X[t,:]; padding rows that close an aligned segment are zeroed. */
int c2r_permute_rows(const c2r_config* cfg, const void* X, const int32_t* row_of_slot, const int32_t* counts,
                     const int32_t* offsets, void* Xp, void* stream);

/* Sec. 3.4 (zero-redundancy all-to-all), carried out on one device in its two stages.
 * Stage 1: every token is copied ONCE to each partition that hosts at least one of its selected
 * experts.  Partition q receives recv_counts[q] rows, in token order, at rows
 * [recv_offsets[q], recv_offsets[q+1]) of Xr; recv_offsets[P] is the number of rows an all-to-all
 * would carry (the `dedup` total of c2r_dispatch_volume, against N*K for the plain dispatch).
 * Stage 2, local to a partition: the per-expert layout of c2r_permute is filled from the receive
 * buffer, Xp[r,:] = Xr[recv_row_of_slot[slot_of_row[r]],:].  With a partition-major expert_rank a
 * partition's rows of Xp read only that partition's segment of Xr.
 * part [E] int32 (expert -> partition, cfg->P partitions); the other inputs as c2r_permute.
 * out: counts, offsets, row_of_slot, slot_of_row, Xp exactly as c2r_permute writes them (bit-exact);
 *      recv_counts [P], recv_offsets [P+1] int32; recv_row_of_slot [N*K] int32; token_of_recv_row
 *      [N*min(K,P)] int32 (-1 beyond recv_offsets[P]); Xr [N*min(K,P), d] T.
 * X == NULL builds the indices only.  Atomic-free and deterministic.  ws: C2R_WS_DISPATCH_DEDUP bytes. */
int c2r_dispatch_dedup(const c2r_config* cfg, const int32_t* idx, const int32_t* part, const int32_t* expert_rank,
                       const void* X, int32_t* counts, int32_t* offsets, int32_t* row_of_slot, int32_t* slot_of_row,
                       int32_t* recv_counts, int32_t* recv_offsets, int32_t* recv_row_of_slot,
                       int32_t* token_of_recv_row, void* Xr, void* Xp, int32_t* status, void* ws, size_t ws_bytes,
                       void* stream);

/* c2r_permute without a workspace argument (an addition of this library; the paper has no
 * counterpart).  Same inputs, same outputs and the same bit-exact results as c2r_permute; the
 * only difference is where the per-block expert counts live: in a fixed array of
 * C2R_PERMUTE_STATIC_SCRATCH_BYTES that is part of the library's device image, so the call (like
 * every call here) performs no cudaMalloc / cudaFree and the caller needs no scratch buffer either.
 *
 * Who needs it: callers that have no way to obtain device scratch at the point of the call --
 * a serving process whose device memory has been handed in full to its own pool, a plug-in
 * running under a host that forbids allocation on its hot path, or code in a latency-critical
 * section where cudaMalloc's device-wide synchronisation is not acceptable.
 *
 * Limit: ceil(N / b) * E * 4 bytes must fit the array, b = 512, 256, 160, 128, 96, 80, 64, 64 tokens
 * for K = 1..8 (a block of the sort owns at most 512 slots), i.e. about N*K <= 2.0 M slots at
 * E = 64 when K is a power of two; a larger batch is refused with C2R_ERR_STATIC_SCRATCH before
 * anything is enqueued.
 * Cost: every GPU that loads the library carries the array (1 MiB) until the process exits.
 * Set-up: the first call on each device looks up the array's device address (with that device
 * current); make that first call outside any stream capture.
 * Sharing: all calls on a device use the same array.  It keeps the previous call's contents,
 * which is harmless (each call writes every entry before reading it), but two calls whose
 * kernels can overlap on the GPU -- different streams, or different host threads on
 * unordered streams -- race on it and must be ordered by the caller. */
#define C2R_PERMUTE_STATIC_SCRATCH_BYTES (1u << 20)
int c2r_permute_static(const c2r_config* cfg, const int32_t* idx, const int32_t* expert_rank, const void* X,
                       int32_t* counts, int32_t* offsets, int32_t* row_of_slot, int32_t* slot_of_row, void* Xp,
                       int32_t* status, void* stream);

/* Weight layout used by the fused SwiGLU kernels (no counterpart in the paper).
 * W1 (gate projection) and W3 (up projection), both [n_experts, I, d] T, are interleaved in
 * blocks of 128 intermediate channels: block j holds rows [128j, 128j+b) of W1 followed by the
 * same rows of W3, b = min(128, I-128j).  W13p [n_experts, 2I, d] T.  unpack is the inverse and
 * also converts a gradient in packed layout back to (dW1, dW3). */
int c2r_pack_weights(const c2r_config* cfg, int n_experts, int I, const void* W1, const void* W3,
                     void* W13p, void* stream);
int c2r_unpack_weights(const c2r_config* cfg, int n_experts, int I, const void* W13p, void* W1,
                       void* W3, void* stream);

/* Options of the two grouped SwiGLU calls below (a NULL pointer to it, or a zeroed struct, selects none).
 *   row_scale / scale_kind: per-row scale s_r of H (C2R_SCALE_*; row_scale [R] float).  With the Eq. 1
 *     weights as row scale, Yp already carries the weight of Sec. 3.1's weighted sum.
 *   X with slot_of_row: the dispatch folded into the GEMMs (the gather-fused form): wherever the calls read
 *     row r of Xp, the kernels read row slot_of_row[r] / K of X [N,d] T instead (zeros where slot_of_row[r] < 0),
 *     so c2r_permute can run with X == NULL and no permuted copy of the hidden states exists (Xp may be NULL).
 *     Same results, bit for bit.  bf16 tensor-core shapes only, else C2R_ERR_UNSUPPORTED_SHAPE.
 *   token_acc with slot_of_row: the combine folded into the GEMM epilogue: the [R,d] float result (Yp forward,
 *     dXp backward) is not stored; row r is added into token_acc[slot_of_row[r] / K, :] ([N,d] float, which the
 *     caller has zeroed or pre-loaded, e.g. with the shared expert's output).  The adds are fp32 atomics: the
 *     order in which a token's K contributions arrive is not fixed, so results may differ in the last bits
 *     from run to run.  Yp / dXp may then be NULL.
 *   qpart (backward only): [c2r_swiglu_qparts(...)][R] float, partial sums whose total over the first index is
 *     q_r = <dH'_r, H_r> = s_r dLoss/ds_r, the gradient w.r.t. the row's scale times the scale (added up in
 *     index order by c2r_route_bwd_scaled); rows outside every expert's segment are not written. */
typedef struct c2r_expert_opts {
  const float* row_scale;
  int32_t scale_kind;
  int32_t reserved;
  const void* X;
  const int32_t* slot_of_row;
  float* token_acc;
  float* qpart;
} c2r_expert_opts;

/* Sec. 3.1: expert evaluation of the routed tokens; expert = SwiGLU MLP without biases.
 * For each expert e on rows [offsets[e], offsets[e]+counts[e]) of Xp:
 *   A = Xp W1_e^T, B = Xp W3_e^T, H = s_r silu(A) * B, Yp = H W2_e^T      (s_r = 1 without a row scale).
 * Xp [R,d] T; counts [n_experts], offsets [n_experts+1] int32 (device); W13p packed (above);
 * W2 [n_experts, d, I] T.  out: AB [R, 2I] T (what the backward pass needs from A and B, in the
 * packed column layout: the local derivatives B silu'(A) in the gate columns and silu(A) in the up
 * columns, without the scale; AB == NULL skips it: forward only, e.g. inference),
 * H [R,I] T (scale included), Yp [R,d] float.
 * R = rows of the buffers.  Padding rows of Xp must be zero.  n_experts = 1 with counts = {R},
 * offsets = {0,R} evaluates the dense shared expert.
 * bf16 runs on the tensor cores (tcgen05) when d % 16 == 0 and, for n_experts > 1, row_align is a
 * multiple of 128; other shapes and fp32 use a CUDA-core kernel.  status (one int32, may be NULL)
 * receives C2R_STATUS_WAIT_TIMEOUT if a bounded wait inside the kernel gave up (results invalid). */
int c2r_grouped_swiglu_fwd(const c2r_config* cfg, int n_experts, int I, int64_t R, const void* Xp,
                           const int32_t* counts, const int32_t* offsets, const void* W13p, const void* W2,
                           void* AB, void* H, void* Yp, const c2r_expert_opts* opts, int32_t* status, void* stream);

/* Backward of the above, given dYp = dLoss/dYp:  dH' = dYp W2 (the gradient w.r.t. the scaled H);
 * dA = s_r dH' B silu'(A); dB = s_r dH' silu(A); dXp = dA W1 + dB W3; dW2_e = dYp^T H; dW1_e = dA^T Xp;
 * dW3_e = dB^T Xp.  dYp [R,d] T (padding rows zero); AB, H as the forward call wrote them;
 * out: dAB [R,2I] T (packed columns), dXp [R,d] float, dW13p [n_experts,2I,d] T (packed rows),
 * dW2 [n_experts,d,I] T.  accumulate != 0 adds into the weight gradients. */
int c2r_grouped_swiglu_bwd(const c2r_config* cfg, int n_experts, int I, int64_t R, const void* Xp,
                           const int32_t* counts, const int32_t* offsets, const void* W13p, const void* W2,
                           const void* AB, const void* H, const void* dYp, void* dAB, void* dXp, void* dW13p,
                           void* dW2, int accumulate, const c2r_expert_opts* opts, int32_t* status, void* stream);

/* First dimension of c2r_expert_opts.qpart for this shape (host function; -1 on a bad argument). */
int c2r_swiglu_qparts(const c2r_config* cfg, int n_experts, int I, int64_t R);

/* Sec. 3.1 (weighted sum of the selected experts' outputs):
 * Y[t,:] = sum_k w[t,k] * Yp[row_of_slot[t*K+k],:]  (k ascending, fp32)
 *          + sigmoid(z[t]) * Ys[t,:] when Ys != NULL (gated shared expert).
 * w == NULL / z == NULL: that factor is 1 (the expert call already applied it as its row scale).
 * Yp == NULL: no such term (the GEMMs already added their rows into Ys: Y is Ys in the storage type).
 * Yp [R,d] float; Ys [N,d] float; out: Y [N,d] T. */
int c2r_combine(const c2r_config* cfg, const void* Yp, const float* w, const int32_t* row_of_slot,
                const void* Ys, const float* z, void* Y, void* stream);

/* Backward of c2r_combine: dYp[row(t,k),:] = w[t,k] dY[t,:] (padding rows zeroed);
 * dw[t,k] = <dY[t,:], Yp[row(t,k),:]>; dYs = sigmoid(z) dY; dz = <dY,Ys> sigmoid'(z).
 * dY [N,d] T; Yp, Ys float; out: dYp [R,d] T; dYs [N,d] T; dw [N,K], dz [N] float.
 * For callers that keep the weights outside the expert calls (c2r_combine with w, z); the layer drivers apply
 * them as the experts' row scale instead and get the same gradients from c2r_permute_rows, the backward expert
 * call's qpart and c2r_route_bwd_scaled, without reading Yp. */
int c2r_combine_bwd(const c2r_config* cfg, const void* dY, const void* Yp, const float* w,
                    const int32_t* row_of_slot, const int32_t* slot_of_row, const void* Ys, const float* z,
                    void* dYp, float* dw, void* dYs, float* dz, void* stream);

/* Backward of Eq. 1's softmax over the kept logits (cfg->renorm must be 1):
 * dl[t,k] = w[t,k] (dw[t,k] - sum_j w[t,j] dw[t,j]) -- the gradient w.r.t. L[t, idx[t,k]];
 * all other entries of dL are zero. */
int c2r_route_bwd(const c2r_config* cfg, const float* w, const float* dw, float* dl, void* stream);

/* c2r_route_bwd for experts that applied the weights themselves (C2R_SCALE_ROW / C2R_SCALE_SIGMOID): from the
 * partial row dots the backward expert call left, q[t,k] = sum_j qpart[j, row_of_slot[t*K+k]] = w dLoss/dw,
 *   dl[t,k] = q[t,k] - w[t,k] sum_j q[t,j]      (identical to the formula above, without dividing by w);
 *   dw[t,k] = q[t,k] / w[t,k] (optional output, 0 where w is 0);
 *   dz[t]   = (sum_j qspart[j,t]) (1 - sigmoid(z[t]))   (shared expert; optional).
 * qpart [nq, c2r_permuted_rows] float; qspart [nqs, N] float. */
int c2r_route_bwd_scaled(const c2r_config* cfg, const float* w, const int32_t* row_of_slot, const float* qpart, int nq,
                         const float* z, const float* qspart, int nqs, float* dw, float* dl, float* dz, void* stream);

/* Gate weight gradients: dWg[e,:] = sum_t dL[t,e] X[t,:], evaluated over expert e's rows of Xp
 * (dl addressed through slot_of_row); dwsg[:] = sum_t dz[t] X[t,:].
 * out: dWg [E,d] float; dwsg [d] float (iff dz != NULL); accumulate != 0 adds into both.
 * ws: C2R_WS_GATE_BWD bytes.
 * bf16 with X and ws given: evaluated as one tensor-core GEMM dL^T X over a dense [N,64] bf16 copy of the
 * gradient w.r.t. the logits (dl and dz rounded to bf16, fp32 accumulation, token splits added in a fixed
 * order); otherwise a row-serial fp32 kernel over Xp.  idx [N,K] (optional): with it the dense copy is written
 * token by token in one pass; without it, it is zeroed and filled expert by expert through slot_of_row. */
int c2r_gate_bwd(const c2r_config* cfg, const void* X, const void* Xp, const int32_t* counts,
                 const int32_t* offsets, const int32_t* slot_of_row, const int32_t* idx, const float* dl,
                 const float* dz, float* dWg, float* dwsg, int accumulate, void* ws, size_t ws_bytes, void* stream);

/* Gradient w.r.t. the hidden states (transpose of the dispatch, done as an atomic-free gather-sum):
 * dX[t,:] = sum_k dXp[row_of_slot[t*K+k],:]  + dXs[t,:]                (shared expert, optional)
 *           + sum_k dl[t,k] Wg[idx[t,k],:] + dz[t] wsg[:]              (gate, optional)
 *           + dX[t,:] when accumulate != 0.
 * dXp [R,d] float (NULL: no such term, e.g. when the GEMMs already added their rows into dXs);
 * dXs [N,d] float; out: dX [N,d] T. */
int c2r_unpermute_grad(const c2r_config* cfg, const void* dXp, const int32_t* row_of_slot, const void* dXs,
                       const int32_t* idx, const float* dl, const void* Wg, const float* dz, const void* wsg,
                       void* dX, int accumulate, void* stream);

/* Sec. 3.4 / Sec. 4.1 (token redundancy of the all-to-all).  part [E] int32 maps expert -> partition,
 * home(t) = floor(t*P/N).  out (device, overwritten):
 *   totals[0] = naive   = N*K rows (one per (token, expert));
 *   totals[1] = dedup   = number of distinct (token, partition) pairs (zero-redundancy scheme);
 *   totals[2], totals[3] = the same two counting only destinations != home(t);
 *   send_naive, send_dedup [P,P] uint64: rows from home partition src to partition dst.
 * redundancy r = 1 - dedup/naive. */
int c2r_dispatch_volume(const c2r_config* cfg, const int32_t* idx, const int32_t* part, uint64_t* totals,
                        uint64_t* send_naive, uint64_t* send_dedup, void* stream);

/* Buffers of one layer for the drivers below.  Unused members may be NULL (no shared expert:
 * every *s member; inference: every backward member). */
typedef struct c2r_layer_buffers {
  /* inputs and parameters */
  const void* X;              /* [N,d] T */
  const void* Wg;             /* [E,d] T */
  const void* wsg;            /* [d] T */
  const void* W13p;           /* [E,2I,d] T packed */
  const void* W2;             /* [E,d,I] T */
  const void* Ws13p;          /* [1,2I_s,d] T packed */
  const void* Ws2;            /* [1,d,I_s] T */
  const uint64_t* mask;       /* [E] collaborator masks, NULL = conventional Top-K */
  const int32_t* expert_rank; /* [E] or NULL */
  const int32_t* part;        /* [E] or NULL (dispatch volume skipped) */
  /* forward state */
  float* L;             /* [N,E] */
  float* z;             /* [N] */
  int32_t* idx;         /* [N,K] */
  float* w;             /* [N,K] */
  int32_t* counts;      /* [E] */
  int32_t* offsets;     /* [E+1] */
  int32_t* row_of_slot; /* [N*K] */
  int32_t* slot_of_row; /* [R] */
  float* w_row;         /* [R]: w of the slot that owns each permuted row */
  void* Xp;             /* [R,d] */
  void* AB;             /* [R,2I]; NULL (with ABs) when no backward pass follows */
  void* H;              /* [R,I], Eq. 1 weight of the row included */
  void* Yp;             /* [R,d] float, weight included */
  void* ABs;            /* [N,2I_s] */
  void* Hs;             /* [N,I_s], gate sigmoid(z) included */
  void* Ys;             /* [N,d] float, gate included */
  int32_t* s_counts;    /* [1]  = {N}   (device) */
  int32_t* s_offsets;   /* [2]  = {0,N} (device) */
  void* Y;              /* [N,d] T: layer output */
  float* Yacc;          /* [N,d] float, only with C2R_FLAG_FUSED_COMBINE (Yp, Ys may then be NULL) */
  uint64_t* volume;     /* [4 + 2*P*P] totals, send_naive, send_dedup */
  int32_t* status;      /* one int32 */
  /* backward */
  const void* dY; /* [N,d] T */
  void* dYp;      /* [R,d]: dY of the row's token */
  void* dAB;      /* [R,2I] */
  void* dXp;      /* [R,d] float */
  void* dABs;     /* [N,2I_s] */
  void* dXs;      /* [N,d] float */
  float* dw;      /* [N,K], may be NULL (informational: the backward pass itself needs only dl) */
  float* dl;      /* [N,K] */
  float* dz;      /* [N] */
  void* dW13p;    /* [E,2I,d] T */
  void* dW2;      /* [E,d,I] T */
  void* dWs13p;   /* [1,2I_s,d] T */
  void* dWs2;     /* [1,d,I_s] T */
  float* dWg;     /* [E,d] */
  float* dwsg;    /* [d] */
  void* dX;       /* [N,d] T */
  float* dXacc;   /* [N,d] float, only with C2R_FLAG_FUSED_COMBINE (dXp, dXs may then be NULL) */
  /* live profiling (c2r_train_step) */
  int32_t* C;          /* [E,E] */
  int32_t* I_T;        /* [E,T] */
  uint64_t* mask_next; /* [E]: sets for the next step */
  /* optional second stream for the shared expert, which depends on nothing the routing chain produces: a
   * cudaStream_t and two cudaEvent_t (created with cudaEventDisableTiming) owned by the caller.  All three
   * non-NULL: the shared expert's GEMMs are enqueued on stream2 between a fork from and a join into the
   * drivers' stream, so they overlap gate -> route -> dispatch and fill the tails of the routed GEMMs. */
  void* stream2;
  void* ev_fork;
  void* ev_join;
  /* scratch */
  void* ws;        /* C2R_WS_LAYER bytes */
  size_t ws_bytes;
} c2r_layer_buffers;

/* Forward of the whole layer, no host synchronisation:
 * gate -> route (C2R or Top-K) -> permute -> grouped SwiGLU (+ shared expert) -> combine
 * (-> dispatch volume when part != NULL).  The Eq. 1 weights and the shared expert's gate are applied
 * inside the expert calls (row scale), so the combine is a plain sum. */
int c2r_layer_fwd(const c2r_config* cfg, const c2r_layer_buffers* b, void* stream);

/* Backward of c2r_layer_fwd (routing decision frozen) using the state it left in `b`.
 * accumulate != 0 adds into every parameter gradient (dW13p, dW2, dWs13p, dWs2, dWg, dwsg); dX is always
 * overwritten. */
int c2r_layer_bwd(const c2r_config* cfg, const c2r_layer_buffers* b, int accumulate, void* stream);

/* Forward, backward, then Eq. 2 and Eq. 4 on this step's routing: C is overwritten from idx and
 * the refreshed sets are written to I_T / mask_next for the next step. */
int c2r_train_step(const c2r_config* cfg, const c2r_layer_buffers* b, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* C2R_H_ */
