/*
 * l2a.h -- C ABI of the B200 (sm_100a) hot path of the L2A conditional attention layer.
 *
 * The layer (paper Section 3.1, Eq. 2-5): every token gets causal sliding-window ("Local")
 * attention s_t; tokens whose routing decision d_t = 1 additionally get exact causal ("Global")
 * attention a_t over the full prefix; the output is o_t = s_t + d_t * a_t.  The kernel-level
 * method (Section 3.2, Algorithm 1): routed queries are compacted into a contiguous buffer with
 * their original positions recorded (Q_idx), attention is tiled over the compact rows with the
 * causal mask taken from the true positions, and the result is scattered back.
 *
 * Conventions shared by every call
 *   - Every pointer is a DEVICE pointer unless its comment says "host".  The caller owns all
 *     buffers, including the workspaces; the library allocates no device memory and never
 *     synchronises the stream (only l2a_workspace_status, l2a_step_host and l2a_step_host_wait do).  State kept between
 *     calls: per-device facts looked up once (SM count, kernel attributes); the fixed device array
 *     and its cached address of l2a_route_compact_static; the per-thread helper streams and events of
 *     l2a_step_host / l2a_step_host_async; the one-shot event registration of l2a_profile_next_call.
 *   - Tensors are contiguous bf16:  Q, O, dO, dQ, S_save, A_c : [B, Lq, Hq, D]
 *                                   K, V, dK, dV              : [B, Lk, Hkv, D]
 *     D contiguous, base pointers 16-byte aligned.  D is 64 or 128.  Hq % Hkv == 0 (GQA: query
 *     head h reads KV head h / (Hq/Hkv)).
 *   - Positions are 0-based.  Query row t sits at position p = t + q_pos_offset; the local
 *     neighbourhood is max(0, p - window) <= j <= p (self plus `window` predecessors, the mask
 *     0 <= i - j <= w of Section 2), the global neighbourhood is 0 <= j <= p.
 *   - Routing is per token and shared by all heads (the router projection has one output, Eq. 3).
 *   - Each call validates its arguments on the host and returns L2A_ERR_* before launching
 *     anything; work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = default).
 *   - Device-side waits are bounded; a wait that runs out is recorded in the workspace's status
 *     word and the kernels finish without writing further results (see l2a_workspace_status).
 */
#ifndef L2A_H_
#define L2A_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  L2A_OK = 0,
  L2A_ERR_INVALID_ARG = -1,    /* NULL pointer, bad shape, misaligned base pointer          */
  L2A_ERR_UNSUPPORTED = -2,    /* valid request this build does not implement               */
  L2A_ERR_WORKSPACE = -3,      /* workspace pointer NULL / misaligned / too small           */
  L2A_ERR_CUDA = -4,           /* a CUDA runtime or driver call failed (launch, encode)     */
  L2A_ERR_DEVICE_TIMEOUT = -5, /* a bounded device-side wait ran out (l2a_workspace_status) */
  L2A_ERR_DEVICE_BOUNDS = -6   /* debug build only (-DL2A_DEBUG): an index derived from q_idx / prefix / tile      */
                               /* metadata fell outside its tensor; the store was skipped (l2a_workspace_status)   */
} l2a_status;

/* l2a_params.flags */
#define L2A_FLAG_SAVE_FOR_BWD 1u  /* forward also writes S_save and A_c (needed by l2a_backward)  */
#define L2A_FLAG_SKIP_LOCAL 2u    /* forward: no local module; O = d * A (the "SWA-0" ablation).   */
                                  /* backward: gradients of the Global Attention module only       */
#define L2A_FLAG_SKIP_GLOBAL 4u   /* forward: local module only; O = S (first phase of the layer, */
                                  /* before the router has seen S).  backward: gradients of the   */
                                  /* Local Attention module only                                  */
#define L2A_FLAG_GLOBAL_PHASE 16u  /* forward: second phase of the layer.  O (and S_save) already hold   */
                                  /* the local output from an earlier L2A_FLAG_SKIP_GLOBAL call; only  */
                                  /* the routed rows' global attention runs and is added into O.       */
                                  /* Lets the caller compute the router decision from S in between     */
                                  /* (Eq. 2 -> 3 -> 4 -> 5 in the order the layer defines them).       */
#define L2A_FLAG_SHARED_WINDOW 64u /* Only for callers that really pass ONE Q/K/V set to both modules (the benchmark     */
                                  /* configurations do; in the paper's layer Global Attention reads the local output   */
                                  /* s_t through its own projections, so its Q/K/V differ from the local module's and   */
                                  /* the flag does not apply).  With one set, a routed row's scores against the keys    */
                                  /* inside its window are the ones the Local pass has already reduced, so Global       */
                                  /* Attention covers only the keys BEFORE the window (positions 0 .. t-W-1) and is     */
                                  /* merged with the local result,                                                      */
                                  /*   a_t = (e^{lse_out} o_out + e^{lse_loc} s_t) / (e^{lse_out} + e^{lse_loc}),       */
                                  /* which is the softmax over the whole prefix.  Saves rho * W pairs per head.         */
                                  /* s_t enters as the stored bf16 value (one extra rounding of relative size 2^-9      */
                                  /* on the window's share of a_t; same tolerance).  Needs lse_loc (also without        */
                                  /* L2A_FLAG_SAVE_FOR_BWD); not combined with L2A_FLAG_SKIP_LOCAL or                   */
                                  /* L2A_FLAG_FORCE_ALL_GLOBAL; ignored by a call that has L2A_FLAG_SKIP_GLOBAL.        */
                                  /* A_c, lse_glb and O mean the same as without it, so the backward does not depend    */
                                  /* on how the forward was run.  Passed to l2a_backward, the flag allows the same       */
                                  /* sharing there: inside the window P_glb = beta_t P_loc with                          */
                                  /* beta_t = exp(lse_loc - lse_glb) and dP = dO V^T is common to both modules, so       */
                                  /* the local tile pairs carry both gradients (row statistics                           */
                                  /* lse' = lse_loc - log(1 + beta), Delta' = (Delta_loc + beta Delta_glb)/(1 + beta))   */
                                  /* and the global ones stop before the window.  Used only when both outputs get the    */
                                  /* same gradient (not l2a_backward_split with its own dS_loc) and without              */
                                  /* FORCE_ALL_GLOBAL / SKIP_*; otherwise ignored.                                       */
#define L2A_FLAG_FORCE_ALL_GLOBAL 8u /* training iterations that invoke Global Attention for every    */
                                  /* token regardless of d_t (Section 3.3: done with a small       */
                                  /* probability so that masked tokens' routers get a gradient).   */
                                  /* O is unchanged (a_t is still multiplied by d_t), but A_c and   */
                                  /* lse_glb are then indexed by ROW t and hold a_t for every t,    */
                                  /* and l2a_backward's dgate covers every token.  Pass the flag to */
                                  /* both calls.  Needs L2A_FLAG_SAVE_FOR_BWD.                      */

/* router_kind of l2a_route_compact */
#define L2A_ROUTER_MASK_U8 0     /* router = uint8 [B, Lq], non-zero => routed                    */
#define L2A_ROUTER_LOGITS_F32 1  /* router = fp32 logits [B, Lq]; d = (z >= logit_threshold)      */
#define L2A_ROUTER_LOGITS_BF16 2 /* router = bf16 logits [B, Lq], compared in fp32 (exact upcast)  */

typedef struct l2a_params {
  int32_t B, Lq, Lk, Hq, Hkv, D;
  int32_t window;       /* W >= 0: keys j with 0 <= p - j <= W                                    */
  int32_t q_pos_offset; /* p = t + q_pos_offset; pass Lk - Lq for bottom-right aligned causality  */
  float softmax_scale;  /* scores are softmax_scale * q.k ; pass 0 for the default 1/sqrt(D)      */
  uint32_t flags;       /* L2A_FLAG_*                                                             */
  /* Optional strides, in elements, of the [B, L, H, D] tensors: {batch stride, token stride}; the heads of
   * a token and the D values of a head stay contiguous (head stride = D).  {0, 0} = dense.  Both must be
   * multiples of 8 (16 bytes), token stride >= H * D, batch stride >= L * token stride.  This is the layout of
   * slices of a fused QKV projection output [B, L, (Hq + 2 Hkv) * D].  q_stride applies to Q and dQ, k_stride to
   * K and dK, v_stride to V and dV, o_stride to O, dO and dS_loc.  S_save, A_c and the workspaces are always
   * dense.  l2a_step_host, l2a_router_backward and the q / O arguments of l2a_decode take dense tensors only
   * (L2A_ERR_UNSUPPORTED otherwise). */
  int64_t q_stride[2], k_stride[2], v_stride[2], o_stride[2];
  /* Packed variable-length batch (optional; NULL = every batch entry is one sequence).  Device pointer to the
   * per-token table written by l2a_pack_sequences: int32 [Lq][2] = {first token of the token's sequence, one past its
   * last token}.  The token axis then holds several sequences back to back and no query attends across a sequence
   * boundary: token t sees the keys max(t - W, first) .. t (Local Attention) and first .. t (Global Attention);
   * key blocks and query tiles that lie wholly in other sequences are not visited.  Needs B == 1, Lq == Lk and
   * q_pos_offset == 0.  Routing, compaction and every output keep their meaning on the packed token axis, and the
   * results are, sequence by sequence, those of one call per sequence (equal up to fp32 rounding: the key blocks are
   * aligned to the packed axis, not to each sequence's start).  The table is read by l2a_forward*, l2a_backward* and
   * l2a_forward_routed; l2a_step_host and l2a_decode reject it (L2A_ERR_UNSUPPORTED).  The paper evaluates padded
   * batches only; this layout is the usual one for training on documents of mixed length. */
  const int32_t* seq_bounds;
} l2a_params;

/* Version / capability string of the loaded library (host pointer, static storage). */
const char* l2a_version(void);

/* Human-readable name of a status code (host pointer, static storage). */
const char* l2a_status_string(l2a_status s);

/*
 * Workspace sizes in bytes for the three calls, for the given shape (worst case over routing:
 * they do not depend on how many tokens are routed).  Any of the three outputs may be NULL.
 * Workspaces must be 256-byte aligned device memory.  Contents need not be preserved between
 * calls, except that the backward reads nothing from the forward's workspace either: everything
 * the backward needs is passed explicitly.
 */
l2a_status l2a_workspace_bytes(const l2a_params* p, size_t* route_ws_bytes, size_t* fwd_ws_bytes,
                               size_t* bwd_ws_bytes);

/*
 * Self-test of the bounded device-side wait (the mechanism behind L2A_ERR_DEVICE_TIMEOUT).  Launches one small
 * kernel in which a warp waits, with a limit of `limit_us` microseconds (1 .. 1000000), for an mbarrier arrival that
 * never comes, while the other warps wait for something else: the first wait runs out, raises the CTA's abort flag,
 * the other warps leave their waits on seeing it, and the CTA writes the status word of workspace `ws` (any 256-byte
 * aligned device buffer of at least 256 bytes) -- the path every kernel of this library takes when a wait runs
 * out.  Afterwards l2a_workspace_status(ws) returns L2A_ERR_DEVICE_TIMEOUT and the context stays usable.  Nothing
 * traps, faults or spins without a limit.  Returns L2A_ERR_INVALID_ARG for a limit outside the range.
 */
l2a_status l2a_selftest_wait_timeout(void* ws, unsigned limit_us, void* stream);

/*
 * Reads the status word the kernels of earlier calls left in workspace `ws` (any of the three).
 * Synchronises `stream`.  Returns L2A_OK, or L2A_ERR_DEVICE_TIMEOUT if a bounded device-side wait
 * ran out in some kernel that used this workspace since it was last used by a successful call, or
 * (debug build) L2A_ERR_DEVICE_BOUNDS if an index check failed.
 */
l2a_status l2a_workspace_status(const void* ws, void* stream);

/*
 * Packed variable-length batches: expands the sequence boundaries into the per-token table that
 * l2a_params.seq_bounds points to.
 *   cu_seqlens  device int32 [n_seq + 1], ascending, cu_seqlens[0] = 0: sequence i holds the tokens
 *               cu_seqlens[i] .. cu_seqlens[i + 1] - 1 of the packed axis
 *   seq_bounds  device int32 [Lq][2], written: {first token, one past the last token} of each token's sequence.
 *               Tokens at or after cu_seqlens[n_seq] (padding at the end of the axis) become sequences of their own.
 * One small kernel on `stream`; no allocation.  Entries of cu_seqlens that are not ascending give masks that
 * correspond to no batch, but no access outside the tensors.
 */
l2a_status l2a_pack_sequences(const int32_t* cu_seqlens, int n_seq, int Lq, int32_t* seq_bounds, void* stream);

/*
 * Routing decision and query compaction (Eq. 3; Section 3.2: the routed queries are gathered into one
 * dense buffer and the sequence position of each is kept; Algorithm 1, step 1).
 *
 *   router      in : [B, Lq] uint8 mask, fp32 logits or bf16 logits, per router_kind.  For logits the decision
 *                    is taken on the logit in fp32, d = (z >= logit_threshold); threshold 0 is
 *                    sigmoid(z) >= 0.5, the tie z == threshold routes, NaN does not.
 *   d_mask      out: [B, Lq] uint8, 0 or 1.
 *   q_idx       out: [B, Lq] int32.  Row b holds the routed row indices t of batch entry b in
 *                    ascending order in its first n_routed[b] entries; the rest is -1.
 *   n_routed    out: [B] int32 (stays on the device; nothing here reads it on the host).
 *   prefix      out: [B, Lq + 1] int32, prefix[b][t] = number of routed rows u < t
 *                    (the compact index of row t if it is routed); prefix[b][Lq] = n_routed[b].
 *   route_ws       : workspace of at least route_ws_bytes.
 * Integer results are exact.  Returns L2A_ERR_INVALID_ARG for NULL/misaligned pointers or a bad
 * router_kind; nothing is launched in that case.
 */
l2a_status l2a_route_compact(const l2a_params* p, const void* router, int router_kind, float logit_threshold,
                             uint8_t* d_mask, int32_t* q_idx, int32_t* n_routed, int32_t* prefix,
                             void* route_ws, size_t route_ws_bytes, void* stream);

/*
 * Router logits from the local output (Eq. 3: d_hat_t = sigmoid(W s_t), one scalar per token), with the
 * sparsity regulariser's sum (Eq. 6) as a by-product.
 *
 *   S           in : bf16 [B, Lq, Hq, D], the local output s_t (as written by l2a_forward); the router sees
 *                    the Hq * D values of a token as one vector.
 *   w           in : fp32 [Hq * D] router weights; bias: scalar added to every logit.
 *   logits      out: fp32 [B, Lq], z_t = w . s_t + bias (fp32 accumulation), ready for
 *                    l2a_route_compact(..., L2A_ROUTER_LOGITS_F32, threshold 0).
 *   sum_sq      out: optional fp32 [B] (may be NULL): sum_t sigmoid(z_t)^2, the un-normalised regulariser
 *                    of Eq. 6 (the caller multiplies by lambda / (n L)).  Accumulated with atomics: the
 *                    last bits depend on the order of addition.
 * HBM-bound: one pass over S.
 */
l2a_status l2a_router_logits(const l2a_params* p, const void* S, const float* w, float bias, float* logits,
                             float* sum_sq, void* stream);

/*
 * Forward of the layer (Eq. 2, 4, 5; Algorithm 1 for the global part).
 *
 *   Q, K, V     in : bf16, layouts above.
 *   d_mask, q_idx, n_routed, prefix
 *               in : exactly as written by l2a_route_compact for the same shape.
 *   O           out: bf16 [B, Lq, Hq, D];  O_t = S_t + d_t * A_t, rounded to bf16 once more after
 *                    the sum for routed rows; rows with d_t = 0 are bit-identical to a run with
 *                    no routed rows at all.
 *   S_save      out: bf16 [B, Lq, Hq, D], the local output s_t.  Required with
 *                    L2A_FLAG_SAVE_FOR_BWD, otherwise may be NULL.
 *   A_c         out: bf16 [B, Lq, Hq, D] worst case; compact row c of batch b (c < n_routed[b])
 *                    holds a_t of row t = q_idx[b][c] (Algorithm 1's O_c).  Rows >= n_routed[b]
 *                    are not written.  Required with L2A_FLAG_SAVE_FOR_BWD, otherwise may be NULL.
 *   lse_loc     out: fp32 [B, Hq, Lq], natural-log log-sum-exp of the local scores of row t.
 *   lse_glb     out: fp32 [B, Hq, Lq], first n_routed[b] entries of each (b, h) row: natural-log
 *                    log-sum-exp of the global scores of compact row c (Algorithm 1's L_c).
 *                    Both lse outputs may be NULL unless L2A_FLAG_SAVE_FOR_BWD is set.
 *   fwd_ws         : workspace of at least fwd_ws_bytes (holds the compact query buffer Q_c).
 * Scores and soft-max run in fp32, probabilities are rounded to bf16 for the second contraction,
 * accumulation is fp32.  Returns L2A_ERR_UNSUPPORTED for D not in {64, 128}.
 */
l2a_status l2a_forward(const l2a_params* p, const void* Q, const void* K, const void* V,
                       const uint8_t* d_mask, const int32_t* q_idx, const int32_t* n_routed,
                       const int32_t* prefix, void* O, void* S_save, void* A_c, float* lse_loc,
                       float* lse_glb, void* fwd_ws, size_t fwd_ws_bytes, void* stream);

/*
 * Backward of the layer: the vector-Jacobian product of l2a_forward with the routing mask held
 * fixed (Section 3.2: gradients only for active queries in the global part, reusing L_c and Q_idx;
 * the local part is a sliding-window attention backward).  With one Q/K/V set feeding both
 * modules, dQ_t = dQ_loc,t + d_t * dQ_glb,t and dK, dV sum both modules' contributions and the
 * query heads of each KV group.
 *
 * When the Global Attention module has its own Q/K/V (its own projections of s_t, Section 3.1), the layer is two
 * calls each way: forward L2A_FLAG_SKIP_GLOBAL with the local set, then L2A_FLAG_GLOBAL_PHASE with the global
 * set; backward L2A_FLAG_SKIP_GLOBAL with the local set (gradients of Q, K, V; d_mask, q_idx, n_routed, prefix,
 * A_c, lse_glb may be NULL) and L2A_FLAG_SKIP_LOCAL with the global set (dQ is zero outside the routed rows;
 * S_save, lse_loc may be NULL).  Both skip flags at once, or either with L2A_FLAG_FORCE_ALL_GLOBAL, is
 * L2A_ERR_INVALID_ARG.
 *
 *   Q, K, V, d_mask, q_idx, n_routed, prefix : as given to l2a_forward.
 *   dO          in : bf16 [B, Lq, Hq, D], gradient of the loss w.r.t. O.
 *   S_save, A_c, lse_loc, lse_glb
 *               in : as written by l2a_forward with L2A_FLAG_SAVE_FOR_BWD.
 *   dQ          out: bf16 [B, Lq, Hq, D].  The contributions of the key blocks meet in fp32 accumulators in the
 *                    workspace through atomic additions, in no fixed order: two runs agree to fp32 rounding of
 *                    the sums (and almost always bit for bit after the bf16 rounding), not by construction.
 *   dK, dV      out: bf16 [B, Lk, Hkv, D].  Accumulated on chip in a fixed order: bit-reproducible.
 *   dgate       out: optional fp32 [B, Lq] (may be NULL): sum over heads of dO_t . a_t -- the
 *                    loss-dependent term of the straight-through router gradient (Eq. 7) -- for
 *                    the rows whose global output was computed: routed rows (0 elsewhere), or
 *                    every row with L2A_FLAG_FORCE_ALL_GLOBAL.
 *   bwd_ws         : workspace of at least bwd_ws_bytes (compact copies of Q and dO, row statistics, and two fp32
 *                    dQ accumulators of B * Hq * ceil(Lq / 128) * 128 * D floats each).
 */
l2a_status l2a_backward(const l2a_params* p, const void* Q, const void* K, const void* V,
                        const uint8_t* d_mask, const int32_t* q_idx, const int32_t* n_routed,
                        const int32_t* prefix, const void* dO, const void* S_save, const void* A_c,
                        const float* lse_loc, const float* lse_glb, void* dQ, void* dK, void* dV,
                        float* dgate, void* bwd_ws, size_t bwd_ws_bytes, void* stream);

/*
 * Forward and backward of a layer whose Global Attention module has its OWN Q/K/V (Section 3.1: both modules are
 * initialised from the base model's attention and have their own projections; Global Attention projects the local
 * output s_t).  (Q, K, V) feed Local Attention, (Qg, Kg, Vg) -- same shapes and strides -- feed Global Attention
 * of the routed rows; o_t = s_t + d_t a_t as before.  All three of Qg, Kg, Vg NULL: one set feeds both modules and the
 * calls are l2a_forward / l2a_backward.  Otherwise they are the two-phase sequences described above in one call,
 * bit for bit (dQ up to the order of its fp32 sums): forward = local phase, then global phase added into O;
 * backward = the local module's gradients into dQ, dK, dV and the global module's into dQg, dKg, dVg (dQg is zero
 * outside the routed rows); dgate as in l2a_backward.  L2A_FLAG_SHARED_WINDOW does not apply to two sets and is
 * ignored; the SKIP / PHASE flags (and, in the backward, FORCE_ALL_GLOBAL) are L2A_ERR_INVALID_ARG.
 */
l2a_status l2a_forward_sets(const l2a_params* p, const void* Q, const void* K, const void* V, const void* Qg,
                            const void* Kg, const void* Vg, const uint8_t* d_mask, const int32_t* q_idx,
                            const int32_t* n_routed, const int32_t* prefix, void* O, void* S_save, void* A_c,
                            float* lse_loc, float* lse_glb, void* fwd_ws, size_t fwd_ws_bytes, void* stream);
l2a_status l2a_backward_sets(const l2a_params* p, const void* Q, const void* K, const void* V, const void* Qg,
                             const void* Kg, const void* Vg, const uint8_t* d_mask, const int32_t* q_idx,
                             const int32_t* n_routed, const int32_t* prefix, const void* dO, const void* S_save,
                             const void* A_c, const float* lse_loc, const float* lse_glb, void* dQ, void* dK, void* dV,
                             void* dQg, void* dKg, void* dVg, float* dgate, void* bwd_ws, size_t bwd_ws_bytes,
                             void* stream);

/*
 * l2a_backward with a separate gradient for the local output.  o_t = s_t + d_t a_t, but s_t also feeds the
 * router (z_t = W s_t + bias, Eq. 3), so in a trained layer dL/ds_t = dL/do_t + dz_t W (Section 3.3, straight-
 * through estimator).  dS_loc (bf16 [B, Lq, Hq, D], e.g. written by l2a_router_backward) drives the Local
 * Attention backward; dO drives the Global Attention backward (da_t = d_t dO_t) and dgate.  Everything else is as
 * in l2a_backward, which is this call with dS_loc = dO.
 */
l2a_status l2a_backward_split(const l2a_params* p, const void* Q, const void* K, const void* V,
                              const uint8_t* d_mask, const int32_t* q_idx, const int32_t* n_routed,
                              const int32_t* prefix, const void* dO, const void* dS_loc, const void* S_save,
                              const void* A_c, const float* lse_loc, const float* lse_glb, void* dQ, void* dK,
                              void* dV, float* dgate, void* bwd_ws, size_t bwd_ws_bytes, void* stream);

/*
 * Router backward under the straight-through estimator (Section 3.3, Eq. 7, with the gradient of the sparsity
 * regulariser of Eq. 6).  With d_hat_t = sigmoid(z_t):
 *     dL/dd_hat_t = dgate_t + 2 reg_coeff d_hat_t,     dz_t = dL/dd_hat_t d_hat_t (1 - d_hat_t),
 *     dw = sum_t dz_t s_t,   dbias = sum_t dz_t,   dS_loc_t = dO_t + dz_t w.
 *
 *   S           in : bf16 [B, Lq, Hq, D] local output (S_save of l2a_forward);  w in: fp32 [Hq * D].
 *   logits      in : fp32 [B, Lq], z_t as written by l2a_router_logits.
 *   dgate       in : optional fp32 [B, Lq] from l2a_backward (NULL = 0: regulariser only).
 *   reg_coeff      : lambda / (n L) of Eq. 6 (n tokens, L layers); 0 disables the regulariser term.
 *   dO, dS_loc     : optional pair (both or neither): bf16 [B, Lq, Hq, D] in / out, dS_loc = dO + dz w rounded to
 *                    bf16 once; dS_loc may alias dO.
 *   dz          out: optional fp32 [B, Lq].
 *   dw, dbias   out: optional fp32 [Hq * D] and [1]; zeroed by this call, then accumulated with atomics (the last
 *                    bits depend on the order of addition).
 * All pointers are device memory.  HBM-bound: one pass over S (and over dO, dS_loc when given).
 */
l2a_status l2a_router_backward(const l2a_params* p, const void* S, const float* w, const float* logits,
                               const float* dgate, float reg_coeff, const void* dO, float* dz, float* dw,
                               float* dbias, void* dS_loc, void* stream);

/*
 * The whole layer forward in its defining order, without the caller in between: Local Attention (Eq. 2) ->
 * router logits z_t = router_w . s_t + router_bias on the local output (Eq. 3) -> d_t = (z_t >= logit_threshold),
 * compaction -> Global Attention of the routed tokens added into O (Eq. 4, 5).  Equal, bit for bit, to
 * l2a_forward(L2A_FLAG_SKIP_GLOBAL), l2a_router_logits, l2a_route_compact, l2a_forward(L2A_FLAG_GLOBAL_PHASE).
 *
 *   p->flags       : L2A_FLAG_SAVE_FOR_BWD and L2A_FLAG_FORCE_ALL_GLOBAL allowed; the SKIP and PHASE flags are not.
 *   logits      out: fp32 [B, Lq];  sum_sq out: optional fp32 [B] (see l2a_router_logits).
 *   d_mask, q_idx, n_routed, prefix: outputs, as in l2a_route_compact; the remaining arguments as in l2a_forward.
 * Nothing is read back to the host: the routed count stays on the device.
 */
l2a_status l2a_forward_routed(const l2a_params* p, const void* Q, const void* K, const void* V,
                              const float* router_w, float router_bias, float logit_threshold, float* logits,
                              float* sum_sq, uint8_t* d_mask, int32_t* q_idx, int32_t* n_routed, int32_t* prefix,
                              void* O, void* S_save, void* A_c, float* lse_loc, float* lse_glb, void* route_ws,
                              size_t route_ws_bytes, void* fwd_ws, size_t fwd_ws_bytes, void* stream);

/*
 * Decode step (Section 3.4): one new token per sequence.  The token attends to the last `window` + 1 keys of
 * the cache (Local Attention) and, only when its routing decision is 1, to the whole cache (Global
 * Attention, skipped entirely otherwise); o = s + d * a.  The full K/V cache is kept either way, because a
 * later routed token may need it.
 *
 *   p           : Lq must be 1; Lk = number of cached tokens INCLUDING the new one; q_pos_offset = position of
 *                 the new token (normally Lk - 1); Hq / Hkv <= 8.
 *   q           in : bf16 [B, 1, Hq, D];  K, V in: bf16 [B, Lk, Hkv, D] (the cache).
 *   d           in : uint8 [B] routing decision of the new token (NULL = not routed); device memory.
 *   O           out: bf16 [B, 1, Hq, D].
 *   ws             : device workspace of l2a_decode_workspace_bytes, 256-byte aligned: a status header (read it
 *                    with l2a_workspace_status) and the partial soft-max results of the key chunks.
 * Keys after q_pos_offset are never used, whatever they hold.  A layer whose Global Attention was pruned keeps
 * only its last window + 1 keys: call with d = NULL, Lk = window + 1 slots (q_pos_offset = Lk - 1); the result
 * does not depend on the order of the slots, so the cache may be a ring buffer.  HBM-bound: reads the local window once and, for
 * routed tokens, the cache once.  Errors: L2A_ERR_INVALID_ARG (Lq != 1, NULL or unaligned pointers),
 * L2A_ERR_UNSUPPORTED (Hq / Hkv > 8), L2A_ERR_WORKSPACE, L2A_ERR_CUDA; a bounded device wait that runs out is
 * reported by the status header, not by the return value.
 */
l2a_status l2a_decode_workspace_bytes(const l2a_params* p, size_t* ws_bytes);
l2a_status l2a_decode(const l2a_params* p, const void* q, const void* K, const void* V, const uint8_t* d,
                      void* O, void* ws, size_t ws_bytes, void* stream);

/*
 * One whole step for callers that hold HOST buffers, so that end-to-end time including the
 * transfers can be measured through the C ABI: copies Q, K, V, the router input (and dO) to the
 * device buffers the caller supplies, runs l2a_route_compact + l2a_forward (+ l2a_backward when
 * host->dO is non-NULL), copies O (and dQ, dK, dV) back, and synchronises the stream.  The transfers overlap
 * the kernels on two helper streams the library creates once per host thread (dO goes up during the
 * forward, O / dK / dV come down during the backward); this is the one call that keeps such state.
 * `host` holds HOST pointers (pinned memory makes the copies asynchronous); `dev` holds DEVICE
 * pointers with the sizes the corresponding arguments of the three calls need.  With a backward,
 * p->flags must contain L2A_FLAG_SAVE_FOR_BWD and every field of `dev` must be set; without one,
 * dO, S_save, A_c, lse_*, dQ, dK, dV and bwd_ws may be NULL.
 */
typedef struct l2a_host_io {
  const void *Q, *K, *V;  /* bf16, layouts above                                   */
  const void* router;     /* [B, Lq] uint8, fp32 or bf16, per router_kind          */
  const void* dO;         /* bf16 [B, Lq, Hq, D] or NULL for a forward-only step   */
  void* O;                /* out                                                   */
  void *dQ, *dK, *dV;     /* out; may be NULL when dO is NULL                      */
} l2a_host_io;

typedef struct l2a_device_io {
  void *Q, *K, *V, *router, *dO;
  uint8_t* d_mask;
  int32_t *q_idx, *n_routed, *prefix;
  void *O, *S_save, *A_c;
  float *lse_loc, *lse_glb;
  void *dQ, *dK, *dV;
  void* route_ws; size_t route_ws_bytes;
  void* fwd_ws;   size_t fwd_ws_bytes;
  void* bwd_ws;   size_t bwd_ws_bytes;
} l2a_device_io;

l2a_status l2a_step_host(const l2a_params* p, const l2a_host_io* host, const l2a_device_io* dev,
                         int router_kind, float logit_threshold, void* stream);

/*
 * The same step, enqueued only: the call returns when its copies and kernels are queued, and l2a_step_host_wait
 * blocks until every step enqueued by this host thread has delivered its results.  For a training loop that keeps
 * two steps in flight on TWO sets of device tensors used alternately (`dev` of step i + 1 differs from that of
 * step i and equals that of step i - 1): the uploads of step i + 1 then run under the kernels of step i and the
 * downloads of step i under the kernels of step i + 1, so that in steady state a step costs its kernels only.
 * Ordering the library provides: the uploads of a step wait for the kernels of the step before the previous one
 * (the last user of the same device tensors), its kernels for that step's downloads; kernels of successive steps
 * run in order on `stream`.  What the caller provides: at most two steps in flight between waits, alternating
 * device sets as above, the same `stream` for every step, and host result buffers of a step that are not read
 * before l2a_step_host_wait returns (successive steps may share them: they are written in step order).
 * Results are those of l2a_step_host.
 */
l2a_status l2a_step_host_async(const l2a_params* p, const l2a_host_io* host, const l2a_device_io* dev,
                               int router_kind, float logit_threshold, void* stream);
l2a_status l2a_step_host_wait(void* stream);

/*
 * l2a_route_compact without any caller-provided scratch (an addition of this library; the paper has
 * no counterpart).  Same inputs, outputs and results as l2a_route_compact, but the per-CTA counts the
 * two kernels exchange live in a fixed device array compiled into the library instead of in
 * `route_ws`, and the call performs no device allocation of any kind.
 *
 * Who needs this: callers that cannot obtain device memory at the point of the call -- code running
 * inside an engine whose allocator has already reserved all of HBM for its own pools, plug-ins that
 * are handed tensors but no allocator, and latency-critical loops that must not touch cudaMalloc
 * (which may synchronise the whole device) once they are running.
 *
 * Limits and rules:
 *   - B * ceil(Lq / 4096) must not exceed L2A_STATIC_ROUTE_SLOTS (4096 counts, 16 KB; e.g. B = 1 up
 *     to Lq = 16,777,216, or B = 128 at Lq = 131,072).  Larger shapes are rejected on the host with
 *     L2A_ERR_UNSUPPORTED before anything is launched; use l2a_route_compact for those.
 *   - The array is static device memory: every GPU that loads the library holds its 16 KB until the
 *     process exits.
 *   - The first call on each device looks up the array's device address (with that device current)
 *     and caches it; make that first call before starting any stream capture.
 *   - All calls on one device share the array and it keeps the previous call's contents.  Nothing in
 *     it needs to start at zero (the first kernel overwrites every count the second one reads), but
 *     two calls whose kernels overlap on the GPU (different streams, no dependency) race on it:
 *     serialise them.
 */
#define L2A_STATIC_ROUTE_SLOTS 4096
l2a_status l2a_route_compact_static(const l2a_params* p, const void* router, int router_kind,
                                    float logit_threshold, uint8_t* d_mask, int32_t* q_idx,
                                    int32_t* n_routed, int32_t* prefix, void* stream);

/*
 * Profiling aid (no counterpart in the paper).  Registers up to 12 cudaEvent_t handles (host array of
 * `n_events` handles created by the caller with timing enabled; the array is copied).  The NEXT
 * l2a_forward or l2a_backward call made by this host thread records event k on its stream at its
 * k-th phase boundary and then clears the registration.  Phase boundaries:
 *   l2a_forward : 0 start | 1 after the query gather | 2 after the local kernel | 3 after the
 *                 global kernel
 *   l2a_backward: 0 start | 1 after the gathers | 2 after the Delta kernel and the clearing of the dQ accumulators |
 *                 3 after the five-GEMM kernel | 4 after the dQ merge (everything final).
 *                 With 7 (11) events the kernel runs as two (four) launches over key-block ranges -- keys below and
 *                 from 3/4 (1/2, 3/4, 7/8) of ceil(Lk / 128) blocks, when there are at least 8 (16) blocks -- each
 *                 followed by the merge of the dQ rows it completes: boundaries 3 + 2 r / 4 + 2 r after the kernel /
 *                 the merge of range r (dK, dV of the range's keys and dQ of the rows that see no later key are final).
 */
l2a_status l2a_profile_next_call(void* const* events, int n_events);

#ifdef __cplusplus
}
#endif
#endif /* L2A_H_ */
