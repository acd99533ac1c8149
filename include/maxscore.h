/*
 * maxscore.h -- C ABI of the MaxScore router for NVIDIA B200 (sm_100a).
 *
 * Maximum Score Routing (arXiv 2508.12801) for one MoE layer and one batch of T tokens:
 *
 *   gate logits      L = H . W_g                                   (Eq. 2)
 *   affinities       A = SoftTopk(L; k, t)                         (Eq. 6)
 *   assignment       P = argmax { sum_ij P_ij A_ij : P binary, every token has exactly k experts,
 *                                 every expert at most C tokens }  (Eq. 7-8, network of Table 1)
 *   capacity         C = ceil(cf * T * k / E)                      (Sec. 2.3; Algorithm 1, step 1)
 *   dispatch/combine tokens into and out of dense [E, C, d_model] expert buffers   (Eq. 1)
 *
 * Conventions that hold for every entry point
 *   - All tensor arguments are DEVICE pointers unless the name ends in _host.  Row-major, contiguous,
 *     16-byte aligned.  The caller owns every buffer; the library allocates no device memory and
 *     keeps no pointer after a call returns other than the workspace handed to maxscore_create.
 *   - cuda_stream is a cudaStream_t passed as void*.  Calls enqueue work and return without
 *     synchronising.  Calls on one context must not overlap on the GPU (they share the workspace).
 *   - Host-detectable errors (NULL pointers, bad sizes, k > E, infeasible capacity, misalignment,
 *     short workspace) return a status before anything is launched.  Conditions only the device sees
 *     (solver gave up, non-finite input) set bits in maxscore_stats.status, which the caller reads
 *     after synchronising.  Nothing aborts, throws or traps.
 *   - Every wait inside a kernel is bounded.  A wait that runs out raises the context's internal-error
 *     flag and the kernel returns with its output incomplete.  maxscore_route_fwd and maxscore_assign
 *     report the flag as MAXSCORE_STAT_INTERNAL in stats.status and clear it; after the calls that write
 *     no stats (maxscore_gate, maxscore_gate_bwd, maxscore_route_bwd) read it with maxscore_check_internal.
 *   - expert_idx[i, :] is ascending.  slot_idx[i, c] is the rank of token i among the tokens of expert
 *     expert_idx[i, c], in ascending token order.  Unused slots of slot_token hold -1.
 *   - If the solver runs out of its budget (MAXSCORE_STAT_NOT_CONVERGED; never seen with the default
 *     budget on the documented workloads) every token still has k distinct experts, but an expert may
 *     hold more than C tokens.  The surplus pairs then have slot_idx >= C: index build leaves them out of
 *     slot_token, dispatch does not write them, combine and the backward passes skip them (they contribute
 *     zero), so nothing is read or written out of bounds.
 *   - Limits of this build: 1 <= k <= 8, k <= E <= 128, bf16 I/O needs d_model % 8 == 0, fp32 I/O
 *     needs d_model % 4 == 0, T * k < 2^31.
 */
#ifndef MAXSCORE_H_
#define MAXSCORE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct maxscore_ctx maxscore_ctx; /* opaque; owns nothing but host bookkeeping */

typedef enum {
  MAXSCORE_OK = 0,
  MAXSCORE_ERR_INVALID_ARG = 1,   /* NULL pointer, non-positive size, misaligned pointer        */
  MAXSCORE_ERR_INFEASIBLE = 2,    /* k > E, or E * min(C, T) < T * k: no assignment exists       */
  MAXSCORE_ERR_WORKSPACE = 3,     /* workspace smaller than maxscore_workspace_bytes()           */
  MAXSCORE_ERR_CUDA = 4,          /* a CUDA runtime / driver call failed (see maxscore_last_cuda_error) */
  MAXSCORE_ERR_NOT_CONVERGED = 5, /* never returned by a call; mirrors the stats bit for readers */
  MAXSCORE_ERR_UNSUPPORTED = 6    /* outside the limits listed above                             */
} maxscore_status;

typedef enum { MAXSCORE_F32 = 0, MAXSCORE_BF16 = 1 } maxscore_dtype;

/* bits of maxscore_stats.status */
#define MAXSCORE_STAT_NOT_CONVERGED 1u /* solver hit max_sweeps; the assignment returned is not certified optimal */
#define MAXSCORE_STAT_NON_FINITE 2u    /* a NaN or Inf was seen in the score matrix                               */
#define MAXSCORE_STAT_INTERNAL 4u      /* an internal bound (a bounded wait, a path search) was hit               */

typedef struct {
  int32_t T;               /* tokens in the batch (the paper's n)                                  */
  int32_t d_model;         /* width of a token row                                                 */
  int32_t E;               /* experts (the paper's e)                                              */
  int32_t k;               /* experts per token                                                    */
  float capacity_factor;   /* c_f of Sec. 2.3; C = ceil(c_f * T * k / E)                           */
  int32_t capacity;        /* > 0 overrides the formula                                            */
  float t;                 /* SoftTopk temperature, > 0                                            */
  int32_t score_mode;      /* 0: maximise the float affinities A, as fixed-point keys              */
                           /*    rne(A * 2^40) + (((i*E + j) * 2654435761 mod 2^32) >> 20): the    */
                           /*    12-bit position hash only separates exact ties (< 4e-9 per pair); */
                           /* 1: maximise integer keys from the logits: q * 2^S + r with           */
                           /*    q = clamp_int16(rne(L * 2^quant_shift)),                          */
                           /*    r = fmix32(i*E + j + tiebreak_seed * 0x9E3779B9) >> 12            */
                           /*        (fmix32 = 32-bit finaliser of MurmurHash3),                   */
                           /*    S = 20 + ceil(log2(T*k))                                          */
  int32_t quant_shift;     /* score_mode 1 only                                                    */
  uint32_t tiebreak_seed;  /* score_mode 1 only                                                    */
  int32_t max_sweeps;      /* bound on price sweeps + augmentations of the solver; 0 = default     */
  int32_t io_dtype;        /* maxscore_dtype of hidden, w_gate, xdisp, yexp, y, dY, dH             */
  int32_t w_gate_layout;   /* 0: w_gate is [d_model, E] as in Eq. 2; 1: [E, d_model]               */
  int32_t softtopk_mode;   /* 0: Eq. 6 read as k masked softmaxes with temperature t (level j runs  */
                           /*    over the entries that are not among the j-1 largest); the default */
                           /* 1: Eq. 6 read literally: y_i = p_i * (beta + t * min(rank_i - delta, */
                           /*    k)), p = Softmax over all experts, rank 1 = largest, ties: lowest */
                           /*    index first                                                       */
                           /* 2: IterTopk of Table 2: y^(l) = y^(l-1) + g(x; 1 - y^(l-1)) for l = 1..k,  */
                           /*    g(x; w) = w e^x / sum(w e^x), y^(0) = 0; Table 2 has no temperature,    */
                           /*    so t is not used in this mode                                     */
  float rankscale_beta;    /* mode 1: 0 = the recursion starts from 0, 1 = it starts from Softmax  */
  int32_t rankscale_delta; /* mode 1: 0 = level j masks the j-1 largest, 1 = the j largest         */
} maxscore_params;

typedef struct {           /* lives in DEVICE memory; written by route_fwd / assign                */
  uint32_t status;         /* MAXSCORE_STAT_* bits                                                 */
  int32_t capacity;        /* C used                                                               */
  int32_t sweeps;          /* price sweeps run                                                     */
  int32_t augmentations;   /* exact augmenting paths applied after the sweeps                      */
  int32_t rounds;          /* candidate-collection rounds used by the exact phase                  */
  int32_t candidates;      /* tokens in the last candidate list                                    */
  int32_t rerouted;        /* token-slots assigned outside the token's own unconstrained top-k     */
  int32_t reserved;
  double total_score;      /* score_mode 0: sum of A over the chosen pairs; mode 1: sum of keys    */
} maxscore_stats;

/* C = ceil(c_f * T * k / E), or params->capacity when that is > 0 (Sec. 2.3).  Returns -1 on NULL. */
int32_t maxscore_capacity(const maxscore_params* params);

/* Bytes of device workspace a context for `params` needs.  Host only. */
maxscore_status maxscore_workspace_bytes(const maxscore_params* params, size_t* bytes);

/* Validate params, record the workspace (device memory, 256-byte aligned, at least the size above,
 * owned by the caller and left untouched by other work while the context lives) and build a context.
 * Performs no device work except one cudaMemsetAsync of the workspace head on the default stream,
 * followed by a synchronise. */
maxscore_status maxscore_create(maxscore_ctx** ctx, const maxscore_params* params, void* workspace,
                                size_t workspace_bytes);
void maxscore_destroy(maxscore_ctx* ctx);

/* Text of the last CUDA error seen by this thread's calls ("" if none). Host only. */
const char* maxscore_last_cuda_error(void);

/* ---- the four calls of the hot path ------------------------------------------------------------ */

/* Forward routing of one batch: Eq. 2, Eq. 6, Eq. 7-8, then the slot indices of the E x C buffers.
 *   hidden      [T, d_model]  io_dtype          in
 *   w_gate      per w_gate_layout, io_dtype     in
 *   expert_bias [E] fp32 or NULL                in   added to the logits (not in the paper; used to
 *                                                    skew the load in tests)
 *   logits      [T, E] fp32                     out  L
 *   scores      [T, E] fp32                     out  A
 *   expert_idx  [T, k] int32                    out  the experts of each token, ascending
 *   slot_idx    [T, k] int32                    out
 *   gate_w      [T, k] fp32                     out  A at the chosen pairs (R(x) of Eq. 1-2, not renormalised)
 *   slot_token  [E, C] int32                    out  token held by each slot, -1 = padding
 *   expert_load [E] int32                       out
 *   stats       device maxscore_stats           out */
maxscore_status maxscore_route_fwd(maxscore_ctx* ctx, const void* hidden, const void* w_gate,
                                   const float* expert_bias, float* logits, float* scores,
                                   int32_t* expert_idx, int32_t* slot_idx, float* gate_w,
                                   int32_t* slot_token, int32_t* expert_load, maxscore_stats* stats,
                                   void* cuda_stream);

/* Dispatch (Eq. 1, input side): dst[e, s, :] = src[slot_token[e, s], :], zero rows where the slot is
 * padding.  src [T, d_model], dst [E, C, d_model], both io_dtype.  Needs slot_idx and expert_idx too:
 * rows are read once per token and written to each of its k slots. */
maxscore_status maxscore_dispatch(maxscore_ctx* ctx, const void* src, const int32_t* expert_idx,
                                  const int32_t* slot_idx, const int32_t* slot_token, void* dst,
                                  void* cuda_stream);

/* Combine (Eq. 1, output side): dst[i, :] = sum_c gate_w[i, c] * src[expert_idx[i, c], slot_idx[i, c], :],
 * summed in ascending expert index in fp32 and rounded once.  gate_w NULL = unit weights (this is the
 * backward of dispatch).  accumulate != 0 adds to dst instead of overwriting it. */
maxscore_status maxscore_combine(maxscore_ctx* ctx, const void* src, const int32_t* expert_idx,
                                 const int32_t* slot_idx, const float* gate_w, void* dst,
                                 int accumulate, void* cuda_stream);

/* Backward of combine, SoftTopk and the gate with the assignment P held constant:
 *   dyexp[e, s, :]   = gate_w * dY[i, :]        (zero rows at padding slots)     [E, C, d_model] io_dtype
 *   dgate_w[i, c]    = <dY[i, :], yexp[e, s, :]>                                 [T, k] fp32
 *   dlogits          = J_SoftTopk^T . scatter(dgate_w)                           [T, E] fp32
 *   dw_gate          = H^T . dlogits            always [d_model, E] fp32
 *   dH               = dlogits . W_g^T          [T, d_model] io_dtype
 * slot_token is needed to zero the padding rows of dyexp. */
maxscore_status maxscore_route_bwd(maxscore_ctx* ctx, const void* dY, const void* yexp,
                                   const void* hidden, const void* w_gate, const float* logits,
                                   const int32_t* expert_idx, const int32_t* slot_idx,
                                   const float* gate_w, const int32_t* slot_token, void* dyexp,
                                   float* dgate_w, float* dlogits, float* dw_gate, void* dH,
                                   void* cuda_stream);

/* ---- single stages (the same kernels route_fwd / route_bwd run), for stage-by-stage checks ------ */

/* Eq. 2 only: logits = hidden . w_gate (+ expert_bias). */
maxscore_status maxscore_gate(maxscore_ctx* ctx, const void* hidden, const void* w_gate,
                              const float* expert_bias, float* logits, void* cuda_stream);

/* Eq. 6 only: scores = SoftTopk(logits; k, t). */
maxscore_status maxscore_softtopk_fwd(maxscore_ctx* ctx, const float* logits, float* scores,
                                      void* cuda_stream);

/* Derivative of Eq. 6: dlogits = J^T g where g is zero except g[i, expert_idx[i, c]] = dgate_w[i, c]. */
maxscore_status maxscore_softtopk_bwd(maxscore_ctx* ctx, const float* logits,
                                      const int32_t* expert_idx, const float* dgate_w,
                                      float* dlogits, void* cuda_stream);

/* Auxiliary load-balance loss, Eq. 9: loss = lambda / (E T^2) * sum_j (sum_i scores[i, j]) * expert_load[j]
 * (the column sum of the binary P is the expert's load), and its gradient with respect to the scores with
 * P held constant, which is the same for every token: dscores_col[j] = lambda * expert_load[j] / (E T^2).
 * scores [T, E] fp32, expert_load [E] int32, loss: one double, dscores_col [E] fp32; all device memory,
 * caller-owned.  Uses the context's workspace (calls on one context must not overlap).  Column sums are
 * accumulated in double with atomics, so the loss is reproducible to rounding (about 1e-15 relative), not
 * bit for bit.  Errors: NULL arguments -> MAXSCORE_ERR_INVALID_ARG. */
maxscore_status maxscore_aux_loss(maxscore_ctx* ctx, const float* scores, const int32_t* expert_load,
                                  float lambda, double* loss, float* dscores_col, void* cuda_stream);

/* maxscore_softtopk_bwd with the auxiliary loss folded in: g[i, j] = dscores_col[j] for every expert j, plus
 * dgate_w[i, c] at j = expert_idx[i, c]; dlogits = J^T g (derivative of Eq. 6 applied to the sum of the
 * gradients of Eq. 1 and Eq. 9). */
maxscore_status maxscore_softtopk_bwd_aux(maxscore_ctx* ctx, const float* logits, const int32_t* expert_idx,
                                          const float* dgate_w, const float* dscores_col, float* dlogits,
                                          void* cuda_stream);

/* Eq. 7-8 only: the solver on a caller-supplied [T, E] fp32 matrix (affinities in score_mode 0,
 * logits in score_mode 1).  Writes expert_idx [T, k], expert_load [E] and stats. */
maxscore_status maxscore_assign(maxscore_ctx* ctx, const float* matrix, int32_t* expert_idx,
                                int32_t* expert_load, maxscore_stats* stats, void* cuda_stream);

/* Algorithm 1 (Sec. 3.2): maximum score routing for top-2 the way the paper trains it.  Needs k = 2.
 *   steps 1-2  c_j = C (the context's capacity; 2n/e in the paper); a = scores (SoftTopk affinities of the caller)
 *   steps 4-6  every token's best expert (ties: lowest index) is fixed; the pair is removed from the second stage;
 *              c_j = max(0, c_j - number of tokens whose best expert is j)
 *   steps 7-9  one more expert per token by Sinkhorn on the residual problem.
 * The paper names Sinkhorn and nothing else; this library's reading: entropic regularisation sinkhorn_eps (in units of
 * score), K_ij = exp(a_ij / eps) over the pairs not fixed in step 4, sinkhorn_iters rounds of
 *     u_i = 1 / sum_j K_ij v_j,   t_j = sum_i u_i K_ij,   v_j = min(1, c_j / t_j)
 * (columns capped at the residual capacity rather than forced to meet it), a last row scaling, then every token takes
 * the arg-max of its plan row (ties: lowest index) and per expert the first c_j such tokens in ascending token index keep
 * it; the others end with one expert only.  Best-expert pairs are never dropped here, even beyond C: index build,
 * dispatch and combine skip what does not fit.  All arithmetic is fp64.
 *   scores [T, E] fp32 in; expert_idx [T, 2] out, ascending, -1 (dropped second expert) last; expert_load [E] out;
 *   plan [T, E] fp64 out or NULL (the row-scaled plan u_i K_ij v_j); counts [2] int32 DEVICE memory out: best-expert
 *   pairs beyond C, second experts dropped.  Uses the context's workspace.  The result approximates the maximum of
 *   Eq. 8; maxscore_assign gives the exact one. */
maxscore_status maxscore_assign_top2_sinkhorn(maxscore_ctx* ctx, const float* scores, float sinkhorn_eps,
                                              int32_t sinkhorn_iters, int32_t* expert_idx, int32_t* expert_load,
                                              double* plan, int32_t* counts, void* cuda_stream);

/* Iterative rerouting (Sec. 2.3, the Switch Transformers paragraph; the assignment of "MaxScore-I", Sec. 4.1):
 * the fast, approximate alternative to the flow of Eq. 7-8 that Sec. 3.2 names for k > 2.
 *   stage 1  top-k by affinity with capacity: choice level 1 of every token is served before level 2, ..., within
 *            a level in ascending token index; a pair is accepted while its expert holds fewer than C tokens;
 *   stage 2  the dropped pairs, in ascending token index and within a token in level order, go to the expert of
 *            highest affinity among those with room that the token does not hold, or stay empty if there is none.
 * Ties in affinity go to the lowest expert index.  The paper fixes neither serving order: both are this library's
 * reading.  scores [T, E] fp32 (finite) in; expert_idx [T, k] out, ascending, empty slots = -1 and last (index build,
 * dispatch and combine skip them); expert_load [E] out; counts [2] int32 DEVICE memory out: pairs dropped in stage 1,
 * slots left empty after stage 2.  Uses the context's workspace.  The result is feasible but in general not the
 * maximum of Eq. 8. */
maxscore_status maxscore_assign_iterative(maxscore_ctx* ctx, const float* scores, int32_t* expert_idx,
                                          int32_t* expert_load, int32_t* counts, void* cuda_stream);

/* Slot indices of an assignment: slot_idx [T, k], slot_token [E, C], expert_load [E]. */
maxscore_status maxscore_index_build(maxscore_ctx* ctx, const int32_t* expert_idx, int32_t* slot_idx,
                                     int32_t* slot_token, int32_t* expert_load, void* cuda_stream);

/* Derivative of Eq. 1 alone (first two outputs of route_bwd). */
maxscore_status maxscore_combine_bwd(maxscore_ctx* ctx, const void* dY, const void* yexp,
                                     const int32_t* expert_idx, const int32_t* slot_idx,
                                     const float* gate_w, const int32_t* slot_token, void* dyexp,
                                     float* dgate_w, void* cuda_stream);

/* Derivative of Eq. 2 alone (last two outputs of route_bwd). */
maxscore_status maxscore_gate_bwd(maxscore_ctx* ctx, const void* hidden, const void* w_gate,
                                  const float* dlogits, float* dw_gate, void* dH, void* cuda_stream);

/* ---- housekeeping (no counterpart in the paper) --------------------------------------------------- */

/* Reads and clears the context's internal-error flag: *flag_out != 0 means that a bounded wait inside one of
 * the tensor-core kernels (gate, gate backward) or the solver's grid barrier gave up since the flag was last
 * cleared, so some output of that call is incomplete.  Synchronises cuda_stream.  flag_out is HOST memory. */
maxscore_status maxscore_check_internal(maxscore_ctx* ctx, uint32_t* flag_out, void* cuda_stream);

/* Kernels launched through this context since maxscore_create (memsets and copies not counted).  Host only. */
long long maxscore_launch_count(const maxscore_ctx* ctx);

/* For tests of the error plumbing only: raises the internal-error flag from the host (one cudaMemsetAsync on
 * cuda_stream), as if a bounded wait had run out.  Nothing waits, hangs or faults. */
maxscore_status maxscore_test_raise_internal(maxscore_ctx* ctx, void* cuda_stream);

/* ---- end-to-end from host memory ---------------------------------------------------------------- */

/* route_fwd + dispatch for callers whose batch lives in HOST memory (pinned for full speed).
 * Copies hidden_host (and w_gate_host, expert_bias_host) to the device buffers given in `dev`,
 * runs maxscore_route_fwd and maxscore_dispatch, copies expert_idx, slot_idx, gate_w and stats back
 * to the *_host outputs and synchronises the stream before returning.  xdisp stays on the device
 * (dev->xdisp) for the experts to consume.
 * The rows of hidden_host go up in as many as eight blocks on a second stream that the context creates on
 * the first call (and maxscore_destroy releases); the gate GEMM and SoftTopk of a block run as soon as it has
 * landed, and the index arrays come back on that stream while the rows are dispatched.  The assignment
 * itself needs every row's scores, so it starts when the last block is in.  Both streams are ordered after
 * what was queued on cuda_stream before the call, and the results are the same as those of
 * maxscore_route_fwd + maxscore_dispatch on the same inputs.  Every dev buffer must be 16-byte aligned. */
typedef struct {
  void* hidden; void* w_gate; float* expert_bias; float* logits; float* scores; int32_t* expert_idx;
  int32_t* slot_idx; float* gate_w; int32_t* slot_token; int32_t* expert_load; maxscore_stats* stats;
  void* xdisp;
} maxscore_device_buffers;

maxscore_status maxscore_route_dispatch_host(maxscore_ctx* ctx, const void* hidden_host,
                                             const void* w_gate_host, const float* expert_bias_host,
                                             const maxscore_device_buffers* dev,
                                             int32_t* expert_idx_host, int32_t* slot_idx_host,
                                             float* gate_w_host, maxscore_stats* stats_host,
                                             void* cuda_stream);

/* ---- index build for callers that cannot allocate device memory ---------------------------------- */

/* The paper has no counterpart to this call; it exists for integration reasons only.
 *
 * Same result as maxscore_index_build (slot_idx [T, k], slot_token [E, C] with -1 padding,
 * expert_load [E]), but it needs neither a context nor a workspace: its scratch (per-block expert
 * counts) lives in a fixed array inside the library's device image.  It is meant for callers that must
 * not allocate while they run: code inside a region where cudaMalloc is forbidden or would
 * synchronise the device (a latency-critical serving loop, a plugin that only receives tensors its
 * host framework owns, a memory pool that is already fully handed out).  It calls no cudaMalloc,
 * cudaFree or any other allocating routine; the caller passes inputs and outputs only.
 *
 *   Limits: T <= MAXSCORE_NOALLOC_MAX_T (1,048,576 tokens), E <= 128, k <= 8, C >= 1.  Larger sizes
 *   return MAXSCORE_ERR_UNSUPPORTED before anything is launched.  The scratch array is 512 KiB and is
 *   held by every GPU that loads the library until the process exits.
 *   First call on a device: looks up the device address of the scratch array (cudaGetSymbolAddress,
 *   with that device current) and caches it for that device; make this first call outside any stream
 *   capture.  The call uses whichever device is current.
 *   Sharing: all calls on a device use the same scratch array.  Nothing in it has to start at zero
 *   (every entry read by a call is first written by that call), but two calls that overlap on the GPU
 *   (different streams, no ordering between them) race on it; order them on one stream or with events. */
#define MAXSCORE_NOALLOC_MAX_T 1048576
maxscore_status maxscore_index_build_noalloc(int32_t T, int32_t E, int32_t k, int32_t C,
                                             const int32_t* expert_idx, int32_t* slot_idx,
                                             int32_t* slot_token, int32_t* expert_load,
                                             void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* MAXSCORE_H_ */
