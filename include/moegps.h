/*
 * moegps.h - C ABI of the B200 (sm_100a) hot path of one Mixture-of-Experts inference layer with
 * prediction-driven expert duplication.
 *
 * The layer is the one whose load balance the MoE-GPS paper studies: tokens are routed to their
 * top-K experts (paper, Section 2), the per-expert token counts form the distribution that
 * Distribution-Only Prediction forecasts (Section 3.2.1, Eq. 1), a duplication plan replicates
 * popular experts (Section 3.1, Algorithm 1), tokens are shuffled to the replica that serves them
 * (the routing all-to-all of Section 2), the experts' SwiGLU FFNs run (Sections 2 and 3.4), and the
 * results are shuffled back to token order (last sentence of the communication paragraph of
 * Section 2).  Here all of it runs on ONE device: the "GPUs" of Algorithm 1 become S logical slots,
 * each holding one expert replica and owning a contiguous bucket of rows.
 *
 * Notation: T tokens, D model width, F expert hidden width, E experts, K experts per token,
 * S slots (S >= E), R = T*K routed pairs with flat index p = t*K + j, A = row_align,
 * Rcap = R + S*(A-1) rows in the permuted buffers.
 *
 * Conventions that hold for every call
 *  - Every tensor pointer is a DEVICE pointer owned by the caller, 16-byte aligned, row-major with
 *    the last dimension contiguous.  bf16 tensors are passed as `const void*` / `void*`.
 *  - The library allocates no device memory after moegps_create, copies nothing to the host and
 *    never synchronises, except in moegps_status.  `stream` is a cudaStream_t passed as void*
 *    (NULL = the legacy default stream).  Calls are asynchronous and ordered by the stream.
 *  - Outputs are fully overwritten unless stated; inputs are never modified.
 *  - Return value: MOEGPS_OK (0) or a negative moegps_error code.  Arguments are validated on the
 *    host before anything is launched; a failing call launches nothing.  Conditions only the device
 *    can see (an expert index out of range, a wait that ran out) are recorded in a device status
 *    word that moegps_status reads; the kernels skip the offending access instead of faulting.
 *  - A context belongs to the device it was created on, and that device must be the calling
 *    thread's current device in every call that launches work (and in moegps_status); otherwise the
 *    call returns MOEGPS_ERR_INVALID_ARG and launches nothing.
 *  - Device-side index checks: a slot extent, row or expert index outside its range is skipped (no
 *    out-of-range read or write is made for it) and MOEGPS_ERR_BAD_INDEX is recorded.
 *  - Weight layouts are "output features x input features", so both GEMM operands are contiguous
 *    along the contraction.
 *  - If the environment variable MOEGPS_TRACE is set (and not "0") when a context is created, every
 *    kernel launch made through that context is logged to stderr (ordinal, launcher, shape).  Host
 *    side only; nothing on the device changes.
 */
#ifndef MOEGPS_H_
#define MOEGPS_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define MOEGPS_API __attribute__((visibility("default")))
#else
#define MOEGPS_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum moegps_error {
  MOEGPS_OK = 0,
  MOEGPS_ERR_INVALID_ARG = -1,         /* null or misaligned pointer, n_slots != S, bad enum value   */
  MOEGPS_ERR_UNSUPPORTED_SHAPE = -2,   /* a dimension outside the limits listed at moegps_shape_t    */
  MOEGPS_ERR_WORKSPACE_TOO_SMALL = -3, /* raised only by a binding that knows the buffer's size: the C calls
                                          take a bare pointer and cannot check it (see moegps_dispatch)  */
  MOEGPS_ERR_CUDA = -4,                /* a CUDA runtime/driver call failed (see moegps_last_cuda_error) */
  MOEGPS_ERR_UNIMPLEMENTED = -5,
  MOEGPS_ERR_BAD_INDEX = -6,           /* device: an expert/row index outside its range was skipped  */
  MOEGPS_ERR_TIMEOUT = -7,             /* device: a bounded wait inside a kernel ran out             */
  MOEGPS_ERR_HIST_MISMATCH = -8,       /* device: `hist` passed to dispatch disagrees with topk_idx  */
  MOEGPS_ERR_STATIC_SCRATCH_EXCEEDED = -9  /* problem too large for moegps_dispatch_static's built-in scratch */
} moegps_error;

/* Problem shape, fixed for the life of a context.
 * Limits: 1 <= K <= min(E, 8); E <= 256; E <= S <= 1024; D and F multiples of 8;
 * T*K + S*(row_align-1) < 2^31; row_align a power of two in [1, 256]. */
typedef struct moegps_shape {
  int32_t T, D, F, E, K, S;
  int32_t gate_mode;   /* 0: softmax over the K selected logits; 1: sigmoid, then renormalise over the K */
  int32_t row_align;   /* A: every slot's first row is a multiple of A                                  */
  int32_t c_max;       /* Algorithm 1's C_max (most copies of one expert); 0 = no cap                   */
} moegps_shape_t;

typedef struct moegps_ctx moegps_ctx_t;   /* opaque: shape, device id, device status word, cached TMA descriptors */

/* Create / destroy a context on CUDA device `device`.  Allocates one small block of device memory
 * (about 1 KiB: the status word and the router's histogram accumulators); this is the only device
 * allocation the library ever makes. */
MOEGPS_API int moegps_create(moegps_ctx_t** out, const moegps_shape_t* shape, int device);
MOEGPS_API int moegps_destroy(moegps_ctx_t* ctx);

/* Number of permuted rows Rcap = T*K + S*(row_align-1) the caller must provide for xp/h_ws/yp/row_pair. */
MOEGPS_API int64_t moegps_rcap(const moegps_shape_t* shape);

/* Bytes of scratch (`workspace`, device, 16-byte aligned) moegps_dispatch needs for this shape. */
MOEGPS_API size_t moegps_workspace_bytes(const moegps_shape_t* shape);

/* route - top-K gating (paper, Section 2: each token goes to its top-K experts; the mapping is
 * never altered afterwards).
 *   logit[t,e] = sum_d x[t,d]*w_router[e,d] + bias[e]   (bf16 inputs, fp32 accumulation)
 *   topk_idx[t,0..K) = the K experts with the largest logits, in descending logit order; equal
 *   logits are ordered by ascending expert index.
 *   topk_w[t,j] = gate weight over the selected K (see moegps_shape_t.gate_mode), fp32.
 * x: bf16 [T,D]; w_router: bf16 [E,D]; bias: fp32 [E] or NULL; topk_idx: int32 [T,K]; topk_w: fp32 [T,K]. */
MOEGPS_API int moegps_route(moegps_ctx_t* ctx, const void* x, const void* w_router, const float* bias,
                 int32_t* topk_idx, float* topk_w, void* stream);

/* route_histogram - moegps_route and moegps_histogram in one kernel: the router's epilogue also
 * counts the selections per expert (the n_e of the paper's Eq. 1 with N = T*K), so the indices are
 * not read back from memory and one launch is saved.  Same arguments and results as moegps_route,
 * plus hist: int32 [E], fully overwritten.  The counts are summed with integer atomics (exact and
 * deterministic) in accumulators that belong to the context; the CTA that finishes last copies them
 * to hist and leaves the accumulators at zero.  Two such calls of ONE context must therefore not
 * overlap on the GPU (issue them on one stream, or order them with events); different contexts are
 * independent.  Bit-identical to moegps_route followed by moegps_histogram. */
MOEGPS_API int moegps_route_histogram(moegps_ctx_t* ctx, const void* x, const void* w_router, const float* bias,
                                      int32_t* topk_idx, float* topk_w, int32_t* hist, void* stream);

/* route_prepare + dispatch_prepared - the same results as moegps_route_histogram followed by
 * moegps_dispatch, in two launches instead of four.  The router's epilogue already holds, per CTA,
 * the per-expert counts of the token rows that CTA owns; route_prepare stores them as the columns of
 * the count matrix that dispatch ranks pairs with (into `workspace`); dispatch_prepared derives
 * slot_row_off from the finished histogram and the plan, ranks, places and copies (and marks padding
 * rows of row_pair with -1).  Copies of an expert share its pairs evenly (as in moegps_dispatch).
 * Bit-identical to the separate calls.
 * route_prepare: x, w_router, bias, topk_idx, topk_w, hist as in moegps_route_histogram; workspace:
 * moegps_workspace_bytes(shape) bytes, written here and read by dispatch_prepared (the layout is
 * private to the library: pass the same buffer, untouched, on the same stream).  Like
 * moegps_route_histogram it sums the counts in accumulators of the context: calls of one context
 * must not overlap on the GPU.
 * dispatch_prepared: arguments as moegps_dispatch, except that workspace is an input. */
MOEGPS_API int moegps_route_prepare(moegps_ctx_t* ctx, const void* x, const void* w_router, const float* bias,
                                    int32_t* topk_idx, float* topk_w, int32_t* hist, void* workspace,
                                    void* stream);
MOEGPS_API int moegps_dispatch_prepared(moegps_ctx_t* ctx, const void* x, const int32_t* topk_idx,
                                        const int32_t* hist, const int32_t* replicas, const int32_t* slot_off,
                                        int32_t* slot_row_off, int32_t* row_pair, int32_t* pair_row,
                                        void* xp, const void* workspace, void* stream);

/* Debug companion of moegps_route: also stores the fp32 logits (fp32 [T,E]) the selection was made on. */
MOEGPS_API int moegps_route_logits(moegps_ctx_t* ctx, const void* x, const void* w_router, const float* bias,
                        float* logits, void* stream);

/* histogram - per-expert counts n_e of the routed pairs (paper, Eq. 1: p_e = n_e / N with
 * N = T*K; this is the distribution that Distribution-Only Prediction estimates).
 * topk_idx: int32 [T*K]; hist: int32 [E].  An index outside [0,E) is skipped and reported as
 * MOEGPS_ERR_BAD_INDEX through the status word. */
MOEGPS_API int moegps_histogram(moegps_ctx_t* ctx, const int32_t* topk_idx, int32_t* hist, void* stream);

/* plan - expert duplication from a predicted histogram (paper, Algorithm 1, with one replica per
 * logical slot and only predicted proportions known, Section 3.2.1): every expert keeps one slot;
 * each of the S-E extra slots goes to the expert with the largest predicted load per replica
 * (exact integer comparison; equal ratios go to the fewer replicas, then the lower index) among
 * experts with fewer than c_max copies.
 * predicted_hist: int32 [E], >= 0; n_slots must equal shape.S.
 * replicas: int32 [E]; slot_off: int32 [E+1] (expert e owns slots slot_off[e]..slot_off[e+1]-1);
 * slot_expert: int32 [S] (-1 for a slot left empty by c_max); bound: int32 [1] = max_e ceil(n_e/r_e). */
MOEGPS_API int moegps_plan(moegps_ctx_t* ctx, const int32_t* predicted_hist, int32_t n_slots,
                int32_t* replicas, int32_t* slot_off, int32_t* slot_expert, int32_t* bound, void* stream);

/* pack - Algorithm 1 of the paper as printed (Section 3.1): G devices, each with room for
 * capacity[g] expert copies (all experts are the same size, so the algorithm's memory test is a
 * count of free places), several experts per device, at most c_max copies of an expert (shape.c_max;
 * 0 = no cap).  Only predicted counts are known before routing (Section 3.2.1), so the dispatch is
 * kept as counts: share[e,g] = tokens of expert e served by device g.  Start: expert e alone on
 * home[e] with all its tokens.  While max_g L_g - min_g L_g > 1: g_h / g_c = most / least loaded
 * device (ties: lowest index), Delta = ceil((L_gh - L_gc)/2), e* = the expert with the most tokens on
 * g_h (ties: lowest index) among those g_c hosts or may still receive; copy e* to g_c if needed and
 * move min(Delta, share[e*,g_h]) of its tokens.  Ends when the loads differ by at most one token or
 * g_c can serve no expert of g_h (the printed algorithm leaves that case open).
 * predicted_hist: int32 [E] >= 0; home: int32 [E] in [0,G); capacity: int32 [G] (>= the experts homed
 * there); n_devices = G in [1,64].
 * placement: int32 [E,G] of 0/1; share: int32 [E,G]; load: int32 [G] (column sums of share);
 * iterations: int32 [1] (moves made).  All device pointers, 16-byte aligned (iterations: 4).
 * A home outside [0,G), a negative count, counts that add up to more than 2^31-1 or an over-full
 * initial placement is reported as MOEGPS_ERR_BAD_INDEX and the outputs then describe the (clamped)
 * initial placement.
 * This call plans only: mapping its placement onto devices and the all-to-all between them are not
 * part of this single-device library. */
MOEGPS_API int moegps_pack(moegps_ctx_t* ctx, const int32_t* predicted_hist, const int32_t* home,
                           const int32_t* capacity, int32_t n_devices, int32_t* placement, int32_t* share,
                           int32_t* load, int32_t* iterations, void* stream);

/* pack_slots - the placement of moegps_pack as the slot tables the rest of the path works on: one
 * slot per (expert, device) copy, experts in ascending order and, within an expert, its devices in
 * ascending order; slot_share[s] = the predicted tokens Algorithm 1's dispatch gave that copy,
 * slot_device[s] = its device; slots beyond the last copy are empty (expert -1, device -1, share 0).
 * placement, share: int32 [E,G] from moegps_pack; n_devices = G.
 * replicas: int32 [E]; slot_off: int32 [E+1]; slot_expert, slot_share, slot_device: int32 [S].
 * More copies than shape.S slots are reported as MOEGPS_ERR_BAD_INDEX (the surplus is not written). */
MOEGPS_API int moegps_pack_slots(moegps_ctx_t* ctx, const int32_t* placement, const int32_t* share,
                                 int32_t n_devices, int32_t* replicas, int32_t* slot_off, int32_t* slot_expert,
                                 int32_t* slot_share, int32_t* slot_device, void* stream);

/* dispatch - the routing shuffle (paper, Section 2 all-to-all; Algorithm 1's dispatch d and its
 * "first tokens" rule): pairs of expert e, in flat pair order, are split into r_e contiguous
 * balanced ranges (replica rho takes stable ranks floor(rho*n_e/r_e) .. floor((rho+1)*n_e/r_e)-1)
 * and token rows are copied into the slot buckets in that order.  Lossless: no capacity, no drops.
 * x: bf16 [T,D]; topk_idx: int32 [T,K]; hist: int32 [E] (actual counts of topk_idx);
 * replicas, slot_off: from moegps_plan.
 * slot_row_off: int32 [S+1], slot s owns rows slot_row_off[s]..slot_row_off[s+1]-1, starts are
 *   multiples of row_align; row_pair: int32 [Rcap] (flat pair of each occupied row, -1 on padding);
 * pair_row: int32 [T,K]; xp: bf16 [Rcap,D] (padding rows are not written).
 * workspace: moegps_workspace_bytes(shape) bytes of scratch, contents irrelevant.  Its size cannot be
 *   checked here (only a pointer is passed): a buffer shorter than that is the caller's error.
 *   Calls that may overlap on the GPU need a workspace each. */
MOEGPS_API int moegps_dispatch(moegps_ctx_t* ctx, const void* x, const int32_t* topk_idx, const int32_t* hist,
                    const int32_t* replicas, const int32_t* slot_off,
                    int32_t* slot_row_off, int32_t* row_pair, int32_t* pair_row,
                    void* xp, void* workspace, void* stream);

/* dispatch_shares - moegps_dispatch for a placement made by moegps_pack / moegps_pack_slots (paper,
 * Algorithm 1: the dispatch d sends different numbers of an expert's tokens to its copies).  The
 * copies of expert e take shares of its ACTUAL pairs in proportion to slot_share (the predicted
 * tokens each copy was given): copy rho takes the stable ranks floor(n_e c_rho / c) ..
 * floor(n_e c_{rho+1} / c) - 1, c_rho = the shares of the copies before it, c their sum; an expert
 * whose shares are all zero (the prediction gave it nothing) is split evenly as in moegps_dispatch.
 * slot_share: int32 [S] >= 0, at most 2^31-1 per expert in total.  Everything else as moegps_dispatch. */
MOEGPS_API int moegps_dispatch_shares(moegps_ctx_t* ctx, const void* x, const int32_t* topk_idx,
                                      const int32_t* hist, const int32_t* replicas, const int32_t* slot_off,
                                      const int32_t* slot_share, int32_t* slot_row_off, int32_t* row_pair,
                                      int32_t* pair_row, void* xp, void* workspace, void* stream);

/* dispatch_static - moegps_dispatch without the `workspace` argument.  (The paper has no
 * counterpart: this is a deployment convenience, not a step of the method.)
 *
 * Who needs it: code that must run the shuffle but cannot obtain device memory at that point -
 * for example a plug-in called inside someone else's serving loop whose memory pool is closed to
 * it, a caller whose device memory is fully pre-partitioned at start-up, or a real-time path in
 * which an allocator call (which may block or synchronise the device) is not acceptable.  For them
 * the scratch that moegps_dispatch takes from the caller is a fixed 1 MiB device array built into
 * the library (262144 int32 counters).  Every GPU that loads the library holds that 1 MiB until the
 * process exits, used or not.
 *
 * Same inputs, outputs, ordering and error reporting as moegps_dispatch, and bit-identical results.
 * Differences:
 *  - Limit: ceil(T*K / 256) * E must not exceed 262144 (the five reference workloads need at most
 *    32768); beyond it the call returns MOEGPS_ERR_STATIC_SCRATCH_EXCEEDED and launches nothing.
 *  - The context's device must be the current device of the calling thread (else INVALID_ARG).
 *  - The first call on each device looks up the array's device address (a host-side query, no
 *    allocation); make that first call before any stream capture begins.
 *  - No allocation of any kind is made, here or in the kernels.
 *  - All calls on a device share the one array, and it keeps whatever the previous call left in
 *    it.  Nothing in it needs to start at zero (every counter is written before it is read), but
 *    two calls that may overlap on the GPU (different streams, or different contexts on the same
 *    device) race on it and corrupt each other: serialise them on one stream or with events. */
MOEGPS_API int moegps_dispatch_static(moegps_ctx_t* ctx, const void* x, const int32_t* topk_idx,
                                      const int32_t* hist, const int32_t* replicas, const int32_t* slot_off,
                                      int32_t* slot_row_off, int32_t* row_pair, int32_t* pair_row,
                                      void* xp, void* stream);

/* expert_ffn - the expert-parallel SwiGLU FFN (paper, Sections 2 and 3.4) over ragged slots:
 * for every row rho of slot s with e = slot_expert[s]:
 *   h = silu(w_gate[e] xp[rho]) * (w_up[e] xp[rho]);   yp[rho] = w_down[e] h
 * bf16 inputs, fp32 accumulation in tensor memory, h and yp rounded to bf16 (nearest even).
 * xp: bf16 [Rcap,D]; slot_row_off: int32 [S+1]; slot_expert: int32 [S];
 * w_gate, w_up: bf16 [E,F,D]; w_down: bf16 [E,D,F]; h_ws: bf16 [Rcap,F] scratch; yp: bf16 [Rcap,D].
 * All rows of a slot's extent are computed (padding rows yield unspecified values); rows outside
 * every slot and slots with slot_expert < 0 are not written.  A slot whose extent in slot_row_off
 * is not inside [0, Rcap] (negative, decreasing, or past the buffers) is skipped entirely and
 * MOEGPS_ERR_BAD_INDEX is recorded. */
MOEGPS_API int moegps_expert_ffn(moegps_ctx_t* ctx, const void* xp, const int32_t* slot_row_off,
                      const int32_t* slot_expert, const void* w_gate, const void* w_up,
                      const void* w_down, void* h_ws, void* yp, void* stream);

/* The two halves of moegps_expert_ffn as separate calls (same arguments, same kernels), for callers
 * that want to time or schedule them apart: gate_up writes h_ws = silu(xp w_gate^T) * (xp w_up^T),
 * down writes yp = h_ws w_down^T.  moegps_expert_ffn is exactly gate_up followed by down. */
MOEGPS_API int moegps_expert_ffn_gate_up(moegps_ctx_t* ctx, const void* xp, const int32_t* slot_row_off,
                              const int32_t* slot_expert, const void* w_gate, const void* w_up,
                              void* h_ws, void* stream);
MOEGPS_API int moegps_expert_ffn_down(moegps_ctx_t* ctx, const void* h_ws, const int32_t* slot_row_off,
                           const int32_t* slot_expert, const void* w_down, void* yp, void* stream);

/* combine - the post-FFN shuffle back to token order (paper, Section 2: the same amount of traffic
 * as the routing shuffle):  out[t,:] = sum_{j<K} topk_w[t,j] * yp[pair_row[t,j],:], fp32
 * accumulation in ascending j, bf16 result (nearest even).
 * yp: bf16 [Rcap,D]; pair_row: int32 [T,K]; topk_w: fp32 [T,K]; out: bf16 [T,D]. */
MOEGPS_API int moegps_combine(moegps_ctx_t* ctx, const void* yp, const int32_t* pair_row, const float* topk_w,
                   void* out, void* stream);

/* predictor_update - state of Distribution-Only Prediction across batches (paper, Section 3.2.1:
 * the maximum-likelihood estimate p_e = n_e / N of Eq. 1, averaged over the batches seen).  state[e] += hist[e]; state / sum(state) is then Eq. 1 over all tokens
 * seen.  predicted_hist = state divided by the smallest power of two that makes its largest entry fit
 * an int32 (the planner only uses proportions) - ready to be passed to moegps_plan for the next
 * batch.  hist: int32 [E] >= 0; state: int64 [E], zeroed by the caller to start or restart;
 * predicted_hist: int32 [E].  All device pointers, 16-byte aligned. */
MOEGPS_API int moegps_predictor_update(moegps_ctx_t* ctx, const int32_t* hist, int64_t* state,
                                       int32_t* predicted_hist, void* stream);

/* predictor_update_ema - the same estimate with geometric forgetting (Section 3.2.1 leaves the
 * weights of its average over batches open; Section 3.1 discusses how often to predict and re-place):
 * state holds per-expert counts in units of 2^-16 tokens and moves towards the new batch by
 * floor((hist*2^16 - state) / 2^shift), i.e. a weight of 2^-shift for the newest batch (shift = 0: the
 * last batch alone).  Integer arithmetic: exact and deterministic.  predicted_hist as above (state
 * scaled down by a power of two to fit int32).  shift in [0,16]; state: int64 [E], zeroed to start. */
MOEGPS_API int moegps_predictor_update_ema(moegps_ctx_t* ctx, const int32_t* hist, int64_t* state, int32_t shift,
                                           int32_t* predicted_hist, void* stream);

/* error_rate - the paper's quality metric of a predicted distribution (Section 3.2.1, with the
 * averaging of Section 3.3): mean over the experts of |p_est_e - p_e| / (1/E), where p_est and p are
 * predicted_hist and hist normalised to sum 1.  fp64, deterministic summation order.
 * error_rate: double [1] on the device (8-byte aligned); 0 if either histogram is empty. */
MOEGPS_API int moegps_error_rate(moegps_ctx_t* ctx, const int32_t* predicted_hist, const int32_t* hist,
                                 double* error_rate, void* stream);

/* Self-test of the library's failure detection (no counterpart in the paper).  Every wait inside the
 * pipelined kernels (route, expert_ffn) is bounded: when it runs out the kernel records
 * MOEGPS_ERR_TIMEOUT in the status word, drains and returns instead of hanging.  This call launches
 * a one-warp kernel that waits on a barrier nobody signals and gives up after `limit_cycles` SM
 * cycles (1e3 .. 4e9); afterwards moegps_status reports MOEGPS_ERR_TIMEOUT and the context and the
 * device are as usable as before. */
MOEGPS_API int moegps_selftest_bounded_wait(moegps_ctx_t* ctx, int64_t limit_cycles, void* stream);

/* Synchronises `stream`, copies the device status word to *host_status (0 = no device-side error,
 * else the first moegps_error recorded) and clears it.  Returns MOEGPS_OK or MOEGPS_ERR_CUDA. */
MOEGPS_API int moegps_status(moegps_ctx_t* ctx, void* stream, int32_t* host_status);

/* Number of kernels this context has launched so far (host-side counter). */
MOEGPS_API int64_t moegps_launch_count(const moegps_ctx_t* ctx);

/* The cudaError_t (as int) of the last failing CUDA call seen by this context, 0 if none. */
MOEGPS_API int moegps_last_cuda_error(const moegps_ctx_t* ctx);

MOEGPS_API const char* moegps_error_string(int code);

#ifdef __cplusplus
}
#endif
#endif  /* MOEGPS_H_ */
