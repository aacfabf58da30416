/*
 * cosmoe.h -- C boundary of the sparse Mixture-of-Experts feed-forward layer
 * (CoSMoEs, arXiv 2503.00245) for NVIDIA B200 (sm_100a).
 *
 * The layer (Section 2.1): a router scores E experts per token, the routing
 * weights are W = softmax(R) (Eq. 2, tau = 1 at inference), each token keeps the
 * top-k experts S = top_k(W, K) (Eq. 3), the selected experts' gated FFNs run on
 * the token (Section 3.1: Llama-style experts, here SwiGLU without biases), and
 * the outputs are summed with the gate's weights (Section 1).  Experts are dense
 * matrices or weight-decomposed M = L x R (Eq. 1).  Experts may live in host
 * memory and be brought to the device on routing (Eq. 8, Section 3.4.2).
 *
 * General rules
 *  - Every call returns a moe_status (int).  Nothing throws, exits or traps.
 *  - "dev" pointers are device memory owned by the caller, 16-byte aligned;
 *    "host" pointers are host memory.  The library allocates device memory only in
 *    moe_create / moe_offload_create (a few KB of state) and never in a hot call.
 *  - `stream` is a cudaStream_t passed as void*.  Hot calls only enqueue work on it;
 *    they return before the work has run.  Faults a kernel detects (an expired
 *    bounded wait, an index out of range) set a device status word that
 *    moe_check() reads; the output of that call is then undefined.
 *  - One moe_ctx serves one stream at a time: calls on the same ctx from two
 *    streams that overlap on the device race on the ctx's barrier state.
 *  - Weights are read-only for the library and may be shared between ctxs.
 *  - Shapes: d_model, d_ff and wd_rank multiples of 8; 1 <= top_k <= n_experts <= 64;
 *    top_k <= 8.  Anything else: MOE_ERR_UNSUPPORTED, nothing is read or written.
 *    The streaming path of dense experts also needs d_model <= 2048.
 *  - The streaming path sums the CTAs' partial outputs with 64-bit fixed-point atomics
 *    (2^-36 resolution, |partial sums| < 2^27; a one-token call of a whole layer keeps the
 *    number of arrivals in the low bits of the same words: 2^-32 resolution, |sums| < 2^23):
 *    integer addition is associative, so results do not depend on the order of arrival and
 *    repeated calls are bit-identical.  Outputs beyond those magnitudes are not supported.
 *
 * Weight layouts.  The mathematical layouts (row-vector convention y = x W) are
 *    w_gate, w_up [E][d][f],  w_down [E][f][d]                       (dense)
 *    gL,uL [E][d][r]  gR,uR [E][r][f]  dL [E][f][r]  dR [E][r][d]    (Eq. 1 factors)
 * The kernels read a packed form.  Dense experts: everything hidden unit c of an
 * expert touches is one contiguous run of 3*d values, so any range of hidden units is
 * one contiguous run of bytes for the copy engines (and for a host->device fetch):
 *    gud [S][f][3][d] : row c = ( w_gate[:, c] , w_up[:, c] , w_down[c, :] )
 * Eq. 1 factors: one output neuron's weights contiguous in every matrix:
 *    wd_a [S][r][2][d] = (gL[:,j], uL[:,j]);  wd_b [S][f][2][r] = (gR[:,c], uR[:,c]);
 *    wd_c [S][r][f] = dL[:,j];                wd_d [S][d][r] = dR[:,n]
 * S = number of expert slots (= E unless an offload cache is used).
 * moe_pack_dense / moe_pack_wd produce the packed form once; packing is not part
 * of the layer and is excluded from timings.
 */
#ifndef COSMOE_H_
#define COSMOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum moe_status {
  MOE_OK = 0,
  MOE_ERR_INVALID_ARG = 1, /* null pointer, negative size, misaligned pointer          */
  MOE_ERR_UNSUPPORTED = 2, /* shape / dtype / path combination no kernel handles        */
  MOE_ERR_WORKSPACE = 3,   /* workspace smaller than moe_workspace_bytes() asked for    */
  MOE_ERR_CUDA = 4,        /* a CUDA runtime call failed (moe_last_cuda_error())        */
  MOE_ERR_TIMEOUT = 5,     /* a bounded device- or host-side wait expired               */
  MOE_ERR_STATE = 6,       /* call order violated, or a kernel flagged an internal fault */
  MOE_ERR_NO_DEVICE = 7    /* no usable CUDA device: there is no CPU fallback           */
} moe_status;

enum { MOE_F32 = 0, MOE_BF16 = 1 };
/* Which kernels run the expert FFN.  AUTO: STREAM for T <= MOE_STREAM_MAX_TOKENS, else TENSOR. */
enum { MOE_PATH_AUTO = 0, MOE_PATH_STREAM = 1, MOE_PATH_TENSOR = 2 };
#define MOE_STREAM_MAX_TOKENS 16
#define MOE_MAX_EXPERTS 64
#define MOE_MAX_TOPK 8

typedef struct moe_config {
  int32_t d_model;   /* d                                                              */
  int32_t d_ff;      /* f, hidden width of one expert                                  */
  int32_t n_experts; /* E                                                              */
  int32_t top_k;     /* k                                                              */
  int32_t wd_rank;   /* r of Eq. 1; 0 = dense experts                                  */
  int32_t x_dtype;   /* MOE_F32 or MOE_BF16: type of x and of y                        */
  int32_t renorm;    /* 1: a token's k gate weights are rescaled to sum to one         */
  int32_t path;      /* MOE_PATH_*                                                     */
} moe_config;

typedef struct moe_weights {
  const void* w_router;       /* dev [d][E] bf16                                       */
  const float* b_router;      /* dev [E] fp32 added to the logits, or NULL             */
  const void* gud;            /* dev packed dense, see above (NULL when wd_rank > 0)   */
  const void* wd_a;           /* dev packed Eq. 1 factors (NULL when wd_rank == 0)     */
  const void* wd_b;
  const void* wd_c;
  const void* wd_d;
  const int32_t* expert_slot; /* dev [E]: slot of the packed arrays that holds expert e
                                 (-1 = not resident), or NULL for slot == expert       */
} moe_weights;

typedef struct moe_ctx moe_ctx;
typedef struct moe_offload moe_offload;

/* ---- library ------------------------------------------------------------------ */
const char* moe_status_string(int status);
/* cudaError_t of the most recent failing CUDA call in this thread (0 if none). */
int moe_last_cuda_error(void);
/* Number of SMs of the current device, or a negative moe_status. */
int moe_device_sm_count(void);

/* ---- context -------------------------------------------------------------------
 * moe_create validates cfg, allocates the ctx's device state (status word, grid
 * barrier) on the current device and returns it.  moe_check copies the status word
 * back on `stream` and waits for that copy only, so call it after the work of
 * interest; it returns MOE_OK, MOE_ERR_TIMEOUT or MOE_ERR_STATE and clears the word
 * (and re-arms the barrier) so the ctx stays usable.                              */
int moe_create(const moe_config* cfg, moe_ctx** out);
int moe_destroy(moe_ctx* ctx);
int moe_check(moe_ctx* ctx, void* stream);
/* Scratch the hot calls need for T tokens (upper bound over all calls and paths). */
int moe_workspace_bytes(const moe_config* cfg, int32_t T, size_t* bytes);
/* Diagnostics, for testing the time-out path without hanging or faulting anything.  Not for production use.
 * moe_set_finaliser_wait: how many SM clock cycles the finalising CTAs of the dense streaming kernel wait for
 * the other CTAs' partial sums before they give up and flag MOE_ERR_TIMEOUT (0 = the default, about two seconds).
 * moe_seed_arrival_counter: overwrites the ctx's arrival counter (which normally runs over launches and is a
 * multiple of the grid size between calls) and waits for `stream`.  Seeded with grid size - 1, the next launch's
 * arrivals straddle a multiple of the grid size, so most of its finalisers wait for a count that launch never
 * reaches: with a short budget they give up, every CTA having streamed its share and exited normally.  (A
 * one-token launch counts arrivals in its accumulator words instead; a value that is not a multiple of the grid
 * size makes those words wait for one arrival more than the launch has, to the same effect.)  The output of
 * such a call is undefined; moe_check reports MOE_ERR_TIMEOUT and re-arms the state.                          */
int moe_set_finaliser_wait(moe_ctx* ctx, long long cycles);
int moe_seed_arrival_counter(moe_ctx* ctx, unsigned long long value, void* stream);
/* Kernels launched by hot calls on this ctx since creation (for accounting). */
int moe_launch_count(moe_ctx* ctx, uint64_t* launches);

/* ---- weight packing (once, outside the layer) ----------------------------------
 * Inputs in the mathematical layouts, outputs in the packed layouts, all dev bf16.
 * n_experts experts are packed into consecutive slots of the outputs.             */
int moe_pack_dense(int32_t d_model, int32_t d_ff, int32_t n_experts, const void* w_gate, const void* w_up,
                   const void* w_down, void* gud_out, void* stream);
int moe_pack_wd(int32_t d_model, int32_t d_ff, int32_t rank, int32_t n_experts, const void* gL, const void* gR,
                const void* uL, const void* uR, const void* dL, const void* dR, void* wd_a_out, void* wd_b_out,
                void* wd_c_out, void* wd_d_out, void* stream);

/* ---- 8-bit storage of packed rows (for the host link) -----------------------------
 * rows x n bf16 values (dev, n a multiple of 8) -> FP8 E4M3 codes (dev [rows][n] bytes) and one fp32 scale per
 * row: scale = max|w| / 448 (1 for an all-zero row), code = e4m3(w / scale) with round-to-nearest-even and
 * saturation, all in fp32.  moe_fp8_dequantize_rows: w' = bf16(value(code) * scale).                      */
int moe_fp8_quantize_rows(const void* w, int64_t rows, int32_t n, void* codes, float* scales, void* stream);
int moe_fp8_dequantize_rows(const void* codes, const float* scales, int64_t rows, int32_t n, void* w, void* stream);

/* ---- the layer, step by step ---------------------------------------------------- */

/* Router logits, softmax over experts (Eq. 2), top-k (Eq. 3), gate weights.
 * x dev [T][d] (cfg.x_dtype).  topk_idx dev [T][k] int32: descending weight, equal
 * weights to the lower expert index.  topk_w dev [T][k] fp32.  probs dev [T][E] fp32
 * or NULL.  fp32 arithmetic.  T >= 0 (T == 0 is a no-op).                          */
int moe_route(moe_ctx* ctx, const void* x, int32_t T, const moe_weights* w, int32_t* topk_idx, float* topk_w,
              float* probs, void* stream);

/* Group the T*k (token, choice) pairs p = t*k + j by expert, stably (token-choice
 * routing gives every expert a discrete set of tokens, Section 2.1).
 * expert_offsets dev [E+1] int32 (exclusive scan of per-expert counts),
 * perm dev [T*k]: perm[slot] = p;  inv dev [T*k]: inv[p] = slot.  Integer-exact.   */
int moe_permute(moe_ctx* ctx, const int32_t* topk_idx, int32_t T, int32_t* expert_offsets, int32_t* perm,
                int32_t* inv, void* stream);

/* Selected experts' FFN per slot (Section 3.1; Eq. 1 for decomposed experts):
 * out_slots[s] = (silu(x_t W_g[e]) * (x_t W_u[e])) W_d[e], t = perm[s] / k, e the
 * expert whose [expert_offsets[e], expert_offsets[e+1]) contains s.  out_slots dev
 * [T*k][d] fp32, unweighted.  ws: dev scratch of moe_workspace_bytes().            */
int moe_expert_ffn(moe_ctx* ctx, const void* x, int32_t T, const moe_weights* w, const int32_t* expert_offsets,
                   const int32_t* perm, float* out_slots, void* ws, size_t ws_bytes, void* stream);

/* Gate-weighted sum (Section 1): y[t] = sum_j topk_w[t][j] * out_slots[inv[t*k+j]],
 * j ascending, fp32, rounded once to cfg.x_dtype.  y dev [T][d].                   */
int moe_combine(moe_ctx* ctx, const float* out_slots, const float* topk_w, const int32_t* inv, int32_t T, void* y,
                void* stream);

/* The whole layer: equals moe_route -> moe_permute -> moe_expert_ffn -> moe_combine
 * but is free to fuse.  topk_idx / topk_w (dev, may be NULL) receive the routing.
 * On the streaming path (T <= MOE_STREAM_MAX_TOKENS) y may also be MAPPED PINNED HOST memory (a device-accessible
 * address): the finalising CTAs store y with ordinary stores, so a decode step then needs no device->host copy,
 * only a wait for `stream` before the host reads y.                                  */
int moe_layer_forward(moe_ctx* ctx, const void* x, int32_t T, const moe_weights* w, void* y, int32_t* topk_idx,
                      float* topk_w, void* ws, size_t ws_bytes, void* stream);

/* The whole layer again, for callers that must not allocate device memory: code that runs where
 * cudaMalloc is off limits -- a plug-in inside a host application that has handed out all of the GPU's
 * memory up front, or a real-time loop in which an allocation (a device-wide synchronising call) is not
 * allowed.  The paper has no counterpart of this call; it is a convenience of this library.
 * No ctx, no workspace: the scratch moe_create would allocate (fixed-point accumulators, status and
 * arrival-counter words) is a 257 KiB __device__ array inside the library, which every GPU that loads the
 * library holds until the process exits.  Limits: dense experts only (wd_rank == 0), d_model <= 2048,
 * T <= 16, streaming path; beyond them the call returns MOE_ERR_UNSUPPORTED and touches nothing.
 * T >= 2 also needs topk_idx and topk_w (dev, [T][k]) for the routing; at T == 1 they may be NULL.
 * The first call on a GPU looks up the array's address (cudaGetSymbolAddress, with that GPU current):
 * make that first call outside any stream capture.  The call itself uses no cudaMalloc / cudaFree and no
 * allocating library routine; it enqueues two small memsets and the kernels on `stream`.
 * All calls on one GPU share the array: it keeps the last call's contents, the call clears what it needs
 * before launching, and two calls that overlap on the GPU (different streams, or different threads)
 * race on it -- issue them in one stream or serialise them yourself.
 * T == 0 does no work: it waits for `stream` and returns what the kernels of earlier calls on this GPU
 * reported (MOE_OK, MOE_ERR_TIMEOUT or MOE_ERR_STATE), clearing the report.  Until it is cleared, a
 * report stays: the kernels of later calls see it and leave their output unwritten, although those
 * calls return MOE_OK (they only enqueue) -- so poll with T == 0 wherever moe_check would be called.
 * The one-off set-up is thread-safe; a device that is not sm_100 gets MOE_ERR_NO_DEVICE.              */
int moe_layer_forward_static(const moe_config* cfg, const void* x, int32_t T, const moe_weights* w, void* y,
                             int32_t* topk_idx, float* topk_w, void* stream);

/* ---- host-resident experts (Eq. 8, Section 3.4.2) --------------------------------
 * All experts of n_layers layers live in pinned host memory in packed form
 * (host_experts[layer*E + e] -> one expert in the gud layout, slot_bytes in total).  The device holds slots_per_layer slots per layer
 * (device_slots: dev, n_layers*slots_per_layer*slot_bytes, caller-owned; on creation
 * slot i of every layer is filled with expert i).  With slots_per_layer == top_k the
 * bookkeeping is exactly Eq. 8; with more slots the least recently used expert that
 * is not selected in the current step is replaced.  Evicted experts are dropped (the
 * host copy is the master), so only host->device bytes move.
 *
 * moe_offload_ensure: host call.  topk_idx_host [n] = the experts layer `layer`
 * selected for this step.  Misses are copied on the offload's copy stream in chunks;
 * compute_stream is made to wait for them (event), the layer's expert_slot table
 * (dev [E] int32, owned by the offload object, moe_offload_slot_table()) is updated
 * in stream order, and the call returns without waiting for the copies.           */
int moe_offload_create(const moe_config* cfg, int32_t n_layers, int32_t slots_per_layer,
                       const void* const* host_experts, void* device_slots, size_t slot_bytes, moe_offload** out);
/* The same with the host copies in 8-bit form (bit-width reduction for the host link; the paper names it only as
 * related work, Section 2.3 / Section 5): host_blobs[layer*E + e] -> pinned memory holding the expert's packed
 * rows as FP8 E4M3 codes, [f][3][d] bytes, followed by one fp32 scale per row, [f][3] (moe_fp8_quantize_rows makes
 * both from the packed bf16 rows).  A fetch moves d_ff * (3 d + 12) bytes instead of 6 d d_ff, lands in a staging
 * area the object owns and is widened into the bf16 slot by a kernel ordered behind the copy (on the compute stream
 * in the stacked steps, so that the copy stream only ever copies); the layer kernels read
 * bf16 slots as before, so the layer computes with w' = bf16(value(code) * scale) in place of w.
 * slot_bytes stays the bf16 size of a slot (6 d d_ff).                                                       */
int moe_offload_create_fp8(const moe_config* cfg, int32_t n_layers, int32_t slots_per_layer,
                           const void* const* host_blobs, void* device_slots, size_t slot_bytes, moe_offload** out);
int moe_offload_destroy(moe_offload* off);
int moe_offload_ensure(moe_offload* off, int32_t layer, const int32_t* topk_idx_host, int32_t n,
                       void* compute_stream);
int moe_offload_slot_table(moe_offload* off, int32_t layer, const int32_t** expert_slot_dev);
/* Host copy of the current slot contents of a layer: slots_host[slots_per_layer]. */
int moe_offload_resident(moe_offload* off, int32_t layer, int32_t* slots_host);
int moe_offload_stats(moe_offload* off, uint64_t* fetches, uint64_t* bytes, uint64_t* hits);

/* One decode step (T = 1) through n_layers stacked MoE layers with offloaded experts.  Per layer:
 * u = h / rms(h) (no learned scale) rounded to cfg.x_dtype, the router on u, y = experts(u) with the gate
 * weights, h += y (fp32, y not rounded in between).  h dev [d] fp32, updated in place.  routers: host array of
 * n_layers moe_weights whose w_router / b_router are set (expert pointers are taken from the offload object).
 * topk_trace_host [n_layers][k] receives each layer's selection.
 * The host must see a layer's selection before it can copy: a small kernel (norm + router) writes it to mapped
 * pinned memory and the host polls for it (bounded: MOE_ERR_TIMEOUT after 10 s) -- no stream synchronisation.
 * Overlap: the resident selected experts of the layer run at once; a missing expert is copied in chunks of about
 * 8 MB on the offload's copy stream, and the launch that computes a chunk's hidden units waits only for that
 * chunk, so compute trails the copy by one chunk and the link goes idle only between the last chunk of a layer
 * and the routing of the next.  All launches of a layer add into the ctx's fixed-point accumulators; the last
 * converts them.  Returns with the work queued; wait for `stream` (or call moe_check) before reading h.     */
int moe_stack_decode_step(moe_offload* off, moe_ctx* ctx, const moe_weights* routers, float* h,
                          int32_t* topk_trace_host, void* ws, size_t ws_bytes, void* stream);

/* The same step with the expert set of every layer prescribed by the caller
 * (sel_host [n_layers][k], distinct experts per layer): the layer's gate weights are
 * the router's probabilities (Eq. 2) of those experts, renormalised over the set.  For
 * replaying routing traces, e.g. traces with a given expert replacement ratio (Eq. 4-5)
 * under the rule of Eq. 8.  Because the host knows the sets, it does not wait for the
 * device at all: a layer's misses are copied on the offload's copy stream while earlier layers
 * compute, and a layer is ONE launch (norm, router, experts, residual add).  Returns with the work queued. */
int moe_stack_decode_step_trace(moe_offload* off, moe_ctx* ctx, const moe_weights* routers, float* h,
                                const int32_t* sel_host, void* ws, size_t ws_bytes, void* stream);

/* Host wall time moe_stack_decode_step has spent so far waiting for routing words (poll_s, over `polls`
 * waits) and queueing copies and launches (issue_s): where a token's time goes besides the link.        */
int moe_offload_host_times(moe_offload* off, double* poll_s, double* issue_s, uint64_t* polls);

/* ---- routing-trace metrics (Eq. 4-5, Section 2.3 / 3.3) ---------------------------
 * topk_trace dev [B][T][k] int32.  Writes H (Eq. 4, summed over experts) to
 * h_total_out dev [1] uint64; replacements = H / 2 and H_norm = (H/2) / (B k (T-1)).
 * A row is read as a set: a repeated id counts once, an id outside [0, n_experts) not at all. */
int moe_expert_replacements(const int32_t* topk_trace, int32_t B, int32_t T, int32_t k, int32_t n_experts,
                            unsigned long long* h_total_out, void* stream);

/* Expert balance of a routing trace (Section 3.3, "delta between the uniform distribution and the realised
 * expert balance"; Table 3 and Fig. 6 report it per layer).  topk_trace dev [B][T][k] int32, one row b per
 * layer.  counts_out dev [B][E] uint64: selections of expert e in row b (integer-exact).  delta_out dev [B+1]
 * fp64: delta_out[b] = 100 * mean_e |counts[b][e] / sum_e counts[b][e] - 1/E|, delta_out[B] = their mean.
 * bad_out dev [1] uint64: ids outside [0, E) met (they are not counted).  The paper prints no formula for
 * this metric: the mean absolute deviation is this library's reading, and no value of the paper pins it.  */
int moe_delta_uniform(const int32_t* topk_trace, int32_t B, int32_t T, int32_t k, int32_t n_experts,
                      unsigned long long* counts_out, double* delta_out, unsigned long long* bad_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* COSMOE_H_ */
