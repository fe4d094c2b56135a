/*
 * remoe.h -- C ABI of the bounded-cache MoE decode step for one NVIDIA B200 (sm_100a).
 *
 * The library runs, per decoded token and per MoE layer, the inference path that the
 * ReMoE paper's router fine-tuning targets: router GEMV, softmax and top-K gating,
 * resolution of the selected experts against a per-layer cache of C fixed HBM slots with
 * LRU replacement, fetch of missing experts from pinned host memory, the SwiGLU expert
 * GEMVs over the resident weights plus always-resident shared experts, the gate-weighted
 * combine, and the step-to-step reuse statistic.
 *
 * Conventions
 *   - Every function returns 0 (REMOE_OK) or a negative REMOE_E_* code; nothing aborts,
 *     throws or traps across this boundary.  remoe_strerror() names a code.
 *   - "dev" pointers are CUDA device pointers owned by the caller; "host" pointers are host
 *     memory owned by the caller.  The handle is owned by the library.
 *   - All tensors are dense, row-major, layer-major: [L, B, ...].
 *   - Device-side errors.  Kernels never trap: a bounded wait that runs out or an index out of range
 *     sets an error word and the kernel returns.  The routing kernel's errors are seen by the decode
 *     call itself; an expert or combine kernel runs after the call has returned, so its error is
 *     reported as REMOE_E_DEVICE_FLAG by the NEXT call on the stack that synchronises: a decode call,
 *     remoe_decode_step_host (which reports its own step), remoe_last_step_trace or one of the
 *     statistics calls.  The outputs of that step are then finite but incomplete.
 *   - After REMOE_E_DEVICE_FLAG or REMOE_E_CUDA from a decode call the cache directory may already hold
 *     the step's admissions while their slots were never filled: call remoe_cache_reset() before the
 *     next step (it also clears the error word).  Nothing else needs to be rebuilt.
 *   - One stack belongs to one device (the one current at creation) and one stream.  A call
 *     may be made with any device current: the library switches to the stack's device for
 *     the call and restores the caller's.  Calls on one stack must not overlap in time.
 *
 * Data layouts
 *   router weights   [N, H]   one row per routed expert, element type = weight_dtype
 *   shared-gate      [H]      element type = weight_dtype
 *   expert block     [I, 3, H] for intermediate channel i three consecutive rows:
 *                    W_gate[i, :], W_up[i, :], W_down[:, i]; 3*I*H elements, contiguous.
 *                    An expert computes y = W_down (silu(W_gate x) * (W_up x)).
 *   hidden states    [L, B, H] float32; layer l reads its own stream: out[l] = MoE_l(in[l]).
 */
#ifndef REMOE_H_
#define REMOE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  REMOE_OK = 0,
  REMOE_E_ARG = -1,          /* null pointer, index out of range, misaligned pointer      */
  REMOE_E_CAPACITY = -2,     /* cache_slots_per_layer < top_k at batch 1 (App. A.2, Assumption 1) */
  REMOE_E_NOT_LOADED = -3,   /* a router, shared expert or requested routed expert is missing */
  REMOE_E_NOT_PINNED = -4,   /* an expert pointer is not page-locked host memory          */
  REMOE_E_CUDA = -5,         /* a CUDA runtime call failed; see remoe_last_cuda_error()   */
  REMOE_E_DEVICE_FLAG = -6,  /* a kernel recorded an internal error (bounded wait ran out, bad index) */
  REMOE_E_UNSUPPORTED = -7,  /* shape outside what the kernels are built for              */
  REMOE_E_NOMEM = -8,        /* host or device allocation failed                          */
  REMOE_E_ORDER = -9         /* REMOE_CHECK_ORDER=1 only: the call enqueued a slot access whose order
                                the streams and events do not guarantee; see remoe_last_cuda_error() */
};

enum { REMOE_F32 = 0, REMOE_BF16 = 1, REMOE_FP8_E4M3 = 2, REMOE_INT4_G32 = 3 };
enum { REMOE_POLICY_LRU = 0, REMOE_POLICY_FIFO = 1, REMOE_POLICY_LFU = 2 };

/* Shape of the stack.  Sec. 3.1: N_r routed experts, Top-K; shared experts always active. */
typedef struct {
  int32_t n_layers;      /* L                                                              */
  int32_t hidden;        /* H; float32: multiple of 128, bf16: multiple of 256; <= 2048    */
  int32_t n_routed;      /* N_r <= 256                                                     */
  int32_t top_k;         /* K <= min(N_r, 32)                                              */
  int32_t inter_routed;  /* I of a routed expert                                           */
  int32_t n_shared;      /* number of shared experts (0 if none)                           */
  int32_t inter_shared;  /* I of each shared expert                                        */
  int32_t shared_gate;   /* 1: shared output is scaled by sigmoid(w_sg . h)                */
  int32_t renorm_topk;   /* 1: top-K gate weights are renormalised to sum to 1             */
  int32_t weight_dtype;  /* REMOE_F32, REMOE_BF16 (router, shared gate, all experts) or    */
                         /* REMOE_FP8_E4M3: expert blocks are OCP FP8 E4M3 bytes, value =  */
                         /* byte * 2^-8; router and shared gate bf16; H multiple of 512.   */
                         /* Halves the bytes a miss moves over the host link.  At batch 1  */
                         /* the slots hold the FP8 bytes; at batch > 1 (I, I_shared        */
                         /* multiples of 64) a fetched block is widened, exactly, to bf16  */
                         /* operand tiles on arrival and the grouped GEMM is the bf16 one. */
                         /* REMOE_INT4_G32 (H 1024 or 2048): 4-bit codes in groups         */
                         /* of 32 consecutive elements of a row, value = (code - 8) * the  */
                         /* group's bf16 scale; a stored row is H/2 bytes of codes (element*/
                         /* 2i in the low half of byte i) then H/32 scales, so a row takes */
                         /* 0.5625 H bytes: 3.6x fewer bytes per miss than bf16.  Router   */
                         /* and shared gate bf16.  At batch > 1 as for FP8: widened to     */
                         /* bf16 operand tiles on arrival (one rounding to bf16 per weight)*/
  int32_t batch;         /* B sequences per step; B > 1 needs bf16, FP8 or 4-bit weights and I, I_shared */
                         /* multiples of 8, B * K <= 1024                                   */
} remoe_shape;

/* Counters of App. E.2.3-E.2.4, summed over steps since creation or the last reset. */
typedef struct {
  uint64_t tok_hits, tok_misses;     /* per routed slot (B*K events per layer-step)        */
  uint64_t uniq_hits, uniq_misses;   /* per distinct requested expert; uniq_misses = #uMiss */
  uint64_t h2d_bytes;                /* bytes fetched from host memory for misses          */
  uint64_t steps;                    /* decode steps taken                                 */
} remoe_cache_counters;

typedef struct remoe_stack remoe_stack;

/*
 * Create a stack with an empty cache of `cache_slots_per_layer` expert slots per layer
 * (Sec. 3.1: per-layer expert cache of capacity C; Sec. 3: request-isolated cold start).
 * `cuda_stream` is the cudaStream_t all kernels are ordered on (NULL = default stream); the
 * library also owns one copy stream.  Allocates the slot pools, directory and scratch on
 * the current device.  Errors: ARG, CAPACITY (B == 1 and C < K), UNSUPPORTED, NOMEM, CUDA.
 * Environment read here: REMOE_BATCHED_KERNEL=mma keeps a batched stack on the mma.sync expert kernel;
 * REMOE_CHECK_ORDER=1 makes every decode call also replay what it enqueues on its streams (launches, copies,
 * event records and waits, host waits) into a host-side ledger that checks, per cache slot, that each write
 * is ordered behind the readers of the previous contents and each read behind the write that filled it; a
 * call that fails the check returns REMOE_E_ORDER (a debugging aid: host work only, no effect on the GPU);
 * REMOE_FAULT_INJECT=lost_copy (failure-detection tests, batch 1) makes the first step's resident-phase
 * expert launch run with a short wait limit and never issue the copy of its first weight row: the
 * consumer's bounded wait runs out, the kernel sets the error word and returns, and the error surfaces as
 * described under "Device-side errors" above.  Later launches of the stack are normal.
 */
int remoe_stack_create(const remoe_shape* shape, int32_t cache_slots_per_layer,
                       void* cuda_stream, remoe_stack** out);

/* Copy layer `layer`'s router weights [N, H] (and, when shape.shared_gate, the gate vector
 * [H]; else pass NULL) from host memory to the device.  Synchronous.  (Sec. 3.1: theta_gate.) */
int remoe_load_router(remoe_stack*, int32_t layer, const void* w_router_host,
                      const void* w_shared_gate_host);

/* Copy shared expert `idx` of `layer` (one expert block, I = inter_shared) to the device,
 * where it stays resident and never enters the cache (Sec. 3.1; App. A.1).  Synchronous. */
int remoe_load_shared(remoe_stack*, int32_t layer, int32_t idx, const void* block_host);

/* Register the host copies of routed experts first_expert .. first_expert+count-1 of
 * `layer`: `pinned_ptrs[i]` points at one expert block in page-locked host memory, 16-byte
 * aligned.  BORROWED: the caller keeps the memory pinned, alive and unchanged until the
 * stack is destroyed; misses are fetched from it (the cache model of Sec. 3.1).
 * Several experts may share one pointer.  Errors: ARG, NOT_PINNED. */
int remoe_load_experts_host(remoe_stack*, int32_t layer, int32_t first_expert, int32_t count,
                            const void* const* pinned_ptrs);

/*
 * One decode step for all L layers and B sequences (Sec. 3.1 routing; App. A.1-A.2 cache
 * model; Eq. 1 reuse).  Inputs/outputs are device pointers:
 *   hidden_in    [L, B, H] float32
 *   hidden_out   [L, B, H] float32   sum_e g_e y_e + shared terms
 *   selected_ids [L, B, K] int32     by descending logit, equal logits by ascending id
 *   gate_weights [L, B, K] float32   softmax probability (renormalised if renorm_topk)
 * Hits and misses are judged against the cache state held before the step; misses are
 * fetched from the registered host blocks into the victim slots (empty slot first, else
 * least recently used) on the copy stream while resident experts are already computed.
 * The call blocks only until the step's miss list is known; on return the remaining work
 * is enqueued and the outputs are complete once the stack's stream has drained.
 * With B > 1 the cache is shared by the batch: the step's distinct requests U = Unique(R)
 * (App. E.2.3) are resolved together, tokens are grouped per expert and the experts run as a
 * tensor-core grouped GEMM (activations rounded to bf16, fp32 accumulation); if U has more
 * experts than there are slots, slots are handed on within the step in request order.
 * Errors: ARG, NOT_LOADED, CUDA, DEVICE_FLAG.
 */
int remoe_decode_step(remoe_stack*, const float* hidden_in_dev, float* hidden_out_dev,
                      int32_t* selected_ids_dev, float* gate_weights_dev);

/*
 * n_steps consecutive decode steps of a batch-1 stack whose inputs are all known up front (replaying a
 * recorded trace of hidden states, teacher-forced evaluation as in Sec. 5.2, benchmarking):
 *   hidden_in [n_steps, L, 1, H], hidden_out [n_steps, L, 1, H], selected_ids / gate_weights
 *   [n_steps, L, 1, K], device pointers; step t reads and writes slice t.
 * Results, cache behaviour, counters and statistics are exactly those of n_steps calls of
 * remoe_decode_step, bit for bit.  The difference is scheduling: a step's routing needs nothing from the
 * previous step's fetches or expert compute (each layer reads its own input stream), so step t+1 is routed
 * on an internal stream while step t is still fetching, and its miss list reaches the host before the copy
 * engine runs out of work.  The host link, which bounds the step at realistic cache sizes, then stays
 * busy across step boundaries (a single call per step leaves it idle for the time of the last expert
 * launch, the combine, the next routing and the host hand-off: about 1 % of a step for a 26-layer stack
 * of 17 MB experts at 28 misses per step).
 * Inputs must be complete when the stack's stream reaches the call; outputs are complete when that
 * stream has drained.  The host blocks until the last step's miss list is known.  The first call
 * allocates a second set of small per-step buffers.  Errors: ARG, NOT_LOADED, UNSUPPORTED (batch > 1),
 * NOMEM, CUDA, DEVICE_FLAG.
 */
int remoe_decode_steps(remoe_stack*, int32_t n_steps, const float* hidden_in_dev, float* hidden_out_dev,
                       int32_t* selected_ids_dev, float* gate_weights_dev);

/*
 * Chained variant of the step: the layers feed each other through a pre-norm residual connection as
 * in a decoder stack, x_l = h_l / sqrt(mean(h_l^2) + 1e-6), h_{l+1} = h_l + MoE_l(x_l), instead of
 * each reading its own stream (the paper treats layers independently, App. A.5; chaining is how they
 * sit in a model; without the norm a randomly initialised stack diverges).
 *   hidden_in    dev [B, H]        h_0
 *   hidden_out   dev [B, H]        h_L
 *   layer_inputs dev [L, B, H]     residual stream h_0 .. h_{L-1} (may be NULL)
 *   selected_ids dev [L, B, K], gate_weights dev [L, B, K]
 * Routing of layer l+1 depends on layer l's output, so the host waits for one small trace per
 * layer instead of one per step, and a layer's fetches cannot start before the layer above it
 * has finished.  With B > 1 the sequences move through the layers together and share each layer's
 * cache as in remoe_decode_step.  Cache, counters and reuse statistics behave exactly as in
 * remoe_decode_step.  Errors: ARG, NOT_LOADED, CUDA, DEVICE_FLAG.
 */
int remoe_decode_step_chained(remoe_stack*, const float* hidden_in_dev, float* hidden_out_dev,
                              float* layer_inputs_dev, int32_t* selected_ids_dev, float* gate_weights_dev);

/* Same step with HOST buffers (pageable or pinned): copies hidden_in to the device, runs
 * the step, copies the three outputs back and returns when they are complete. */
int remoe_decode_step_host(remoe_stack*, const float* hidden_in_host, float* hidden_out_host,
                           int32_t* selected_ids_host, float* gate_weights_host);

/* Cache trace of the most recent step, to host arrays (any may be NULL).  Per layer the
 * distinct requests U in first-occurrence order (App. E.2.3), padded to B*K entries:
 *   requests/hit/slot/evicted [L, B*K] int32 (evicted = -1 when nothing was displaced),
 *   n_unique [L].  Waits for the stack's stream. */
int remoe_last_step_trace(remoe_stack*, int32_t* requests, int32_t* hit, int32_t* slot,
                          int32_t* evicted, int32_t* n_unique);

/* The directory of one layer as it stands after the most recent step (a debugging aid; App. A.1: the cache
 * state C_{t+1}).  Host arrays, any may be NULL: expert_of_slot [C] (-1 = empty slot), stamp [C] (the slot's
 * place in the layer's touch order: last touch under LRU and LFU, insertion under FIFO; 0 = never used),
 * use_count [C] (selections since insertion; decides under LFU).  Waits for the stack's stream. */
int remoe_cache_snapshot(remoe_stack*, int32_t layer, int32_t* expert_of_slot, uint64_t* stamp, uint32_t* use_count);

/* Counters for one layer, or summed over layers with layer = -1 (App. E.2.4: #uMiss, uHR =
 * uniq_hits / (uniq_hits + uniq_misses), tHR likewise).  Waits for the stack's stream; like the
 * other statistics calls it fills its outputs and returns DEVICE_FLAG if a kernel has set the error word. */
int remoe_cache_stats(remoe_stack*, int32_t layer, remoe_cache_counters* out);

/* Reuse statistic (Eq. 1): overlap_sum = sum over counted (step, sequence) pairs of
 * |E_t n E_{t-1}|, pairs_counted = number of such pairs (steps t >= 2 since the last
 * reset), so EOR = overlap_sum / (K * pairs_counted).  `last_ir` (host, [L, B] or NULL; with
 * layer >= 0: [B]) receives IR_t of the most recent step, -1 where t = 1.  layer = -1 sums. */
int remoe_reuse_stats(remoe_stack*, int32_t layer, uint64_t* overlap_sum,
                      uint64_t* pairs_counted, float* last_ir);

/* Reuse mass (Eq. 2): m_t = (1/K) * sum over k in E_{t-1} of P_t^(k), the probability the current
 * router puts on the previous step's experts.  mass_sum = sum of m_t over the counted (step,
 * sequence) pairs of the layer (layer = -1: all layers), pairs = their number, last_mass (host,
 * [L, B] or [B], may be NULL) = m_t of the most recent step, -1 where t = 1. */
int remoe_reuse_mass(remoe_stack*, int32_t layer, double* mass_sum, uint64_t* pairs, float* last_mass);

/* Expert load since the last reset (Sec. 4.4 "Routing imbalance"; Sec. 5.2 reports entropy and CV of
 * the routing).  counts (host, [N] for one layer, [L, N] for layer = -1, may be NULL) receives how
 * often each routed expert was selected (token level: B*K selections per layer-step).  From them,
 * per layer: the normalised entropy H(p) / log N of the load distribution p_e = n_e / sum n (1 = even
 * load), the coefficient of variation std(n) / mean(n) with the population standard deviation (0 =
 * even load), and the number of experts selected at least once.  With layer = -1 the three figures
 * are means over the layers (visited rounded down).  Before any step: entropy 1, cv 0, visited 0.
 * The paper prints entropy and CV without formulas; these definitions reproduce the relation its
 * printed pairs obey.  Any output may be NULL.  Waits for the stack's stream. */
int remoe_expert_load(remoe_stack*, int32_t layer, uint64_t* counts, double* norm_entropy, double* cv,
                      int32_t* experts_visited);

/* Per-step aggregates over all layers since the last reset (App. E.2.6): for steps first ..
 * first+count-1, umiss[i] = #uMiss^(all) of the step and tok_hits[i] = H_tok^(all) (either may be
 * NULL); n_steps receives how many steps are recorded.  Host-side bookkeeping, no device work. */
int remoe_step_history(remoe_stack*, int32_t first, int32_t count, uint32_t* umiss, uint32_t* tok_hits,
                       int32_t* n_steps);

/* I/O-time and TPOT proxy of App. E.2.6 / F.1: io_ms[i] = umiss[i] * expert_bytes / bandwidth * 1000
 * with bandwidth_gbps in 10^9 bytes/s, TPOT_i = tpot_compute_ms + io_ms[i] / batch.  io_ms ([n], may
 * be NULL) receives the per-step I/O time, tpot_p50_p95_p99 ([3], may be NULL) the percentiles of
 * TPOT over the n steps (linear interpolation between order statistics).  Pure host arithmetic. */
int remoe_tpot_proxy(const uint32_t* umiss, int32_t n, uint64_t expert_bytes, double bandwidth_gbps,
                     int32_t batch, double tpot_compute_ms, double* io_ms, double* tpot_p50_p95_p99);

/* Empty every layer's cache, forget E_{t-1} and zero all counters (Sec. 3: each request
 * starts from a cold expert cache). */
int remoe_cache_reset(remoe_stack*);

/* Replacement policy for subsequent steps (App. A.5 names LRU, LFU, FIFO); resets the cache. */
int remoe_set_policy(remoe_stack*, int32_t policy);

/* Cache-aware rerouting (App. F.2): add `beta` to the pre-top-K logits of experts resident
 * before the step; 0 (default) leaves routing untouched.  Gate weights still come from the
 * unbiased softmax. */
int remoe_set_reroute_beta(remoe_stack*, float beta);

/* Kernel timing aid: with `on` != 0 every launch of the expert-streaming kernel is bracketed
 * by CUDA events on the stream it runs on.  remoe_kernel_time returns, for phase 0 (resident
 * experts: cache hits + shared, one launch per step) or phase 1 (just-fetched experts, one
 * launch per layer with misses), the summed duration in ms, the number of launches and the
 * expert-weight bytes they streamed since profiling was switched on.  Waits for the events. */
int remoe_set_profiling(remoe_stack*, int32_t on);
int remoe_kernel_time(remoe_stack*, int32_t phase, double* ms_sum, uint64_t* launches,
                      uint64_t* weight_bytes);

/* Ordering checker of a stack created with REMOE_CHECK_ORDER=1 (see remoe_stack_create): how many pairs of
 * operations it has compared so far and how many were found unordered; both 0 on other stacks. */
int remoe_order_check_counts(remoe_stack*, uint64_t* comparisons, uint64_t* violations);

/* Number of kernels this stack has launched since creation (all kinds). */
int remoe_launch_count(remoe_stack*, uint64_t* launches);

/*
 * Gate-weighted SwiGLU expert sum of ONE layer without any allocation (the paper has no
 * counterpart: this exists for embedders, not for the method).
 *
 *     hidden_out[0:H] = sum_{e < n_experts} scales[e] * W_down^e (silu(W_gate^e h) * (W_up^e h))
 *
 * For callers that cannot call cudaMalloc where they use this library -- a serving loop whose
 * device memory is handed out once at start-up by someone else, worker threads on which the
 * host framework bans allocator calls, a device that is already full.  The stack-based entry
 * points above allocate their scratch at remoe_stack_create; this one keeps its scratch (one
 * partial output vector per CTA) in a fixed device array inside the library image, 1.25 MiB on
 * every GPU that loads the library, held until the process exits.  A call makes no cudaMalloc,
 * no cudaFree and no allocating library call; it launches two kernels on `cuda_stream`.
 *
 *   hidden, weight_dtype   as in remoe_shape; hidden <= REMOE_STATIC_MAX_HIDDEN
 *   n_experts              1 .. REMOE_STATIC_MAX_EXPERTS (routed and shared alike)
 *   expert_blocks_dev      HOST array of n_experts DEVICE pointers, each one expert block in
 *                          the [I, 3, H] layout above, 16-byte aligned, owned by the caller
 *   inter                  HOST array: I of each block, 1 .. REMOE_STATIC_MAX_INTER
 *   scales                 HOST array: gate weight (or shared-expert scale) of each block
 *   hidden_in_dev          DEVICE [H] float32;  hidden_out_dev  DEVICE [H] float32 (overwritten;
 *                          may be the same buffer as hidden_in_dev)
 *
 * The host arrays are read before the call returns.  The result is complete when `cuda_stream`
 * reaches the end of the call's work.  Sizes beyond the limits above, a hidden width the kernels
 * are not built for, or REMOE_FP8_E4M3 blocks are refused with REMOE_E_UNSUPPORTED before anything
 * is launched; bad pointers and unknown element types with REMOE_E_ARG.  The first call on each device also looks up the scratch
 * array's device address and sets kernel attributes for that device (with that device
 * current), so make that first call outside any stream capture.  All calls on a device share
 * the one scratch array: calls whose kernels could run at the same time (different streams
 * without ordering, or several host threads) race on it and must be serialised by the caller.
 * Each call overwrites the part of the scratch it reads, so earlier contents never matter.  If
 * an internal bounded wait ever runs out, the output is filled with NaN rather than a wrong
 * value.
 */
#define REMOE_STATIC_MAX_EXPERTS 16
#define REMOE_STATIC_MAX_HIDDEN 2048
#define REMOE_STATIC_MAX_INTER 65536
int remoe_expert_ffn_static(int32_t hidden, int32_t weight_dtype, int32_t n_experts,
                            const void* const* expert_blocks_dev, const int32_t* inter,
                            const float* scales, const float* hidden_in_dev, float* hidden_out_dev,
                            void* cuda_stream);

/* Text of the last CUDA runtime error, or of the last device-flag / trace-validation failure,
 * seen by this stack ("" if none). */
const char* remoe_last_cuda_error(const remoe_stack*);

void remoe_stack_destroy(remoe_stack*);
const char* remoe_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* REMOE_H_ */
