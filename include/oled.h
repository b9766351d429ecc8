/*
 * oled.h — C ABI of the B200 MoE denoise-step library.
 *
 * One context holds, for an L-layer MoE stack, a bounded GPU expert cache per layer (every
 * layer has a cache pool of its own, paper Sec. 4.1), the host expert store (borrowed pinned
 * host memory, where the experts that are not cached live, Sec. 2.2) and the scratch the step
 * needs.  A call to oled_denoise_step() performs one layer execution of one
 * denoising iteration over a block of tokens (Sec. 2.1, Sec. 4.1 per-layer flow):
 *
 *   gate -> top-k expert ids + gate scores -> token->expert permutation -> hits/misses
 *   against the resident set before execution (Sec. 4.2: A, R, M = A \ R) -> misses copied
 *   host->HBM on a side stream -> grouped SwiGLU expert FFN through the expert->slot table
 *   -> gate-weighted combine -> reuse priority (Sec. 4.3 priority equation) and the cache
 *   update R' = Top_C(R u G, p) (Sec. 4.2 cache-update equation) with G = M.
 *
 * There is no CPU execution path for misses: every missed expert is fetched and computed on
 * the GPU.  Offloading is lossless (Sec. 5.1): the output does not depend on the capacity.
 *
 * Conventions
 *   - Every function returns OLED_OK (0) or a negative oled_status; nothing aborts or throws.
 *   - "device" pointers are CUDA device memory of the current device; "host" pointers are
 *     ordinary host memory unless "pinned" is stated.
 *   - bf16 tensors are row-major arrays of 16-bit bfloat16 values.
 *   - One context is used by one host thread at a time.  Work is ordered on the stream given
 *     to oled_create(); oled_denoise_step() blocks the host until the gate results of the step
 *     are known (a few hundred bytes are read back to plan the copies), not until the step ends.
 *   - Shape limits: hidden a multiple of 256, at most 16384; intermediate a multiple of 128;
 *     1 <= top_k <= 32, top_k <= n_experts <= OLED_MAX_EXPERTS, max_tokens <= 65535.
 */
#ifndef OLED_H_
#define OLED_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define OLED_MAX_EXPERTS 512
#define OLED_MAX_TOPK 32

typedef enum {
  OLED_OK = 0,
  OLED_ERR_INVALID_ARG = -1,    /* null pointer, bad shape, layer out of range, aliasing       */
  OLED_ERR_NOT_PINNED = -2,     /* host expert store is not page-locked host memory             */
  OLED_ERR_NOT_REGISTERED = -3, /* step before the layer's router / experts were registered    */
  OLED_ERR_TOO_MANY_TOKENS = -4,/* n_tokens > max_tokens                                        */
  OLED_ERR_OOM = -5,            /* device or host allocation failed                             */
  OLED_ERR_CUDA = -6,           /* a CUDA call failed; see oled_last_cuda_error()               */
  OLED_ERR_TIMEOUT = -7,        /* a bounded device-side wait ran out; the step's out is invalid */
  OLED_ERR_NO_SLOT = -8,        /* staging_slots too small for this step's misses               */
  OLED_ERR_STALE_DEBUG = -9,    /* oled_debug_last(): the last step was on another layer        */
  OLED_ERR_SELF_CHECK = -10     /* OLED_OPT_SELF_CHECK found a violation; oled_self_check_report() */
} oled_status;

typedef struct oled_ctx oled_ctx; /* opaque, owned by the library */

typedef struct {
  int32_t n_layers;
  int32_t hidden;          /* H */
  int32_t n_experts;       /* E */
  int32_t top_k;           /* k */
  int32_t intermediate;    /* I (SwiGLU) */
  int32_t max_tokens;      /* upper bound on n_tokens of any step */
  int32_t has_router_bias; /* 1: oled_register_router() takes a per-expert fp32 bias */
  int32_t staging_slots;   /* transient slots for misses beyond capacity; 0 = E - 1, which can never
                              run out; a smaller value s stops layer-adaptive sizing from shrinking
                              a layer below E - s slots (a layer with C slots can need E - C
                              transient ones while it executes) */
  int32_t expert_format;   /* OLED_EXPERTS_BF16 (0) or OLED_EXPERTS_FP8 */
} oled_model_shape;

/* Expert blob formats of the host store and of the HBM slots (a blob is copied as it is).
 *   OLED_EXPERTS_BF16: gate[I,H] | up[I,H] | down[H,I] in bf16; 3*H*I*2 bytes.
 *   OLED_EXPERTS_FP8:  the same three matrices as fp8 e4m3 codes (1 byte each), followed by one
 *     fp32 scale per weight row, s_gate[I] | s_up[I] | s_down[H]; a weight is code * scale of its
 *     row.  3*H*I + 4*(2*I+H) bytes, padded to a multiple of 256.  Half the host-link and HBM
 *     traffic per expert (the paper names quantisation as the complementary lever for H2D volume).
 *     Token tiles of at most 32 rows (hidden and intermediate multiples of 128, steps of at most
 *     4096 token-expert assignments): the tensor cores read the codes as they are; a bf16 token
 *     row, scaled by a power of two, enters as the sum of two e4m3 terms, which represents every
 *     element within 2^-14 of the row's largest magnitude exactly (OLED_OPT_FP8_DIRECT).
 *     Otherwise the codes are widened to bf16 on chip (exactly) and the arithmetic is the bf16
 *     path's. */
#define OLED_EXPERTS_BF16 0
#define OLED_EXPERTS_FP8 1
/* Bytes of one expert blob in the given format. */
size_t oled_expert_blob_bytes(int32_t hidden, int32_t intermediate, int32_t expert_format);

/* Cumulative counters (Sec. 5.1 metrics: cache utilisation = hits / capacity per execution). */
typedef struct {
  uint64_t steps;          /* layer executions                                   */
  uint64_t hits;           /* sum of #(A n R), R taken before execution (Sec. 4.2) */
  uint64_t misses;         /* sum of #(A \ R)                                    */
  uint64_t bytes_moved;    /* host->HBM bytes: misses * blob bytes               */
  uint64_t evictions;      /* sum of #(R \ R')                                   */
  uint64_t active_experts; /* sum of #A                                          */
  uint64_t assignments;    /* sum of n_tokens * k                                */
  uint64_t fills_reused;   /* fetched experts that were retained and activated again at the
                              layer's next execution (Sec. 5.3 effective transfer ratio =
                              fills_reused / misses)                               */
  uint64_t ideal_hits;     /* sum of min(C_l, #A): hits of the clairvoyant cache bound of
                              Sec. 5.1 under the same capacity                     */
} oled_stats_t;

/* Create a context on the current CUDA device.
 *   shape           host; copied.
 *   cache_capacity  host int32[n_layers]; slots C_l per layer, 1 <= C_l <= E ("Cache" in Sec. 5.1).
 *   cuda_stream     a cudaStream_t (may be 0) on which every step is enqueued; borrowed.
 *   out_ctx         receives the context; the library owns it until oled_destroy().
 * Allocates the slot pool (sum C_l + staging slots, each one expert blob), router weights and
 * scratch in device memory.  Errors: INVALID_ARG, OOM, CUDA. */
int oled_create(const oled_model_shape* shape, const int32_t* cache_capacity, void* cuda_stream,
                oled_ctx** out_ctx);

/* Give a layer its gate, which yields the routed expert ids and the gate scores of every token
 * (Sec. 4.1).  w_router: [E,H] bf16, host or device, copied by the call.  bias: fp32[E] host or
 * device, or NULL (must be non-NULL iff has_router_bias). */
int oled_register_router(oled_ctx* ctx, int32_t layer, const void* w_router, const float* bias);

/* Give a layer its host expert store (Sec. 2.2, Sec. 4.1).  host_blob is PINNED host memory,
 * borrowed until oled_destroy() and never written; expert e starts at
 * host_blob + e*expert_stride_bytes and holds one blob in the context's expert_format
 * (stride >= oled_expert_blob_bytes() and a multiple of 16).  Errors: NOT_PINNED, INVALID_ARG. */
int oled_register_experts(oled_ctx* ctx, int32_t layer, const void* host_blob,
                          size_t expert_stride_bytes);

/* One layer execution of one denoising iteration (Sec. 4.1 per-layer flow; Sec. 4.2-4.3).
 *   hidden       device [n_tokens,H] bf16, read only.
 *   confidences  device fp32[n_tokens], token confidences c_t in [0,1] (Sec. 4.3).
 *   n_tokens     0 <= n_tokens <= max_tokens.
 *   out          device [n_tokens,H] bf16: sum_j g[t,j]*FFN_{e(t,j)}(hidden[t]); must not alias hidden.
 * hidden and out must be 16-byte aligned (rows are moved with 16-byte vector accesses),
 * confidences 4-byte aligned; a misaligned pointer is rejected with INVALID_ARG, nothing is launched.
 * Buffers are borrowed until the enqueued work completes on the context's stream.  The layer's
 * resident set and the counters are updated before the call returns.
 * Non-finite activations do not break the step: a NaN gate logit ranks as -inf (the k expert
 * ids of a token stay distinct), a NaN gate*confidence product adds nothing to the reuse score,
 * the outputs of the affected tokens are NaN and those of the other tokens are unaffected.
 * Errors: INVALID_ARG, NOT_REGISTERED, TOO_MANY_TOKENS, NO_SLOT, CUDA, TIMEOUT (reported by
 * the next call that synchronises). */
int oled_denoise_step(oled_ctx* ctx, int32_t layer, const void* hidden, const float* confidences,
                      int32_t n_tokens, void* out);

/* Same step with HOST buffers: hidden/confidences are copied host->device, out device->host,
 * on the context's stream; the call returns after out has arrived.  Pinned buffers make the
 * copies asynchronous with respect to the expert fills. */
int oled_denoise_step_host(oled_ctx* ctx, int32_t layer, const void* host_hidden,
                           const float* host_confidences, int32_t n_tokens, void* host_out);

/* One denoising iteration of the whole stack (Sec. 2.1: one iteration = one forward over the
 * block): layers 0..L-1 in order, x_{l+1} = bf16(x_l + out_l).  hidden / hidden_out are device
 * [n_tokens,H] bf16 (hidden_out may not alias hidden), confidences device fp32[n_tokens] and are
 * used for every layer of the iteration.  Errors as oled_denoise_step(). */
int oled_denoise_iteration(oled_ctx* ctx, const void* hidden, const float* confidences,
                           int32_t n_tokens, void* hidden_out);

/* The same with HOST buffers (copied in and out on the context's stream; returns after
 * hidden_out has arrived). */
int oled_denoise_iteration_host(oled_ctx* ctx, const void* host_hidden,
                                const float* host_confidences, int32_t n_tokens,
                                void* host_hidden_out);

/* Counters of one layer, or summed over layers for layer = -1.  Synchronises the stream. */
int oled_stats(oled_ctx* ctx, int32_t layer, oled_stats_t* out);

/* Parity aid: results of the most recent step, which must have been on `layer`.  All outputs
 * are host buffers and may be NULL to skip: ids int32[T*k], gate fp32[T*k], perm int32[T*k]
 * (perm[r] = t*k+j of sorted row r), counts int32[E], scores uint64[E] (integer numerators of
 * the Sec. 4.3 priority), resident_before / resident_after uint8[E] (0/1).  Synchronises. */
int oled_debug_last(oled_ctx* ctx, int32_t layer, int32_t* ids, float* gate, int32_t* perm,
                    int32_t* counts, uint64_t* scores, uint8_t* resident_before,
                    uint8_t* resident_after);

/* Parity aid, the permutation's other two products of the most recent step (host buffers, NULL
 * to skip): offsets int32[E+1], the exclusive scan of the counts (sorted rows of expert e are
 * offsets[e] .. offsets[e+1]-1), and pos int32[T*k], the inverse of perm (pos[t*k+j] = sorted row
 * of assignment (t,j)).  Synchronises. */
int oled_debug_perm(oled_ctx* ctx, int32_t layer, int32_t* offsets, int32_t* pos);

/* Tracing aid: the device-side timeline of the most recent step on `layer` that ran with
 * OLED_OPT_TIMELINE on.  times: host uint64[3 * OLED_TIMELINE_SLOTS], nanoseconds of the GPU's
 * global timer: [slot] earliest kernel entry, [SLOTS + slot] earliest pass of the dependency
 * wait, [2*SLOTS + slot] latest CTA end; a slot that did not run holds UINT64_MAX / 0.
 * Synchronises. */
int oled_debug_timeline(oled_ctx* ctx, int32_t layer, uint64_t* times);

/* Gate logits fp32[T*E] of the most recent step (host buffer).  Synchronises. */
int oled_debug_logits(oled_ctx* ctx, int32_t layer, float* logits);

/* Back to the cold state: every layer's resident set empty, counters zero.  Synchronises. */
int oled_reset_cache(oled_ctx* ctx);

/* y = bf16(x + r) elementwise over n bf16 values on the context's stream (the residual
 * between the layers of a stack is the caller's; this is a convenience kernel). */
int oled_residual_add(oled_ctx* ctx, const void* x, const void* r, void* y, size_t n);

/* Options.  OLED_OPT_FFN_IMPL: 0 = tcgen05 tensor-core kernels (default), 1 = plain-FMA
 * bring-up kernels.  OLED_OPT_MISS_CHUNK: size of the last fill group of a step, the only one whose
 * FFN runs after all copies have landed (default 4).
 * OLED_OPT_PROFILE: 1 = bracket every kernel launch with CUDA events on the context's stream
 * (adds two event records per launch; off by default).
 * OLED_OPT_POLICY: retention value used by the cache update of every layer (OLED_POLICY_*).
 * OLED_OPT_ADAPT_PERIOD: n > 0 makes oled_denoise_iteration() call oled_adapt_capacity() after
 * every n-th iteration (the paper refreshes every five); 0 = fixed capacities (default).
 * OLED_OPT_TEST_WITHHOLD_LOADS: test aid for the failure path.  1 = the tensor-core FFN kernels'
 * load producers issue nothing, so the consumers' bounded waits (2 s) run out: the kernels set
 * the status word, free their TMEM and return, and the next synchronising call reports
 * OLED_ERR_TIMEOUT.  The context stays usable; oled_clear_status() re-arms it. */
#define OLED_OPT_FFN_IMPL 1
#define OLED_OPT_MISS_CHUNK 2
#define OLED_OPT_PROFILE 3
#define OLED_OPT_POLICY 4
#define OLED_OPT_ADAPT_PERIOD 5
#define OLED_OPT_TEST_WITHHOLD_LOADS 6
/* OLED_OPT_SELF_CHECK: 1 = every step also runs two checking kernels (the paper has no counterpart;
 * they stand in for a memory checker): after the permutation, the invariants all later addressing
 * relies on (OLED_CHECK_* below); after the combine, the guard words behind the step's scratch
 * buffers.  A violation is sticky like a time-out: the next synchronising call returns
 * OLED_ERR_SELF_CHECK, oled_self_check_report() tells what was found, oled_clear_status() re-arms.
 * OLED_OPT_TEST_CORRUPT_PERM: test aid for that path.  1 = the first two rows of the sorted order
 * are exchanged after the permutation (both stay valid rows; the step's output is wrong). */
#define OLED_OPT_SELF_CHECK 7
#define OLED_OPT_TEST_CORRUPT_PERM 8
/* Launch-structure switches, all on by default; the results do not depend on them (they exist
 * to measure what each one buys):
 * OLED_OPT_SPLIT_LAST_FILL: the step's last expert blob is copied in two parts, gate|up first,
 *   so that the last group's gate/up kernel runs while its down-projection weights still arrive.
 * OLED_OPT_FUSE_COMBINE: inside oled_denoise_iteration(), steps of at most 1024 tokens leave a
 *   layer's combine and residual to the next layer's gate kernel (one kernel boundary and one
 *   reload of the hidden states less per layer).
 * OLED_OPT_FUSE_FFN: 0 = gate/up and down projection of an expert group always as two launches;
 *   1 (default) = as ONE launch where few work items per SM are expected (bf16 stores, token tiles
 *   of at most 32 rows): SMs that run out of gate/up items go on with the down projection of
 *   experts that are complete instead of idling until the whole gate/up launch has ended;
 *   2 = one launch wherever that form exists.
 * OLED_OPT_PDL: programmatic dependent launch between the kernels of a few-token step
 *   (process-wide, not per context). */
#define OLED_OPT_SPLIT_LAST_FILL 9
#define OLED_OPT_FUSE_COMBINE 10
#define OLED_OPT_FUSE_FFN 11
#define OLED_OPT_PDL 12
/* OLED_OPT_TIMELINE: 1 = the kernels of every step record, per kernel, when its first CTA entered,
 * when the first one got past its dependency wait and when the last one finished (GPU global
 * timer); read with oled_debug_timeline().  Off by default (a few atomics per CTA). */
#define OLED_OPT_TIMELINE 13
/* OLED_OPT_FP8_DIRECT (fp8 expert stores): 1 (default) = token tiles of at most 32 rows take the
 * form whose MMAs read the e4m3 codes directly; 0 = every tile widens the codes to bf16. */
#define OLED_OPT_FP8_DIRECT 14
/* OLED_OPT_FFN_PAIRS: 1 (default) = many-token steps (token tiles of 256 rows, bf16 stores,
 * intermediate a multiple of 256, hidden a multiple of 512) run the expert FFN on pairs of CTAs
 * that share a token tile (tcgen05 cta_group::2); 0 = always one CTA per tile. */
#define OLED_OPT_FFN_PAIRS 15
/* OLED_OPT_L2_PREFETCH: 1 (default) = inside oled_denoise_iteration(), while a layer whose previous
 * execution had no miss runs its gate and permutation kernels (the HBM is idle then), the weights
 * of the first experts its FFN will stream - the residents activated at that previous execution,
 * adjacent iterations activating mostly the same experts (Sec. 3.3) - are called into L2 from
 * the side stream, provided that execution streamed at least 320 MB of experts (shorter streams
 * were measured to lose); 2 = the same without that condition; 0 = off. */
#define OLED_OPT_L2_PREFETCH 16
/* OLED_OPT_GATHER_IN_FFN: 1 (default) = a many-token step whose FFN launches all run on CTA pairs
 * has no gather kernel: each gate/up launch copies its own experts' token rows into sorted order
 * while its first items run (one thread per CTA, bulk copies through shared memory, a counter
 * per expert that the items wait for); 0 = a gather kernel in front, as for every other step. */
#define OLED_OPT_GATHER_IN_FFN 17
#define OLED_TIMELINE_SLOTS 12 /* 0 gate, 1 permutation, 2 gather (not recorded),
                                  3..10 the step's FFN launches in order, 11 combine */
#define OLED_CHECK_ID_RANGE 0x01u      /* an expert id outside [0, E)                               */
#define OLED_CHECK_ID_DUPLICATE 0x02u  /* a token routed twice to one expert                        */
#define OLED_CHECK_OFFSETS 0x04u       /* offsets are not the exclusive scan of the counts          */
#define OLED_CHECK_PERM_RANGE 0x08u    /* a sorted row names no assignment                          */
#define OLED_CHECK_INVERSE 0x10u       /* pos is not the inverse of perm                            */
#define OLED_CHECK_ROW_EXPERT 0x20u    /* a sorted row lies outside the range of its expert         */
#define OLED_CHECK_ORDER 0x40u         /* the rows of an expert are not in ascending (token, rank)  */
#define OLED_POLICY_PRIORITY 0 /* confidence- and gate-guided priority, Sec. 4.3 (default) */
#define OLED_POLICY_LRU 1      /* comparison point: least recently used (Sec. 5.1 Naive-LRU)  */
#define OLED_POLICY_LFU 2      /* comparison point: least frequently used (Sec. 5.3)          */
int oled_set_option(oled_ctx* ctx, int32_t option, int64_t value);

/* Layer-adaptive cache sizing (Sec. 4.3): w_l = a_l * u_l with a_l the activation ratio and u_l
 * the cache utilisation of layer l over the layer executions since the previous call (smoothed
 * over calls by halving), C_l = C_total * w_l / sum_j w_j with C_total the sum of the capacities
 * given to oled_create(), every C_l in [1, E].  A layer left with more residents than slots
 * evicts its lowest-valued ones at once (a table update).  new_capacity: host int32[n_layers]
 * or NULL.  Host-side only; no GPU work. */
int oled_adapt_capacity(oled_ctx* ctx, int32_t* new_capacity);

/* Current per-layer capacities (host int32[n_layers]). */
int oled_get_capacity(oled_ctx* ctx, int32_t* capacity);

/* Per-kernel timing collected while OLED_OPT_PROFILE is on.  bytes / flops are the ALGORITHMIC
 * figures of the launches (weights of each expert once, token rows in, result rows out), not
 * measured traffic. */
#define OLED_KERNEL_ROUTE 0
#define OLED_KERNEL_PERMUTE 1
#define OLED_KERNEL_GATHER 2
#define OLED_KERNEL_FFN_GATE_UP 3
#define OLED_KERNEL_FFN_DOWN 4
#define OLED_KERNEL_COMBINE 5
#define OLED_KERNEL_FFN_FUSED 6 /* gate/up + SwiGLU + down projection in one launch */
#define OLED_N_KERNELS 7
typedef struct {
  uint64_t launches;
  double ms;       /* sum of CUDA-event durations */
  uint64_t bytes;
  uint64_t flops;
} oled_kernel_profile;
/* Synchronises, folds pending event pairs into the totals and returns those of `kernel`;
 * reset != 0 clears them afterwards. */
int oled_profile_read(oled_ctx* ctx, int32_t kernel, int32_t reset, oled_kernel_profile* out);

/* Clears a recorded device-side time-out (OLED_ERR_TIMEOUT is sticky until then).  Synchronises. */
int oled_clear_status(oled_ctx* ctx);

/* What OLED_OPT_SELF_CHECK has found since the status was last cleared.  Synchronises.
 *   flags        OR of OLED_CHECK_* (0 = nothing).
 *   first_index  the smallest offending index (assignment, expert or sorted row, by flag), -1 if none.
 *   guard_mask   bit b set = the guard words behind scratch buffer b were overwritten (order:
 *                logits, ids, gate, offsets, perm, pos, sorted token rows, intermediate, outputs).
 * Any pointer may be NULL. */
int oled_self_check_report(oled_ctx* ctx, uint32_t* flags, int32_t* first_index, uint32_t* guard_mask);

/* Host time spent in the cache policy (hit/miss resolution, Top-C retention, slot plan) so far, in
 * nanoseconds, and the number of policy runs - the "policy overhead" of Sec. 5.4. */
int oled_policy_time(oled_ctx* ctx, uint64_t* nanoseconds, uint64_t* runs);

/* Number of kernels the library has launched on this context so far. */
int oled_launch_count(oled_ctx* ctx, uint64_t* out);

/* Wait for the context's streams; returns TIMEOUT if a device-side wait ran out. */
int oled_synchronize(oled_ctx* ctx);

void oled_destroy(oled_ctx* ctx);

const char* oled_strerror(int code);

/* The CUDA error code of the last OLED_ERR_CUDA on this context (cudaError_t as int). */
int oled_last_cuda_error(oled_ctx* ctx);

/* Routing of one step without any allocation.  The paper has no counterpart: this exists for
 * hosts that cannot let a library allocate device memory - a server that gives all of it to its
 * own arena at start-up, or a decode loop that cannot afford the device-wide synchronisation
 * hidden in cudaMalloc/cudaFree.  It runs the same gate, top-k, gate-score and permutation
 * kernels as oled_denoise_step(), needs no context, and keeps its scratch (gate logits, inverse
 * permutation, reuse-score accumulators; about 0.55 MB) in a fixed array inside the library
 * image, which every GPU that loads the library holds until the process exits.
 *   hidden [n_tokens,hidden_dim] bf16, w_router [n_experts,hidden_dim] bf16, bias fp32[n_experts]
 *   or NULL, confidences fp32[n_tokens]: device, read only.
 *   ids int32[n_tokens*top_k], gate fp32[n_tokens*top_k], counts int32[n_experts],
 *   offsets int32[n_experts+1], perm int32[n_tokens*top_k]: device, written; caller-owned.
 *   n_tokens <= OLED_NOALLOC_MAX_TOKENS, else OLED_ERR_TOO_MANY_TOKENS; other limits as above.
 *   hidden, w_router and ids must be 16-byte aligned (they are accessed with 16-byte vectors), the
 *   other arrays 4-byte aligned; a misaligned pointer is rejected with OLED_ERR_INVALID_ARG before
 *   anything is launched.
 * The launches use programmatic dependent launch when the calling thread's most recent
 * oled_denoise_step() did (steps of at most 4096 token-expert assignments), and by default if the
 * thread has run no step; either way the results are the same.
 * The work is enqueued on cuda_stream.  The first call on a device looks up the array's device
 * address (one-time set-up under a lock); make that first call before any stream capture.
 * All calls share the one array, which still holds the previous call's data: the accumulators
 * are cleared on the stream at the start of every call, and two calls whose work overlaps on
 * the GPU (different streams, no ordering between them) race on it.  Calls cudaMemsetAsync and
 * kernel launches only: no cudaMalloc, cudaFree or allocating library routine. */
#define OLED_NOALLOC_MAX_TOKENS 256
int oled_route_noalloc(const void* hidden, const void* w_router, const float* bias,
                       const float* confidences, int32_t n_tokens, int32_t hidden_dim,
                       int32_t n_experts, int32_t top_k, void* cuda_stream, int32_t* ids,
                       float* gate, int32_t* counts, int32_t* offsets, int32_t* perm);

/* ---- host-only policy simulator (no GPU needed): the same C++ policy code the step uses,
 * driven by recorded counts and integer scores.  For tests of the host logic. ---- */
typedef struct oled_policy oled_policy;
int oled_policy_create(int32_t n_experts, int32_t capacity, int32_t pool_slots, oled_policy** out);
/* counts int32[E], scores uint64[E] -> resident_before/after uint8[E], slot_of int32[E] (slot of
 * every activated expert during the step, -1 otherwise), n_hits/n_misses/n_evictions. */
int oled_policy_step(oled_policy* p, const int32_t* counts, const uint64_t* scores,
                     uint8_t* resident_before, uint8_t* resident_after, int32_t* slot_of,
                     int32_t* n_hits, int32_t* n_misses, int32_t* n_evictions);
/* The layers of a simulated STACK: n_layers simulators that share one slot pool sized by the rule
 * oled_create() uses (sum of the capacities + staging; staging_slots = 0 takes the default), with
 * the same floor on the capacities oled_policy_adapt() may hand out.  out: oled_policy*[n_layers],
 * each destroyed with oled_policy_destroy(); pool_slots (may be NULL) receives the pool size. */
int oled_policy_create_stack(int32_t n_layers, int32_t n_experts, const int32_t* capacity,
                             int32_t staging_slots, oled_policy** out, int32_t* pool_slots);
void oled_policy_destroy(oled_policy* p);
/* Retention value of the simulator's layer (OLED_POLICY_*). */
int oled_policy_set_policy(oled_policy* p, int32_t policy);
/* fills_reused counter of the simulator's layer. */
int oled_policy_fills_reused(oled_policy* p, uint64_t* out);
/* Layer-adaptive sizing over n simulated layers (one oled_policy each): as oled_adapt_capacity(). */
int oled_policy_adapt(oled_policy** layers, int32_t n_layers, int32_t total_capacity,
                      int32_t* new_capacity);

#ifdef __cplusplus
}
#endif
#endif /* OLED_H_ */
