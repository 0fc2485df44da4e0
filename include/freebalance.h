/*
 * freebalance.h - C ABI of the B200 (sm_100a) FreeBalance hot path.
 *
 * One call sequence per MoE layer l, following the paper's four-stage overview
 * (Method, "Motivation and Overview") and Algorithm 1:
 *
 *   1. fb_predict_load      early router pass g_l(h_{l-1}) (Eqs. 2, 4), the model's
 *                           top-k rule, predicted expert workload n_e (Eq. 5)
 *   2. fb_plan_swaps        rank loads under the placement pi (Alg. 1 line 2), cost
 *                           model (Eq. 9), budgets (Eq. 10), deterministic greedy
 *                           pairwise swaps under the load objective (Eqs. 6-8)
 *      fb_predict_and_plan  1 + 2 in a single kernel launch
 *      fb_layer_step        1 + 2 + 4 for one layer: both router passes in one launch
 *   3. fb_apply_swaps       the accepted swaps applied to the expert weights (logical ranks
 *                           on one GPU: an exchange of slot images inside one buffer)
 *   4. fb_route_dispatch    normal router pass g_l(H_l) (Eq. 3), authoritative top-k
 *                           and routing weights, and the token -> expert dispatch
 *                           index under the committed placement pi'
 *
 * Expert-parallel ranks are logical: a placement maps expert e to a physical slot
 * p = expert_to_slot[e] in [0, E); slot p belongs to rank p / (E / R).  Everything
 * runs on one GPU.
 *
 * Conventions
 *   - "dev" pointers are device memory owned by the caller, 16-byte aligned,
 *     dense row-major.  "host" pointers are ordinary host memory.
 *   - Structs (fb_config, fb_router, fb_budget) are host structs read during the call.
 *   - Calls enqueue work on `stream` and return without synchronising, except
 *     fb_layer_step_host and fb_device_status, which block until the stream drains,
 *     fb_apply_swaps_staged (waits for the plan) and fb_calibrate_exchange (times itself).
 *   - The method's device calls (fb_predict_load, fb_plan_swaps, fb_predict_and_plan,
 *     fb_route_dispatch, fb_layer_step, the dispatch-index helpers) allocate nothing,
 *     query nothing and keep no per-launch state on the host that a kernel depends on,
 *     so after one ordinary call with the same arguments (which builds the tensor maps
 *     and loads the kernels) they may be captured into a CUDA graph and the graph
 *     replayed on new contents of the same buffers.  Budgets and shapes are frozen into
 *     the graph at capture; fb_device_status is not capturable (it synchronises).
 *   - No call throws or aborts.  Argument and shape problems are reported by the
 *     return value and nothing is launched.  Problems only the device can see (a
 *     placement that is not a bijection, count sums beyond the planner's range, a
 *     bounded wait inside a kernel that expired) set a device status word which
 *     fb_device_status returns; outputs of that call are then unspecified but every
 *     write stays inside the caller's buffers.
 *   - There is no CPU fallback: without a CUDA device fb_create fails.
 */
#ifndef FREEBALANCE_H_
#define FREEBALANCE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fb_ctx fb_ctx;              /* opaque; owns a few KB..MB of device scratch */
typedef void* fb_stream;                   /* a cudaStream_t (NULL = default stream)      */

typedef enum {
  FB_OK = 0,
  FB_ERR_INVALID_ARG = 1,                  /* NULL pointer, negative size, bad struct field   */
  FB_ERR_UNSUPPORTED_SHAPE = 2,            /* shape outside the limits listed at fb_create    */
  FB_ERR_CUDA = 3,                         /* a CUDA runtime / driver call failed             */
  FB_ERR_BAD_PLACEMENT = 4,                /* device: expert_to_slot is not a bijection       */
  FB_ERR_TIMEOUT = 5,                      /* device: a bounded wait inside a kernel expired  */
  FB_ERR_RANGE = 6,                        /* device: sum of counts exceeds FB_MAX_COUNT_SUM  */
  FB_ERR_INTERNAL = 7                      /* device, builds with -DFB_DEBUG only: an index the */
                                           /* kernels were about to write was out of range      */
} fb_status;

/* The model's "original top-k rule" applied to the router logits (text after Eq. 4). */
typedef enum {
  FB_GATE_SOFTMAX_TOPK = 0,                /* key = logit; weights = softmax probabilities    */
  FB_GATE_SIGMOID_GROUP_TOPK = 1           /* key = sigmoid(logit) + select_bias, restricted  */
                                           /* to the topk_group best of n_group expert groups */
} fb_gate;

#define FB_MAX_EXPERTS   256
#define FB_MAX_RANKS     64
#define FB_MAX_TOPK      8
#define FB_MAX_GROUPS    32
#define FB_MAX_COUNT_SUM (1u << 21)        /* planner: sum of counts <= 2^21                  */
#define FB_MAX_GAMMA_NUM (1u << 20)
#define FB_BUDGET_OFF    UINT64_MAX        /* a residual budget that is not enforced          */

typedef struct {
  int32_t T_max;        /* largest token count any call will pass                              */
  int32_t d;            /* hidden size; multiple of 8                                          */
  int32_t E;            /* routed experts, 1..256                                              */
  int32_t k;            /* experts per token, 1..min(E, 8)                                     */
  int32_t R;            /* logical ranks, 1..64, divides E                                     */
  int32_t gate;         /* fb_gate                                                             */
  int32_t n_group;      /* sigmoid gate: number of contiguous expert groups (divides E, <=32)  */
  int32_t topk_group;   /* sigmoid gate: groups kept per token (1..min(n_group, 8))            */
  int32_t renorm;       /* 1: routing weights divided by their sum over the k chosen           */
  float   route_scale;  /* sigmoid gate: factor applied to the routing weights                 */
} fb_config;

/* The frozen router of the target layer, shared by both invocations (Eqs. 2-4). */
typedef struct {
  const void*  W;            /* dev bf16 [E][d]: row e = column e of the paper's W (K-major)   */
  const float* logit_bias;   /* dev fp32 [E] or NULL: b of Eq. 4                               */
  const float* select_bias;  /* dev fp32 [E] or NULL: added to the sigmoid score for selection */
                             /* only (never to the routing weight); ignored by the softmax gate */
} fb_router;

/* How the planner walks the candidates ("Budgeted Expert-Swap Planning").  The paper's
 * Algorithm 1 loops and re-enumerates after every accepted swap; its prose describes one
 * enumeration and one sorted pass; its last paragraph restricts the candidates to the most
 * and the least loaded rank "in practice".  The default follows Algorithm 1 on that narrow
 * frontier; the other two modes are the readings left over, kept for comparison. */
typedef enum {
  FB_PLAN_LOOP = 0,    /* Algorithm 1: most -> least loaded rank, re-enumerated per accepted swap      */
  FB_PLAN_SWEEP = 1,   /* one enumeration on the initial frontier, one sort by benefit / cost, one     */
                       /* pass: a pair is accepted if both experts are unselected and the budgets hold */
                       /* (later pairs keep the score of the initial loads, so the maximum can rise)   */
  FB_PLAN_WIDE = 2     /* Algorithm 1 with frontier_width ranks at each end of the load order; a       */
                       /* source must carry strictly more than its destination; ties also by ranks     */
} fb_plan_mode;

/* Planner parameters: Algorithm 1's budget B and threshold tau, the weight gamma of
 * Eq. 8 and the cost model of Eq. 9 in integer units so that every rank (and the CPU
 * oracle) reproduces the same plan bit for bit. */
typedef struct {
  uint32_t max_swaps;        /* hard cap on accepted swaps (0 keeps the placement), <= E/2     */
  uint64_t global_ns;        /* residual budgets, initial value B_l of Eq. 10: one for the     */
  uint64_t rank_ns;          /*   whole plan, one per rank, one per link.  Every accepted swap */
  uint64_t link_ns;          /*   is charged C(s) to each it touches; FB_BUDGET_OFF disables.  */
  uint32_t tau_tokens;       /* loop only while max_r L_r - min_r L_r > tau_tokens             */
  uint32_t gamma_num;        /* gamma = gamma_num / gamma_den (<= FB_MAX_GAMMA_NUM / any);     */
  uint32_t gamma_den;        /*   gamma_den == 0 means gamma = 0                               */
  uint64_t alpha_ns[2];      /* alpha of Eq. 9: [0] same node, [1] different nodes             */
  uint64_t fs_per_byte[2];   /* 1 / beta of Eq. 9 in femtoseconds per byte, same indexing      */
  int32_t  ranks_per_node;   /* <= 0: all ranks in one node                                    */
  uint64_t expert_bytes;     /* S(e) when every expert has the same size                       */
  const uint64_t* expert_bytes_table; /* dev u64 [E] per-expert S(e), or NULL for the uniform size */
  int32_t  mode;             /* fb_plan_mode; 0 (all-zero tail of the struct) is Algorithm 1's loop */
  int32_t  frontier_width;   /* FB_PLAN_WIDE: 1..4 ranks from each end (values outside are clamped)  */
} fb_budget;

/* One accepted swap: expert_src leaves src_rank (the overloaded one) for dst_rank,
 * expert_dst travels the other way. */
typedef struct { int32_t src_rank, dst_rank, expert_src, expert_dst; } fb_swap;

/* ------------------------------------------------------------------------------------
 * Context.  fb_create allocates all device scratch the other calls need (sized from
 * T_max and E) on `device`; fb_destroy frees it.  No other call allocates, except the
 * first fb_layer_step_host and fb_apply_swaps_staged (their staging buffers).
 * Limits (FB_ERR_UNSUPPORTED_SHAPE otherwise): 1 <= E <= 256, 1 <= k <= min(E, 8),
 * 1 <= R <= 64 with R | E, d >= 8 with 8 | d, 0 <= T <= T_max < 2^31 / max(E, k);
 * sigmoid gate: n_group | E, n_group <= 32, 1 <= topk_group <= min(n_group, 8),
 * topk_group * (E / n_group) >= k.
 * ------------------------------------------------------------------------------------ */
fb_status fb_create(fb_ctx** out, const fb_config* cfg, int device);
fb_status fb_destroy(fb_ctx* ctx);

/* Eq. 10: B = max(0, t_attn - delta), all in nanoseconds.  Pure host arithmetic. */
uint64_t fb_budget_ns(uint64_t t_attn_ns, uint64_t delta_ns);

/* ---- attention profiling for the budget of Eq. 10 ("Budgeted Expert-Swap Planning": attention
 * is profiled once per attention type and the measurement is reused for later layers of that
 * type; r(l) is the first layer that uses the attention mechanism of layer l) ----
 * The caller brackets the attention of every layer with fb_attention_begin / fb_attention_end
 * on the stream the attention kernels run on.  For the first layer of an attention type (its
 * r(l)) the pair records two CUDA events around the region; for every later layer of a type
 * that already has a measurement (or one under way) both calls do nothing, so they cost nothing
 * in steady state.  attn_type is a caller-chosen id in [0, FB_MAX_ATTENTION_TYPES): 0 for a
 * homogeneous model, one id per mechanism (full, linear, sparse, ...) for a hybrid one.
 *   fb_layer_budget_ns   B_l = max(0, T_attn[r(l)] - delta_ns) for a layer of that type, in
 *                        *budget_ns; *profiled_layer (optional) receives r(l).  The first
 *                        query after a measurement waits for its closing event (blocking, once
 *                        per type); FB_ERR_INVALID_ARG if the type has never been profiled.
 *   fb_attention_set_time_ns  installs a measurement taken elsewhere (or replaces one).
 *   fb_attention_reset   forgets every measurement (the input shape changed).
 * Host-side bookkeeping plus event records; nothing is launched. */
#define FB_MAX_ATTENTION_TYPES 8
fb_status fb_attention_begin(fb_ctx* ctx, int32_t layer_id, int32_t attn_type, fb_stream stream);
fb_status fb_attention_end(fb_ctx* ctx, int32_t layer_id, int32_t attn_type, fb_stream stream);
fb_status fb_layer_budget_ns(fb_ctx* ctx, int32_t attn_type, uint64_t delta_ns, uint64_t* budget_ns,
                             int32_t* profiled_layer);
fb_status fb_attention_set_time_ns(fb_ctx* ctx, int32_t attn_type, int32_t layer_id, uint64_t t_attn_ns);
fb_status fb_attention_reset(fb_ctx* ctx);

/* Eq. 9 for a pair of ranks with uniform expert size: C = alpha + 2 S / beta in whole
 * nanoseconds (transfer term rounded up, total at least 1).  Pure host arithmetic;
 * returns 0 if the product overflows 64 bits. */
uint64_t fb_swap_cost_ns(const fb_budget* budget, int32_t rank_a, int32_t rank_b);

/* Stage 1 - residual workload prediction (Eqs. 2, 4, 5).
 *   x           dev bf16 [T][d]  residual hidden states h_{l-1}
 *   counts      dev u32 [E]      out: n_e = number of tokens whose top-k contains e
 *   topk_ids    dev i32 [T][k]   out, optional (NULL to skip): chosen experts per token,
 *                                descending selection key, equal keys -> lower id first
 *   logits      dev f32 [T][E]   out, optional debug dump of g(x) (NULL to skip)
 * T == 0 writes zero counts. */
fb_status fb_predict_load(fb_ctx* ctx, const fb_router* router, const void* x, int32_t T,
                          uint32_t* counts, int32_t* topk_ids, float* logits, fb_stream stream);

/* Stage 2 - budgeted expert-swap planning (Algorithm 1 lines 2-8; Eqs. 6-9).
 * Each iteration takes the most and the least loaded rank (lowest index on ties),
 * enumerates pairs of their experts not yet moved in this call, drops pairs whose
 * benefit Phi(L) - Phi(L') (Eq. 8) is not positive or whose cost C(s) exceeds a
 * residual budget, and accepts the pair with the largest benefit / cost (compared
 * exactly; ties -> smallest (expert_src, expert_dst)).  It stops when max - min load
 * <= tau_tokens, after max_swaps swaps, or when no pair survives.
 *   counts              dev u32 [E]        predicted workload
 *   expert_to_slot      dev i32 [E]        current placement pi (a bijection onto 0..E-1)
 *   expert_to_slot_out  dev i32 [E]        out: pi' (may alias expert_to_slot)
 *   swaps               dev fb_swap [max_swaps]  out: accepted swaps in order
 *   n_swaps             dev i32 [1]        out
 *   load_before/after   dev u32 [R]        out: rank loads under pi / pi'
 * An empty plan leaves pi' == pi. */
fb_status fb_plan_swaps(fb_ctx* ctx, const uint32_t* counts, const int32_t* expert_to_slot,
                        const fb_budget* budget, int32_t layer_id,
                        int32_t* expert_to_slot_out, fb_swap* swaps, int32_t* n_swaps,
                        uint32_t* load_before, uint32_t* load_after, fb_stream stream);

/* Stages 1 + 2 in one launch: the thread block that finishes last runs the planner. */
fb_status fb_predict_and_plan(fb_ctx* ctx, const fb_router* router, const void* x, int32_t T,
                              const int32_t* expert_to_slot, const fb_budget* budget,
                              int32_t layer_id, uint32_t* counts, int32_t* expert_to_slot_out,
                              fb_swap* swaps, int32_t* n_swaps,
                              uint32_t* load_before, uint32_t* load_after, fb_stream stream);

/* Stage 4 - normal routing (Eq. 3) and the dispatch index under pi'.  Never looks at
 * the prediction: the normal router alone decides the assignments.
 *   x             dev bf16 [T][d]   H_l, the router's normal input
 *   topk_ids      dev i32 [T][k]    out: chosen experts (order as in fb_predict_load)
 *   topk_w        dev f32 [T][k]    out: routing weights of those experts
 *   slot_offsets  dev u32 [E+1]     out: exclusive prefix sums of tokens per physical slot
 *   rank_offsets  dev u32 [R+1]     out: rank_offsets[r] = slot_offsets[r * E / R]
 *   perm          dev i32 [T*k]     out: perm[pos] = i*k + j, ordered by (slot, token i)
 *   inv_perm      dev i32 [T*k]     out: inv_perm[i*k + j] = pos
 *   rank_load     dev u32 [R]       out: realised tokens per rank
 *   logits        dev f32 [T][E]    out, optional debug dump (NULL to skip) */
fb_status fb_route_dispatch(fb_ctx* ctx, const fb_router* router, const void* x, int32_t T,
                            const int32_t* expert_to_slot, int32_t* topk_ids, float* topk_w,
                            uint32_t* slot_offsets, uint32_t* rank_offsets,
                            int32_t* perm, int32_t* inv_perm, uint32_t* rank_load,
                            float* logits, fb_stream stream);

/* ---- the path on several GPUs (token-sharded; "Budgeted Expert-Swap Planning": the ranks
 * exchange only the compact load statistics and then reproduce the same plan locally) ----
 * Every GPU holds a contiguous token range, in rank order.  Prediction and planning need one
 * exchange: fb_predict_load on the local tokens, a sum all-reduce of the E counts among the
 * ranks (the caller's collective, e.g. NCCL), fb_plan_swaps on the summed counts - every rank
 * arrives at the same plan.  The dispatch index needs one more: fb_route_dispatch on the local
 * tokens gives local positions; fb_dispatch_slot_counts turns the local slot_offsets into the E
 * per-slot counts; the ranks all-gather them (world x E words); fb_dispatch_globalize then
 * rewrites the local inv_perm into positions in the dispatch order of the WHOLE batch (by slot,
 * then by token, earlier ranks' tokens first) and writes the whole batch's slot_offsets,
 * rank_offsets and rank_load, identical on every rank.  An assignment at whole-batch position
 * pos goes to the rank r with rank_offsets[r] <= pos < rank_offsets[r+1], to row
 * pos - rank_offsets[r] of its receive buffer.
 *   slot_counts_all     dev u32 [world][E]  the gathered counts, row r from rank r
 *   slot_offsets_local  dev u32 [E+1]       as written by fb_route_dispatch on the local tokens
 *   topk_ids            dev i32 [T_local][k], expert_to_slot dev i32 [E]: as given to / written by that call
 *   inv_perm            dev i32 [T_local*k] in: local positions; out: whole-batch positions
 * Errors: FB_ERR_INVALID_ARG (NULL pointer, rank outside [0, world), world outside [1, 4096]),
 * FB_ERR_UNSUPPORTED_SHAPE (T_local > T_max).  The whole batch must stay below 2^31 assignments. */
fb_status fb_dispatch_slot_counts(fb_ctx* ctx, const uint32_t* slot_offsets, uint32_t* slot_counts, fb_stream stream);
fb_status fb_dispatch_globalize(fb_ctx* ctx, int32_t T_local, int32_t world, int32_t rank,
                                const uint32_t* slot_counts_all, const uint32_t* slot_offsets_local,
                                const int32_t* topk_ids, const int32_t* expert_to_slot, int32_t* inv_perm,
                                uint32_t* slot_offsets, uint32_t* rank_offsets, uint32_t* rank_load,
                                fb_stream stream);

/* One whole layer with device buffers: stages 1, 2 and 4 in one call.  Same results, bit for
 * bit, as fb_predict_and_plan followed by fb_route_dispatch under the new placement, but
 * both router passes (the early one on h_prev, the normal one on H) run in ONE kernel
 * launch: the tiles of the normal pass follow those of the early pass on the same blocks
 * (or in the same grid), so the selection and planning tail of the early pass is hidden
 * behind the normal pass.  The dispatch index follows in a second launch.  Arguments as in
 * the two calls it replaces; h_prev and H must be different buffers of [T][d] bf16 each,
 * and expert_to_slot_out must not alias expert_to_slot.  Errors as in those calls. */
fb_status fb_layer_step(fb_ctx* ctx, const fb_router* router, const void* h_prev, const void* H, int32_t T,
                        const int32_t* expert_to_slot, const fb_budget* budget, int32_t layer_id,
                        uint32_t* counts, int32_t* expert_to_slot_out, fb_swap* swaps, int32_t* n_swaps,
                        uint32_t* load_before, uint32_t* load_after, int32_t* topk_ids, float* topk_w,
                        uint32_t* slot_offsets, uint32_t* rank_offsets, int32_t* perm, int32_t* inv_perm,
                        uint32_t* rank_load, fb_stream stream);

/* One whole layer (fb_layer_step) with HOST buffers for the per-step tensors: h_prev, H, expert_to_slot
 * are copied to the device, every output pointer receives host data, and the call
 * returns after the stream has drained.  The router stays on the device (frozen
 * weights).  Device staging is allocated on the first call.  Any output pointer may
 * be NULL to skip its copy.  Pinned host memory makes the copies asynchronous. */
fb_status fb_layer_step_host(fb_ctx* ctx, const fb_router* router,
                             const void* h_prev_host, const void* H_host, int32_t T,
                             const int32_t* expert_to_slot_host, const fb_budget* budget,
                             int32_t layer_id,
                             uint32_t* counts, int32_t* expert_to_slot_out, fb_swap* swaps,
                             int32_t* n_swaps, uint32_t* load_before, uint32_t* load_after,
                             int32_t* topk_ids, float* topk_w, uint32_t* slot_offsets,
                             uint32_t* rank_offsets, int32_t* perm, int32_t* inv_perm,
                             uint32_t* rank_load, fb_stream stream);

/* fb_predict_load for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a deployment variant of stage 1, same computation.)
 *
 * Who needs it: code that runs after an inference server has frozen its memory pool
 * and forbids any further cudaMalloc (allocations there synchronise the device and
 * fragment the pool), code inside a region where allocation is illegal, and hosts that
 * link the library but may not create an fb_ctx because fb_create allocates.  This call
 * takes no context and performs no cudaMalloc / cudaFree and calls no allocating library
 * routine; the caller passes inputs and outputs as for fb_predict_load (`logits` is not
 * offered).
 *
 * The kernel's scratch - FB_STATIC_MAX_EXPERTS histogram counters, the finished-block
 * ticket and a status word, 1280 bytes - is a fixed array inside the library image, so
 * every GPU that loads the library holds those bytes until the process exits.
 *   - cfg->E above FB_STATIC_MAX_EXPERTS is refused with FB_ERR_UNSUPPORTED_SHAPE; the
 *     other limits are those of fb_create.
 *   - The first call on a device looks up the array's device address and raises the
 *     kernels' shared-memory ceiling (once per device); a change of cfg only redoes host
 *     arithmetic.  Make that first call before starting any stream capture.
 *   - What the call cannot rule out is the driver's own work: with lazy module loading the
 *     first launch of a kernel variant on a device places its code (and this array) there.
 *     The guarantee "takes nothing from the device" therefore holds from the second call
 *     with a given gate type on; make one warm-up call before the memory pool is frozen.
 *   - All calls on a device share the one array.  Each call clears it on `stream` before
 *     its kernel, so a call is not disturbed by what an earlier one left behind, but two
 *     calls that overlap on the GPU (different streams) race on it: serialise them.
 *   - status_word: dev i32 [1] or NULL.  If given (zeroed by the caller), device-detected
 *     problems are recorded there as by fb_device_status; if NULL they go unreported.
 * Not thread-safe. */
#define FB_STATIC_MAX_EXPERTS 256
fb_status fb_predict_load_static(const fb_config* cfg, int device, const fb_router* router,
                                 const void* x, int32_t T, uint32_t* counts, int32_t* topk_ids,
                                 int32_t* status_word, fb_stream stream);

/* Synchronises `stream`, returns the device status word in *word (FB_OK, or the
 * first FB_ERR_BAD_PLACEMENT / FB_ERR_TIMEOUT / FB_ERR_RANGE raised since the last
 * query) and clears it. */
fb_status fb_device_status(fb_ctx* ctx, int32_t* word, fb_stream stream);

/* ---- stage 3 on one device (Method overview, "Weight Transfer"): apply a plan to the weights ----
 * slot_weights is a device buffer of E slot images of expert_bytes each (slot p at byte
 * offset p * expert_bytes; 16-byte aligned, expert_bytes a multiple of 16); slot p holds the
 * weights of the expert placed there.  For each of the *n_swaps accepted swaps (device
 * scalar and device array as written by fb_plan_swaps / fb_predict_and_plan / fb_layer_step;
 * max_swaps = capacity of the array) the images of the two experts' slots UNDER
 * expert_to_slot - the placement BEFORE the plan, i.e. the planner's input - are exchanged
 * in place, so that afterwards every expert's weights sit in the slot the planner's output
 * placement names.  One launch for the whole plan (swaps of one plan touch disjoint slots);
 * no staging memory; nothing is read on the host, so the call can follow the planner on the
 * same stream, or run on another stream behind an event, beside the attention kernels.
 * The caller keeps the weights unused by other work on the device until the call completes.
 * status_word (device, optional) receives FB_ERR_RANGE / FB_ERR_BAD_PLACEMENT if a swap or
 * the placement is out of range (that swap is skipped).  Traffic: 4 * expert_bytes per swap. */
fb_status fb_apply_swaps(void* slot_weights, uint64_t expert_bytes, int32_t E, const int32_t* expert_to_slot,
                         const fb_swap* swaps, const int32_t* n_swaps, int32_t max_swaps, int32_t* status_word,
                         fb_stream stream);

/* Cost-model calibration ("Budgeted Expert-Swap Planning": the parameters of Eq. 9 are
 * calibrated during runtime initialisation).  fb_fit_cost_model fits C = alpha + 2 S / beta
 * through two timed exchanges of experts of bytes_small and bytes_large each (host
 * arithmetic, exact): *fs_per_byte = 1/beta in femtoseconds per byte rounded up, *alpha_ns
 * rounded down and not below zero - the units of fb_budget.  FB_ERR_INVALID_ARG unless
 * bytes_large > bytes_small and t_large_ns > t_small_ns.
 * fb_calibrate_exchange takes the two timings itself: it exchanges two slot images of
 * bytes_small and of bytes_large bytes (slot_weights: device buffer of 2 * bytes_large
 * bytes, 16-byte aligned; its contents are not preserved),
 * reps times each after two warm-up runs, keeps the fastest, and fits.  Blocking (it waits
 * for its own events); allocates no device memory.  Runs on the device that holds
 * slot_weights, whichever device is current (so does fb_apply_swaps).
 * t_small_ns_out / t_large_ns_out (optional) receive the two timings. */
fb_status fb_fit_cost_model(uint64_t t_small_ns, uint64_t t_large_ns, uint64_t bytes_small, uint64_t bytes_large,
                            uint64_t* alpha_ns, uint64_t* fs_per_byte);
fb_status fb_calibrate_exchange(void* slot_weights, uint64_t bytes_small, uint64_t bytes_large, int32_t reps,
                                uint64_t* alpha_ns, uint64_t* fs_per_byte, uint64_t* t_small_ns_out,
                                uint64_t* t_large_ns_out, fb_stream stream);

/* The same exchange issued from the host as device-to-device copies, the way a serving engine
 * moves expert weights between ranks: the plan (n_swaps, swaps) and the placement before the
 * plan are copied to the host on plan_stream, the call WAITS for that stream, and then
 * enqueues, for every swap, the pairwise exchange through a staging buffer of at most
 * staging_bytes (0 = one whole expert) on copy_stream: stage <- A, A <- B, B <- stage, piece
 * by piece.  No kernel of the library runs, so the transfer does not compete for SMs with the
 * attention kernels it is meant to hide behind.  Returns after the copies are enqueued; the
 * staging buffer (owned by ctx, grown on demand) and a small pinned host buffer are allocated
 * on first use.  Traffic: 6 * expert_bytes per swap.  Errors: FB_ERR_RANGE /
 * FB_ERR_BAD_PLACEMENT for a swap or placement out of range (copies of earlier swaps may
 * already be enqueued), FB_ERR_CUDA. */
fb_status fb_apply_swaps_staged(fb_ctx* ctx, void* slot_weights, uint64_t expert_bytes, const int32_t* expert_to_slot,
                                const fb_swap* swaps, const int32_t* n_swaps, int32_t max_swaps,
                                uint64_t staging_bytes, fb_stream plan_stream, fb_stream copy_stream);

/* ---- prediction-quality metrics (Evaluation, "Metrics"); not part of the per-layer hot path ---- */
#define FB_DTYPE_BF16 0
#define FB_DTYPE_F32 1
/* Mean over the rows (tokens) of the cosine similarity between row i of a and row i of b:
 * the paper's hidden-state cosine (a = h_prev, b = H, bf16 [rows][n]) and logit cosine
 * (a, b = the two router invocations' logits, f32 [rows][n], as dumped by fb_predict_load
 * and fb_route_dispatch).  A row that is zero on either side contributes 0.  All pointers
 * are device pointers; row_scratch (double[rows]) receives the per-row cosines, mean_out
 * (one double) their mean; sums are formed in double precision in a fixed order.  rows = 0
 * gives 0.  Errors: FB_ERR_INVALID_ARG for a bad size, dtype or NULL pointer. */
fb_status fb_row_cosine_mean(const void* a, const void* b, int64_t rows, int32_t n, int32_t dtype,
                             double* row_scratch, double* mean_out, fb_stream stream);
/* Numerator of the top-k hit rate: the number of (token, expert) assignments of ids_b
 * ([T][k], the normal pass) that also appear in ids_a ([T][k], the early pass); the hit
 * rate is that number / (T k).  Device pointers; hits_out is one uint32. */
fb_status fb_topk_hits(const int32_t* ids_a, const int32_t* ids_b, int32_t T, int32_t k, uint32_t* hits_out,
                       fb_stream stream);

/* Limit on the SM pairs the router kernel may occupy (0 = no limit, the default).  The
 * prediction pass is meant to run beside the previous layer's attention (stage 1 of the
 * method is hidden behind it), so a caller may want to leave SMs free.  A call with more
 * 256-row tile pairs than the limit (or than fit on the GPU at once, fb_max_pairs) runs
 * the persistent kernel, where each block pair walks several tiles (on as few block pairs as
 * the resulting number of rounds needs: 128 tile pairs run on 64 block pairs, not on all 74);
 * results do not depend on the limit.  Honoured for the gate shapes that kernel supports (E a multiple of 32 up
 * to 256; sigmoid gates with 32-expert groups and topk_group <= 4, or softmax gates whose
 * weights are renormalised); other shapes ignore it.  Returns FB_ERR_INVALID_ARG for a
 * negative limit. */
fb_status fb_set_pair_limit(fb_ctx* ctx, int32_t pairs);
/* k-range split of the router kernel (on by default).  When a call has fewer 256-row tile pairs
 * than block pairs fit on the GPU (and the persistent kernel is not used), the spare pairs sum
 * the tail of every tile's k-range into partial tiles that the tiles' owners add before their
 * epilogue, so that every SM's tensor core works through the whole main loop (128 tiles leave
 * 20 of 148 SMs idle otherwise; the smaller shapes leave more than half).  The schedule is a
 * function of the shape and of the number of pairs only: a call is reproducible, but its logits
 * differ from an unsplit call's in the order of the fp32 additions (both stay within the
 * library's tolerance of the fp64 product), so a token whose k-th and (k+1)-th keys are closer
 * than that rounding may be routed differently by the two.  mode 0 switches the split off, 1 on;
 * owner_bias_kblocks tunes how many k-blocks more than an even share a tile's owner keeps
 * (-1: built-in choice).  FB_ERR_INVALID_ARG for other values. */
fb_status fb_set_split(fb_ctx* ctx, int32_t mode, int32_t owner_bias_kblocks);
/* Block pairs of the persistent router kernel that fit on the GPU at once (0 when the
 * configuration does not support that kernel). */
int32_t fb_max_pairs(const fb_ctx* ctx);
/* Text for a status code; never NULL. */
const char* fb_status_string(fb_status s);

#ifdef __cplusplus
}
#endif
#endif  /* FREEBALANCE_H_ */
