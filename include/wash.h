/*
 * wash.h -- C ABI of the B200 WASH population library (libwash.so).
 *
 * A population is N copies of one model, held on one GPU as a "stack": every model's
 * learnable tensors laid end to end in a row of padded_P elements (each tensor starts
 * on a multiple of 8 elements), the N rows stored either model-major, [N][padded_P],
 * or coordinate-major, [padded_P][N].  The library runs, in hand-written sm_100a
 * kernels, the population operators of the WASH paper (Fournier et al., "WASH: Train
 * your Ensemble with Communication-Efficient Weight Shuffling, then Average"):
 *
 *   wash_shuffle / _opt_state / _both   the shuffling step, Eq. 3 and Algorithm 1
 *   papa_ema                            PAPA's pull toward the consensus, Eq. 1
 *   population_average                  the averaged model, output of Algorithm 1
 *   papa_all                            PAPA-all / DART: every model := the average
 *   wash_consensus_sq                   squared distances to the consensus (Fig. 2)
 *
 * Conventions common to all calls
 *   - Every function returns a wash_status (0 = success, negative = error) and never
 *     throws, aborts or traps.  wash_last_error() gives a message for the last failure
 *     of the calling thread.
 *   - Pointers are HOST pointers unless the comment says DEVICE.  Stacks are DEVICE
 *     memory BORROWED from the caller: the library never frees, moves or resizes
 *     them.  The context owns only its small tables.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Kernel
 *     launches are asynchronous on it; argument errors are reported before any launch.
 *     Calls on one context must be issued on one stream at a time (the context's
 *     tables are rewritten in stream order when the probabilities change).
 *   - Randomness is a pure function of (seed, step, tensor index, coordinate index)
 *     through Philox4x32-10, so a result does not depend on layout, dtype, grid size,
 *     kernel variant, or on which of the shuffle entry points produced it.
 *   - Padding elements of a row are not coordinates: no call reads them into a result
 *     or writes them.
 */
#ifndef WASH_H_
#define WASH_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct wash_ctx wash_ctx; /* opaque; made by wash_create*, released by wash_destroy */

enum wash_status {
    WASH_OK = 0,
    WASH_ERR_ARG = -1,         /* invalid argument (range, NULL, NaN, size mismatch)      */
    WASH_ERR_STATE = -2,       /* call not valid now (e.g. stack not bound)               */
    WASH_ERR_ALLOC = -3,       /* host or device allocation failed                        */
    WASH_ERR_CUDA = -4,        /* a CUDA runtime call or a launch failed                  */
    WASH_ERR_UNSUPPORTED = -5, /* valid request the library has no kernel for             */
    WASH_ERR_DEVICE_CHECK = -6 /* a device-side consistency check tripped (wash_check)    */
};
enum wash_layout { WASH_LAYOUT_NP = 0 /* [N][padded_P] */, WASH_LAYOUT_PN = 1 /* [padded_P][N] */ };
enum wash_dtype { WASH_F32 = 0, WASH_BF16 = 1 };
enum wash_stack { WASH_STACK_PARAMS = 0, WASH_STACK_OPT = 1 };
enum wash_schedule { WASH_SCHEDULE_DECREASING = 0, WASH_SCHEDULE_CONSTANT = 1, WASH_SCHEDULE_INCREASING = 2 };
enum wash_mode {
    WASH_MODE_STREAM = 0, /* one pass that reads the whole stack and writes the selected
                             coordinates; the stack travels global -> shared memory by
                             per-thread asynchronous copies (cp.async).  Default.            */
    WASH_MODE_SPARSE = 1, /* draws the mask first; touches only selected coordinates          */
    WASH_MODE_AUTO = 2             /* SPARSE when the call's probabilities select, in expectation,
                                      less than a share of the coordinates that depends on layout
                                      and N, else STREAM.  [N][padded_P]: max(3 %, 35 % / N);
                                      [padded_P][N]: 30 % up to N = 8, 10 % above (the measured
                                      crossovers on B200: in the second layout the N values of a
                                      coordinate share a DRAM access; a small population leaves
                                      the streaming kernel bound by issue slots)                 */
};

#define WASH_MAX_N 64            /* largest population                                     */
#define WASH_ALIGN_ELEMS 8       /* tensors start on a multiple of this many elements      */

/* Counters a shuffle ADDS to (Table 1's "communication volume", measured):
 *   selected_coords  coordinates that drew "shuffle" (each stands for N values routed
 *                    through a permutation);
 *   moved_values     among those, values whose model index changed, i.e. the sum over
 *                    selected i of #{n : pi_i(n) != n}.
 * Counted once per coordinate, whether one stack or two were shuffled. */
typedef struct {
    uint64_t selected_coords;
    uint64_t moved_values;
} wash_stats;

/* ---- context ------------------------------------------------------------------- */

/* Describe a population of N models (2 <= N <= WASH_MAX_N) made of n_tensors tensors,
 * tensor t holding numel[t] coordinates (0 < numel[t] < 2^32); the tensor's index t
 * is what the paper's Algorithm 1 calls the layer l when per-layer probabilities are
 * given.  `device` is the CUDA device ordinal that owns the stacks.  On success *out
 * is a new context.  Errors: WASH_ERR_ARG, WASH_ERR_ALLOC, WASH_ERR_CUDA. */
int wash_create(wash_ctx **out, int32_t N, int32_t n_tensors, const int64_t *numel,
                int32_t layout, int32_t device);

/* As wash_create, for a SHARD of a larger population: segment s holds numel[s]
 * coordinates that are coordinates coord_begin[s] .. coord_begin[s]+numel[s]-1 of the
 * global tensor tensor_id[s].  Because the random draws are keyed by the global
 * (tensor, coordinate), shards processed on different GPUs reproduce the unsharded
 * result exactly and need no communication.  coord_begin[s] must be a multiple of 4
 * and coord_begin[s] + numel[s] <= 2^32.  tensor_id / coord_begin may be NULL
 * (meaning s and 0). */
int wash_create_segments(wash_ctx **out, int32_t N, int32_t n_segments, const int64_t *numel,
                         const uint32_t *tensor_id, const int64_t *coord_begin,
                         int32_t layout, int32_t device);

/* Release the context's tables.  Bound stacks are the caller's and are left alone. */
int wash_destroy(wash_ctx *ctx);

/* Row geometry: *padded_P = elements per model row; offsets[t] (array of n_tensors,
 * may be NULL) = element offset of tensor t inside a row.  A stack is N * padded_P
 * elements; element (n, e) lives at n*padded_P + e (WASH_LAYOUT_NP) or e*N + n
 * (WASH_LAYOUT_PN). */
int wash_stack_elems(const wash_ctx *ctx, int64_t *padded_P, int64_t *offsets);

/* Lend a DEVICE buffer of n_elems == N * padded_P elements of `dtype` to the context
 * as its parameter stack or optimizer-state stack.  The pointer must be 16-byte
 * aligned.  Passing dev_ptr == NULL unbinds. */
int wash_bind(wash_ctx *ctx, int32_t stack, int32_t dtype, void *dev_ptr, int64_t n_elems);

/* Which kernel family the shuffle entry points launch (default WASH_MODE_STREAM).
 * Results are bit-identical across modes. */
int wash_set_mode(wash_ctx *ctx, int32_t mode);

/* Launch shape override for tuning: threads per block (multiple of 32 in 32..256;
 * 0 = each kernel's default) and grid style: blocks_per_sm == 0 each kernel's default,
 * > 0 a persistent grid of SM count x min(blocks_per_sm, resident blocks per SM) blocks
 * that stride over the groups, < 0 one group of 4 coordinates per thread.  For
 * WASH_MODE_STREAM blocks_per_sm = 1 or 2 fixes the number of groups a thread takes
 * (default: 2 when a group of all models is at most 64 bytes, else 1); blocks_per_sm = -2 / -3
 * forces the streaming kernel's lean / early flavour (early draws the permutations while the
 * stack's copies are in flight and serves populations of more than 16 models densely; by
 * default it is launched for N > 16 when the call's probabilities select 30 % or more);
 * blocks_per_sm = -4 / -5 forces / excludes the streaming kernel for small groups (a
 * resident grid of warps walking tiles through two shared-memory stages; by default
 * it is launched when a group of all models of both stacks is at most 48 bytes and the
 * call's probabilities select at most 30 %, and for groups of up to 64 bytes when they
 * select between 0.7 % and 5 %; it ignores `threads`).  Results do not
 * depend on any of this. */
int wash_set_launch(wash_ctx *ctx, int32_t threads, int32_t blocks_per_sm);

/* ---- the shuffling step ----------------------------------------------------------- */

/* Layer-wise probabilities (section "Layer-wise adaptation via WASH"): writes out[l],
 * l = 0..L-1, as p*(1 - l/(L-1)) (DECREASING, the paper's schedule: first layer p,
 * last layer never shuffled), p (CONSTANT) or p*l/(L-1) (INCREASING; the two variants
 * of Table 4).  L == 1 gives out[0] = p.  Host-only helper. */
int wash_layer_probs(int32_t L, double p, int32_t schedule, double *out);

/* One shuffling step on the parameter stack (Eq. 3; Algorithm 1, "Shuffling step").
 * Every coordinate i of tensor t is selected with probability p_layer[t] (or p when
 * p_layer is NULL; probabilities in [0,1]; realised as word < floor(p*2^32) on a
 * 32-bit Philox word), one draw per coordinate shared by all models; for a selected
 * coordinate a permutation pi_i, uniform over the N! permutations, is drawn and the N
 * values are rearranged in place as new[n] = old[pi_i(n)], as raw bits.  Unselected
 * coordinates are not written.
 *   step   < 2^56, the training step; seed: any 64-bit value.
 *   stats  DEVICE-accessible pointer (device memory or mapped pinned host memory) to a
 *          wash_stats the kernel atomically adds to; may be NULL.
 * Errors: WASH_ERR_ARG (p out of range / NaN, step too large), WASH_ERR_STATE (stack
 * not bound), WASH_ERR_UNSUPPORTED, WASH_ERR_CUDA. */
int wash_shuffle(wash_ctx *ctx, uint64_t step, double p, const double *p_layer,
                 uint64_t seed, void *stream, wash_stats *stats);

/* The same step applied to the optimizer-state stack (WASH+Opt, section "Training
 * methods"): with equal (seed, step, p) it selects the same coordinates and applies
 * the same permutations as wash_shuffle, so the momentum follows its parameter. */
int wash_shuffle_opt_state(wash_ctx *ctx, uint64_t step, double p, const double *p_layer,
                           uint64_t seed, void *stream, wash_stats *stats);

/* Both stacks in one launch; equal to wash_shuffle followed by wash_shuffle_opt_state
 * with the same arguments, with the draws made once. */
int wash_shuffle_both(wash_ctx *ctx, uint64_t step, double p, const double *p_layer,
                      uint64_t seed, void *stream, wash_stats *stats);

/* The shuffling step with the distance to the consensus gathered in the same pass.
 * The streaming shuffle already brings every coordinate's N values on chip; this call
 * also sums, per model and per range of tensors, the squared deviation from the mean over
 * the models (the quantity of Eq. 2 and Eq. 5; Fig. 2 plots its square root averaged over
 * models, Fig. 4 the same per quarter of the parameters) -- no second read of the stack.
 * The values are those before the exchange; by Eq. 5 the exchange leaves the total over the
 * models unchanged.
 *   stacks         WASH_STACK_PARAMS, WASH_STACK_OPT or WASH_STACK_BOTH: what is shuffled
 *                  (as wash_shuffle / wash_shuffle_opt_state / wash_shuffle_both); the
 *                  statistic is taken on the first of them (the parameters unless only the
 *                  optimizer state is shuffled);
 *   n_ranges       1 .. WASH_MAX_CONSENSUS_RANGES;
 *   tensor_bounds  HOST array of n_ranges + 1 ascending tensor indices in [0, n_tensors]:
 *                  range r covers tensors tensor_bounds[r] .. tensor_bounds[r+1]-1 (tensors
 *                  outside every range are shuffled but not measured);
 *   dev_sq_out     DEVICE array [n_ranges][N] of doubles the caller has zeroed:
 *                  dev_sq_out[r][n] += sum over the range's coordinates of
 *                  (x_n^i - mean^i)^2, in binary64 (sums arrive through atomics, so the
 *                  last bits depend on their order).
 * Always runs the streaming kernel, whatever wash_set_mode says.  Other arguments, errors
 * and the bits of the stacks: as wash_shuffle. */
#define WASH_STACK_BOTH 2
#define WASH_MAX_CONSENSUS_RANGES 8
int wash_shuffle_consensus(wash_ctx *ctx, int32_t stacks, uint64_t step, double p, const double *p_layer,
                           uint64_t seed, void *stream, wash_stats *stats, int32_t n_ranges,
                           const int32_t *tensor_bounds, double *dev_sq_out);

/* ---- comparison operators --------------------------------------------------------- */

/* PAPA's EMA (Eq. 1), in place on the chosen stack, 0 < alpha < 1:
 *     m = (((x_0 + x_1) + x_2) + ... + x_{N-1}) / N ;  x_n <- alpha*x_n + (1-alpha)*m
 * evaluated in binary32 with every operation rounded to nearest even once (no fused
 * multiply-add), terms added in the order n = 0..N-1.  bf16 stacks are widened,
 * computed in binary32 and rounded back to nearest even. */
int papa_ema(wash_ctx *ctx, int32_t stack, float alpha, void *stream);

/* The averaged model (output of Algorithm 1): dev_out[e] = m as defined above for
 * every coordinate; dev_out is a DEVICE row of padded_P elements of out_dtype
 * (16-byte aligned), laid out like one model's row; its padding is not written. */
int population_average(wash_ctx *ctx, int32_t stack, void *dev_out, int32_t out_dtype, void *stream);

/* PAPA-all / DART step (section "Reducing distance to consensus"): every model's
 * coordinates are overwritten by m. */
int papa_all(wash_ctx *ctx, int32_t stack, void *stream);

/* Squared distance of every model to the consensus (the quantity of Eq. 2 and Eq. 5,
 * whose square root averaged over models is plotted in Fig. 2), over tensors
 * [tensor_lo, tensor_hi):  dev_sq_out[n] += sum_i (x_n^i - mean^i)^2, accumulated in
 * binary64.  dev_sq_out is a DEVICE array of N doubles the caller has zeroed. */
int wash_consensus_sq(wash_ctx *ctx, int32_t stack, int32_t tensor_lo, int32_t tensor_hi,
                      double *dev_sq_out, void *stream);

/* ---- whole step over HOST buffers ------------------------------------------------- */

enum wash_step_ops { WASH_OP_SHUFFLE = 1, WASH_OP_EMA = 2, WASH_OP_AVERAGE = 4 };

/* One pass of the selected operators over stacks that live in HOST memory (pinned
 * memory makes the copies asynchronous): copies host_params (and host_opt, if not
 * NULL) into the bound device stacks, runs, in this order, the shuffle (both stacks
 * when host_opt is given), papa_ema on the parameters and population_average, copies
 * the stacks back to the same host buffers and the average (row of padded_P elements
 * of the parameter dtype) to host_avg (may be NULL unless WASH_OP_AVERAGE), and waits
 * for the stream.  host_stats (may be NULL) receives this call's counters.  The
 * device stacks must be bound; they serve as staging and hold the results too.
 * Populations of 2^20 coordinates per model and more are processed in eight coordinate
 * ranges on two internal copy streams, so that the copy in of one range, the kernels on
 * the previous one and the copy out of the one before overlap; the result is the same. */
int wash_step_host(wash_ctx *ctx, int32_t ops, void *host_params, void *host_opt, void *host_avg,
                   uint64_t step, double p, const double *p_layer, uint64_t seed, float alpha,
                   void *stream, wash_stats *host_stats);

/* ---- one model per device ----------------------------------------------------------
 *
 * The deployment the paper describes (Introduction: a permutation is drawn and models
 * communicate their parameters peer to peer following it; section "WASH": each model
 * communicates p*d parameters per step in expectation): worker n holds model n only.
 * Every worker derives the same mask and the same permutations from the shared
 * (seed, step), so nothing but values crosses the link, and in a fixed order that needs
 * no indices:
 *
 *   worker n owns a STAGING buffer.  The selected coordinates with pi_i(n) != n, taken
 *   in the order of Algorithm 1's shuffling loop (tensor by tensor, coordinate by
 *   coordinate), occupy its slots 0, 1, 2, ...; the slot of coordinate i is filled by
 *   worker pi_i(n) with its own value of i (Eq. 3 read as a gather).  Fixed points of
 *   pi_i do not travel.
 *
 * A step is  wash_exchange_plan  ->  wash_exchange_send  ->  (all workers have sent)  ->
 * wash_exchange_receive  on every worker; the result equals wash_shuffle (or
 * wash_shuffle_both when both rows are bound) on the stacked population, bit for bit.
 * The library performs no inter-device synchronisation: between send and receive the
 * caller orders the workers (a barrier of the process group enqueued on the same
 * stream, or stream/event order when one process drives several workers).
 * Two staging sets (parity 0 and 1) may be registered; a step uses set (step & 1) if it
 * is registered, else set 0.  With both registered one barrier per step suffices (a
 * worker can start sending step s+1 while a slower peer still reads step s's set).
 *
 * The context is created with wash_create / wash_create_segments as usual (N = size of
 * the population, the tensor table of ONE model; layout is ignored).  Rows of 2^32 and
 * more elements are not supported in this form (WASH_ERR_UNSUPPORTED). */

/* Declares this context worker `self` (0 <= self < N) and borrows the worker's model:
 * dev_row is a DEVICE row of padded_P elements (n_elems must say so) of `dtype`, 16-byte
 * aligned, for `stack` (WASH_STACK_PARAMS, or WASH_STACK_OPT for the optimizer state,
 * which then follows the same mask and permutations).  NULL unbinds.  The first call
 * allocates the plan's tables (about padded_P/4 bytes + 4 (N+1) padded_P/4096 bytes). */
int wash_exchange_bind(wash_ctx *ctx, int32_t self, int32_t stack, int32_t dtype, void *dev_row, int64_t n_elems);

/* Registers staging set `parity` (0 or 1) of `stack`: buffers is a HOST array of N
 * pointers, entry n = worker n's staging buffer for this stack, each holding
 * capacity_elems elements of the stack's dtype, 4-byte aligned, and accessible from this
 * device (entry `self` is this worker's own buffer; the others are peer mappings, or
 * plain device buffers when one process emulates all workers).  The pointers are copied;
 * the buffers stay the caller's.  A step that needs more slots than capacity_elems writes
 * and reads nothing beyond the buffers and makes wash_check fail. */
int wash_exchange_staging(wash_ctx *ctx, int32_t stack, int32_t parity, void *const *buffers, int64_t capacity_elems);

/* The same registration for workers that live in different processes (one per GPU).
 * wash_exchange_staging_create allocates this worker's buffer of set `parity` for `stack`
 * (the row must be bound; capacity_elems elements of its dtype; owned and freed by the
 * context) and writes its inter-process handle, WASH_IPC_HANDLE_BYTES bytes, to the HOST
 * buffer handle_out.  The processes exchange the handles (any host channel) and every
 * worker passes all N of them, in worker order, to wash_exchange_staging_open, which maps
 * the peers' buffers into this process (entry `self` is ignored; peer access over NVLink
 * is enabled as needed) and registers the set.  All workers must use one capacity.
 * The mappings are closed by wash_destroy: destroy every context of the group only after
 * all workers have finished their last step. */
#define WASH_IPC_HANDLE_BYTES 64
int wash_exchange_staging_create(wash_ctx *ctx, int32_t stack, int32_t parity, int64_t capacity_elems, void *handle_out);
int wash_exchange_staging_open(wash_ctx *ctx, int32_t stack, int32_t parity, const void *handles);

/* Draws the step: mask, permutations, and the slot offsets of every worker's buffer.
 * Reads no model data.  step, p, p_layer, seed as for wash_shuffle; every worker must
 * pass the same values. */
int wash_exchange_plan(wash_ctx *ctx, uint64_t step, double p, const double *p_layer, uint64_t seed, void *stream);

/* Stores this worker's values into the other workers' staging buffers, for every bound
 * stack, according to the last plan. */
int wash_exchange_send(wash_ctx *ctx, void *stream);

/* Copies this worker's slots from its own staging buffer into its model, for every bound
 * stack.  stats (DEVICE-accessible, may be NULL): selected_coords += coordinates selected
 * in the step (the same on every worker), moved_values += values this worker received
 * (summed over workers: wash_shuffle's moved_values). */
int wash_exchange_receive(wash_ctx *ctx, void *stream, wash_stats *stats);

/* Waits for `stream` and reports the last plan: host_need[n] (HOST array of N, may be
 * NULL) = slots worker n's buffer needs, *host_selected (may be NULL) = selected
 * coordinates. */
int wash_exchange_counts(wash_ctx *ctx, uint64_t *host_need, uint64_t *host_selected, void *stream);

/* ---- for callers that must not allocate ------------------------------------------- */

#define WASH_NOALLOC_MAX_TENSORS 1024                 /* most tensors per model            */
#define WASH_NOALLOC_MAX_ROW_ELEMS (1ll << 26)        /* longest padded row, in elements   */

/* The paper has no counterpart to this call; it exists for deployment reasons only.
 *
 * wash_create puts the context's lookup tables in device memory with cudaMalloc.  Two
 * kinds of caller cannot afford that: a process in which a framework's memory pool has
 * already taken the whole GPU (an allocation from this library would fail or compete
 * with the pool), and a loop in which cudaMalloc / cudaFree, which
 * synchronise the whole device, would stall work that other streams have in flight.
 * wash_shuffle_noalloc runs the same streaming shuffle as wash_shuffle on ONE stack
 * without any context and without allocating device or pinned memory: its tables live
 * in a fixed 296 KiB array inside the library image (32 KiB segment table, 256 KiB tile
 * index, 8 KiB of partial sums for the counters), which every GPU that loads libwash.so holds until the process exits.
 *
 *   N, n_tensors, numel, layout     as for wash_create (row geometry is the same:
 *                                   tensors start on multiples of 8 elements);
 *   dtype, dev_stack, n_elems       as for wash_bind: a DEVICE stack of N * padded_P
 *                                   elements, 16-byte aligned, borrowed for the call;
 *   step, p, p_layer, seed, stats   as for wash_shuffle (stats: DEVICE-accessible,
 *                                   added to, may be NULL);
 *   device                          ordinal of the GPU that owns dev_stack.
 *
 * Limits: n_tensors <= WASH_NOALLOC_MAX_TENSORS and padded_P <=
 * WASH_NOALLOC_MAX_ROW_ELEMS; anything larger is refused with WASH_ERR_ARG (use a
 * context instead).  The result is bit-identical to wash_shuffle with the same
 * arguments.  The message of a failure is returned by wash_noalloc_last_error().
 *
 * Sharing: all calls on a GPU use the one array.  Each call rewrites the tables it
 * needs in full and zeroes the partial sums, in stream order, so the previous call's
 * contents never leak into the next; but two calls that can overlap on
 * the GPU (different streams without an ordering between them, or two host threads)
 * race on the tables and give undefined results.  Issue them on one stream, or order
 * them with events.
 *
 * First use: the first call on each device looks up that device's address of the array
 * (cudaGetSymbolAddress, with the device made current for the duration of the call).
 * Make that first call before any stream capture begins.
 *
 * Every call uploads its two tables (up to 288 KiB) with two host-to-device copies from
 * ordinary pageable host memory, ordered on `stream`; the host arrays are freed when the
 * call returns, so a stream that is in capture mode is refused with WASH_ERR_STATE.
 *
 * Device-side checks: the kernel is given no status word, so a group that falls outside
 * the tables (which this call builds itself from numel) would be skipped without a report;
 * there is no wash_check for this entry point. */
int wash_shuffle_noalloc(int32_t N, int32_t n_tensors, const int64_t *numel, int32_t layout,
                         int32_t dtype, void *dev_stack, int64_t n_elems, uint64_t step, double p,
                         const double *p_layer, uint64_t seed, int32_t device, void *stream,
                         wash_stats *stats);

/* Message for the calling thread's most recent wash_shuffle_noalloc failure. */
const char *wash_noalloc_last_error(void);

/* ---- diagnostics ------------------------------------------------------------------ */

/* Waits for `stream` and returns WASH_ERR_DEVICE_CHECK if a kernel recorded an
 * inconsistency (an index outside its table) since the last check, else WASH_OK. */
int wash_check(wash_ctx *ctx, void *stream);

/* Message for the calling thread's most recent error (never NULL). */
const char *wash_last_error(void);

/* Integer-pipe ceiling of the shuffle's mask: a kernel that does nothing but draw
 * n_blocks Philox4x32-10 blocks (the mask of 4*n_blocks coordinates, counters as in
 * wash_shuffle for tensor 0 at step 0 with key = seed) and folds them into one word,
 * which it adds to *dev_checksum (DEVICE, uint32, caller-zeroed; may be NULL).  Timing it
 * gives the rate at which masks can be drawn when memory costs nothing, i.e. the bound
 * that takes over from HBM for small N.  A thread draws four blocks (four independent
 * chains, the form that measured fastest).  No stack is touched.  Diagnostic only. */
int wash_philox_probe(uint64_t n_blocks, uint64_t seed, uint32_t *dev_checksum, int32_t device, void *stream);

/* Number of kernels this library has launched in this process. */
uint64_t wash_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* WASH_H_ */
