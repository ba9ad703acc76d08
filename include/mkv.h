/*
 * mkv -- Moment-KV decode hot path for NVIDIA B200 (sm_100a), C ABI.
 *
 * One context holds, for `layers` attention layers and `batch` sequences, the
 * frozen prefill K/V pool, the budget-bounded decode K/V pool, one importance
 * score and one position id per decode-pool token.  mkv_decode_step() performs,
 * for one layer and all sequences, one pass of Algorithm 1 of the Moment-KV
 * paper (Sec. 4.2) minus the Q/K/V projection: append, attention over prefill U
 * decode pool, head mean, momentum update of the importance, lowest-score
 * eviction and in-place compaction.  Everything runs in CUDA kernels on the
 * caller's stream; there is no CPU fallback.
 *
 * Conventions (all entry points)
 *   - Return value: mkv_status.  No exceptions, no abort, no device trap.
 *   - "device pointer": memory of the context's GPU, owned by the caller, only
 *     read/written during the call's kernels (stream order); never retained.
 *   - "host pointer": ordinary host memory, read/written before return unless
 *     stated otherwise.
 *   - `stream` is a cudaStream_t passed as void* (NULL = legacy default stream).
 *   - The library allocates NO device memory: the caller passes one workspace of
 *     mkv_workspace_bytes() bytes, 256-byte aligned, which must outlive the
 *     context.  mkv_destroy() frees host state only.
 *   - Tensor layouts are row-major with the last index contiguous.
 *     q, out: [batch][q_heads][head_dim]; k_new, v_new: [batch][kv_heads][head_dim].
 *   - Query head h reads KV head h / (q_heads / kv_heads).
 *   - Errors found on the host are returned at once; errors found by a kernel
 *     (a count beyond capacity, a bounded wait that expired) set a sticky device
 *     status word that mkv_status_sync() reads.
 *   - One host thread at a time per context, and all calls of a context on one stream (or
 *     ordered by the caller in some other way): the layers of a context share the per-step
 *     scratch, and a step may begin while the previous kernel of its stream is still ending.
 *   - Stream capture: mkv_decode_step() and mkv_attend_only() only enqueue kernels, so a
 *     sequence of them (any number, any layers) can be recorded into a CUDA graph and replayed
 *     any number of times; step numbers, pool counts and the work-sharing state live on the
 *     device (Algorithm 1 has no host-side state).  A recording holds the pointers, the budget
 *     and the launch plan of the moment: record again after mkv_prefill*() or mkv_set_budget().
 *     mkv_prefill*(), the *_host entry points and the mkv_get_*() readers synchronise or copy
 *     from pageable memory and cannot be recorded.  mkv_launch_count() counts enqueued
 *     kernels, not replays.
 *   - The kernels are persistent: the CTAs of a launch hand work to one another and a unit's
 *     finishing part waits (bounded) for tiles that other CTAs deliver, so all CTAs of a launch
 *     must be resident at once.  mkv_create() sizes the grid from the occupancy the device
 *     reports for the kernel (SM count x resident CTAs per SM, see mkv_grid_limit()), which
 *     holds as long as the GPU's SMs are not shared with other work for the length of a step:
 *     kernels of other streams or processes that occupy SMs meanwhile can delay a step up to
 *     the wait limit (MKV_OPT_WAIT_LIMIT_US), after which it ends with MKV_ERR_TIMEOUT.
 *   - Several layers per launch: the layers of a context are independent instances of
 *     Algorithm 1, and mkv_decode_step_layers() steps a run of consecutive layers with one
 *     kernel launch (inputs stacked by layer).  Small per-layer batches fill the GPU that way.
 */
#ifndef MKV_H_
#define MKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif
#if defined(__GNUC__)
#pragma GCC visibility push(default) /* the only exported symbols of libmkv.so */
#endif

typedef struct mkv_ctx mkv_ctx; /* opaque, host-owned */

typedef enum {
    MKV_OK = 0,
    MKV_ERR_INVALID_ARG = 1,  /* NULL pointer, value out of range                     */
    MKV_ERR_BAD_STATE = 2,    /* e.g. decode step on a layer that was never prefilled */
    MKV_ERR_CAPACITY = 3,     /* prefill longer than max_prefill, budget above create */
    MKV_ERR_WORKSPACE = 4,    /* workspace too small or misaligned                    */
    MKV_ERR_UNSUPPORTED = 5,  /* shape/dtype combination without a kernel             */
    MKV_ERR_CUDA = 6,         /* a CUDA runtime call failed (no device, launch error) */
    MKV_ERR_TIMEOUT = 7,      /* device: a bounded wait inside a kernel ran out       */
    MKV_ERR_DEVICE_CHECK = 8  /* device: an internal consistency check failed         */
} mkv_status;

typedef enum { MKV_BF16 = 0, MKV_F32 = 1 } mkv_dtype;

/* Which heads Eq. 4 (Sec. 4.2, "Momentum-Based Attention Aggregation") averages. */
typedef enum {
    MKV_SCORE_GROUP_MEAN = 0, /* per KV head: mean over its G query heads; each KV head
                                 scores and evicts on its own                           */
    MKV_SCORE_LAYER_MEAN = 1  /* as printed: mean over all H heads, one score vector per
                                 (layer, sequence), all KV heads evict the same tokens  */
} mkv_score_mode;

/* Kernel family used for the attention pass. */
typedef enum {
    MKV_KERNEL_AUTO = 0, /* tensor-core path where it exists, else the scalar path      */
    MKV_KERNEL_SIMT = 1, /* scalar fp32 FMA path: every dtype / head_dim                */
    MKV_KERNEL_MMA = 2   /* bf16, head_dim 128, G <= 8: bulk-copy pipeline + mma        */
} mkv_kernel;

/* flags for mkv_create */
#define MKV_FLAG_RECORD_PROBS 1u /* keep the head-averaged decode probabilities of the last
                                    step (Eq. 4) and their position ids, for
                                    mkv_get_last_probs() and mkv_recency_diagnostics()  */
#define MKV_FLAG_INPUTS_READY 2u /* a promise by the caller: q, k_new and v_new of every
                                    mkv_decode_step*() / mkv_attend_only*() call are final in
                                    device memory when the call is made -- nothing still pending
                                    on any stream writes them.  A step may then begin its
                                    attention over the frozen prompt rows while the previous
                                    kernel of the stream (normally the previous step) is still
                                    finishing.  And a step whose layers are all different from
                                    those of the context's previous step on the same stream
                                    shares nothing with it (layers are independent instances of
                                    Algorithm 1): it runs alongside that step from its start and
                                    only its end is ordered behind it, so steps still complete
                                    in stream order.  Such neighbours must therefore be given
                                    different `out` buffers.  Without the flag a step reads q
                                    only after every earlier kernel of the stream has completed.
                                    (The *_host entry points ignore the flag.)               */
#define MKV_FLAG_REPRODUCIBLE 4u /* same inputs, same bits: work is split among the CTAs by a
                                    fixed table instead of run-time counters and partial results
                                    are combined in a fixed order.  Costs some load balance;
                                    meant for debugging and for race hunting (two runs must
                                    agree bit for bit).  Without it `out` and the scores can
                                    differ in their last bits from run to run.               */

/* options for mkv_set_option */
typedef enum {
    MKV_OPT_RING_STAGES = 1,   /* tensor-core kernel: stages of its shared-memory ring, 2..6
                                  (default 3; 32 KB each).  The grid is re-sized from the
                                  occupancy that results (4 or more stages leave room for one
                                  CTA per SM instead of two).  Layers must be prefilled again. */
    MKV_OPT_HEAD_TILES = 2,    /* 64-row prompt tiles a CTA owns outright where it starts, 0..16
                                  (default 3): they are fetched, and with MKV_FLAG_INPUTS_READY
                                  also attended, before the previous step has ended.  Layers
                                  must be prefilled again.                                    */
    MKV_OPT_WAIT_LIMIT_US = 3, /* limit of every wait inside a kernel, microseconds
                                  (default 2,000,000); on expiry the step ends early and the
                                  sticky status becomes MKV_ERR_TIMEOUT                       */
    MKV_OPT_OVERLAP = 4,       /* 1 (default): consecutive steps on a stream overlap their
                                  start-up with the previous step's end (programmatic
                                  dependent launch); 0: plain stream order                    */
    MKV_OPT_GRID_SHARE = 5     /* percent (10..100) of the CTAs the GPU can keep resident that a
                                  single-layer step uses.  Default 100, and 75 with
                                  MKV_FLAG_INPUTS_READY: steps of different layers then run side
                                  by side, and a step that leaves a quarter of the CTA slots
                                  free lets its successor begin streaming at once instead of
                                  waiting for slots.  A context with that flag whose steps all
                                  go to the same layer should set 100.  Steps over several
                                  layers always use all slots.  Layers must be prefilled again. */
} mkv_option;

/*
 * Size in bytes of the workspace mkv_create() needs for these parameters
 * (0 if the parameters are invalid).  Pure host arithmetic.  Per cached token and
 * layer it accounts 2 * kv_heads * head_dim * sizeof(element) bytes (K and V), the
 * figure Sec. 1 of the paper quotes as 128 KB per token for Llama-3.1-8B at 16 bit.
 */
size_t mkv_workspace_bytes(int layers, int batch, int q_heads, int kv_heads, int head_dim,
                           int budget, int max_prefill, int kv_dtype, int score_mode);

/*
 * The start table mkv_prefill() builds for the kernels, as pure host arithmetic (for
 * inspection and tests).  The rows of a (sequence, KV head) unit form 64-row tiles, prefill
 * tiles first; CTAs are spread over the units in proportion to the units' tile counts and
 * each owns up to head_tiles reserved prefill tiles where it starts, the rest being handed out by
 * per-unit counters at run time, unit_chunk tiles per pull.  At most 32 CTAs start in one
 * unit (the grid shrinks when few, long units would draw more), and a unit's chunk is sized so
 * that the CTAs starting there plus the pulls of its counter stay within the 64 partial results
 * a unit has room for.
 *   prefill_lens    host, [batch]
 *   n_ctas_max      upper bound of the grid (1..2048)
 *   n_ctas          host out: CTAs used
 *   head_tiles      tiles a CTA reserves where it starts (0..16; the library's default is 3)
 *   cta_unit0/head0/headn   host out, [n_ctas_max]: unit a CTA starts in, its first reserved
 *                   tile there, and how many tiles it has reserved (0 or head_tiles)
 *   unit_next0      host out, [batch*kv_heads]: reserved tiles per unit = start value of the
 *                   unit's counter
 *   unit_chunk      host out, [batch*kv_heads]: tiles per pull of the unit's counter (>= 2)
 */
mkv_status mkv_plan_starts(int batch, int kv_heads, int budget, const int32_t* prefill_lens, int n_ctas_max,
                           int head_tiles, int32_t* n_ctas, int32_t* cta_unit0, int32_t* cta_head0,
                           int32_t* cta_headn, int32_t* unit_next0, int32_t* unit_chunk);

/*
 * The table of the reproducible mode (MKV_FLAG_REPRODUCIBLE), as pure host arithmetic: the
 * units' tiles (a full decode pool assumed) form one global sequence, which is cut into n_ctas
 * contiguous ranges of near-equal length; CTA c covers tiles [cta_t0[c], cta_t0[c+1]) and its
 * partial result for a unit goes to slot c - unit_cta0[unit].
 *   cta_t0      host out, [n_ctas_max + 1];  tile_begin  host out, [batch*kv_heads + 1]
 *   unit_cta0   host out, [batch*kv_heads]: first CTA whose range reaches into the unit
 */
mkv_status mkv_plan_ranges(int batch, int kv_heads, int budget, const int32_t* prefill_lens, int n_ctas_max,
                           int32_t* n_ctas, int32_t* cta_t0, int32_t* tile_begin, int32_t* unit_cta0);

/*
 * Upper bound of a launch's grid: sm_count x min(resident_per_sm, wanted_per_sm), at most 2048;
 * 0 when the kernel does not fit an SM at all (resident_per_sm < 1).  resident_per_sm is what
 * the CUDA occupancy query reports for the kernel with its shared memory; wanted_per_sm is the
 * design point (2 for the tensor-core kernel, 8 for the scalar one).  Pure host arithmetic;
 * mkv_create() and MKV_OPT_RING_STAGES use it and fail with MKV_ERR_UNSUPPORTED on 0.
 */
int mkv_grid_limit(int sm_count, int resident_per_sm, int wanted_per_sm);

/* K+V bytes one cached token occupies over all layers (the paper's 128 KB/token). */
size_t mkv_kv_bytes_per_token(int layers, int kv_heads, int head_dim, int kv_dtype);

/*
 * Create a context (Algorithm 1 "Require": decoding budget B_d = `budget`, momentum
 * factor alpha = `beta`).
 *   layers, batch            >= 1
 *   q_heads % kv_heads == 0; G = q_heads / kv_heads <= 8
 *   head_dim                 64 or 128
 *   budget                   >= 1; also the largest budget mkv_set_budget accepts
 *   beta                     in [0, 1]  (paper: (0,1); 0 and 1 are the limits)
 *   max_prefill              >= 0, longest prompt any sequence may have
 *   kv_dtype                 element type of the cache and of q, k_new, v_new
 *   out_dtype                element type of `out` (MKV_F32 allowed with a bf16 cache)
 *   score_mode, kernel, flags  see the enums above
 *   workspace                device pointer, 256-byte aligned, >= mkv_workspace_bytes();
 *                            its first use zero-fills it on `device`'s legacy stream
 *   device                   CUDA device ordinal
 *   out_ctx                  host pointer receiving the context
 * Errors: INVALID_ARG, UNSUPPORTED (kernel family cannot do this shape, or its CTAs do not
 * fit the device), WORKSPACE, CUDA.
 */
mkv_status mkv_create(int layers, int q_heads, int kv_heads, int head_dim, int budget, float beta,
                      int batch, int max_prefill, int kv_dtype, int out_dtype, int score_mode,
                      int kernel, unsigned flags, void* workspace, size_t workspace_bytes,
                      int device, mkv_ctx** out_ctx);

/* Frees host state.  The workspace stays with the caller.  NULL is ignored. */
void mkv_destroy(mkv_ctx* ctx);

/*
 * Change one of the mkv_option settings.  Options that shape the launch plan put every layer
 * back to "not prefilled".  Errors: INVALID_ARG (unknown option, value out of range),
 * UNSUPPORTED (option of the other kernel family; ring that does not fit), CUDA.
 */
mkv_status mkv_set_option(mkv_ctx* ctx, int option, long long value);

/*
 * Prefill phase (Sec. 4.1): store the prompt's K_P, V_P of one layer in the frozen
 * prefill pool and empty that layer's decode pool (scores, positions, step counter).
 *   K, V          device pointers, [batch][kv_heads][src_rows][head_dim], kv_dtype
 *   prefill_lens  host pointer, [batch]; sequence b uses rows [0, prefill_lens[b])
 *   src_rows      row count of the source arrays' third index (>= every length)
 * Asynchronous on `stream`.  Errors: INVALID_ARG, CAPACITY (a length > max_prefill), CUDA.
 */
mkv_status mkv_prefill(mkv_ctx* ctx, int layer, const void* K, const void* V,
                       const int32_t* prefill_lens, int src_rows, void* stream);

/*
 * The same with one prompt length per (sequence, KV head) unit: the shape of a frozen pool
 * that a per-head prefill compressor (SnapKV- or PyramidKV-like; Sec. 6.3 of the paper runs
 * Moment-KV on top of such pools) has already thinned out.  The compressors themselves are
 * not part of this library: K and V hold, for unit (b, g), its retained rows first.
 *   unit_lens     host pointer, [batch * kv_heads]; unit (b, g) uses rows [0, unit_lens[b*kv_heads+g])
 * Errors as mkv_prefill; UNSUPPORTED with MKV_SCORE_LAYER_MEAN and several KV heads unless
 * the KV heads of a sequence have equal lengths.
 */
mkv_status mkv_prefill_units(mkv_ctx* ctx, int layer, const void* K, const void* V,
                             const int32_t* unit_lens, int src_rows, void* stream);

/*
 * One decode step of Algorithm 1 for one layer, all sequences:
 *   append (k_new, v_new) with importance 0; attention of q over prefill U decode pool
 *   (Eq. 2), fresh token included; per decode token the head-averaged probability
 *   (Eq. 4); I <- beta * I + abar (Eq. 5); if the pool holds more than `budget` tokens,
 *   remove the overflow-many lowest-I tokens (Eq. 7-9; ties: smaller position id first)
 *   and close the holes.  `out` is the attention output over the pool BEFORE eviction.
 *   q, k_new, v_new   device pointers, kv_dtype;  out  device pointer, out_dtype
 * Asynchronous, no allocation, no host synchronisation.
 * Errors: INVALID_ARG, BAD_STATE (layer not prefilled), CUDA.
 */
mkv_status mkv_decode_step(mkv_ctx* ctx, int layer, const void* q, const void* k_new,
                           const void* v_new, void* out, void* stream);

/*
 * The same step for layers [layer0, layer0 + n_layers) with ONE kernel launch: Algorithm 1 runs
 * per layer and the layers' inputs are independent, so their (sequence, KV head) units simply
 * share the grid.  Meant for small per-layer batches, where one layer alone cannot fill the GPU.
 *   q, out            device pointers, [n_layers][batch][q_heads][head_dim]
 *   k_new, v_new      device pointers, [n_layers][batch][kv_heads][head_dim]
 * Every layer of the range must have been prefilled.  The first call for a range (and the first
 * after one of its layers was prefilled again) builds the range's launch plan with copies on
 * `stream`: make it outside stream capture.  Calls for single layers and for ranges may be
 * mixed freely.  Errors: INVALID_ARG, BAD_STATE, CUDA.
 */
mkv_status mkv_decode_step_layers(mkv_ctx* ctx, int layer0, int n_layers, const void* q, const void* k_new,
                                  const void* v_new, void* out, void* stream);

/* mkv_attend_only for a run of layers with one launch; q and out as in mkv_decode_step_layers. */
mkv_status mkv_attend_only_layers(mkv_ctx* ctx, int layer0, int n_layers, const void* q, void* out,
                                  void* stream);

/*
 * Same step with HOST buffers: copies q, k_new, v_new to the device, runs the step,
 * copies `out` back; all on `stream`, asynchronous when the host buffers are pinned
 * (the caller synchronises the stream before reading `out` or reusing the inputs).  When
 * q, k_new and v_new lie back to back in host memory they travel as one copy.  Pinned,
 * 16-byte aligned host buffers are reached by the GPU in place: the inputs are fetched by a
 * small kernel ahead of the step and `out` is written by the step's kernel itself, instead
 * of copy operations before and after it; pageable buffers take staged copies.  Either way
 * `out` is complete once the stream has been synchronised.  Whether a host buffer is pinned is
 * looked up once per (address, size) and remembered until mkv_reset() or mkv_destroy(): do not
 * unpin a buffer and hand the same address to the same context again as pageable memory.
 */
mkv_status mkv_decode_step_host(mkv_ctx* ctx, int layer, const void* q_host, const void* k_new_host,
                                const void* v_new_host, void* out_host, void* stream);

/*
 * Plain decode attention (Eq. 2) of q over the pools as they are: no append, no score
 * update, no eviction.  The timing baseline the score/evict overhead is measured against.
 */
mkv_status mkv_attend_only(mkv_ctx* ctx, int layer, const void* q, void* out, void* stream);

/*
 * Change the decode budget B_d (1 <= budget <= the value given to mkv_create).  A
 * smaller budget makes the next step evict overflow = count - budget > 1 tokens (the
 * general arg-min of Eq. 8).
 */
mkv_status mkv_set_budget(mkv_ctx* ctx, int budget);

/* Back to "no layer prefilled"; pools keep their bytes but are treated as empty.  Waits for the
 * device, then clears the sticky device status. */
mkv_status mkv_reset(mkv_ctx* ctx);

/* Synchronise `stream`, then return the sticky device status (MKV_OK if clean). */
mkv_status mkv_status_sync(mkv_ctx* ctx, void* stream);

/*
 * Plain decode attention (softmax(q K^T / sqrt(d)) V) for callers that cannot allocate
 * device memory.  The paper has no counterpart of this call: it exists for hosts that are
 * handed input and output buffers only -- code running after a serving process has given
 * all device memory to its own pool, plug-ins without access to an allocator, processes
 * where allocation is forbidden once serving has begun.  It needs no context and no
 * workspace.  What its CTAs exchange (split-KV partials, tickets) lives in a fixed array
 * inside the library image, about 4.3 MB that every GPU loading the library holds until
 * the process exits; that array bounds the problem size:
 *     batch * kv_heads                         <= MKV_NOALLOC_MAX_UNITS
 *     batch * q_heads * ceil(n_tokens / 256)   <= MKV_NOALLOC_MAX_PART_ROWS
 *     n_tokens                                 <= 16384
 * Larger problems are refused with MKV_ERR_CAPACITY.
 *   q    device pointer [batch][q_heads][head_dim], kv_dtype
 *   K,V  device pointers [batch][kv_heads][kv_rows][head_dim], kv_dtype, plain row order;
 *        every sequence attends rows [0, n_tokens)
 *   out  device pointer [batch][q_heads][head_dim], out_dtype
 *   head_dim 64 or 128, q_heads / kv_heads <= 8, device = CUDA ordinal of the buffers
 * Asynchronous on `stream`.  The call allocates nothing and frees nothing.  The first call
 * on a device looks up the device address of the built-in array; make that first call
 * before starting any stream capture.  All calls share the one array, which keeps the
 * previous call's contents (tickets are cleared on `stream` at the start of every call):
 * calls whose kernels may overlap on the GPU -- different streams, several host threads --
 * race on it and must be ordered by the caller.
 * Errors: INVALID_ARG, UNSUPPORTED (head_dim, group size), CAPACITY, CUDA.
 */
#define MKV_NOALLOC_MAX_UNITS 2048
#define MKV_NOALLOC_MAX_PART_ROWS 8192
mkv_status mkv_attend_noalloc(const void* q, const void* K, const void* V, void* out, int batch,
                              int q_heads, int kv_heads, int head_dim, int n_tokens, int kv_rows,
                              int kv_dtype, int out_dtype, int device, void* stream);

/* Number of kernels this context has launched so far (host counter). */
int64_t mkv_launch_count(const mkv_ctx* ctx);

/* The grid of `layer`'s launches (0 before its prefill) and the number of CTAs the GPU keeps
 * resident, which bounds every grid.  layer == the context's layer count asks for the grid of
 * the launches over several layers (0 before the first such launch). */
mkv_status mkv_get_grid(const mkv_ctx* ctx, int layer, int32_t* n_ctas, int32_t* n_ctas_max);

/*
 * Test hook for the error path of the kernels' bounded waits; nothing traps, faults or spins
 * without bound.  Tensor-core kernel only (the scalar kernel has no waits): otherwise
 * MKV_ERR_UNSUPPORTED.  Synchronises the device.  The layer's results are undefined afterwards:
 * call mkv_reset() and prefill again.
 *   MKV_INJECT_LOST_TILE   one tile of unit (b, kv_head) counts as never delivered from now on, so
 *                          in the layer's next step the unit's finishing part waits for a count
 *                          that cannot come, gives up at the wait limit (MKV_OPT_WAIT_LIMIT_US)
 *                          and sets MKV_ERR_TIMEOUT; the rest of the step completes.
 */
#define MKV_INJECT_LOST_TILE 0
mkv_status mkv_debug_inject(mkv_ctx* ctx, int layer, int what, int b, int kv_head);

/*
 * Recency-window attention diagnostics of the last decode step of `layer` (the analysis of
 * Sec. 3.2 and Sec. 7.1 of the paper: how a step's attention is spread over the most recently
 * decoded tokens), from the probabilities the step recorded (MKV_FLAG_RECORD_PROBS, else
 * MKV_ERR_BAD_STATE).  The paper shows figures, no formulas; the quantities are defined here.
 * For every (sequence, KV head) unit u = b * kv_heads + kv_head, with t the id of the last step
 * and the window = the cached decode tokens (before that step's eviction) whose position id
 * lies in (t - window, t]:
 *   count[u]          number of tokens in the window (<= window)
 *   mass[u]           attention they received together, head-averaged as in Eq. 4 (a share
 *                     of 1; the rest went to older decode tokens and to the prompt)
 *   curve[u][j]       share of mass[u] held by the j+1 most attended tokens of the window,
 *                     j < count[u]; entries from count[u] to window-1 are set to 0.  Uniform
 *                     attention would give (j+1)/count[u].
 * In the score mode MKV_SCORE_LAYER_MEAN the values are those of the whole layer, equal in
 * every KV head of a sequence.  Before the first step all outputs are 0.
 * mass: device float [batch*kv_heads]; count: device int32 [batch*kv_heads]; curve: device
 * float [batch*kv_heads][window]; all owned by the caller, written by a kernel on `stream`
 * (asynchronous, allocation-free).  window >= 1; min(window, budget + 1) <= 8192, else
 * MKV_ERR_UNSUPPORTED.  Not part of the decode step: nothing is computed unless called.
 */
mkv_status mkv_recency_diagnostics(mkv_ctx* ctx, int layer, int window, float* mass, int32_t* count,
                                   float* curve, void* stream);

/* ---- inspection: synchronous (device-wide sync + D2H), for tests and debugging ---- */

/* Decode pool of (layer, b, kv_head): *n tokens; pos/score (host, `cap` entries) may be
 * NULL.  Order is the physical slot order, which compaction permutes. */
mkv_status mkv_get_decode_state(mkv_ctx* ctx, int layer, int b, int kv_head, int32_t* n,
                                int32_t* pos, float* score, int cap);
/* Tokens the last step evicted from that pool, with their scores at eviction. */
mkv_status mkv_get_last_evicted(mkv_ctx* ctx, int layer, int b, int kv_head, int32_t* k,
                                int32_t* pos, float* score, int cap);
/* Eq. 4 values of the last step per slot, pre-eviction order, and the position ids of those
 * slots (needs MKV_FLAG_RECORD_PROBS; abar, pos: host, `cap` entries, either may be NULL);
 * *n receives the pre-eviction token count. */
mkv_status mkv_get_last_probs(mkv_ctx* ctx, int layer, int b, int kv_head, int32_t* n,
                              float* abar, int32_t* pos, int cap);
/* Copy a pool's rows out in plain [token][head_dim] layout (kv_dtype).  pool 0 = prefill,
 * 1 = decode.  *n receives the token count; at most cap_tokens rows are written. */
mkv_status mkv_read_kv(mkv_ctx* ctx, int layer, int b, int kv_head, int pool, int32_t* n,
                       void* K_host, void* V_host, int cap_tokens);
/* Decode steps completed on a layer since its prefill. */
mkv_status mkv_get_step(mkv_ctx* ctx, int layer, int64_t* step);

const char* mkv_status_string(mkv_status s);

#if defined(__GNUC__)
#pragma GCC visibility pop
#endif
#ifdef __cplusplus
}
#endif
#endif /* MKV_H_ */
