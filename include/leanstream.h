/*
 * leanstream.h -- C ABI of the B200 (sm_100a) speculate-and-refine sparse FFN decode library.
 *
 * One FFN layer of a decoder at batch 1 (small batches allowed) is executed the way Section 2.1 of the
 * LeanStream paper describes: a predictor scores the layer's hidden neurons from a residual feature
 * (speculate), the selected neurons are computed in K priority-ordered stages (Eq. 1), and after every stage the
 * partial residual feature (Eq. 2) re-scores the neurons of the next layer (refine).  Weights of layers that do
 * not fit in HBM live in pinned host memory and are served through an HBM neuron cache (Section 3.3.3, cache
 * eviction task; Section 4.3, cache miss ratio).
 *
 * Conventions
 *  - Every function returns an int32_t status: LS_OK (0) or a negative LS_ERR_* code; ls_last_error() gives a
 *    text for the calling thread's last failure.  Nothing throws, aborts or traps.
 *  - Pointers named d_* and every pointer inside ls_selection / ls_step_trace are DEVICE pointers owned by the
 *    caller; the library neither frees nor keeps them after the call has been enqueued.  Pointers inside
 *    ls_layer_desc are HOST pointers read only during ls_layer_create().
 *  - `stream` arguments carry a cudaStream_t (0 = the legacy default stream).  Work is enqueued asynchronously;
 *    argument validation is synchronous.  Calls on fully resident layers never synchronise or allocate and may be
 *    captured in a CUDA graph; calls on layers with a cache (cache_rows > 0) do not synchronise either (except where a
 *    result is returned to the host) but use a second stream and events and are not meant for capture.
 *  - A layer handle is not thread safe: one call at a time per layer; per-layer scratch is reused by every call.
 *  - Neuron i of a layer owns gate row i, up row i and down-projection row i (column i of the paper's W_gate /
 *    W_up, row i of W_down).  Index lists are int32, masks hold neuron i at bit (i & 31) of word (i >> 5).
 */
#ifndef LEANSTREAM_H_
#define LEANSTREAM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LS_OK 0
#define LS_ERR_INVALID (-1)  /* bad argument (null pointer, size out of range, unsupported combination) */
#define LS_ERR_NOMEM (-2)    /* host or device allocation failed */
#define LS_ERR_CUDA (-3)     /* a CUDA runtime call failed; ls_last_error() has the CUDA message */
#define LS_ERR_STATE (-4)    /* call not valid for this layer (e.g. cache call on a resident layer) */
#define LS_ERR_CAPACITY (-5) /* wanted + protected neurons exceed the cache capacity, or a list exceeds its cap */
#define LS_ERR_TIMEOUT (-6)  /* a bounded wait (miss copies, a barrier inside a kernel) gave up */
#define LS_ERR_INTERNAL (-7) /* a kernel's self-check failed (reported through ls_layer_status) */

#define LS_ACT_RELU 0
#define LS_ACT_SILU 1 /* the activation Eq. 1 prints: g * sigmoid(g); no exact zeros, so every selected neuron needs all its rows */
#define LS_WDTYPE_BF16 0
#define LS_WDTYPE_FP16 1
#define LS_NORM_RMS 0
#define LS_NORM_NONE 1

typedef struct ls_layer ls_layer;

/*
 * Problem statement of one FFN layer: the operands of Eq. 1 plus the layer's neuron predictor.
 *   act(h W_gate) * (h W_up) W_down with act = ReLU (the sparsity source of Section 2.1) or SiLU (as Eq. 1 prints it);
 *   gated = 0 gives the two-matrix form act(h W_fc1 + b) W_fc2 + b_down.  h = rmsnorm(x) without gain (norm = LS_NORM_RMS) or h = x.
 *   Predictor (Section 3.3.3: projection of the feature, then the scorer): s = pred_b^T (pred_a^T h) + pred_c.
 * All weight matrices are 16-bit (wdtype), row-major, HOST memory, copied by ls_layer_create():
 *   w_gate, w_up, w_down_t: [d_ff][d_model] (w_down_t is neuron-major, i.e. the transposed down projection);
 *   pred_a: [d_model][pred_rank];  pred_b: [pred_rank][d_ff];  b_gate, pred_c: float [d_ff] or NULL (zeros);
 *   b_down: float [d_model] or NULL.  d_model and pred_rank must be multiples of 8; d_model <= 16384.
 * cache_rows = 0 keeps every neuron in HBM.  cache_rows > 0 keeps the weights in library-owned pinned host memory
 *   and gives the layer an HBM cache of that many neuron bundles (gate, up, down rows of one neuron).
 * max_batch (default 1 when 0, at most 8) and max_sel (default d_ff when 0) size the per-layer scratch: the largest
 *   batch and the longest selection list any call will pass.
 */
typedef struct {
  uint32_t struct_size; /* sizeof(ls_layer_desc), checked */
  int32_t device;       /* CUDA device ordinal */
  int32_t d_model, d_ff;
  int32_t gated, act, wdtype, norm;
  float norm_eps;
  int32_t pred_rank;
  const void *w_gate, *w_up, *w_down_t;
  const float *b_gate, *b_down;
  const void *pred_a, *pred_b;
  const float *pred_c;
  int64_t cache_rows;
  int32_t max_batch, max_sel;
} ls_layer_desc;

/* Creates a layer on desc->device (weights uploaded before return).  *out is owned by the library until
 * ls_layer_destroy().  Errors: LS_ERR_INVALID (shape/flags), LS_ERR_NOMEM, LS_ERR_CUDA; *out is NULL on failure. */
int32_t ls_layer_create(const ls_layer_desc *desc, ls_layer **out);
/* Waits for the layer's own streams, frees everything the layer owns.  NULL is accepted. */
int32_t ls_layer_destroy(ls_layer *layer);

/*
 * A selection of neurons (caller-allocated device buffers).
 *   scores: [d_ff] priority of every neuron (batch > 1: max over the batch), fp64; NULL = not wanted.
 *   mask:   [ceil(d_ff/32)] membership bitmask; NULL = not wanted.
 *   idx:    [cap] the selected neurons in RANK ORDER (highest priority first; equal scores: lower index first),
 *           so that stage c of K is the slice [c*m, min(count,(c+1)*m)), m = ceil(count/K).
 *   count:  [1] number of selected neurons (k at batch 1, size of the union otherwise).
 */
typedef struct {
  double *scores;
  uint32_t *mask;
  int32_t *idx;
  int32_t *count;
  int32_t cap;
} ls_selection;

/*
 * Speculate (Section 2.1, Fig. 2; Section 3.3.3 neuron-activation prediction): scores every neuron of `layer`
 * from d_feature [batch][d_model] (float, un-normalised residual-like feature; the library applies the layer's
 * norm), accumulating in fp64, and selects per token the k best under the total order (score descending, index
 * ascending; NaN ranks last, -0 equals +0); batch > 1 returns the union ordered by the per-neuron maximum score.
 * The layer keeps the priorities as its cache-retention priorities.  0 <= k <= d_ff; out->idx and out->count are
 * required and out->cap >= min(batch*k, d_ff).  Errors: LS_ERR_INVALID; device-side problems (a list longer than
 * its cap) are reported through ls_layer_status().
 */
int32_t ls_predict(ls_layer *layer, const float *d_feature, int32_t batch, int32_t k, ls_selection *out,
                   void *stream);

/*
 * Optional validation outputs of ls_sparse_ffn_step (device pointers, each may be NULL).
 *   xtilde:        [n_chunks+1][batch][d_model] partial residual features x~^(j), j = 0..K (Eq. 2)
 *   refine_masks:  [n_chunks+1][ceil(d_ff_next/32)] refined sets C^(j) for the next layer
 *   refine_counts: [n_chunks+1] their sizes
 *   survive_mask:  [ceil(d_ff/32)] selected neurons whose activation is nonzero for some token
 *   exec_idx:      [count] the order in which the selected neurons were executed (differs from the rank order
 *                  only on cached layers: residents first, then misses, each in rank order)
 */
typedef struct {
  float *xtilde;
  uint32_t *refine_masks;
  int32_t *refine_counts;
  uint32_t *survive_mask;
  int32_t *exec_idx;
} ls_step_trace;

/*
 * One layer's speculate-and-refine step (Section 2.1, Eq. 1 and Eq. 2; Section 3.2.2 permutation-invariant
 * execution): h = norm(x); the neurons listed in `sel` (rank order, *sel->count of them) run in n_chunks stages;
 * stage c adds dm^(c) = sum_i a_i W_down[i] over its neurons with a_i = relu(w_gate[i].h + b_i) * (w_up[i].h),
 * reading down rows only where a_i != 0; x~^(0) = x (+ b_down), x~^(j) = x~^(j-1) + dm^(j); d_x_out = x~^(K).
 * When `next` is given, every x~^(j), j = 0..K, is scored by next's predictor and the top k_next set C^(j) is
 * formed; C^(K) is returned in sel_next (required when next != NULL) and next's retention priorities are updated
 * at each stage.  When `next` has a cache, the first ceil(count_j (j+1)/(K+1)) ranks of C^(j), j < K, are reserved
 * in it (miss copies start on next's copy stream).  When `layer` has a cache, the whole selection is reserved
 * first, residents run before misses, and the stages that need copied rows wait for them on the device.
 * d_x, d_x_out: float [batch][d_model]; d_x_out may alias d_x.  next may equal layer.
 * Errors: LS_ERR_INVALID, LS_ERR_CAPACITY (cached layer: sel->cap larger than the cache; a list whose actual count
 * overflows is reported through ls_layer_status), LS_ERR_CUDA.
 */
int32_t ls_sparse_ffn_step(ls_layer *layer, ls_layer *next, const float *d_x, float *d_x_out, int32_t batch,
                           const ls_selection *sel, int32_t n_chunks, int32_t k_next, ls_selection *sel_next,
                           ls_step_trace *trace, void *stream);

/*
 * HBM neuron cache (Section 3.3.3 cache-eviction task; Section 4.3 cache miss ratio).  Residency is logical: a
 * neuron is resident once a slot is assigned to it; its bytes arrive on the layer's copy stream (LS_OPT_MISS_PATH) and
 * the kernels that read them wait on the device until they have landed.  All calls return LS_ERR_STATE on a layer
 * created with cache_rows = 0.
 *
 * ls_cache_lookup: d_slot[j] = slot of neuron d_idx[j] or -1 (miss); *d_nhit = number of residents.  n <= max_sel.
 *
 * ls_cache_reserve: makes the first `admit_ranks` entries (< 0: all) of want->idx resident.  The new resident set
 *   is the cache_rows best of (residents + wanted) under the key (wanted or protected first, then retention
 *   priority descending, then index ascending); the rest are evicted and their slots given to the misses, whose
 *   bundles are brought from pinned host memory on the layer's copy stream.  When want->scores is given it first
 *   replaces the layer's retention priorities.  d_protect_mask (nullable) marks neurons that must not be evicted.
 *   *h_nmiss (nullable, HOST) receives the number of misses: for it the call waits on the calling thread for the decision
 *   (not for the copies), at most LS_OPT_HOST_WAIT_MS (LS_ERR_TIMEOUT otherwise; the request stays enqueued).
 *   LS_ERR_CAPACITY if wanted + protected exceed cache_rows (nothing changes).
 *   (ls_sparse_ffn_step reserves through the same machinery without waiting on the host at all; with the gather
 *   transport its refine-driven requests for the next layer are decided on that layer's copy stream, and every entry
 *   point here first makes its stream wait for such pending decisions, so callers see them as if they had run in order.)
 *
 * ls_cache_evict: evicts lowest-priority unprotected residents until at least min_free slots are free (fewer when
 *   only protected ones remain); d_evicted (nullable, [cache_rows]) and d_nevicted (nullable) receive them.  Asynchronous.
 */
int32_t ls_cache_lookup(ls_layer *layer, const int32_t *d_idx, int32_t n, int32_t *d_slot, int32_t *d_nhit,
                        void *stream);
int32_t ls_cache_reserve(ls_layer *layer, const ls_selection *want, int32_t admit_ranks,
                         const uint32_t *d_protect_mask, int32_t *h_nmiss, void *stream);
int32_t ls_cache_evict(ls_layer *layer, int32_t min_free, const uint32_t *d_protect_mask, int32_t *d_evicted,
                       int32_t *d_nevicted, void *stream);
/* d_resident_mask [ceil(d_ff/32)] <- current logical resident set (for parity checks). */
int32_t ls_cache_snapshot(ls_layer *layer, uint32_t *d_resident_mask, void *stream);
/* Makes `stream` wait (on the device, bounded) until the rows of every request made so far for this layer have landed. */
int32_t ls_cache_wait(ls_layer *layer, void *stream);

typedef struct {
  int64_t hits, misses, evictions; /* counted over reserve calls (wanted entries found / not found resident) */
  int64_t h2d_bytes;               /* bytes brought from pinned host memory into cache slots */
  int64_t h2d_copies;              /* copy operations issued for them: cudaMemcpyAsync calls (I/O lane) or gather launches */
  int64_t resident;                /* current number of resident neurons */
} ls_cache_stats_t;
/* Counters kept on the device by the decision kernels; the call synchronises the device. */
int32_t ls_cache_stats(ls_layer *layer, ls_cache_stats_t *host_out);

/* Reads and clears the layer's device-side status word (0 = no problem seen by any kernel since the last read;
 * otherwise the first LS_ERR_* code a kernel recorded, e.g. an out-of-range neuron index, which kernels skip
 * rather than dereference).  Synchronises the device. */
int32_t ls_layer_status(ls_layer *layer, int32_t *host_status);

/*
 * Whole-token decode of a stack of fully resident layers (Section 2.1 applied layer after layer: x_{n+1} = x~_n^(K), and
 * the final refined set C^(K) of layer n is the selection of layer n+1).  ls_stack_decode runs every layer's
 * speculate-and-refine step (exactly what ls_sparse_ffn_step computes at batch 1) inside ONE cooperative kernel, so a
 * layer boundary costs a grid barrier instead of a kernel launch.  The last layer refines a weight-tied copy of itself.
 *
 * ls_stack_create: `layers` (HOST array of n_layers handles) must be resident (cache_rows = 0), on one device, with one
 *   d_model and one weight type; the handles are borrowed and must outlive the stack.  LS_ERR_STATE if a layer does not
 *   qualify.  The stack owns small device buffers (per-layer argument table, residual and selection ping-pong).
 * ls_stack_decode: d_x, d_x_out float [d_model] (may alias); sel_first = selection of layer 0 in rank order (from
 *   ls_predict); n_chunks in [1, 16]; sel_out receives the final refined set of the last layer (idx, count required;
 *   mask, scores optional).  Never synchronises or allocates; may be captured in a CUDA graph.  Calls on one device
 *   must not overlap (they share one scratch).  The kernel is bitwise repeatable (every sum has a fixed order).
 *
 * `trace` (nullable; every member nullable) exports what a layer boundary and every refinement produced, for checking
 * and profiling:
 *   x            [n_layers+1][d_model]  the residual entering each layer and leaving the last
 *   sel_idx      [n_layers+1][sel_cap], sel_count [n_layers+1]: the selection entering each layer (rank order) and
 *                the final refined one
 *   xtilde       [n_layers][n_chunks+1][d_model]  the partial residual features x~^(j) of every layer (Eq. 2)
 *   refine_masks [n_layers][n_chunks+1][mask_words]  the refined sets C^(j) of every layer (Section 2.1), j = 0..K;
 *                mask_words >= ceil(d_ff/32) of every layer
 *   phase_ns     [n_layers][SMs][LS_STACK_NSTAMP] nanosecond time stamps (GPU global timer) of every CTA at the ends
 *                of the kernel's phases: 0 layer start, 1 partial output written, 2 barrier 1 passed, 3 features and
 *                partial latents written, 4 barrier 2 passed, 5 latents summed, 6 barrier 3 passed, 7 scores written,
 *                8 barrier 4 passed, 9 own slice of the next selection known, 10 layer end
 */
#define LS_STACK_NSTAMP 12
typedef struct ls_stack ls_stack;
typedef struct {
  float *x;
  int32_t *sel_idx;
  int32_t *sel_count;
  int32_t sel_cap;
  float *xtilde;
  uint32_t *refine_masks;
  int32_t mask_words;
  long long *phase_ns;
} ls_stack_trace;
int32_t ls_stack_create(ls_layer *const *layers, int32_t n_layers, ls_stack **out);
int32_t ls_stack_destroy(ls_stack *stack);
int32_t ls_stack_decode(ls_stack *stack, const float *d_x, float *d_x_out, const ls_selection *sel_first, int32_t n_chunks,
                        int32_t k_next, ls_selection *sel_out, ls_stack_trace *trace, void *stream);

/*
 * Top-k selection that allocates nothing (the paper has no counterpart; it exists for callers that must not allocate).
 *
 * Some callers cannot call cudaMalloc or anything that may call it for them: code running while a stream is being
 * captured into a CUDA graph, a latency-critical serving loop that must never meet the implicit device synchronisation
 * of an allocation, a process whose device memory has been handed out completely to a memory pool, or a callback of
 * another runtime in which allocating is simply forbidden.  For them this entry point selects the k highest scores of a
 * caller-provided device array with the same rule as ls_predict (score descending, equal scores by ascending index,
 * NaN last, -0 equal to +0) using only memory that already exists: its candidate lists live in a fixed array inside
 * the library image (LS_STATIC_TOPK_MAX_N x 12 bytes = 384 KB, held on every GPU that has loaded the library until
 * the process exits).  It calls no cudaMalloc, no cudaFree and no allocating library routine, and needs no ls_layer.
 *
 *   d_scores [n] fp64 (device, read only); d_idx [k] receives the selected positions in rank order; d_mask
 *   [ceil(n/32)] (nullable) the membership bits; d_count [1] the number selected (= k).  All caller-owned.
 *   1 <= n <= LS_STATIC_TOPK_MAX_N and 0 <= k <= n, otherwise LS_ERR_INVALID with an explanatory ls_last_error().
 *
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress) and opts the kernel in to its
 * shared memory; make that first call outside any stream capture.  Every call runs on the device that owns d_scores
 * (d_idx, d_mask and d_count must live there too), whatever device is current.  All calls on a
 * device share the one array: two calls that overlap on the GPU (different streams) race on it, so order them; the
 * array keeps whatever the last call left there, which is harmless because every entry is written before it is read.
 */
#define LS_STATIC_TOPK_MAX_N 32768
int32_t ls_topk_select_static(const double *d_scores, int32_t n, int32_t k, int32_t *d_idx, uint32_t *d_mask,
                              int32_t *d_count, void *stream);

/*
 * Process-wide options (no counterpart in the paper).  LS_OPT_FUSED (default 1): steps that qualify (batch 1, layer and
 * next layer fully resident, a next layer given, n_chunks <= 16, d_model <= 8192, shared memory fits) run as ONE
 * cooperative kernel, the same one ls_stack_decode runs over a whole stack; 0 forces the stage-by-stage kernels, which
 * compute the same thing.  Both paths add partial outputs in a fixed order (no floating-point atomics) and are bitwise
 * repeatable; the two orders differ, so their features may differ in the last fp32 bits.  The selected sets are always
 * the exact top-k of the features that were actually produced.  Fused steps and ls_stack_decode share one working
 * scratch per device: issue them on one stream, or order the streams that issue them.
 */
#define LS_OPT_FUSED 1
/*
 * LS_OPT_MISS_PATH: how the misses of a cached layer travel from pinned host memory to their cache slots.  Either way the
 * calling thread only enqueues work and the stages that need copied rows wait on the device (bounded) for a word the copy
 * stream raises; set the option before the first call on a cached layer and do not change it while requests are in flight.
 *   LS_MISS_PATH_LANE:   Section 3.2.1 / Algorithm 1 of the paper re-targeted: the decision kernel writes its miss list
 *     and a sequence flag to mapped pinned memory; a host thread of the library (the paper's I/O lane) polls the flag and
 *     issues one cudaMemcpyAsync per run of adjacent neurons and slots on the layer's copy stream.  The calling thread
 *     lets at most two requests of a layer be in flight and enqueues the stages of a step once the lane has issued the
 *     copies of the step's own request (bounded host waits on the lane's acknowledgement word, never on the stream).
 *   LS_MISS_PATH_GATHER (default): the list stays on the device and one kernel on the copy stream reads the missing
 *     bundles straight from the mapped pinned store over the host link; no host thread takes part.
 * LS_OPT_HOST_WAIT_MS (default 30000): how long ls_cache_reserve waits on the calling thread for the number of misses
 * before it returns LS_ERR_TIMEOUT.  A request that timed out stays enqueued and takes effect when its stream reaches it.
 */
#define LS_OPT_MISS_PATH 2
#define LS_MISS_PATH_LANE 0
#define LS_MISS_PATH_GATHER 1
#define LS_OPT_HOST_WAIT_MS 3
int32_t ls_set_option(int32_t option, int32_t value);

/*
 * Kernel timing for roofline accounting (no counterpart in the paper).  While enabled (process-wide, off by default)
 * the launches of the named kernel groups are bracketed by CUDA events on the stream they are launched on; not valid
 * during stream capture.  ls_timing_read() waits for the recorded events of one group, returns their number and summed
 * duration in milliseconds, and forgets them.
 */
#define LS_TIMED_GATEUP 0  /* gate/up gather-GEMV + activation of one stage */
#define LS_TIMED_DOWN 1    /* sparse down projection of one stage */
#define LS_TIMED_PREDICT 2 /* latent + scores + top-k of one predictor evaluation */
#define LS_TIMED_FUSED 3   /* the fused per-layer step kernel */
#define LS_TIMED_STACK 4   /* the whole-token kernel of ls_stack_decode */
int32_t ls_timing_enable(int32_t on);
int32_t ls_timing_read(int32_t kind, int64_t *launches, double *total_ms);

/*
 * Stacked learnable hashing predictor, inference (Section 3.3.1 - 3.3.3): an alternative to the linear predictor of
 * ls_layer_desc for ranking a layer's neurons.  Layer k computes y_k = T_k[phi_tau(sign(x_k (*) W_k))]: the first layer
 * hashes the PCA-projected feature with real hyperplanes (decided in fp64), the others are binary (XNOR and bitcount); a
 * neuron's priority is the XNOR-and-bitcount inner product of the last layer's output with the neuron's binary code.
 * Sign vectors are packed one bit per component: +1 -> 1, -1 -> 0, component c at bit (c & 31) of word (c >> 5).
 * phi_tau takes the FIRST component of a code as the most significant bit (the convention of the structured matrix Z of
 * Section 3.3.2); sign(0) = +1.
 *   pca     HOST [d_model][rank] 16-bit (wdtype)      w1      HOST float [rank][tau]
 *   w       HOST uint32 [n_layers-1][tau][d_code/32]   tables  HOST uint32 [n_layers][2^tau][d_code/32]
 *   codes   HOST uint32 [d_ff][d_code/32]
 *   d_model, rank multiples of 8; 1 <= tau <= 16; d_code a multiple of 32, at most 1024; 1 <= n_layers <= 16.
 * ls_hash_predict: scores every neuron from d_feature [d_model] (float, un-normalised: a hyperplane hash does not see a
 *   positive scale) and selects the k best under the same total order as ls_predict; `out` as there (scores are the
 *   integer priorities as fp64).  d_layer_idx (nullable, DEVICE int32 [n_layers]) receives every layer's bucket number.
 */
typedef struct ls_hash_predictor ls_hash_predictor;
typedef struct {
  uint32_t struct_size;
  int32_t device;
  int32_t d_model, rank, tau, d_code, n_layers, d_ff, wdtype;
  const void *pca;
  const float *w1;
  const uint32_t *w, *tables, *codes;
} ls_hash_predictor_desc;
int32_t ls_hash_predictor_create(const ls_hash_predictor_desc *desc, ls_hash_predictor **out);
int32_t ls_hash_predictor_destroy(ls_hash_predictor *pred);
int32_t ls_hash_predict(ls_hash_predictor *pred, const float *d_feature, int32_t k, ls_selection *out, int32_t *d_layer_idx,
                        void *stream);

/*
 * Streaming controller (Section 3.2.3: state q_n = Q(R_n), coordination plan phi_n, finite-horizon stochastic dynamic
 * programme solved offline, LUT[n, q] looked up at every layer boundary).  Host-side: every pointer is HOST memory.
 * In this library a plan is an index into a caller-defined list of candidates (for instance stage counts n_chunks).
 *
 * ls_controller_quantize: q = Q(R): the remaining-load volume cut into n_states equal bins over [0, vmax] (0 = nothing
 *   left; the last state collects everything from vmax on).  Returns the state, or LS_ERR_INVALID.
 * ls_controller_build: Bellman backward recursion V_n^h(q) = min_a [ t_bar[n][q][a] + mean_s V_{n+1}^{h-1}(next_state[n][q][a][s]) ],
 *   V^0 = 0 and V = 0 beyond the last layer.  t_bar [n_layers][n_states][n_plans]: profiled time of layer n from state q
 *   under plan a (infinite or negative: plan not allowed in that state).  next_state [n_layers][n_states][n_plans][n_samples]:
 *   the profiled samples of the next layer's state (negative entries are unused).  lut [n_layers][n_states] receives the
 *   minimising plan at h = horizon (lowest index among equals, -1 when none is allowed); value (nullable, same shape)
 *   receives V_n^horizon(q).  LS_ERR_INVALID on bad sizes or a sample outside [0, n_states).
 */
int32_t ls_controller_quantize(double remaining, double vmax, int32_t n_states);
int32_t ls_controller_build(int32_t n_layers, int32_t n_states, int32_t n_plans, int32_t n_samples, int32_t horizon, const double *t_bar,
                            const int32_t *next_state, int32_t *lut, double *value);

/* Number of kernels launched by this library in the calling process since load (for launch accounting). */
int64_t ls_kernel_launches(void);
/* Copies the calling thread's last error text (NUL terminated, truncated to n) and returns its length. */
size_t ls_last_error(char *buf, size_t n);
/* Library ABI version (major * 1000 + minor). */
int32_t ls_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LEANSTREAM_H_ */
