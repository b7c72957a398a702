/*
 * choco.h -- C interface of libchoco: the CHOCO-Gossip / CHOCO-SGD step for n simulated
 * workers on one GPU (Koloskova, Lin, Stich, Jaggi, "Decentralized Deep Learning with
 * Arbitrary Communication Compression", ICLR 2020).
 *
 * State (caller-owned DEVICE memory, float32, row-major, row pitch `ld` elements):
 *     X    [n, ld]   private iterates x_i                       (Algorithm 1)
 *     Xhat [n, ld]   public copies x^_i                          (Algorithm 1)
 *     S    [n, ld]   neighbour sums s_i = sum_j w_ij x^_j        (the "3 vectors per
 *                    node" storage of Section 3, last paragraph)
 *     G    [n, ld]   stochastic gradients g_i, read-only          (Algorithm 1)
 * A fresh run starts from Xhat = S = 0 (Algorithm 1, input); any state with
 * S = W Xhat resumes one.  Only the first d elements of each row are used.
 *
 * One step call performs, for every worker i at once,
 *     q_i    = Q(x_i - x^_i)                     Algorithm 1: compression
 *     x^_i  += q_i                               update of the public copy (j = i)
 *     s_i   += sum_j w_ij q_j                    the same for all neighbours j, folded into s_i
 *     x_i    = (x_i - eta g_i) + gamma (s_i - x^_i)
 *                                                gradient step, then the gossip step of the next iteration
 *                                                (sum_j w_ij (x^_j - x^_i) = s_i - x^_i as
 *                                                rows of W sum to one)
 * i.e. the gossip scheme h of Appendix A.1 ("Example: CHOCO-SGD"), with the communication
 * and gradient parts in the rotated order that Appendix A.1 notes only shifts the initial
 * values.  The messages q_i are written to library-owned device buffers in compressed form
 * and read back from there by every neighbour.
 *
 * Arithmetic: float32, round to nearest, no fused multiply-add, neighbours accumulated in
 * CSR column order from +0, norms summed as a pairwise tree over the coordinate index.
 * Results are deterministic: same inputs, seed and step number give the same bits.
 *
 * All functions return 0 on success or a negative choco_status; on error nothing has been
 * enqueued.  Calls on one context must be issued in stream order, from one host thread at
 * a time.  `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 * Step calls are asynchronous: they enqueue kernels on `stream` and return.
 *
 * Device-side waits.  The kernels stage their tiles with asynchronous copies and wait for them
 * with a bounded number of polls (about 4 million, seconds of wall time; a copy normally lands
 * within microseconds).  A block whose wait runs out counts it in choco_stats.device_timeouts,
 * waits once more (again bounded) for its copies in flight and returns without writing its part
 * of X, Xhat and S: nothing hangs and nothing faults, but the arrays are then no valid state.
 * Step calls do not synchronise and therefore cannot report this themselves; every call that
 * does synchronise `stream` (choco_get_stats, choco_read_message, choco_consensus_error,
 * choco_sgd_step_host) reads the counter and returns CHOCO_ERR_TIMEOUT once it is non-zero, and
 * from then on every step call on the context returns CHOCO_ERR_TIMEOUT without enqueuing
 * anything.  Recover by restoring X, Xhat and S from a checkpoint into a fresh context
 * (choco_set_step resumes the generator).
 *
 * Memory reads: rows that are not 16-byte aligned (base pointer or ld * 4 not a multiple of 16, or
 * d not a multiple of 4) are staged in whole 16-byte units, so up to 12 bytes before the first and
 * after the last element of a row are read (never written, and never used): the arrays must lie in
 * memory that is readable up to the enclosing 16-byte boundaries, which holds for anything
 * cudaMalloc or a caching allocator hands out.
 *
 * L2 residency (TOPK / RANDK contexts): choco_init raises the device's persisting-L2 limit
 * (cudaLimitPersistingL2CacheSize) if it is below what the context's message arena needs, and never
 * lowers it; the selection and update kernels are launched with an access-policy window over that
 * arena (a per-launch attribute: no stream attribute is left on `stream`).  choco_destroy calls
 * cudaCtxResetPersistingL2Cache, which returns all persisting lines on the device to normal.
 */
#ifndef CHOCO_H_
#define CHOCO_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct choco_ctx choco_ctx; /* opaque; owns the CSR copy of W, messages, workspace */

typedef enum {
    CHOCO_OK = 0,
    CHOCO_ERR_INVALID_ARG = -1, /* null pointer, n < 1, d < 1, ld < d, k outside [1, d], ...  */
    CHOCO_ERR_BAD_W = -2,       /* W violates Assumption 1 or the CSR rules below             */
    CHOCO_ERR_ALLOC = -3,       /* device or host allocation failed                           */
    CHOCO_ERR_CUDA = -4,        /* a CUDA runtime call failed (see choco_last_cuda_error)      */
    CHOCO_ERR_MISALIGNED = -5,  /* a state pointer is not 4-byte aligned                       */
    CHOCO_ERR_UNSUPPORTED = -6, /* valid in the paper, not built (e.g. an odd QSGD bucket)     */
    CHOCO_ERR_TOO_LARGE = -7,   /* a size exceeds a documented limit                           */
    CHOCO_ERR_TIMEOUT = -8      /* a bounded wait inside a kernel ran out: the state arrays are */
                                /* no longer a valid CHOCO state (see "Device-side waits")      */
} choco_status;

/* Compression operator Q (Appendix C, "Compression Schemes"). */
typedef enum {
    CHOCO_Q_IDENTITY = 0, /* q = v: exact gossip, the delta = 1 case of Theorem 4.1           */
    CHOCO_Q_TOPK = 1,     /* top_a: k largest |v|, ties to the lower index                    */
    CHOCO_Q_RANDK = 2,    /* random_a, biased form v (.) u, ||u||_1 = k                        */
    CHOCO_Q_QSGD = 3,     /* gsgd_b with s = 2^(b-1) levels, dithered, per block               */
    CHOCO_Q_SIGN = 4      /* (||v||_1 / d) sgn(v), one bit per coordinate                      */
} choco_q_kind;

typedef struct {
    int32_t kind;        /* choco_q_kind                                                       */
    int32_t s;           /* QSGD: number of levels 2^(b-1), a power of two in [2, 32768]; the  */
                         /*       level of a coordinate is stored in 1, 2, 4, 8 or 16 bits     */
    int32_t bucket;      /* QSGD: block length for the norm; 0 = whole row, else a power of    */
                         /*       two in [128, 1024] (the last block of a row may be shorter)  */
    int32_t qsgd_biased; /* QSGD: 1 = divide by tau = 1 + min(len/s^2, sqrt(len)/s) (the       */
                         /*       delta = 1/tau operator CHOCO uses), 0 = unbiased form        */
    int64_t k;           /* TOPK / RANDK: entries kept per row, floor(a d), in [1, d]          */
} choco_params;

/*
 * choco_init -- Algorithm 1, "input": the communication graph with its mixing matrix W
 * (Assumption 1), the compression operator and the random seed that sender and receiver of a
 * random_a message share (Appendix C: the receiver regenerates the positions from it).
 *   n, d, ld     workers, coordinates per worker, row pitch of all state arrays (ld >= d;
 *                d < 2^31).
 *   w_row_ptr[n+1], w_col[nnz], w_val[nnz]   HOST pointers to W in CSR; copied.  Every row
 *                must list its columns in strictly ascending order and include the diagonal;
 *                weights in [0, 1], row sums within 1e-5 of one, W symmetric within 1e-6.
 *   p            Q and its parameter (copied).
 *   seed         keys the counter-based generator (Philox4x32-10) together with
 *                (step, worker, coordinate); used by RANDK and QSGD.
 * Allocates all device memory the steps need on the current device; steps allocate nothing.
 * The step counter starts at 0.  On success *out owns the context; free with choco_destroy.
 */
int choco_init(choco_ctx** out, int32_t n, int64_t d, int64_t ld, const int32_t* w_row_ptr,
               const int32_t* w_col, const float* w_val, const choco_params* p, uint64_t seed);

/* Frees everything choco_init allocated.  Synchronises the device first. */
int choco_destroy(choco_ctx* ctx);

/*
 * choco_gossip_step -- one application of CHOCO-Gossip (the averaging scheme h of Appendix
 * A.1: X+ = X + gamma Y (W - I), Y+ = Y + Q(X+ - Y), Y = Xhat) in the rotated order given at
 * the top: compress, update Xhat and S, then x_i += gamma (s_i - x^_i).  No gradient.
 * X, Xhat, S: DEVICE pointers, updated in place.  Advances the step counter by one.
 */
int choco_gossip_step(choco_ctx* ctx, float* X, float* Xhat, float* S, float gamma, void* stream);

/*
 * choco_sgd_step -- Algorithm 1: iteration t from its compression step to its gradient step,
 * followed by the gossip step of iteration t+1, with g_i = G[i] the gradient the caller
 * evaluated at the current x_i.
 * G: DEVICE pointer, read-only.  Advances the step counter by one.
 */
int choco_sgd_step(choco_ctx* ctx, float* X, float* Xhat, float* S, const float* G, float eta,
                   float gamma, void* stream);

/*
 * choco_sgd_momentum_step -- Algorithm 2 (CHOCO-SGD with momentum): the gradient step becomes
 *     m_i = (g_i + lambda x_i) + beta m_i ;   x_i = (x_i - eta m_i) + gamma (s_i - x^_i)
 * with M [n, ld] the local momentum memory (DEVICE, updated in place, starts at 0).
 */
int choco_sgd_momentum_step(choco_ctx* ctx, float* X, float* Xhat, float* S, const float* G,
                            float* M, float eta, float gamma, float lambda, float beta,
                            void* stream);

/*
 * choco_set_nesterov -- Appendix D remarks that Nesterov momentum can be adapted in the same way
 * as Algorithm 2 and gives no formula.  With enable = 1 the momentum step calls of this context
 * keep Algorithm 2's memory update and take the step along the look-ahead direction,
 *     m_i = (g_i + lambda x_i) + beta m_i ;   x_i = (x_i - eta ((g_i + lambda x_i) + beta m_i)) + gamma (s_i - x^_i)
 * (the new m_i on the right), the form common in deep-learning optimisers.  enable = 0 (the
 * default) restores Algorithm 2.  Steps captured into CUDA graphs are dropped.
 */
int choco_set_nesterov(choco_ctx* ctx, int32_t enable);

/*
 * choco_sgd_step_host -- the same step as choco_sgd_step on HOST arrays (pageable or
 * pinned): copies X, Xhat, S, G to library-owned device staging buffers (allocated on the
 * first such call), runs the step, copies X, Xhat, S back and synchronises `stream` before
 * returning.  G may be NULL for a gossip-only step.  The copies run on two streams of the
 * context beside `stream` (created on the first such call; they start after what `stream` holds
 * at the call and `stream` waits for them): all of X and Xhat first, then S and G in eight chunks
 * of rows, each chunk updated as soon as it has arrived and copied back while the next ones are
 * still on their way, so that with pinned host arrays the link carries both directions at once.
 */
int choco_sgd_step_host(choco_ctx* ctx, float* X, float* Xhat, float* S, const float* G,
                        float eta, float gamma, void* stream);

/*
 * The library may carry work across calls: while forming x_i of this step it can already
 * prepare the next step's compression from the registers it holds.  That is valid only if
 * the caller leaves X and Xhat untouched between two step calls and passes the same
 * pointers; a change of pointers is detected, a change of contents is not.
 * choco_invalidate -- call after modifying X or Xhat outside the library (for example
 * when loading a checkpoint into the same buffers).
 * choco_set_carry -- enable = 0 turns the carrying off (every step then compresses from X
 * and Xhat as it finds them, at the cost of one more pass over both); default on.  The
 * results are the same either way.
 */
int choco_invalidate(choco_ctx* ctx);
int choco_set_carry(choco_ctx* ctx, int32_t enable);

/*
 * Small problems (n d <= 4 194 304), where a step is a few short kernels whose launches take
 * longer than their work, replay their steady-state step from a CUDA graph: the second time a
 * step call is seen with a given set of arguments (array pointers, eta, gamma, lambda, beta) in
 * the state that repeats (see choco_invalidate above) its kernels are captured, later calls
 * launch the graph; up to 16 graphs per context.  (A caller that passes a newly allocated
 * gradient array every step therefore never triggers a capture, and gains nothing.)  Results
 * are the same bits either way.  Not used on the legacy default stream (NULL), which cannot be
 * captured, nor while `stream` is itself being captured, nor while choco_profile_enable is
 * recording.  QSGD and RANDK contexts that replay keep the step number in device memory and
 * bump it with one tiny kernel per step.
 * choco_set_graphs -- enable = 0 / 1 turns this off / on for a context of any size.
 */
int choco_set_graphs(choco_ctx* ctx, int32_t enable);

/*
 * TOPK keeps, per row, a list of candidate coordinates gathered while the previous step formed
 * x_i, under a key bound guessed for the next step.  When the guess misses (fewer than k, or
 * more than the list holds) the row is selected exactly from the dense row, by one thread block:
 * cheap for short rows, tens of milliseconds for a row of 25 M coordinates.  For rows of at
 * least 4 194 304 coordinates every step therefore enqueues six more kernels after the
 * selection kernel (two rounds of histogram and bound, collection, selection again) that return
 * at once unless a row missed, in which case they rebuild that row's candidates with all SMs.  The result is the
 * same either way.  choco_set_rescue -- enable = 0 / 1 turns these kernels off / on for a
 * context of any row length (TOPK only; CHOCO_ERR_UNSUPPORTED for other operators).
 */
int choco_set_rescue(choco_ctx* ctx, int32_t enable);

/*
 * The kernel that selects the k entries of a row among its candidates runs one thread block per
 * row, or -- for rows with many candidates (capacity of 32 768 or more) when the workers are few
 * enough that all SMs would not be busy otherwise -- a cluster of 2 or 4 blocks per row that
 * share the row through distributed shared memory.  choco_set_select_blocks -- blocks = 1, 2 or
 * 4 overrides that choice for the context (TOPK / RANDK only; CHOCO_ERR_UNSUPPORTED otherwise).
 * The result is the same either way.  Implies choco_invalidate (the candidates the last step
 * collected are arranged for the other kernel).
 */
int choco_set_select_blocks(choco_ctx* ctx, int32_t blocks);

/* Step counter t (keys the generator).  Setting it, together with restoring X, Xhat and S,
 * resumes a run bit-exactly; choco_set_step implies choco_invalidate. */
int choco_get_step(const choco_ctx* ctx, uint64_t* t);
int choco_set_step(choco_ctx* ctx, uint64_t t);

/*
 * Message size of one step by the paper's accounting (Appendix C): TOPK 2*32*k bits per
 * worker, RANDK 32*k, SIGN d + 32 (stored: 4*ceil(d/32) + 4 bytes), QSGD 32 bits per block
 * plus one sign bit and one level field (1, 2, 4 or 8 bits) per coordinate, IDENTITY 32*d.
 */
int choco_message_bytes(const choco_ctx* ctx, int64_t* per_worker, int64_t* total);

/*
 * Debug access to the message most recently formed for `worker` (valid until the next step
 * call).  plane: 0 = indices (u32[k]) or packed sign bits (u32[ceil(d/32)]); 1 = values
 * (f32[k]), the sign scale (f32[1]), QSGD block norms (f32[blocks]) or the dense q
 * (IDENTITY, f32[d]); 2 = QSGD level fields (bytes).  Returns a DEVICE pointer into
 * library-owned memory and its size; a plane the operator does not use gives nbytes = 0.
 */
int choco_get_message(const choco_ctx* ctx, int32_t worker, int32_t plane, const void** dev_ptr,
                      int64_t* nbytes);

/* Same planes, copied to a HOST buffer of `capacity` bytes after synchronising `stream`;
 * *nbytes receives the plane's size (nothing is copied if it exceeds the capacity). */
int choco_read_message(choco_ctx* ctx, int32_t worker, int32_t plane, void* host_dst,
                       int64_t capacity, int64_t* nbytes, void* stream);

/* Consensus distance of Section 6 times n: sum_i ||x_i - xbar||^2, accumulated in float64.
 * X: DEVICE pointer.  Synchronises `stream`; *out is a HOST double. */
int choco_consensus_error(choco_ctx* ctx, const float* X, double* out, void* stream);

/*
 * choco_consensus_error_noalloc -- the same quantity as choco_consensus_error for callers
 * that are not allowed to allocate device memory.  (The paper has no counterpart to this
 * call; it exists for the sake of such callers only.)  Examples: code that runs while a
 * memory pool or a capture session owns all allocation on the device, monitoring hooks
 * inside a training loop whose allocator must not be disturbed, or a process that has
 * handed its whole memory budget to someone else.  It needs no context: choco_init is
 * itself an allocating call.
 *   X        DEVICE pointer, float32 [n, ld], read-only; n >= 1, 1 <= d <= ld.
 *   out_dev  DEVICE pointer to one double, caller-owned; receives sum_i ||x_i - xbar||^2
 *            when the work enqueued on `stream` has finished (no host synchronisation).
 * Limit: d <= 4 194 304.  The per-block partial sums (one double per 256 coordinates) are
 * kept in a fixed 128 KiB array that is part of the library image on every GPU that loads
 * it, for the life of the process; larger d returns CHOCO_ERR_TOO_LARGE and enqueues nothing.
 * The call performs no cudaMalloc / cudaFree and uses no allocating library routine.
 * First use on a device looks up the address of that array (a one-time query, done with that
 * device current).  With CUDA's lazy module loading that first use may also load the kernels'
 * code and the array itself onto the device, which takes device memory: make one warm-up call
 * at start-up, while memory is still to be had and before starting any stream capture.  The
 * looked-up address is cached per device for the life of the process and is not refreshed
 * after cudaDeviceReset.
 * All calls on a device share the array.  Each call overwrites every partial it later reads,
 * so nothing carries over from one call to the next, but two calls whose kernels overlap on
 * the GPU (different streams, no ordering between them) race on it: order them.
 */
int choco_consensus_error_noalloc(const float* X, int32_t n, int64_t d, int64_t ld,
                                  double* out_dev, void* stream);

/*
 * Per-layer compression -- Section 5, "Setup": in the paper's experiments every compression
 * scheme is applied to every layer of the network separately.  The first d = layer_off[n_layers]
 * coordinates of a row are cut into n_layers consecutive layers, layer l = coordinates
 * [layer_off[l], layer_off[l+1]), and Q acts on each layer as a vector of its own:
 *   TOPK / RANDK   k_l = max(1, floor(a d_l)) entries per layer, a = a_num / a_den in (0, 1]
 *                  (p->k is ignored; floor(a d_l) = 0 would never transmit a small layer, so
 *                  at least one entry is kept);
 *   SIGN           one scale ||v_l||_1 / d_l per layer;
 *   QSGD           norms per block inside each layer (blocks restart at the layer's first
 *                  coordinate; a layer shorter than p->bucket is one block of its own length);
 *   the generator of layer l is keyed with seed + l and the coordinate's index inside the layer.
 * Everything else (Algorithm 1 / 2, arithmetic, determinism) is as for the plain calls: a
 * layered step gives the same bits as running choco_*_step with d = d_l, seed + l and
 * pointers advanced by layer_off[l] for every layer.  One library context per layer holds the
 * layer's parameters, messages and workspace.  For TOPK, SIGN and QSGD with blocks, when the
 * layers are small enough for launches to dominate (at most 32 768 tiles of 2048 coordinates
 * over all layers and workers, at most 512 layers), the steady-state step of all layers
 * together is two or three kernel launches whose blocks look their layer up in a table (layers whose rows start at odd elements, which those kernels do
 * not take for the dense operators, run their own few launches beside them).  First steps, steps
 * after choco_layers_invalidate and the other operators run layer by layer, their kernels spread
 * over a few internal streams that fork from and join `stream`; for those operators a
 * steady-state step is captured into a CUDA graph the second time it is seen with a given set
 * of arguments (the array pointers, eta, gamma, lambda, beta) and replayed by one graph launch
 * afterwards; up to 32 such graphs are kept.  (Whole-row QSGD and RANDK contexts of a layered
 * context keep the step number in device memory for this and bump it with one more tiny kernel
 * per step.)  A step call made while `stream` is itself being captured, or on the legacy default
 * stream, which cannot be captured, is enqueued kernel by kernel instead.
 *   layer_off[n_layers + 1]   HOST, strictly increasing from 0; ld >= layer_off[n_layers].
 *   a_num, a_den              used by TOPK / RANDK only.
 * Errors are those of choco_init; on error nothing is left allocated.
 */
typedef struct choco_layers choco_layers;
int choco_layers_init(choco_layers** out, int32_t n, int32_t n_layers, const int64_t* layer_off, int64_t ld,
                      const int32_t* w_row_ptr, const int32_t* w_col, const float* w_val, const choco_params* p,
                      int64_t a_num, int64_t a_den, uint64_t seed);
int choco_layers_destroy(choco_layers* layers);
/* The three step calls, with the meaning of choco_gossip_step, choco_sgd_step and
 * choco_sgd_momentum_step; X, Xhat, S, G, M are the whole [n, ld] DEVICE arrays. */
int choco_layers_gossip_step(choco_layers* layers, float* X, float* Xhat, float* S, float gamma, void* stream);
int choco_layers_sgd_step(choco_layers* layers, float* X, float* Xhat, float* S, const float* G, float eta,
                          float gamma, void* stream);
int choco_layers_sgd_momentum_step(choco_layers* layers, float* X, float* Xhat, float* S, const float* G,
                                   float* M, float eta, float gamma, float lambda, float beta, void* stream);
/* Sum over the layers of choco_message_bytes. */
int choco_layers_message_bytes(const choco_layers* layers, int64_t* per_worker, int64_t* total);
/* The context that serves one layer (owned by `layers`; for choco_get_message, choco_get_stats
 * and the like), the layer's first coordinate and its length.  Any output may be NULL. */
int choco_layers_get_layer(const choco_layers* layers, int32_t layer, choco_ctx** ctx, int64_t* offset,
                           int64_t* length);
/* enable = 0 / 1 turns the graph replay described above off / on (default on), a negative
 * value leaves it as it is; *replays (may be NULL) receives the number of steps replayed so far. */
int choco_layers_set_graphs(choco_layers* layers, int32_t enable, uint64_t* replays);
/* Number of step calls so far that were enqueued as the combined launches described above. */
int choco_layers_combined_steps(const choco_layers* layers, uint64_t* steps);
/* choco_invalidate / choco_set_step / choco_set_nesterov for every layer. */
int choco_layers_invalidate(choco_layers* layers);
int choco_layers_set_step(choco_layers* layers, uint64_t t);
int choco_layers_set_nesterov(choco_layers* layers, int32_t enable);

/* Counters since choco_init (HOST struct filled after synchronising `stream`). */
typedef struct {
    uint64_t steps;            /* step calls enqueued                                         */
    uint64_t prepared_rows;    /* rows whose compression was prepared by the previous step     */
    uint64_t recompressed_rows;/* rows compressed by a separate pass over X and Xhat           */
    uint64_t exact_rows;       /* rows that needed the slow exact selection                    */
    uint64_t kernel_launches;  /* kernels the step calls have enqueued                         */
    uint64_t device_timeouts;  /* bounded waits inside kernels that ran out (must stay 0)      */
    uint64_t graph_replays;    /* step calls served by replaying a captured CUDA graph          */
    uint64_t rescued_rows;     /* rows re-collected by the grid-wide kernels (choco_set_rescue) */
} choco_stats;
/* Fills *out; returns CHOCO_ERR_TIMEOUT (with *out filled) if device_timeouts is non-zero. */
int choco_get_stats(choco_ctx* ctx, choco_stats* out, void* stream);

/*
 * Test hook for the timeout path described at the top: the number of polls a kernel of this
 * context spends on its first wait before it gives up (default 4 194 304).  With 0 every block
 * gives up at once, then sits out its copies in the second, still bounded, wait and returns --
 * the only way to see CHOCO_ERR_TIMEOUT without a stalled memory system.  The state arrays are
 * invalid after such a step.  Not for production use.
 */
int choco_debug_set_wait_polls(choco_ctx* ctx, uint32_t polls);

/*
 * Test hook.  When a cluster of blocks selects a row (choco_set_select_blocks), the update kernel
 * that collects the next step's candidates puts those of a 2048-coordinate tile into the tile's
 * own slot of the candidate arrays, and only a tile with more candidates than the slot holds
 * reserves room behind the slots with an atomic add.  The slot is sized at choco_init (three
 * times a tile's share of 3 k candidates, at least 16); this call makes it smaller, `slot` >= 1
 * (values above the initial size are clamped to it), so that a test reaches the path behind the
 * slots and its exhaustion.  The result of a step does not depend on it.  TOPK contexts with
 * more than one block per row only; CHOCO_ERR_UNSUPPORTED otherwise.  Implies choco_invalidate.
 */
int choco_debug_set_candidate_slot(choco_ctx* ctx, int32_t slot);

/*
 * Optional timing of the update kernel (the one pass that streams X, Xhat, S and G): after
 * choco_profile_enable the next `max_steps` step calls record a CUDA event before and after
 * that kernel on the step's stream.  choco_profile_read synchronises `stream` and returns
 * how many steps were recorded and the sum of their update-kernel durations in
 * milliseconds, then clears the record.  Not part of the method; used by benchmarks.
 */
int choco_profile_enable(choco_ctx* ctx, int32_t max_steps);
/* Record only every `stride`-th step call (default 1): the events sit between the step's
 * kernels and keep them from overlapping, so timing every step slows the steps down. */
int choco_profile_set_stride(choco_ctx* ctx, int32_t stride);
int choco_profile_read(choco_ctx* ctx, int32_t* steps_recorded, double* update_ms_total,
                       void* stream);

const char* choco_strerror(int code);
/* cudaError_t of the last failing CUDA call on this context (0 if none). */
int choco_last_cuda_error(const choco_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* CHOCO_H_ */
