/*
 * nb.h - C ABI of the Non-blocking SGD aggregate-and-update library (CUDA, sm_100a).
 *
 * The library runs, on ONE GPU, the per-iteration aggregate-and-update of Non-blocking SGD
 * (He & Dube, "Accelerating Parallel Stochastic Gradient Descent via Non-blocking Mini-batches")
 * for K learners that are held as a batch dimension in device memory:
 *
 *   1. every learner i sums the gradients of the n_i mini-batches it finished before the fastest
 *      learner raised the terminal signal; the unfinished ones are abandoned   (Alg. 1 inner loop;
 *      Sec. 3.2 "Compute gradients"; Eq. 19);
 *   2. the sum is scaled by a per-learner factor s_i                            (Sec. 3.2 "Adjust
 *      learning rate"; Alg. 2 update step);
 *   3. the learners' models are combined through a mixing matrix W:
 *      x_half_i = sum_j W_ij x_j                                                (Alg. 2 averaging step;
 *      Eq. 4-5 for the all-reduce mean; Eq. 6 for D-PSGD; Sec. 6.1 for MATCHA's activated matchings);
 *   4. a momentum-SGD step follows: v_i <- mom v_i + s_i acc_i, x_i <- x_half_i - lr v_i
 *      (Alg. 2 update step; momentum is this library's addition, mom = 0 gives the paper's rule).
 *
 * Notation: the paper writes P for the number of learners, d for the parameter dimension and N for
 * the number of mini-batches; this header uses K learners, P parameters, M mini-batches.
 *
 * Conventions for every entry point
 *   - returns an nb_status; nothing throws, aborts or prints across the boundary;
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream); device work
 *     is enqueued on it and the call returns without waiting, except where stated;
 *   - pointers marked "host" are read or written on the CPU before the call returns and are never
 *     retained; pointers marked "device" must stay valid until `stream` has passed the call's work;
 *   - a context is bound to the device that was current at nb_create and must be used from one host
 *     thread at a time;
 *   - a CUDA failure is reported as NB_ERR_CUDA and is sticky for that context;
 *   - the kernels' internal waits are bounded.  One that runs out (a defect, never seen in normal
 *     operation) abandons the remaining tiles and records a code in a device word.  That word is
 *     read only where the host already waits for the device: copies to host memory
 *     (nb_get_params, nb_get_momentum, nb_get_accumulator, nb_get_mean_params with a host dst),
 *     nb_step_fused_host and nb_check_guards, the explicit query.  It then becomes a sticky
 *     NB_ERR_CUDA; models and momentum produced since the previous such point are invalid.  Calls
 *     that only enqueue work (nb_accumulate, nb_step, nb_step_fused, outputs to device memory)
 *     return NB_OK without looking at it.
 */
#ifndef NB_H_
#define NB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define NB_MAX_K 64          /* learners                                                     */
#define NB_MAX_MATCHINGS 32  /* matchings of a MATCHA topology (activation bits fit a word)  */
#define NB_MAX_NNZ 1024      /* non-zeros of a sparse mixing matrix                          */

typedef struct nb_ctx nb_ctx; /* opaque; owned by the library */

enum nb_status {
  NB_OK = 0,
  NB_ERR_ARG = -1,         /* invalid argument (nb_last_error says which)               */
  NB_ERR_STATE = -2,       /* call order violated (e.g. nb_step without nb_accumulate)  */
  NB_ERR_CUDA = -3,        /* a CUDA call failed; sticky                                 */
  NB_ERR_NOMEM = -4,       /* device or host allocation failed                           */
  NB_ERR_UNSUPPORTED = -5  /* valid request outside the library's limits                 */
};

/* How the learners are combined (step 3 above). */
enum nb_variant {
  NB_ALLREDUCE = 0,   /* W = (1/K) 1 1^T: mean over learners (Eq. 4-5)                              */
  NB_DPSGD = 1,       /* fixed sparse doubly-stochastic W (Eq. 6; Alg. 2)                           */
  NB_MATCHA = 2,      /* W(t) = I - alpha * sum of the Laplacians of the matchings active at t      */
  NB_CENTRALIZED = 3  /* one parameter-server model shared by all learners (Alg. 3).  The server    */
                      /* applies the MEAN of the learners' terms, (1/K) sum_i s_i acc_i (Eq. 2's    */
                      /* 1/P), where Alg. 3 as printed sums them; pass lr * K to get the sum.        */
};

enum nb_dtype { NB_F32 = 0, NB_BF16 = 1 }; /* element type of the gradient stream */

enum nb_topology_kind {
  NB_TOPO_FULL = 0,           /* complete graph, W_ij = 1/K                                          */
  NB_TOPO_RING = 1,           /* W_ii = W_i,i+1 = W_i,i-1 = 1/3 (indices mod K)                      */
  NB_TOPO_CSR = 2,            /* explicit W in CSR form                                              */
  NB_TOPO_MATCHINGS = 3,      /* explicit matchings (partner table)                                  */
  NB_TOPO_RANDOM_REGULAR = 4  /* seeded random `degree`-regular graph, greedily split into matchings */
};

/* Topology description, host memory, copied by the callee.  Unused fields are ignored. */
typedef struct nb_topology {
  int32_t kind;            /* nb_topology_kind                                                     */
  int32_t degree;          /* RANDOM_REGULAR: vertex degree (K*degree even, degree < K)            */
  uint64_t seed;           /* RANDOM_REGULAR: graph seed; MATCHA: also seeds the activation draws  */
  const int32_t *row_ptr;  /* CSR: [K+1]                                                           */
  const int32_t *col_idx;  /* CSR: [row_ptr[K]], any order inside a row                            */
  const float *val;        /* CSR: [row_ptr[K]]; rows and columns must sum to 1 within 1e-5        */
  int32_t n_matchings;     /* MATCHINGS: number of matchings, <= NB_MAX_MATCHINGS                  */
  const int32_t *partner;  /* MATCHINGS: [n_matchings*K], partner[c*K+v] = v's partner, -1 = none  */
  float alpha;             /* MATCHA: W = I - alpha * sum_active L_j, 0 <= alpha <= 1 (rows and     */
                           /* columns always sum to 1; a diagonal entry is negative where alpha *   */
                           /* active degree > 1)                                                    */
  float act_prob;          /* MATCHA: each matching is active with this probability, per step      */
  const float *act_probs;  /* MATCHA: optional [number of matchings] per-matching probabilities    */
                           /* (replace act_prob; for RANDOM_REGULAR learn the number of matchings  */
                           /* from nb_topology_matchings first); NULL = act_prob for all           */
} nb_topology;

/* nb_set_option keys and values */
enum nb_option {
  NB_OPT_NORM = 0,   /* NB_NORM_MEAN (default) | NB_NORM_PAPER */
  NB_OPT_ORDER = 1,  /* NB_ORDER_MIX_THEN_UPDATE (default) | NB_ORDER_UPDATE_THEN_MIX */
  NB_OPT_KERNEL = 2,    /* NB_KERNEL_AUTO (default) | NB_KERNEL_DIRECT */
  NB_OPT_STREAMING = 3  /* NB_STREAMING_ACCUMULATE (default) | NB_STREAMING_HOLD; see nb_accumulate_minibatch */
};
enum nb_norm {
  NB_NORM_MEAN = 0,  /* s_i = 1/n_i: mean of the finished mini-batch gradients (s_i = 0 if n_i = 0)        */
  NB_NORM_PAPER = 1  /* s_i = n_i/M: the learning-rate adjustment eta*n/N of Alg. 2 applied to the sum     */
};
enum nb_order {
  NB_ORDER_MIX_THEN_UPDATE = 0, /* Alg. 2: x_i <- sum_j W_ij x_j - lr v_i                                   */
  NB_ORDER_UPDATE_THEN_MIX = 1  /* Eq. 4-6: x_i <- sum_j W_ij (x_j - lr v_j)                                */
};

enum nb_streaming {
  NB_STREAMING_ACCUMULATE = 0, /* every delivered mini-batch gradient is added to the accumulator at once   */
  NB_STREAMING_HOLD = 1        /* deliveries are only recorded; nb_step reads the vectors where they lie     */
};
enum nb_kernel {
  NB_KERNEL_AUTO = 0,   /* bulk-copy pipeline kernels wherever they apply, direct-load kernels elsewhere */
  NB_KERNEL_DIRECT = 1  /* direct-load kernels only (same bits, slower): a cross-check for tests        */
};

/* ------------------------------------------------------------------------------------------------
 * Host straggler simulator: stands in for the terminal signal of Alg. 1 (the first learner to
 * finish its M mini-batches ends the iteration; the others abandon what they have not finished).
 * One mini-batch time tau_i per learner per iteration (Sec. 4.1), constant speed inside an
 * iteration (Sec. 4.3): n_i = max(1, #{j in 1..M : j*tau_i <= M*min_i tau_i}).
 * Pure functions of (configuration, step): no context, no GPU.
 * ---------------------------------------------------------------------------------------------- */
enum nb_straggler_model {
  NB_STRAG_UNIFORM_COUNT = 0,       /* n_i uniform on {1..M}; no parameters                               */
  NB_STRAG_SHIFTED_EXP = 1,         /* tau_i = 1 + Exp(mean params[0])                                    */
  NB_STRAG_SHIFTED_EXP_SLOWSET = 2  /* floor(params[0]*K) learners, re-drawn every step, have mean        */
                                    /* params[1]; the rest have mean params[2]                             */
};
typedef struct nb_straggler {
  int32_t model;     /* nb_straggler_model */
  uint64_t seed;
  double params[4];
} nb_straggler;

/* finished: host out [K].  mask: host out [K*M] (mask[i*M+m] = m < n_i) or NULL.
 * tau: host out [K] mini-batch times, or NULL (written as 0 for UNIFORM_COUNT).
 * Errors: NB_ERR_ARG for K<1, K>NB_MAX_K, M<1, unknown model, negative means. */
int nb_straggler_sample(const nb_straggler *cfg, int K, int M, int64_t step, int32_t *finished,
                        uint8_t *mask, double *tau);

/* Run-time figures of the straggler model over `steps` iterations starting at step0 (Sec. 4.2-4.3):
 * per-iteration run-time of Non-blocking SGD, M*min_i tau_i (Lemma 1: the first order statistic),
 * and of a blocking method, M*max_i tau_i; their ratio (Theorem 1); the throughput ratio
 * Y*X_{K:K}/K with Y = sum_i 1/tau_i (Theorem 5); the data fraction Y*X_{1:K}/K that Corollary 1
 * predicts for fractional mini-batches, and the fraction sum_i n_i/(K*M) the floor rule yields.
 * Host only.  NB_ERR_UNSUPPORTED for NB_STRAG_UNIFORM_COUNT (it has no times). */
typedef struct nb_runtime_report {
  double mean_t_nonblocking;    /* mean of M * min_i tau_i                     */
  double mean_t_blocking;       /* mean of M * max_i tau_i                     */
  double ratio;                 /* mean_t_nonblocking / mean_t_blocking        */
  double mean_throughput_ratio; /* mean of Y * max_i tau_i / K                 */
  double mean_fractional_data;  /* mean of Y * min_i tau_i / K                 */
  double mean_finished_fraction;/* mean of sum_i n_i / (K*M)                   */
  double mean_min_tau, mean_max_tau;
  int64_t steps;
} nb_runtime_report;
int nb_runtime_report_compute(const nb_straggler *cfg, int K, int M, int64_t step0, int64_t steps,
                              nb_runtime_report *out);

/* ------------------------------------------------------------------------------------------------
 * Host topology helpers (no context, no GPU).
 * ---------------------------------------------------------------------------------------------- */

/* Matchings of a MATCHINGS or RANDOM_REGULAR topology.  partner: host out [NB_MAX_MATCHINGS*K]
 * (first n*K entries written); n_matchings: host out; attempts: host out or NULL (graph draws
 * rejected + 1).  Errors: NB_ERR_ARG for an impossible degree, a partner table that is not an
 * involution or repeats an edge; NB_ERR_UNSUPPORTED if more than NB_MAX_MATCHINGS are needed. */
int nb_topology_matchings(const nb_topology *topo, int K, int32_t *partner, int32_t *n_matchings,
                          int32_t *attempts);

/* MATCHA's design problem for the matchings of `topo` (MATCHINGS or RANDOM_REGULAR; Sec. 6.1: a
 * communication budget c_b = mean activation frequency of the links, probabilities that favour the
 * links that matter for connectivity, a step size alpha).  With L_bar(p) = sum_j p_j L_j:
 *   probs  maximise lambda_2(L_bar(p)) subject to 0 <= p_j <= 1 and sum_j p_j <= budget * m
 *          (projected supergradient ascent, `iters` iterations, 0 = 1000);
 *   alpha  minimises rho = || E[W^T W] - (1/K) 1 1^T ||_2 for W = I - alpha * sum_j B_j L_j with
 *          independent B_j ~ Bernoulli(p_j) (golden-section search on [0, 1]; rho is convex).
 * Host out: probs[m] (m from nb_topology_matchings), *alpha, *lambda2, *rho (each may be NULL).
 * budget = 1 gives p = 1: every matching always active, i.e. vanilla decentralized SGD.
 * Errors: NB_ERR_ARG (bad topology, budget outside (0, 1]). */
int nb_matcha_optimize(const nb_topology *topo, int K, float budget, int iters, float *probs, float *alpha,
                       float *lambda2, float *rho);

/* The mixing matrix a context created with (variant, topo, K) uses at `step`, dense row-major
 * host out [K*K]; bits: host out or NULL, the MATCHA activation word (bit j = matching j active).
 * Same validation as nb_create. */
int nb_mixing_matrix(const nb_topology *topo, int variant, int K, int64_t step, float *W_dense,
                     uint32_t *bits);

/* ------------------------------------------------------------------------------------------------
 * Context
 * ---------------------------------------------------------------------------------------------- */

/* Creates a context on the current device: K learners, P parameters each, M mini-batches per
 * batch; allocates the models X[K,P], the momentum V[K,P] (zeroed) and the accumulator acc[K,P]
 * in fp32 (NB_CENTRALIZED: one model and one momentum vector; acc still [K,P]).
 * topo may be NULL for NB_ALLREDUCE and NB_CENTRALIZED.  NB_DPSGD takes RING, FULL or CSR;
 * NB_MATCHA takes MATCHINGS or RANDOM_REGULAR.
 * Errors: NB_ERR_ARG (K<1, P<1, M<1, bad topology, W not doubly stochastic within 1e-5),
 * NB_ERR_UNSUPPORTED (K>NB_MAX_K, nnz>NB_MAX_NNZ), NB_ERR_NOMEM, NB_ERR_CUDA.  *out is NULL on error. */
int nb_create(nb_ctx **out, int K, int64_t P, int M, float lr, float mom, int variant,
              const nb_topology *topo);

/* Frees everything the context owns (waits for the device first).  NULL is accepted. */
int nb_destroy(nb_ctx *c);

/* Last error text of this context (or of the last failed nb_create when c is NULL). */
const char *nb_last_error(const nb_ctx *c);

int nb_set_option(nb_ctx *c, int key, int64_t value);
int nb_set_lr(nb_ctx *c, float lr);

/* Loads the models: per_learner = 0: x0[P] is given to every learner (all learners start from
 * one common model: initialisation line of Alg. 1); per_learner = 1: x0[K,P] dense.  x0: host or device.
 * Zeroes the momentum and the step counter.  NB_CENTRALIZED accepts only per_learner = 0. */
int nb_set_params(nb_ctx *c, const float *x0, int per_learner, void *stream);

/* Masked accumulate (step 1): acc[i,p] = sum_{m < finished[i]} grads[i,m,p], fp32 accumulation in
 * ascending m; rows m >= finished[i] are never read.
 * grads: device, element (i,m,p) at grads[i*ld_k + m*ld_m + p], dtype NB_F32 or NB_BF16;
 * ld_m, ld_k in elements, 0 = dense (ld_m = P, ld_k = M*P); grads must be aligned to its element
 * size.  Alignment decides the kernel, never the result (all paths give identical bits): the
 * bulk-copy pipeline kernels cover all full 512-column tiles of any stream - rows that are 16-byte
 * aligned (grads, ld_m and ld_k multiples of 16 bytes) travel as tensor-map boxes, other rows as one
 * bulk copy each of their 16-byte aligned superset (a few per cent slower; when grads itself is not
 * 16-byte aligned the first tile goes to the direct kernels too); the direct kernels take the
 * ragged tail with 128-bit / 64-bit loads where 4-element alignment allows and scalar loads elsewhere.
 * (Rows whose pitch is a multiple of 2 KB stream 1-2 % faster than other 16-byte multiples.)
 * finished: host [K], each in [0, M].  Errors: NB_ERR_ARG. */
int nb_accumulate(nb_ctx *c, const void *grads, int dtype, int64_t ld_m, int64_t ld_k,
                  const int32_t *finished, void *stream);

/* Row pitch, in elements, at which a gradient stream of P columns of `dtype` streams fastest: the
 * smallest multiple of 2 KB that holds P elements.  Every 512-column tile segment of every row then
 * lies inside one 2 KB block of device memory (measured on B200, P = 138,000,000 bf16: dense rows,
 * whose segments straddle those blocks, run 1 to 3 % below rows at this pitch).  Pass it as ld_m (and
 * M * pitch, or more, as ld_k).  Purely advisory: any pitch >= P is accepted.  Returns 0 for P < 1
 * or an unknown dtype. */
int64_t nb_recommended_pitch(int64_t P, int dtype);

/* Streaming form of step 1 (Alg. 1 inner loop as the gradients arrive): a learner hands over one
 * finished mini-batch gradient at a time.  nb_begin_iteration clears the per-learner counts and the
 * terminal signal.  nb_accumulate_minibatch adds grad[P] (device, NB_F32 or NB_BF16) to learner i's
 * accumulator in fp32 - the same sums, in the same order, as nb_accumulate - and counts it; when a
 * learner has delivered all M mini-batches it is the first finisher and the terminal signal is
 * raised (Alg. 1, inner loop: the learner whose count reaches N tells the others); every later
 * call of the iteration returns NB_ABANDONED (a status, not an error) without touching anything
 * (Alg. 1: the other learners leave their loop and drop what they have not finished).  nb_step
 * then runs on the counts collected.  nb_get_finished reports them.
 * With NB_OPT_STREAMING = NB_STREAMING_HOLD (set between iterations) a delivery is only recorded: the
 * caller promises that every delivered vector stays valid and unchanged until `stream` has passed the
 * work of the following nb_step, which then runs the FUSED step on the recorded vectors (no
 * accumulator read-modify-write per delivery: the iteration moves the algorithmic bytes only, as
 * nb_step_fused does; measured 2.6x the throughput of the accumulate mode at K = 16, P = 25.6M, M = 8).  Vectors
 * must be 16-byte aligned and of one dtype per iteration (NB_ERR_ARG otherwise); results are
 * bit-identical to the accumulate mode; nb_get_accumulator is not meaningful in this mode. */
#define NB_ABANDONED 1
int nb_begin_iteration(nb_ctx *c);
int nb_accumulate_minibatch(nb_ctx *c, int learner, const void *grad, int dtype, void *stream);
int nb_get_finished(const nb_ctx *c, int32_t *finished /* host out [K] */, int32_t *terminal /* host out or NULL */);

/* Steps 2-4 on what the last nb_accumulate stored; advances the step counter.
 * NB_ERR_STATE if there has been no nb_accumulate since the last step. */
int nb_step(nb_ctx *c, void *stream);

/* Steps 1-4 in a single pass over the gradient stream without the acc round trip.  The result is
 * bit-identical to nb_accumulate followed by nb_step.  Arguments as nb_accumulate.
 * CUDA graphs: nb_accumulate, nb_step and nb_step_fused only enqueue kernels on `stream` (no
 * allocation, copy or synchronisation), so they may be called while `stream` is being captured;
 * the finished counts, the pointers and (MATCHA) the step index are fixed in the captured launches,
 * and the host-side step counter advances once per call, not per replay.  (Not nb_step after
 * deliveries in NB_STREAMING_HOLD mode: it uploads the table of delivered vectors first.) */
int nb_step_fused(nb_ctx *c, const void *grads, int dtype, int64_t ld_m, int64_t ld_k,
                  const int32_t *finished, void *stream);

/* As nb_step_fused with the gradient stream in HOST memory (pinned for speed): copies only the
 * finished mini-batch rows into a staging buffer the context allocates on first use ([K,M,P]
 * elements of the widest dtype seen), runs the fused step and, when mean_out is not NULL, writes
 * the mean model (Alg. 1 "Output") to host memory mean_out[P].  The columns are processed in up to
 * 8 chunks so that the host-to-device copies, the kernels and the device-to-host copy of the mean
 * overlap (two internal streams and a few events are created on first use; the kernels run on
 * `stream`).  Waits for all of it before it returns.  Same result as nb_step_fused, bit for bit. */
int nb_step_fused_host(nb_ctx *c, const void *grads_host, int dtype, int64_t ld_m, int64_t ld_k,
                       const int32_t *finished, float *mean_out, void *stream);

/* Outputs.  dst is host or device memory, dense.  Copies to pageable host memory wait for `stream`. */
int nb_get_params(nb_ctx *c, float *dst /* [K,P] ([P] for NB_CENTRALIZED) */, void *stream);
int nb_get_momentum(nb_ctx *c, float *dst /* as nb_get_params */, void *stream);
int nb_get_accumulator(nb_ctx *c, float *dst /* [K,P] */, void *stream);
/* Average of all learners' models (Alg. 1 / Alg. 2 "Output"), summed in ascending learner order. */
int nb_get_mean_params(nb_ctx *c, float *dst /* [P] */, void *stream);

/* Checkpoint / resume: loads models, momentum (dense, host or device, shaped as nb_get_params
 * returns them) and the step counter.  All randomness is a function of (seed, step), so a restored
 * run continues bit-identically. */
int nb_set_state(nb_ctx *c, int64_t step, const float *X, const float *V, void *stream);
int nb_get_step(const nb_ctx *c, int64_t *step);

/* The mixing matrix this context uses at `step` (host-side computation), dense host out [K*K]. */
int nb_get_W(nb_ctx *c, int64_t step, float *W_dense);
/* MATCHA: the activation word the host computes for `step`. */
int nb_get_matcha_activation(nb_ctx *c, int64_t step, uint32_t *bits);
/* MATCHA: what the DEVICE-side builder produced for the most recent step: its activation word and
 * its W, densified (host out [K*K]).  Waits for `stream`.  NB_ERR_STATE before the first step. */
int nb_get_device_mixing(nb_ctx *c, uint32_t *bits, float *W_dense, void *stream);

/* Counters of the most recent step: sum of finished counts, algorithmic bytes
 * P*(e_g*sum n_i + 16*K) (e_g = bytes per gradient element; NB_CENTRALIZED: 16 instead of 16*K),
 * and the number of kernels this library has launched on this context so far. */
int nb_get_stats(const nb_ctx *c, int64_t *sum_finished, double *algorithmic_bytes,
                 int64_t *kernel_launches);

/* Self-check: X, V and the accumulator are allocated between guard bands of a fixed byte pattern;
 * this waits for `stream`, reads the bands back and returns NB_ERR_STATE (with the array and offset
 * in nb_last_error) if any kernel wrote outside its array, NB_ERR_CUDA if a kernel reported a wait
 * that ran out, NB_OK otherwise. */
int nb_check_guards(nb_ctx *c, void *stream);

/* Self-test of the kernels' bounded waits: runs one warp that waits, with a limit of about a
 * millisecond, on a barrier nothing will complete, and checks that every lane gave up, that the
 * device error word carried the wait's code and that the kernel returned normally.  The error word
 * is cleared again: the context stays usable.  Waits for `stream`.  NB_OK if all of that held,
 * NB_ERR_STATE otherwise.  (The waits of the production kernels use the same code with a limit of
 * about a second; when one runs out the context reports a sticky NB_ERR_CUDA.) */
int nb_selftest_wait_timeout(nb_ctx *c, void *stream);

/* Bounds-checked build.  A library compiled with -DNB_DEBUG (python -m paper_2211_00889_b200.build
 * --debug writes it next to the shipped one) checks, inside every kernel, that each tile coordinate,
 * ring slot, shared-memory offset, table index and global address it is about to use lies inside
 * the array it belongs to; a failed check skips the access and records a code in the device error
 * word (100 + kind), which nb_check_guards and the host-memory outputs then report as NB_ERR_CUDA.
 * Nothing traps.  nb_debug_build returns 1 in such a library, 0 in the shipped one.  The two
 * functions below run the kernels' own range predicates on the host (any build): 0 if the byte span
 * [addr, addr+bytes) lies inside [lo, hi) / if 0 <= index < count, otherwise the code a kernel
 * would have recorded. */
int nb_debug_build(void);
int nb_debug_span_code(uint64_t addr, uint64_t bytes, uint64_t lo, uint64_t hi);
int nb_debug_index_code(int64_t index, int64_t count);

/* Which kernel shape ran the most recent step (for reports and tests), host out plan[12]:
 * [0] 1 if the bulk-copy pipeline kernel covered the full tiles, 0 if the direct-load kernel did
 * everything; [1] tile width in columns; [2] consumer groups per CTA; [3] ring slots per CTA;
 * [4] gradient rows per ring item; [5] CTAs launched; [6] dynamic shared memory per CTA in bytes;
 * [7] tiles covered; [8] 0 if the gradient rows travelled as tensor-map boxes, 1 if as one bulk
 * copy per row (rows not 16-byte aligned), 2 if as one bulk copy per held vector (NB_STREAMING_HOLD);
 * [9] columns before the first covered tile (they, and the
 * columns after [9] + [7]*[1], went to the direct-load kernel); [10] buffers of the old-model stage
 * (1-3; 0 for the centralized step, which has none); [11] columns a consumer thread owns (4 or 8). */
int nb_get_kernel_plan(const nb_ctx *c, int32_t *plan);

/* ------------------------------------------------------------------------------------------------
 * Allocation-free variant (no counterpart in the paper: it exists for deployment reasons only).
 *
 * For callers that may not allocate device memory while they run - a process whose framework pool
 * already owns the whole GPU, a serving loop that cannot take the device-wide stall of an
 * allocation, a deployment that forbids allocation after start-up.  It runs one all-reduce-variant
 * iteration (masked accumulate, mean normalisation, mean over learners, momentum step, Alg. 2
 * order) entirely on memory the caller passes in, plus ONE piece of scratch: the fp32 accumulator
 * between the accumulate kernel and the update kernel, which is a fixed array inside the library
 * image of NB_STATIC_MAX_ELEMS floats (16 MiB; every GPU that loads the library holds it until the
 * process exits).  No context is needed, and no call after the first on a device allocates or
 * frees anything, through the CUDA runtime or any library (the first call resolves the array's
 * address, which is also when a lazily loading driver brings the library's code and this array onto
 * the device).
 *
 *   X, V      device, in/out, [K, ld] fp32 models and momentum, 16-byte aligned, ld >= P and a
 *             multiple of 4; columns [P, ld) of each row are padding the call may overwrite
 *   grads, dtype, ld_m, ld_k, finished   as nb_accumulate
 *
 * Limits and behaviour
 *   - K*ld must not exceed NB_STATIC_MAX_ELEMS: larger problems are rejected with
 *     NB_ERR_UNSUPPORTED and a message (nb_last_error(NULL)); nothing is launched.
 *   - The first call on each device resolves the array's device address (once, with that device
 *     current); make that first call during set-up, before any stream capture is begun.  The
 *     address is cached per device ordinal and is stale after cudaDeviceReset.
 *   - All calls on a device share the one array.  A call overwrites every element it later reads,
 *     so no state leaks from one call to the next, but two calls whose kernels overlap on the GPU
 *     (different streams, different threads, different contexts of the library) race on it:
 *     serialise them.
 *   - Results are bit-identical to nb_accumulate + nb_step on an NB_ALLREDUCE context.
 * Errors: NB_ERR_ARG, NB_ERR_UNSUPPORTED, NB_ERR_CUDA; text through nb_last_error(NULL).
 * ---------------------------------------------------------------------------------------------- */
#define NB_STATIC_MAX_ELEMS (1 << 22)
int nb_step_static(int K, int64_t P, int M, float lr, float mom, float *X, float *V, int64_t ld,
                   const void *grads, int dtype, int64_t ld_m, int64_t ld_k, const int32_t *finished,
                   void *stream);

#ifdef __cplusplus
}
#endif
#endif /* NB_H_ */
