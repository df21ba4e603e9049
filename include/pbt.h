/*
 * pbt.h -- C ABI of the lockstep Population Based Training library for one
 * NVIDIA B200 (sm_100a).
 *
 * The library trains a whole population of small networks concurrently on one
 * GPU, each member with its own hyperparameter vector h, and interleaves the
 * paper's exploit / explore step (Algorithm 1 of "Population Based Training of
 * Neural Networks", executed in the partial-synchrony form of Appendix A.1: all
 * members advance the same number of steps, then exploit-and-explore runs).
 *
 * Conventions
 *   - Every function returns a pbt_status; none throws or aborts.
 *     pbt_last_error() gives a human-readable reason for the last failure.
 *   - "device" pointers are CUDA device addresses on the current device;
 *     "host" pointers are ordinary host memory.  The library allocates no device
 *     memory: the caller passes one workspace (size from pbt_query_workspace)
 *     and the data pools, and keeps both alive until pbt_destroy.
 *   - All work is enqueued on the stream given to pbt_create.  The calls of
 *     the training loop only enqueue and return: pbt_step, pbt_eval,
 *     pbt_step_subset, pbt_exploit_explore(_ready) under every exploit rule, pbt_set_batch,
 *     pbt_prefetch_host_batch, pbt_step_prefetched / pbt_step_host without a
 *     loss buffer, pbt_grouped_gemm.  Calls that move data between ordinary
 *     host memory and the device synchronise that stream before they return:
 *     pbt_create, every pbt_get_*, and pbt_set_state / pbt_set_fitness /
 *     pbt_set_hparams / pbt_set_history (their host arguments may be reused
 *     at once).
 *   - A handle belongs to the device that was current in pbt_create; make
 *     that device current for every later call on it.  Several handles on
 *     several devices may live in one process.
 *   - There is no CPU fallback: without a CUDA device every call that would
 *     launch work fails with PBT_ERR_CUDA.
 *
 * Canonical parameter order ("flat order") used by pbt_state_view: for stack 0
 * then stack 1, for each layer l in order: W_l as [out][in] row-major, then
 * b_l[out].  P = total count.  The toy model's flat vector is theta itself.
 */
#ifndef PBT_H_
#define PBT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PBT_MAX_LAYERS 8   /* weight layers per stack */
#define PBT_MAX_NH 8       /* hyperparameter slots per member */
#define PBT_HISTORY 10     /* scores kept per member for t-test selection (Section 4.1.1, exploit (a)) */
#define PBT_N_SCALARS 4    /* Adam running beta products: c1,c2 of stack 0; c1,c2 of stack 1 */

typedef enum pbt_status {
  PBT_OK = 0,
  PBT_ERR_INVALID_ARG = 1,
  PBT_ERR_UNSUPPORTED = 2, /* a combination the kernels do not implement (never a silent CPU path) */
  PBT_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small */
  PBT_ERR_CUDA = 4,        /* a CUDA call failed */
  PBT_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired (status word set by a kernel) */
  PBT_ERR_STATE = 6        /* call not valid in the handle's current state */
} pbt_status;

typedef enum pbt_dtype {
  PBT_FP64_TOY = 0,        /* toy quadratic, everything in double */
  PBT_FP32 = 1,            /* fp32 weights, fp32 GEMMs */
  PBT_BF16_FP32MASTER = 2  /* bf16 GEMM operands (weights shadow, activations, deltas), fp32 masters and optimiser state */
} pbt_dtype;

typedef enum pbt_model { PBT_TOY_QUADRATIC = 0, PBT_MLP = 1, PBT_GAN_PAIR = 2 } pbt_model;

typedef enum pbt_loss {
  PBT_LOSS_TOY = 0,
  PBT_LOSS_MSE = 1,        /* mean_i sum_j (z_ij - y_ij)^2 */
  PBT_LOSS_CE_HARD = 2,    /* softmax cross-entropy, int32 class labels */
  PBT_LOSS_CE_SOFT = 3,    /* cross-entropy against a target distribution */
  PBT_LOSS_GAN_LOGISTIC = 4, /* non-saturating logistic GAN losses */
  PBT_LOSS_WGAN_GP = 5       /* Section 4.3.1: Wasserstein critic with gradient penalty,
                                L_D = mean D(G(z)) - mean D(x) + gp_lambda mean_b (||grad_x D(xhat_b)||_2 - 1)^2,
                                xhat_b = eps_b x_b + (1 - eps_b) G(z_b);  L_G = -mean D(G(z)) */
} pbt_loss;

typedef enum pbt_optimizer {
  PBT_OPT_SGD_PLAIN = 0, /* theta <- theta - lr g (Section 3's example of step); no optimiser state */
  PBT_OPT_SGDM = 1,      /* v <- mu v + g, theta <- theta - lr v */
  PBT_OPT_ADAM = 2,
  PBT_OPT_RMSPROP = 3 /* ms <- rho ms + (1-rho) g^2, theta <- theta - lr g / (sqrt(ms) + eps); rho = const_beta2; ms in opt1 */
} pbt_optimizer;

/* prior of a hyperparameter slot, used by the resample explore rule (Section 4.1.1, explore (b)) */
typedef enum pbt_prior { PBT_PRIOR_FIXED = 0, PBT_PRIOR_UNIFORM = 1, PBT_PRIOR_LOG_UNIFORM = 2 } pbt_prior;

/* exploit / explore switches ("PBT targets" ablation, Section 4.4) */
#define PBT_COPY_WEIGHTS 1u  /* exploit copies weights and optimiser state */
#define PBT_COPY_HPARAMS 2u  /* exploit copies the donor's hyperparameters */
#define PBT_EXPLORE 4u       /* members that copied perturb their hyperparameters */

/*
 * Description of a population (plain data, copied by pbt_create).
 *
 * Networks: stack s has n_layers[s] weight layers; layer l maps
 * widths[s][l] -> widths[s][l+1], ReLU after every layer but the last.
 * PBT_MLP uses stack 0 only.  PBT_GAN_PAIR: stack 0 is the generator
 * (noise -> sample), stack 1 the discriminator (sample -> one logit);
 * widths[1][0] must equal the generator's output width.
 * PBT_TOY_QUADRATIC: theta and h both have nh components, n_layers ignored.
 *
 * Hyperparameter slots: slot_* is the column of h that holds the quantity for
 * each member, or -1 when the quantity is the same constant for everybody
 * (const_*).  The toy model uses all nh columns as h itself.
 */
typedef struct pbt_spec {
  int32_t n_members;
  int32_t dtype;      /* pbt_dtype */
  int32_t model;      /* pbt_model */
  int32_t loss;       /* pbt_loss */
  int32_t optimizer;  /* pbt_optimizer */
  int32_t n_layers[2];
  int32_t widths[2][PBT_MAX_LAYERS + 1];
  int32_t batch;        /* training rows per member per update */
  int32_t eval_batch;   /* rows of the held-out set (GAN: generated samples scored) */
  int32_t pool_rows;    /* rows of every training pool */
  int32_t gan_d_steps;  /* K discriminator updates per step (Section 4.3.1: 5) */
  int32_t nh;
  int32_t slot_lr;      /* learning rate (generator's for a GAN) */
  int32_t slot_lr_d;    /* discriminator learning rate */
  int32_t slot_momentum;
  int32_t slot_beta1;
  int32_t slot_wd;
  uint32_t perturb_mask; /* bit k set: explore may perturb slot k */
  uint32_t flags;        /* PBT_COPY_WEIGHTS | PBT_COPY_HPARAMS | PBT_EXPLORE */
  int32_t trunc_num, trunc_den; /* truncation fraction, 1/5 in the paper */
  int32_t keep_grad; /* 1: weight gradients are also stored (pbt_get_state .grad is then valid for every tensor);
                        0: layers whose Adam update is fused into the weight-gradient GEMM never write theirs */
  int32_t fuse_adam; /* 1: apply Adam inside the epilogue of tensor-core weight-gradient GEMMs (the gradient of those
                        layers never goes to HBM); 0: weight gradients are written once and one streaming pass over
                        the slabs applies the update.  Results are bit-identical; only the traffic pattern differs. */
  int32_t programmatic_launches; /* 0 (default): plain stream order.  1: kernels are launched with programmatic stream
                        serialization: a kernel may be scheduled while its predecessor drains and waits on the device
                        until the predecessor's results are visible (same dependences, bit-identical results).  On a
                        B200 this was not faster than replaying the captured step in stream order.  The setting of
                        the handle used last applies to the process. */
  int32_t backward_streams; /* Back-propagation of one layer is three independent launches that all read the layer's
                        delta: the data gradient (which the next layer waits for), the weight gradient and the bias
                        gradient.  0 (default) or 2: the bias gradient, and the weight gradient unless its Adam update
                        is fused into it (that launch must follow the data gradient, which reads the old weights),
                        are enqueued on a second stream owned by the handle, forked from and joined to the handle's
                        stream inside each layer, so they run beside the data gradient; the replayed step graph
                        captures them as parallel branches.  1: everything in the handle's stream.  Same kernels on
                        the same inputs either way: results are bit-identical.  On the legacy default stream (NULL)
                        the setting is ignored and one stream is used. */
  int32_t member_base;  /* this handle holds members [member_base, member_base + n_members) of a larger population that
                           is sharded over several handles (one per GPU).  Everything that is drawn per member (initial
                           weights, training rows, interpolation coefficients, donors, explore draws) is keyed by the
                           member's index in the WHOLE population, so a sharded run takes exactly the steps of the
                           unsharded one.  0 for an ordinary population. */
  int32_t n_global;     /* members of the whole population (0: n_members, i.e. not sharded; at most 1024) */
  int32_t exploit_rule; /* 0: truncation selection (Section 4.1.1 (b)); 1: binary tournament (Section 4.3.1 (b)): every
                           member draws one other member uniformly and copies it if its fitness is strictly higher;
                           2: t-test selection (Section 4.1.1, exploit (a)): one other member drawn uniformly is
                           copied if its mean over its last PBT_HISTORY scores is higher and Welch's t-test rejects
                           equal means at level ttest_alpha (two-sided).  pbt_eval records the scores. */
  int32_t explore_rule; /* 0: perturb (Section 4.1.1, explore (a)); 1: resample (Section 4.1.1, explore (b)): each
                           slot of perturb_mask whose prior is not PBT_PRIOR_FIXED is redrawn from its prior with
                           probability resample_prob, else the copied value is kept; clamped either way */
  int32_t prior_kind[PBT_MAX_NH]; /* pbt_prior of each slot (resample only) */
  double const_lr, const_momentum, const_beta1, const_beta2, const_eps, const_wd;
  double toy_eta;                 /* toy step size */
  double toy_theta0[PBT_MAX_NH];  /* toy initial theta (same for all members) */
  double factor_lo, factor_hi;    /* perturbation factors, 0.8 / 1.2 */
  double clamp_lo[PBT_MAX_NH], clamp_hi[PBT_MAX_NH]; /* applied after perturbation; +-inf = none */
  double ttest_alpha;    /* significance level of the t-test (the paper states none; 0.05 is customary) */
  double resample_prob;  /* probability that explore redraws a slot (the paper states none) */
  double prior_lo[PBT_MAX_NH], prior_hi[PBT_MAX_NH]; /* range of each slot's prior; log-uniform needs 0 < lo <= hi */
  double gp_lambda;      /* PBT_LOSS_WGAN_GP: weight of the gradient penalty (10 in the paper that introduced it) */
} pbt_spec;

/*
 * Caller-owned device data (kept by reference).  Element type of x/z/soft
 * targets: float for PBT_FP32, bfloat16 (raw 16-bit) for PBT_BF16_FP32MASTER.
 *   MLP : x_pool [pool_rows][in],  y_pool: MSE float [pool_rows][out],
 *         CE_HARD int32 [pool_rows], CE_SOFT x-type [pool_rows][out];
 *         x_eval / y_eval the same with eval_batch rows.
 *   GAN : x_pool real samples [pool_rows][d], z_pool noise [pool_rows][zdim],
 *         x_eval fixed evaluation noise [eval_batch][zdim]; y_* unused (NULL).
 *   TOY : all NULL.
 * Each (member, step) trains on the contiguous rows [off, off + batch) of the
 * pools, off a multiple of 128 drawn from the batch stream of the counter-based
 * generator, so the rows are reproducible from (seed, member, step).
 */
typedef struct pbt_data {
  const void* x_pool;
  const void* y_pool;
  const void* z_pool;
  const void* x_eval;
  const void* y_eval;
} pbt_data;

/*
 * Host-side view of one member's record (theta, h, p, t) plus optimiser state.
 * Every pointer is caller-owned host memory and may be NULL to skip that part.
 * w/opt1/opt2/grad hold P elements in flat order: float (double for the toy).
 * `grad` (last gradient applied) is filled by pbt_get_state, ignored by set.
 * step is the member's own step count t (equal for all members as long as only
 * pbt_step is used); round, the number of ready points passed, is population-wide:
 * setting it through any member sets it for the population.
 */
typedef struct pbt_state_view {
  void* w;
  void* opt1;       /* SGD momentum buffer, or Adam first moment */
  void* opt2;       /* Adam second moment */
  void* grad;
  double* scalars;  /* [PBT_N_SCALARS] */
  double* hparams;  /* [nh] */
  double* fitness;  /* [1] */
  int64_t* step;
  int64_t* round;
} pbt_state_view;

typedef struct pbt_handle pbt_t;

/* Bytes of device workspace pbt_create needs for this spec (256-byte aligned base). */
int pbt_query_workspace(const pbt_spec* spec, size_t* bytes);

/* Number of parameters P of one member in flat order. */
int pbt_param_count(const pbt_spec* spec, int64_t* count);

/*
 * Build the initial population P (Algorithm 1, input): member-major slabs in
 * the workspace; weights U(-a, a), a = sqrt(6 / fan_in), drawn on the device from
 * the init stream of Philox4x32-10 keyed by `seed`; biases and optimiser state
 * zero; h from init_hparams (host, [n_members][nh] doubles, row-major).
 * `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 * On failure *out is NULL.
 */
int pbt_create(pbt_t** out, const pbt_spec* spec, const double* init_hparams, uint64_t seed,
               const pbt_data* data, void* workspace, size_t workspace_bytes, void* stream);

/* Release the handle (host memory only; the workspace stays the caller's). */
int pbt_destroy(pbt_t* p);

/*
 * theta <- step(theta | h) for every member, k times in lockstep (Eq. 2, chained
 * as in Eq. 3).  MLP: forward, loss, backward, optimiser update with the member's
 * own h.  GAN: K discriminator updates then one generator update per step
 * (Section 4.3.1), on the logistic losses or on the WGAN-GP objective; for the
 * latter, row b of discriminator update j of a step interpolates with
 * eps_b = ((w >> 9) + 1/2) / 2^23, w = word b mod 4 of Philox block
 * j * 65536 + b div 4 of stream 4 at counter (member, step).
 * Toy: one gradient-ascent step on the surrogate objective.
 */
int pbt_step(pbt_t* p, int k);

/*
 * Members at their own pace (Algorithm 1 is a loop per member; Section 3 lets the workers run asynchronously,
 * and Appendix A.1's partial synchrony exists to tolerate workers that are pre-empted): k steps for the members
 * whose byte in active_host (n_members bytes of host memory) is non-zero, none for the others, whose records
 * stay untouched.  Every member counts its own steps t (pbt_state_view.step): the rows it trains on and its
 * interpolation draws are keyed by (member, its own t), so a member that sat out some calls continues exactly
 * where it stopped, and a call with every byte set equals pbt_step(k).  `ready(p, t, P)` for such a population
 * is a matter of the member's own t; give the ready members to pbt_exploit_explore_ready.  Consecutive active
 * members share their launches (one pass of the step's kernels per run of consecutive active members).
 * PBT_ERR_STATE if a batch set by pbt_set_batch is pending.  Only enqueues.
 */
int pbt_step_subset(pbt_t* p, const uint8_t* active_host, int k);

/*
 * p <- eval(theta) for every member (Eq. 1): minus the held-out loss, the toy's
 * true objective Q(theta), or minus the energy distance between eval_batch
 * generated samples and the eight-mode ring.  Result stays on the device
 * (read it with pbt_get_fitness).
 */
int pbt_eval(pbt_t* p);

/*
 * One ready point for the whole population (Algorithm 1: exploit, the
 * theta != theta' guard, explore, population update): selection by
 * exploit_rule on the current fitness vector (or score histories), slab copy
 * donor -> recipient of weights, optimiser state and (flag) hyperparameters,
 * explore_rule applied to the recipients' h, p[b] <- p[src[b]] (and the score
 * history with it), round <- round + 1.  Every copy reads the donor's record
 * as it was before this ready point.
 */
int pbt_exploit_explore(pbt_t* p);

/*
 * The same ready point for a population whose members are not all ready together (Algorithm 1 tests
 * `ready(p, t, P)` member by member; under the asynchronous execution of Section 3 the ready points of the
 * workers are staggered).  ready_host: n_members bytes of host memory, non-zero = this member is ready and may
 * exploit and explore now; NULL = everybody (pbt_exploit_explore).  Members that are not ready keep their whole
 * record, but they are ranked with the others and can be copied from.  The ready-point counter advances by
 * one per call whatever the mask, so the random draws of successive calls differ.
 */
int pbt_exploit_explore_ready(pbt_t* p, const uint8_t* ready_host);

/*
 * Ready point of a population that is sharded over several handles (Algorithm 1's exploit / explore; the exchange
 * takes the place of the shared store of Appendix A.1).  The per-member records that selection looks at are small,
 * so every shard decides for the WHOLE population and all shards reach the same decisions:
 *   fitness_global_host  [n_global] doubles, in: p of every member (each shard's pbt_get_fitness, all-gathered);
 *                        out: after p[b] <- p[src[b]]
 *   hparams_global_host  [n_global][nh] doubles, in: h of every member; out: after copy and explore
 *   ready_global_host    n_global bytes or NULL (everybody), as for pbt_exploit_explore_ready
 *   src_global_out_host  [n_global] int32: the copy map, in indices of the whole population
 *   level_global_out_host [n_global] int32: copy pass of each recipient (0 under truncation selection; under the
 *                        tournament rule a donor that is itself a recipient has a higher pass than its readers)
 *   n_levels_out_host    number of passes
 * The call runs the same selection / explore kernel as pbt_exploit_explore on these vectors (same draws, keyed by
 * the ready-point counter, which advances by one), writes the rows of this shard's members back into its own h and
 * p, and translates the copy map for the shard (pbt_get_copy_map then gives, per local member, its donor's LOCAL
 * index, or the member itself if it keeps its record or its donor lives on another shard).  It moves no weights.
 * The caller then goes through the passes in order: for pass L, every slab copy whose recipient has level L is
 * carried out, the local ones by pbt_copy_members_level(p, L), the ones that cross shards by sending the donor's
 * slabs (pbt_member_slabs) into the recipient's slabs on the other device (peer copy or send / receive; the data
 * lands in the recipient's own memory before any kernel reads it).  Within a pass no recipient is anybody's donor.
 * All three exploit rules; for t-test selection the whole population's score histories have to be given first
 * (pbt_set_global_history, else PBT_ERR_STATE), and the rows of this shard's members, with the histories that
 * moved with a copy, are written back into the shard's own history.  Synchronises the stream (it returns data to
 * the host).
 */
int pbt_exploit_explore_global(pbt_t* p, double* fitness_global_host, double* hparams_global_host,
                               const uint8_t* ready_global_host, int32_t* src_global_out_host,
                               int32_t* level_global_out_host, int32_t* n_levels_out_host);

/*
 * T-test selection on a sharded population: the score histories of ALL members (each shard's pbt_get_history,
 * all-gathered), hist [n_global][PBT_HISTORY] doubles oldest first, count [n_global] int32; consumed by the next
 * pbt_exploit_explore_global.  Both host.
 */
int pbt_set_global_history(pbt_t* p, const double* hist_global_host, const int32_t* count_global_host);

/* The local slab copies of one pass of the copy map left by pbt_exploit_explore_global.  Only enqueues. */
int pbt_copy_members_level(pbt_t* p, int level);

/*
 * Device addresses of the arrays that make up one local member's copied record, in a fixed order: fp32 master
 * weights, first optimiser state, second optimiser state (Adam), bf16 shadow (bf16 populations), Adam's running
 * beta products; the toy: theta.  ptrs_out_host and bytes_out_host hold up to 5 entries, *count_out_host says how
 * many are used.  The memory belongs to the caller's workspace; the addresses stay valid until pbt_destroy.
 */
int pbt_member_slabs(pbt_t* p, int member, void** ptrs_out_host, size_t* bytes_out_host, int32_t* count_out_host);

/* Read / overwrite one member's record.  get synchronises the stream. */
int pbt_get_state(pbt_t* p, int member, pbt_state_view* out_host);
int pbt_set_state(pbt_t* p, int member, const pbt_state_view* in_host);

/* fitness vector p[n_members] as doubles (host).  set allows a test to inject a
 * fitness vector so that selection can be compared bit for bit. */
int pbt_get_fitness(pbt_t* p, double* out_host);
int pbt_set_fitness(pbt_t* p, const double* in_host);

/*
 * Score history used by t-test selection (Section 4.1.1, exploit (a)): hist[n_members][PBT_HISTORY] doubles, oldest
 * first, the first count[m] entries of row m valid (the rest read as 0); count[n_members] int32.  Both host.
 * pbt_eval appends to it when exploit_rule == 2 (dropping the oldest of PBT_HISTORY); a copy at a ready point
 * moves the donor's history with its weights.  set lets a test inject histories so that the decisions can be
 * compared bit for bit; counts outside [0, PBT_HISTORY] are PBT_ERR_INVALID_ARG.  Either pointer may be NULL in get.
 */
int pbt_get_history(pbt_t* p, double* hist_out_host, int32_t* count_out_host);
int pbt_set_history(pbt_t* p, const double* hist_in_host, const int32_t* count_in_host);

/* h[n_members][nh] as doubles (host). */
int pbt_get_hparams(pbt_t* p, double* out_host);
int pbt_set_hparams(pbt_t* p, const double* in_host);

/* copy map of the last ready point: src[i] == i for members that kept their state. */
int pbt_get_copy_map(pbt_t* p, int32_t* src_out_host);

/* argmax_i p[i], lowest index on ties (Algorithm 1, return value). */
int pbt_get_best(pbt_t* p, int32_t* member_out_host);

/* per-member training loss of the last step: [n_members][2] doubles
 * (column 0: MLP loss or generator loss; column 1: discriminator loss). */
int pbt_get_last_loss(pbt_t* p, double* out_host);

/*
 * Use the caller's rows for the next step instead of a pool window: x is
 * [n_members][batch][in], y the matching targets, both device pointers in the
 * pools' element types; copied before the call returns to the stream.  MLP only.
 */
int pbt_set_batch(pbt_t* p, const void* x_device, const void* y_device);

/*
 * One step fed from host memory, end to end: copies the caller's rows for every
 * member (x_host [n_members][batch][in], y_host the matching targets, both in the
 * pools' element types; pinned memory makes the copies asynchronous), runs one
 * lockstep `step` (Eq. 2) on them, and, if loss_out_host is not NULL, copies the
 * per-member training loss back ([n_members][2] doubles) and synchronises.  MLP only.
 */
int pbt_step_host(pbt_t* p, const void* x_host, const void* y_host, double* loss_out_host);

/*
 * The same step with the upload taken off the critical path: pbt_prefetch_host_batch starts copying the
 * next step's rows (same layout as pbt_step_host; use pinned memory) into a spare buffer on a copy stream of the
 * library's own and returns at once; pbt_step_prefetched makes the stream wait for that copy and enqueues one
 * training step on it.  With loss_out_host == NULL it returns without synchronising, so the caller can prefetch
 * the rows of step t+1 while step t runs and read the losses afterwards (pbt_get_last_loss); otherwise it copies
 * the losses back and synchronises.  PBT_ERR_STATE if nothing was prefetched, or if a prefetched batch is still
 * waiting to be consumed.  MLP only.
 */
int pbt_prefetch_host_batch(pbt_t* p, const void* x_host, const void* y_host);
int pbt_step_prefetched(pbt_t* p, double* loss_out_host);

/* Kernel launches issued by the last pbt_step / pbt_eval / pbt_exploit_explore call. */
int pbt_get_launch_count(const pbt_t* p, int64_t* count);

/*
 * Elapsed device time, in milliseconds, of one named kernel class accumulated
 * since pbt_profile_begin: "gemm", "wgrad_adam" (weight gradient with the Adam update fused in),
 * "optimizer" (the separate update pass), "loss", "copy", "select", "other".
 * Profiling brackets each launch with events on the handle's stream and
 * therefore slows the step down; it is off unless begun.  While it is on, steps are not replayed from the
 * captured graph and the backward pass stays in one stream (pbt_spec.backward_streams), so that every launch is
 * timed alone: the class times of a step can then add up to a little more than an unprofiled step takes.
 */
int pbt_profile_begin(pbt_t* p);
int pbt_profile_end(pbt_t* p);
int pbt_profile_get(pbt_t* p, const char* kernel_class, double* ms_total, int64_t* launches);

/*
 * The member-batched GEMM of the training step on its own (forward, data-gradient and
 * weight-gradient contractions of Eq. 2's gradient step all have this form):
 *   C_b[m][n] = epilogue( sum_k A_b(m,k) * B_b(n,k) ),  b = 0..batch-1.
 * a_mn == 0: A_b(m,k) = A[b*strideA + m*lda + k] (K contiguous); a_mn == 1: A[b*strideA + k*lda + m].
 * B likewise over (n,k).  Operands are float (in_bf16 == 0) or bfloat16; accumulation is fp32;
 * C is float or bfloat16 (out_bf16).  Epilogue, in this order: + bias[b*strideBias + n] (if bias),
 * max(.,0) (if relu), zero where mask[b*strideMask + m*ldmask + n] <= 0 (if mask; operand type).
 * Strides are in elements; a stride of 0 shares the operand between all problems.
 * engine: 0 = choose (tensor cores when operands are bf16 and the shape fills the tiles),
 * 1 = FP32-ALU kernels, 2 = tcgen05 kernel, one CTA per tile, 3 = tcgen05 kernel with CTA pairs (M, N >= 256);
 * PBT_ERR_UNSUPPORTED if the shape does not qualify for the engine asked for.
 * status_device: 32 zeroed bytes of device memory; a bounded wait that expires inside the
 * tensor-core kernel stores PBT_ERR_TIMEOUT in the int32 at byte offset 16.  All pointers are
 * device pointers; the call only enqueues work on `stream`.
 */
typedef struct pbt_gemm_desc {
  int32_t M, N, K, batch;
  int32_t in_bf16, out_bf16;
  int32_t a_mn, b_mn;
  int32_t relu, engine;
  const void* A; int64_t lda, strideA;
  const void* B; int64_t ldb, strideB;
  void* C; int64_t ldc, strideC;
  const float* bias; int64_t strideBias;
  const void* mask; int64_t ldmask, strideMask;
  void* status_device;
} pbt_gemm_desc;
int pbt_grouped_gemm(const pbt_gemm_desc* desc, void* stream);

/*
 * Failure-detection self-test.  Every wait inside the tensor-core kernels (on a TMA transfer, an MMA commit, a
 * partner CTA) is bounded: when its poll limit runs out the kernel stores PBT_ERR_TIMEOUT in the status word, every
 * role leaves its loop, and the kernel returns normally, so the context stays usable and the next pbt_get_* call
 * reports the error (a population's workers being lost or pre-empted is part of the paper's setting, Appendix A.1;
 * here the only thing that can go missing is a signal inside a kernel).  This call runs that same wait in a
 * one-CTA kernel on a barrier that nothing signals, with `polls` polls (1..100000; a few thousand last well under
 * a second), so the expiry path can be exercised without provoking a fault: afterwards the int32 at byte offset 16
 * of status_device (32 zeroed bytes of device memory, as for pbt_grouped_gemm) holds PBT_ERR_TIMEOUT.
 */
int pbt_selftest_bounded_wait(void* status_device, int polls, void* stream);

/*
 * Allocation-free scorer (no counterpart in the paper: it exists for callers that are not
 * allowed to allocate device memory, e.g. a plug-in inside an application that owns the
 * whole device through its own arena, and so cannot provide the workspace pbt_create wants).
 * Computes, for each of n_members sets of n two-dimensional points, the same fitness
 * pbt_eval gives a GAN population: minus the energy distance between the set and the
 * eight-mode unit ring.
 *   x_device            [n_members][n][2] floats, device memory, caller-owned (input)
 *   fitness_out_device  [n_members] floats, device memory, caller-owned (output)
 *   stream              cudaStream_t as void* (NULL = default stream); the call only enqueues
 * The partial sums of the reduction live in a fixed 1 MiB array inside the library image
 * (held by every GPU that loads the library until the process exits), so the call performs
 * no cudaMalloc / cudaFree.  Limits and rules:
 *   - n_members * 2 * ceil(n / 256) must not exceed 131072 and n_members must not exceed 65535,
 *     else PBT_ERR_WORKSPACE with a message naming the size; NULL pointers, non-positive sizes,
 *     or buffers that are not device memory of the CURRENT device give PBT_ERR_INVALID_ARG
 *     (the scratch that is used, and the GPU the kernels run on, are the current device's);
 *   - the array is shared by all calls and keeps the previous call's contents; nothing in it
 *     needs clearing, every slot read is first rewritten by the same call;
 *   - calls that overlap on the GPU (other streams or threads) race on that array: serialise them;
 *   - the first call on each device resolves the array's device address; make that first call
 *     before starting any stream capture.
 */
int pbt_energy_fitness_static(const float* x_device, int n, int n_members, float* fitness_out_device,
                              void* stream);

const char* pbt_last_error(const pbt_t* p); /* p may be NULL: error of the last failed create/query */

#ifdef __cplusplus
}
#endif
#endif /* PBT_H_ */
