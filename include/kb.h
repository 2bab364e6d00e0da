/*
 * kb.h -- C ABI of the batched bandit step (KernelBand decision layer) for
 * NVIDIA B200 (sm_100a).
 *
 * One bandit step scores every arm (candidate kernel k, optimisation strategy
 * s) of the action space A_t = P_t x S (Sec. 2.2) for B independent search
 * instances:
 *
 *   kb_normalize        z-score of the trace features phi(k)       (Sec. 3.2)
 *   kb_cluster_assign   K-Means nearest-centroid assignment        (Sec. 3.3)
 *   kb_cluster_update   K-Means centroid update                    (Sec. 3.3)
 *   kb_prune            roofline bound + saturation mask M_{i,s}   (Assumption 1, Sec. 3.4)
 *   kb_score_select     cluster statistics, masked-UCB index with a
 *                       Lipschitz term, arm selection    (Sec. 3.4, Assumption 2)
 *
 * and, around the step, the other lines of Algorithm 1 that run on the device:
 *
 *   kb_seed_kmeanspp    k-means++ rows to start the clustering from (Sec. 3.5)
 *   kb_best_restart     the run with the smallest inertia among n_init
 *   kb_select_pair      masked-UCB choice of (I_t, S_t) from the K x S tables
 *   kb_sample_member    softmax draw of k_t inside the chosen cluster (Sec. 3.4)
 *   kb_record_outcome   reward clip, N <- N + 1, running mean      (Sec. 2.2, Algorithm 1)
 *   kb_cluster_radius   per-cluster radius, bounds diam(C_i)       (Theorem 1)
 *   kb_select_top_m     the M best arms instead of one
 *
 * Conventions (all entry points unless stated otherwise)
 *  - Arrays are dense, row-major, batch-major: X[B][N][D], C[B][K][D],
 *    labels[B][N], pulls[B][N][S], hsig[B][K][R].  B instances, N candidates,
 *    D features, K clusters, S <= 32 strategies, R hardware resources.
 *  - Every array pointer is a DEVICE pointer, borrowed: the caller allocates
 *    and frees it; the library neither keeps nor frees it once the work queued
 *    by the call has run.  fp32 arrays must be 16-byte aligned.
 *  - Calls are asynchronous on the context's CUDA stream, allocate nothing and
 *    do not synchronise with the host.  Scratch memory comes from the workspace
 *    the caller registers with kb_set_workspace; calls that share a workspace
 *    must be ordered on one stream.
 *  - Outputs marked "nullable" are skipped when NULL.  Inputs and outputs must
 *    not overlap unless stated.
 *  - Return value: KB_OK or an error code; on error nothing has been queued.
 *    B == 0 or N == 0 is valid: outputs that do not depend on candidates are
 *    still written (counts 0, best_arm -1, ...).
 *  - Non-finite inputs give unspecified results.  Ties go to the lowest index.
 */
#ifndef KB_H_
#define KB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kb_ctx kb_ctx;

typedef int kb_status;
#define KB_OK 0
#define KB_ERR_INVALID_ARG 1 /* null pointer, negative size, label/target out of contract */
#define KB_ERR_UNSUPPORTED 2 /* valid request outside the implemented range (e.g. S > 32) */
#define KB_ERR_WORKSPACE 3   /* no workspace registered or it is too small */
#define KB_ERR_CUDA 4        /* a CUDA runtime call failed; see kb_last_error */
#define KB_ERR_TIMEOUT 5     /* a bounded device-side wait expired (device status word) */

/* ---- context ------------------------------------------------------------ */

/* Creates a context bound to `device` and to `cuda_stream` (a borrowed
 * cudaStream_t; NULL = the legacy default stream).  Allocates a few bytes of
 * device memory for the status word; that is the only allocation the library
 * ever makes.  `out` is a host pointer. */
kb_status kb_create(kb_ctx** out, int device, void* cuda_stream);
kb_status kb_destroy(kb_ctx* ctx);
/* Rebinds the context to another stream (borrowed). */
kb_status kb_set_stream(kb_ctx* ctx, void* cuda_stream);

/* Bytes of scratch the five calls, kb_cluster_fit, kb_bandit_step and the
 * calls around the step (kb_seed_kmeanspp, kb_sample_member, kb_select_top_m
 * up to KB_TOP_M_MAX) need for these sizes (host pointer `out`).
 * kb_bandit_step_host needs kb_step_workspace_bytes. */
kb_status kb_workspace_bytes(int B, int N, int D, int K, int S, size_t* out);
/* Registers a device buffer (borrowed, 256-byte aligned) as scratch.  Its
 * contents need not be initialised and are not preserved between calls. */
kb_status kb_set_workspace(kb_ctx* ctx, void* dev_ptr, size_t bytes);

const char* kb_status_string(kb_status s);
/* Text of the last failure on this context (host string owned by the context). */
const char* kb_last_error(kb_ctx* ctx);
/* Conditions that only the device can see are OR-ed into the context's device
 * status word; the call that queued the work has long returned KB_OK by then.
 *
 *   bit     set by                                   meaning
 *   0x001   update, score, prune, radius kernels     a label outside [0, K): the row / candidate was skipped
 *                                                    (prune: treated as cluster 0)
 *   0x002   prune, sample, select_pair kernels       a target[s] outside [0, R): the arm / pair was masked
 *   0x004   init_centroids, sample, record kernels   a row, member or pair index out of range: nothing written for it
 *   0x008   append_candidate kernel                  a frontier was full: the verified kernel was dropped (no error)
 *   0x100   tensor-core assign kernel                a bounded wait between its roles expired; the CTA drained and
 *                                                    left; labels of that launch are unspecified
 *   0x200   cooperative fit kernel                   its bounded grid-wide barrier expired; results unspecified
 *
 * kb_get_device_status synchronises the stream (not for the hot path), stores
 * the word in *out (host pointer) and returns KB_ERR_TIMEOUT if 0x100 or 0x200
 * is set, else KB_OK (the contract bits 0x001..0x004 are the caller's to read).
 * The word keeps its bits until kb_clear_device_status queues its clearing on
 * the stream.  After a timeout the context stays usable: clear and call again. */
#define KB_STATUS_BAD_LABEL 0x001
#define KB_STATUS_BAD_TARGET 0x002
#define KB_STATUS_BAD_INDEX 0x004
#define KB_STATUS_FRONTIER_FULL 0x008
#define KB_STATUS_TIMEOUT_ASSIGN 0x100
#define KB_STATUS_TIMEOUT_FIT 0x200
kb_status kb_get_device_status(kb_ctx* ctx, int* out);
kb_status kb_clear_device_status(kb_ctx* ctx);
/* Test hook for the bounded device-side waits (no counterpart in the paper).
 * Kernels whose roles or CTAs wait on one another -- the tensor-core assign
 * kernel (mbarrier waits between its roles) and the cooperative fit (its
 * grid-wide barrier) -- give every wait a limit; when it runs out the CTA
 * raises its abort flag, every role drains, copies in flight are awaited,
 * tensor memory is freed, the kernel returns and the status word carries 0x100
 * or 0x200.  polls != 0 replaces the limit (a wait of a few hundred polls takes
 * well under a millisecond); leave_one_out != 0 makes one participant stay
 * away -- the B-operand loader of CTA 0 of the assign kernel, the last CTA of
 * the cooperative fit -- so that the others' waits do run out.  That is how a
 * test sees the expiry path run: nothing spins without a limit, nothing
 * faults.  polls = 0, leave_one_out = 0 restores normal operation. */
kb_status kb_debug_wait_limit(kb_ctx* ctx, unsigned polls, int leave_one_out);
/* Input check for debugging (no counterpart in the paper).  The calls take
 * finite inputs on trust; this one counts the entries of a device array of n
 * floats that are NaN or +-inf and hands the count to the host (*out; it
 * synchronises the stream, so it does not belong on the hot path).  Uses the
 * spare words behind the status word, no workspace.  n = 0 gives 0. */
kb_status kb_debug_count_nonfinite(kb_ctx* ctx, const float* x /* device */, size_t n, uint64_t* out /* host */);
/* The mapping itself, as a pure host function (no context, no device): the
 * kb_status that a status word stands for -- KB_ERR_TIMEOUT for a timeout bit;
 * with contract_bits_too != 0 also KB_ERR_INVALID_ARG for 0x001..0x004, which
 * is what kb_bandit_step_host returns; else KB_OK. */
kb_status kb_status_of_device_word(int word, int contract_bits_too);
/* Number of kernels of this library the context has queued since creation
 * (`kernels`) and of memset nodes (`memsets`, nullable).  Host pointers. */
kb_status kb_get_launch_count(kb_ctx* ctx, uint64_t* kernels, uint64_t* memsets);

/* Per-call device timing, a diagnostic that is off by default.  While on,
 * each of the calls below brackets the work it queues with a pair of CUDA
 * events on the context's stream (events come from a pool created by
 * kb_timing_enable, so the calls still allocate nothing; calls beyond the
 * pool's 4096 pairs between two reads go unrecorded).  kb_timing_read
 * synchronises the stream, adds up the recorded pairs per class into
 * ms[KB_T_COUNT] / calls[KB_T_COUNT] (host arrays) and empties the pool. */
#define KB_T_NORMALIZE 0
#define KB_T_ASSIGN 1
#define KB_T_UPDATE 2
#define KB_T_PRUNE 3
#define KB_T_SCORE 4
#define KB_T_INIT 5
#define KB_T_FIT 6 /* kb_cluster_fit when it runs as one fused launch (small instances) */
#define KB_T_ASSIGN_KERNEL 7 /* the tensor-core contraction kernel alone (nested inside KB_T_ASSIGN or KB_T_FIT) */
#define KB_T_SAMPLE 8 /* kb_sample_member, kb_record_outcome, kb_cluster_radius */
#define KB_T_PREP 9   /* once per tensor-path kb_cluster_fit: the conversion of Z to its pre-split fp16 image */
#define KB_T_COUNT 10
kb_status kb_timing_enable(kb_ctx* ctx, int on);
kb_status kb_timing_read(kb_ctx* ctx, double* ms, int64_t* calls);

/* Arithmetic ceilings of the device the context is bound to, measured in the
 * instruction shapes this library's kernels use (a benchmark's denominators;
 * the paper has no counterpart).  fp32: independent register-resident FMA
 * chains on every SM.  Tensor cores: back-to-back tcgen05.mma M = 128, N = 128,
 * A from tensor memory, B from shared memory, fp32 accumulation, one CTA per SM,
 * for kind::f16 (K = 16) and kind::tf32 (K = 8).  Three launches of about a
 * millisecond each (after a warm-up launch each) on the context's stream;
 * synchronises; no workspace.  `out` is a host pointer.  Every wait in the
 * probe kernels is bounded; KB_ERR_TIMEOUT if the products did not retire. */
typedef struct {
    double ffma_tflops, mma_f16_tflops, mma_tf32_tflops; /* 2 flop per multiply-add */
    float ffma_ms, mma_f16_ms, mma_tf32_ms;              /* duration of the timed launch */
    /* one SM's view of its own stream of products: SM cycles per instruction, and the SM clock it ran at
     * (cycles / nanoseconds of the global timer) -- the power cap lowers the clock under tensor load */
    float mma_f16_cycles_per_instr, mma_tf32_cycles_per_instr, mma_f16_sm_mhz, mma_tf32_sm_mhz;
} kb_peak_probe;
kb_status kb_probe_peaks(kb_ctx* ctx, kb_peak_probe* out);

/* ---- the five calls ----------------------------------------------------- */

/* Feature normalisation (Sec. 3.2 / App. A.1 say the features are normalised;
 * the workloads fix the reading): per instance and column, the population
 * z-score z = (x - mean) / std, std over N rows with divisor N; a column whose
 * std is below 1e-12 gets scale 1 (it becomes all zeros).
 *   x     [B][N][D] in
 *   z     [B][N][D] out; may be the same pointer as x (in place)
 *   mean  [B][D]    out, nullable
 *   scale [B][D]    out, nullable (the divisor actually used) */
kb_status kb_normalize(kb_ctx* ctx, int B, int N, int D, const float* x, float* z, float* mean,
                       float* scale);

/* Hardware-aware pruning.
 *   roofline floor   T_lb(k,s) = max(flops[k] / peak_flops[s], bytes[k] / peak_bw[s])
 *                    (the roofline model Assumption 1 cites for B(k,s))
 *   keep bit s of keep[b][k] =  T_lb(k,s) < t_incumbent[b]
 *                          AND  hsig[b][labels[b][k]][target[s]] < theta_sat
 *                    (second factor: the mask equation of Sec. 3.4, strict <;
 *                     applied only when labels, hsig and target are all given)
 *   bound[b][k][s]   = clip((t_cur[k] - T_lb(k,s)) / t_cur[k], 0, 1)
 *                    (Assumption 1: gap between current performance and the limit)
 *   flops, bytes  [B][N] in;  peak_flops, peak_bw [S] in;  t_incumbent [B] in
 *   t_cur         [B][N] in, nullable unless `bound` is requested
 *   labels [B][N], hsig [B][K][R] (percent), target [S] (values in [0,R)): in,
 *                 nullable together
 *   keep          [B][N] out;  kept_count [B] out, nullable (number of set bits)
 *   bound         [B][N][S] out, nullable */
kb_status kb_prune(kb_ctx* ctx, int B, int N, int S, int K, int R, const float* flops,
                   const float* bytes, const float* peak_flops, const float* peak_bw,
                   const float* t_incumbent, const float* t_cur, const int32_t* labels,
                   const float* hsig, const int32_t* target, float theta_sat, uint32_t* keep,
                   uint32_t* kept_count, float* bound);

/* K-Means assignment (Sec. 3.3; the KMeans line of Algorithm 1): for every
 * row, the nearest centroid in squared Euclidean distance (the norm of
 * Assumption 2); the lowest centroid id wins a tie.
 *   z [B][N][D], centroids [B][K][D] in
 *   labels  [B][N] out
 *   dist2   [B][N] out, nullable: squared distance to the chosen centroid
 *   inertia [B]    out, nullable: sum of dist2 over the instance
 *   rep     [B][K] out, nullable: the member nearest its centroid (the
 *           "centroid kernel" that Sec. 3.3 profiles), lowest k on ties,
 *           -1 for an empty cluster */
kb_status kb_cluster_assign(kb_ctx* ctx, int B, int N, int D, int K, const float* z,
                            const float* centroids, int32_t* labels, float* dist2, float* inertia,
                            int32_t* rep);

/* K-Means centroid update (Sec. 3.3; "Update centroids" in Algorithm 1): each
 * centroid becomes the mean of its members; an empty cluster keeps its
 * previous centroid.  labels must lie in [0,K).
 *   centroids [B][K][D] in: previous, out: new;  counts [B][K] out, nullable */
kb_status kb_cluster_update(kb_ctx* ctx, int B, int N, int D, int K, const float* z,
                            const int32_t* labels, float* centroids, int32_t* counts);

typedef struct {
    float c;            /* exploration weight of the masked-UCB index (paper: 2.0) */
    float lipschitz_L;  /* L of Assumption 2; 0 reproduces the paper's index exactly */
    float prior_pulls;  /* N_{i,s} before any pull (Algorithm 1: 1) */
    float prior_mean;   /* mu_{i,s} before any pull (Algorithm 1: 0.5) */
    int cap_with_bound; /* non-zero: U(k,s) = min(U(k,s), bound[k][s]) (Assumption 1) */
} kb_score_params;

/* Cluster statistics, optimistic index and selection.
 *   N_{i,s}  = prior_pulls + sum over members k of cluster i of pulls[k][s]
 *   mu_{i,s} = (prior_pulls*prior_mean + sum of reward_sum[k][s]) / N_{i,s}
 *              (closed form of Algorithm 1's running-mean lines)
 *   U_cl(i,s) = mu_{i,s} + c*sqrt(ln t / N_{i,s})      (masked-UCB equation, Sec. 3.4)
 *   U(k,s)   = U_cl(labels[k], s) + L*sqrt(dist2[k])    (Assumption 2), optionally
 *              capped by bound[k][s]
 *   best_arm         = lowest k*S+s maximising U over arms whose keep bit is set
 *                      (-1, best_val = -inf if none)
 *   best_cluster_arm = lowest i*S+s maximising U_cl over pairs with at least
 *                      one kept member arm (-1 if none)
 *   labels [B][N] in; dist2 [B][N] in, nullable iff L == 0
 *   pulls [B][N][S] (>= 0), reward_sum [B][N][S] in
 *   keep [B][N] in, nullable = every arm valid; bound [B][N][S] in, nullable
 *   t [B] in, >= 1
 *   cl_pulls, cl_mean, cl_index [B][K][S] out
 *   arm_index [B][N][S] out, nullable (-inf for a pruned arm)
 *   best_arm, best_val, best_cluster_arm [B] out
 * Instances of at most 1024 candidates with S in {4, 8, 16, 32}, K*S <= 8192
 * and 16-byte aligned per-arm arrays run as ONE launch (one CTA per instance,
 * no workspace); larger ones as a memset node and four kernels. */
kb_status kb_score_select(kb_ctx* ctx, int B, int N, int K, int S, kb_score_params p,
                          const int32_t* labels, const float* dist2, const int32_t* pulls,
                          const float* reward_sum, const uint32_t* keep, const float* bound,
                          const int32_t* t, float* cl_pulls, float* cl_mean, float* cl_index,
                          float* arm_index, int32_t* best_arm, float* best_val,
                          int32_t* best_cluster_arm);

/* Within-cluster draw of the kernel k_t (Sec. 3.4, "Action selection";
 * Algorithm 1, "Sample k_t in C_{I_t}"): once the pair (I_t, S_t) is chosen,
 * k_t is drawn from the members of cluster I_t with
 *   P(k) proportional to exp(V_hw(k, S_t)),  V_hw(k, s) = theta_sat - h(k)[Target(s)].
 * The draw is a Gumbel-max: every member gets V_hw + G, G = -ln(-ln u), and the
 * largest perturbed value wins (lowest index on ties), which samples exactly
 * that softmax.  u comes from the counter-based generator Philox4x32 (10
 * rounds): counter = (candidate index, instance index, t[b], 0), key = (low,
 * high 32 bits of seed), u = ((first output word >> 9) + 0.5) * 2^-23.  The
 * same seed and t repeat the draw; the result does not depend on the launch
 * shape.  fp32 arithmetic (logf); no temperature (the paper states none).
 *   labels [B][N] in: the candidates' clusters
 *   cluster_arm [B] in: I_t*S + S_t as kb_score_select writes best_cluster_arm;
 *                       negative = no pair chosen, member = -1
 *   h_cand [B][N][R] in: the signature h(k) of every candidate (the paper
 *                       profiles only representatives: a caller without
 *                       per-candidate profiles passes its estimate); a NaN
 *                       entry (or a potential of -inf) is never drawn
 *   target [S] in, values in [0, R);  t [B] in: the step counter (draw index)
 *   member [B] out: the drawn candidate in [0, N), or -1 (no pair, or no
 *                       drawable member in the cluster)
 *   member_val [B] out, nullable: its perturbed value (-inf if none)
 * All arrays in DEVICE memory; seed by value.  cluster_arm >= K*S sets bit 4,
 * a target outside [0, R) bit 2 of the device status word (member = -1).
 * Needs the workspace of kb_workspace_bytes when an instance spans several
 * CTAs (more than 4096 candidates). */
kb_status kb_sample_member(kb_ctx* ctx, int B, int N, int K, int S, int R, const int32_t* labels,
                           const int32_t* cluster_arm, const float* h_cand, const int32_t* target,
                           float theta_sat, uint64_t seed, const int32_t* t, int32_t* member,
                           float* member_val);

/* k-means++ seeding (Arthur & Vassilvitskii, SODA'07; the initialisation of
 * the "scikit-learn's KMeans" of Sec. 3.5, without its extra greedy trials):
 * rows[b][0] is a row of instance b drawn uniformly, rows[b][j] a row drawn
 * with probability D(x)^2 / sum D^2, D(x) = distance of x to the nearest of
 * the j centres chosen before.  Each draw is a Gumbel-max over the weights w
 * (1 in round 0, D^2 after): the row with the largest ln(w) + G, G = -ln(-ln u),
 * u from Philox4x32-10 at counter (row, instance, round, 1), key = the halves
 * of seed, u = ((first word >> 9) + 0.5) * 2^-23.  Rows of weight 0 (chosen
 * rows, their duplicates) are never drawn; when every weight is 0 (fewer
 * distinct rows than K) the round draws uniformly among all rows.  The result
 * feeds kb_init_centroids or the init_rows of kb_bandit_step.
 *   z [B][N][D] in (N >= 1);  rows [B][K] out, values in [0, N)
 * DEVICE memory; seed by value.  K launches (one per round, each reading z
 * once); needs the workspace of kb_workspace_bytes (4 bytes per row plus 20
 * per centre).  Many small instances (N <= 1024, B at least half the number
 * of SMs) run all rounds in one launch, one CTA per instance, no workspace.
 * fp32 distances in the direct form. */
kb_status kb_seed_kmeanspp(kb_ctx* ctx, int B, int N, int D, int K, const float* z, uint64_t seed,
                           int32_t* rows);

/* Restarts (the n_init of the "scikit-learn's KMeans" of Sec. 3.5): a search
 * instance is clustered n_init times from different seeds as n_init
 * CONSECUTIVE instances of the batch (kb_seed_kmeanspp draws differently for
 * each: the instance index is part of its counter), and the run with the
 * smallest inertia is kept:
 *   best[g] = index in [0, n_init) of the smallest inertia[g*n_init + .],
 *             lowest index on ties; NaN is never chosen (-1 if all are NaN).
 *   inertia [G*n_init] in, as kb_cluster_fit writes it;  best [G] out
 * DEVICE memory.  One launch, no workspace. */
kb_status kb_best_restart(kb_ctx* ctx, int G, int n_init, const float* inertia, int32_t* best);

/* The M best arms of every instance by the per-arm index (the masked argmax
 * of Sec. 3.4 taken M times, for generating M candidates per iteration):
 * top_arm[b][j] = flat index k*S + s of the arm with the j-th largest
 * arm_index[b], larger value first, lower flat index first among equal
 * values; pruned arms (-inf) and NaN entries never appear; when fewer than M
 * arms are valid the tail is -1 (top_val -inf).  top_arm[b][0] is
 * kb_score_select's best_arm.  Exact: comparisons only.
 *   arm_index [B][N][S] in, as kb_score_select writes it
 *   top_arm [B][M] out;  top_val [B][M] out, nullable;  0 <= M <= KB_TOP_M_MAX
 * DEVICE memory.  arm_index is read ONCE, whatever M: every CTA keeps the M
 * largest keys of its slice (a shared-memory buffer cut back to M by a sort
 * whenever it fills; after the first cut only about M keys in a few thousand
 * still pass its threshold), a second launch merges the slices (skipped when
 * an instance is one slice).  Needs the workspace of kb_workspace_bytes. */
#define KB_TOP_M_MAX 128
kb_status kb_select_top_m(kb_ctx* ctx, int B, int N, int S, int M, const float* arm_index, int32_t* top_arm,
                          float* top_val);

/* Cluster radius: radius[b][i] = max over the members k of cluster i of
 * sqrt(dist2[b][k]), 0 for an empty cluster.  Theorem 1's bound carries the
 * term L * max_i diam(C_i); through the centroid diam(C_i) <= 2 radius[i], so
 * 2 L max_i radius[i] bounds it with one pass over the candidates.
 *   labels [B][N] in, values in [0, K) (others set bit 1 of the device status
 *   word and are skipped);  dist2 [B][N] in as kb_cluster_assign writes it
 *   (entries that are not positive, NaN included, add nothing)
 *   radius [B][K] out
 * DEVICE memory.  One memset node and one launch, no workspace. */
kb_status kb_cluster_radius(kb_ctx* ctx, int B, int N, int K, const int32_t* labels, const float* dist2,
                            float* radius);

/* Outcome of one iteration (Sec. 2.2 "Formal Model": r_t = Clip((L(k_t) -
 * L(k'_t)) / L(k_t), 0, 1); Algorithm 1, "Generation & update": N <- N + 1,
 * mu <- mu + (r_t - mu) / N for the chosen pair).  The statistics are kept per
 * arm as (pulls, reward_sum), from which kb_score_select forms N_{i,s} and
 * mu_{i,s} per cluster in closed form; the update of the pair (I_t, S_t)
 * through its drawn member k_t is
 *   pulls[k_t][S_t] += 1,  reward_sum[k_t][S_t] += r_t,  t += 1.
 * A regression, a NaN ratio or L(k_t) <= 0 gives r_t = 0.  When verification
 * failed (verified[b] == 0): failures_count == 0 leaves the statistics alone
 * (Algorithm 1), non-zero records one pull with reward 0 (the formal model's
 * "zero reward ... to compilation failures").  t advances in every case (it
 * is the loop index); member[b] < 0 (nothing drawn) changes nothing else.
 *   member [B] in: k_t as kb_sample_member writes it
 *   cluster_arm [B] in: I_t*S + S_t as kb_score_select writes best_cluster_arm
 *   t_cur [B][N] in: L(k) of every candidate;  t_new [B] in: L(k'_t)
 *   verified [B] in, nullable = every k'_t passed
 *   pulls, reward_sum [B][N][S] in/out;  t [B] in/out
 *   reward [B] out, nullable: r_t as recorded (0 where nothing was updated)
 *   cl_pulls, cl_mean [B][K][S] in/out, nullable (both or neither): the
 *     cluster tables kept alongside, updated for the chosen pair by
 *     Algorithm 1's two lines literally (N <- N + 1, mu <- mu + (r_t - mu)/N)
 *     whenever a pull is recorded, so that kb_select_pair can choose the next
 *     pair without a pass over the candidates
 * All arrays in DEVICE memory.  member >= N, a negative cluster_arm beside a
 * drawn member, or (with tables) cluster_arm >= K*S sets bit 4 of the device
 * status word and updates nothing.  One launch, no workspace; meant to be
 * chained after the selection and kb_sample_member on one stream (or inside
 * one CUDA graph). */
kb_status kb_record_outcome(kb_ctx* ctx, int B, int N, int K, int S, int failures_count, const int32_t* member,
                            const int32_t* cluster_arm, const float* t_cur, const float* t_new,
                            const int32_t* verified, int32_t* pulls, float* reward_sum, int32_t* t,
                            float* reward, float* cl_pulls, float* cl_mean);

/* The masked-UCB choice of the pair from the cluster tables alone (Sec. 3.4,
 * masked-UCB equation; Algorithm 1, "Select (I_t, S_t)"):
 *   pair[b] = lowest i*S + s maximising mu_{i,s} + c*sqrt(ln t / N_{i,s})
 *             over the pairs with M_{i,s} = 1 (-1 if none),
 *   M_{i,s} = [ hsig[b][i][target[s]] < theta_sat ]   (Algorithm 1,
 *             "Hardware-constrained selection"); hsig null: no pair is masked.
 * With tables that kb_score_select produced once after a (re-)clustering and
 * kb_record_outcome keeps current, an iteration costs K*S entries instead of
 * a pass over all arms.
 *   cl_pulls, cl_mean [B][K][S] in;  t [B] in, >= 1
 *   hsig [B][K][R] in, nullable;  target [S] in (required with hsig)
 *   cl_index [B][K][S] out, nullable;  pair [B] out
 * DEVICE memory.  One launch (one CTA per instance), no workspace.  A target
 * outside [0, R) sets bit 2 of the device status word (pair masked). */
kb_status kb_select_pair(kb_ctx* ctx, int B, int K, int S, int R, float c, const float* cl_pulls,
                         const float* cl_mean, const int32_t* t, const float* hsig, const int32_t* target,
                         float theta_sat, float* cl_index, int32_t* pair);

/* Which kernel kb_cluster_assign uses.
 *   path: 0 = automatic (tensor cores when K >= 128, D a multiple of 32 and
 *             <= 128 and there are at least 4096 rows; else the fp32 row-wise
 *             kernel), 1 = always the fp32 row-wise kernel, 2 = always the
 *             tensor-core kernel with the fp16 split (what "automatic" picks;
 *             KB_ERR_UNSUPPORTED where it cannot run), 3 = the tensor-core
 *             kernel with the tf32 split (3xTF32).
 *             Both splits carry 22 significant bits per operand (two pieces of
 *             11 bits) and three products per k-step; the fp16 one runs at
 *             twice the tensor rate and scales rows and centroids by exact
 *             powers of two to stay inside fp16's range.
 *   tc_eps:   the tensor-core kernel ranks centroids by the split product's
 *             squared distance; a row whose best and second-best values differ
 *             by no more than tc_eps * (||z||^2 + ||c||^2) (||c||^2: of the
 *             chosen centroid for the tf32 split, the largest of the instance
 *             for the fp16 split) is re-evaluated exactly (direct form, fp32).
 *             <= 0 keeps the default 2^-16.
 * kb_get_assign_path reports what the last kb_cluster_assign ran (1, 2 or 3).
 * kb_get_assign_presplit reports (1 or 0) whether that assignment, if it ran
 * the fp16 tensor-core kernel, multiplied out of a pre-split image of Z:
 * kb_cluster_fit (and kb_bandit_step through it) converts Z to its fp16 pieces
 * once, keeps the image in the workspace for the duration of the fit and lets
 * every assignment of the loop read it; a lone kb_cluster_assign splits the
 * rows on the fly. */
kb_status kb_set_assign_options(kb_ctx* ctx, int path, float tc_eps);
kb_status kb_get_assign_path(kb_ctx* ctx, int* out);
kb_status kb_get_assign_presplit(kb_ctx* ctx, int* out);

/* Diagnostic for the tensor-core assign kernel: runs it on (z, centroids) and
 * returns, besides the labels, the expanded-form squared distance it ranked
 * by (approx_dist2 [B][N], nullable) and the number of rows that went through
 * the exact re-evaluation (flagged, two int32 in DEVICE memory, nullable:
 * rows compared against their runner-up, rows re-evaluated against all K).
 * Same workspace as kb_cluster_assign. */
kb_status kb_assign_tc_probe(kb_ctx* ctx, int B, int N, int D, int K, const float* z,
                             const float* centroids, int32_t* labels, float* approx_dist2,
                             int32_t* flagged);

/* kb_cluster_update for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of the centroid update above.)
 *
 * Some hosts of this library own every byte of device memory themselves: a serving process
 * whose memory plan is fixed when it starts, a plug-in running inside another framework's
 * arena, a latency-critical loop that must never hit the implicit device-wide
 * synchronisation of an allocation call.  Such a caller can neither cudaMalloc a workspace
 * nor hand one over.  This entry point therefore takes no context and no workspace: its
 * scratch (sums and counts) is a fixed array compiled into the library, which every GPU
 * that loads the library carries until the process exits (about 0.27 MB).  It calls no
 * cudaMalloc / cudaFree and no allocating library routine.
 *
 *   single instance (B = 1); same meaning of z [N][D], labels [N], centroids [K][D]
 *   (in: previous, out: new) and counts [K] (nullable) as kb_cluster_update; all DEVICE
 *   pointers on the CURRENT device; cuda_stream is a borrowed cudaStream_t.
 *   Limits: K * D <= KB_NOALLOC_MAX_KD and K <= KB_NOALLOC_MAX_K; anything larger
 *   returns KB_ERR_UNSUPPORTED and queues nothing.
 *   The first call on a device looks up the scratch array's device address and reads two
 *   device attributes; make that first call before any stream capture begins.
 *   Every call on a device shares the one array (the call clears what it needs first), so
 *   two calls that overlap on the GPU -- different streams, no ordering -- race: order them.
 *   (The per-device look-up itself is idempotent: two host threads making the first call at
 *   once store the same values.)
 *   A label outside [0, K) is skipped (it adds to no sum and no count) and sets bit 1 of the
 *   array's own status word -- there is no context to carry it.  The call still returns KB_OK:
 *   read the word with kb_cluster_update_noalloc_status. */
#define KB_NOALLOC_MAX_KD 65536
#define KB_NOALLOC_MAX_K 4096
kb_status kb_cluster_update_noalloc(void* cuda_stream, int N, int D, int K, const float* z,
                                    const int32_t* labels, float* centroids, int32_t* counts);
/* Reads the status word of the allocation-free update on the CURRENT device into *out (host
 * pointer; 0 = fine, bit 1 = a label outside [0, K) was skipped since the last read) and clears
 * it.  Synchronises `cuda_stream` (so it sees every call queued there before it); allocates
 * nothing.  Not for the hot path. */
kb_status kb_cluster_update_noalloc_status(void* cuda_stream, int* out);

/* ---- conveniences built from the five calls ----------------------------- */

/* centroids[b][i][:] = z[b][rows[b][i]][:]  (plain Lloyd started from K data
 * rows chosen by the caller; the paper leaves the initialisation open).
 * rows [B][K] in, values in [0,N). */
kb_status kb_init_centroids(kb_ctx* ctx, int B, int N, int D, int K, const float* z,
                            const int32_t* rows, float* centroids);
/* rows[b][i] == -1 (here and in init_rows of kb_bandit_step for instances of at
 * most 512 rows) marks cluster i of instance b as UNUSED: its centroid is put
 * at 1e18 in every coordinate, out of every row's reach, so it stays empty
 * (count 0, rep -1, never selected) and keeps that centroid through every
 * update.  Instances with fewer than K clusters can so share one batch -- the
 * K in {1, 2, 3, 5} sensitivity study of Sec. 4 as four instances of one call
 * with K = 5.  Meant for the fp32 kernels (K < 128 or small instances); the
 * tensor-core kernel stays exact but sends every row through its fp32
 * re-evaluation, because the far centroid spoils the instance's fp16 scale. */

/* iters x (assign, update) followed by a final assign, so that labels/dist2
 * are consistent with the returned centroids (Sec. 3.3).  Same arguments as
 * the two calls it is made of; counts are those of the last update.
 * Instances of at most 512 rows with D in {16, 32, 64} run the whole loop in one launch
 * (one CTA per instance, the instance resident on chip); a single instance of up to about
 * 75 000 rows with D in {16, 32, 64} that is too small for the tensor-core kernel (K < 128)
 * runs it in one cooperative launch (its rows spread over the SMs and kept on chip, one
 * grid-wide barrier per iteration); both unless kb_set_assign_options forces an assign path. */
kb_status kb_cluster_fit(kb_ctx* ctx, int B, int N, int D, int K, int iters, const float* z,
                         float* centroids, int32_t* labels, float* dist2, float* inertia,
                         int32_t* rep, int32_t* counts);

/* kb_cluster_fit with the tolerance stop of the "scikit-learn's KMeans" of
 * Sec. 3.5: per instance, after every update shift = sum_j ||c_j(new) -
 * c_j(old)||^2; the instance stops after the first update with shift <= tol
 * (that update stays) or after max_iter updates; one more assignment then makes
 * labels / dist2 / inertia / rep belong to the returned centroids.  Unchanged
 * labels give shift 0, so "labels repeat" is covered.  (scikit-learn's own
 * `tol` is relative: multiply it by the mean column variance of z, which is 1
 * for z-scored features without constant columns.)  Instances stop
 * independently; everything stays on the device.
 *   tol >= 0;  n_iter [B] out: updates done per instance;  counts: the members
 *   at the instance's last update;  other arguments as kb_cluster_fit.
 * Instances of at most 512 rows with D in {16, 32, 64} stop inside their
 * one-CTA launch.  Otherwise the loop of calls runs all max_iter iterations and
 * a small kernel after every update undoes the updates of instances that have
 * stopped (the result of stopping, not its saving); needs the workspace of
 * kb_workspace_bytes. */
kb_status kb_cluster_fit_tol(kb_ctx* ctx, int B, int N, int D, int K, int max_iter, float tol, const float* z,
                             float* centroids, int32_t* labels, float* dist2, float* inertia, int32_t* rep,
                             int32_t* counts, int32_t* n_iter);

/* Sizes and inputs/outputs of one whole bandit step.  Every pointer is a
 * device pointer for kb_bandit_step and a HOST pointer for kb_bandit_step_host. */
typedef struct {
    int B, N, D, K, S, R, iters;
    float theta_sat;
    kb_score_params score;
    /* inputs */
    const float* x;             /* [B][N][D] raw features */
    const int32_t* init_rows;   /* [B][K] */
    const float* flops;         /* [B][N] */
    const float* bytes;         /* [B][N] */
    const float* peak_flops;    /* [S] */
    const float* peak_bw;       /* [S] */
    const float* t_incumbent;   /* [B] */
    const float* t_cur;         /* [B][N] */
    const float* hsig;          /* [B][K][R] */
    const int32_t* target;      /* [S] */
    const int32_t* pulls;       /* [B][N][S] */
    const float* reward_sum;    /* [B][N][S] */
    const int32_t* t;           /* [B] */
    /* outputs (kb_bandit_step: all required except arm_index and bound;
     * kb_bandit_step_host: any may be NULL and is then not copied back) */
    float* z;                   /* [B][N][D] */
    float* centroids;           /* [B][K][D] */
    int32_t* counts;            /* [B][K] */
    int32_t* labels;            /* [B][N] */
    float* dist2;               /* [B][N] */
    float* inertia;             /* [B] */
    int32_t* rep;               /* [B][K] */
    uint32_t* keep;             /* [B][N] */
    uint32_t* kept_count;       /* [B] */
    float* bound;               /* [B][N][S], nullable */
    float* cl_pulls;            /* [B][K][S] */
    float* cl_mean;             /* [B][K][S] */
    float* cl_index;            /* [B][K][S] */
    float* arm_index;           /* [B][N][S], nullable */
    int32_t* best_arm;          /* [B] */
    float* best_val;            /* [B] */
    int32_t* best_cluster_arm;  /* [B] */
    /* expanding frontier (both nullable; see kb_append_candidate): */
    const int32_t* n_active;    /* [B] candidates per instance: the arrays keep N rows per instance (the
                                 * capacity), the step sees the first n_active[b] of them */
    const int32_t* run_mask;    /* [B] instances with 0 are skipped: none of their outputs is touched */
} kb_step_args;

/* The whole step on device-resident data: normalise, seed centroids, fit,
 * prune (both masks, after the final assign because the saturation mask is
 * indexed by the candidate's cluster), score and select.  Needs the workspace
 * of kb_workspace_bytes.  Instances of at most 512 rows with D in {16, 32, 64}
 * (and 16-byte aligned x, z, centroids) go from raw features to labels in one
 * launch: normalisation and the gather of the initial centroids then happen
 * inside the clustering kernel, with the results kb_normalize and
 * kb_init_centroids would give; a single instance that kb_cluster_fit would
 * run as one cooperative launch does the same there (column statistics across
 * all its CTAs, one more grid barrier).  Instances of at most 1024 candidates with S in
 * {4, 8, 16, 32}, K*S <= 8192 and 16-byte aligned per-arm arrays are pruned,
 * scored and selected by one more launch (one CTA per instance, the arithmetic
 * of kb_prune and kb_score_select). */
kb_status kb_bandit_step(kb_ctx* ctx, const kb_step_args* args);

/* ---- the expanding frontier ------------------------------------------------
 * Sec. 2.2: the action space A_t = P_t x S grows with the frontier P_t, which
 * is what sets the problem apart from a fixed-arm bandit; Algorithm 1: "P <-
 * {k_0}, C <- {P}" (one initial cluster) and, inside "if Verify(k'_t)", "P <- P
 * U {k'_t}"; re-partition "if t mod tau = 0 and |P| >= 2K".
 *
 * The frontier of every search lives in arrays of a fixed capacity N_cap rows
 * per instance; n_active[b] of them are candidates, the rest is padding whose
 * label the caller initialises to -1 (so that no padding row is ever drawn).
 * kb_bandit_step and kb_bandit_step_tail take n_active (and run_mask) in
 * kb_step_args for instances that run as one CTA each (at most 512 rows with D
 * in {16, 32, 64} for the clustering, at most 1024 with S in {4, 8, 16, 32} for
 * the tail; KB_ERR_UNSUPPORTED otherwise): features are z-scored over the
 * active rows only, initial rows must be active, outputs of padding rows are
 * not written.  kb_sample_member needs no change (a padding row's label -1 is
 * no cluster), kb_record_outcome and kb_select_pair neither. */

/* Appends the verified kernel k'_t of every search to its frontier.  Where
 * verified[b] != 0 (null: all), parent[b] >= 0 (the drawn k_t, as
 * kb_sample_member wrote it) and n_active[b] < N_cap, row j = n_active[b]
 * becomes the new candidate:
 *   x[b][j] = x_new[b], t_cur[b][j] = t_new[b]; flops, bytes, h_cand rows from
 *   flops_new, bytes_new, h_new (each pair nullable together);
 *   pulls[b][j][.] = 0, reward_sum[b][j][.] = 0 (nobody has played it);
 *   labels[b][j] = labels[b][parent[b]], dist2[b][j] = dist2[b][parent[b]]
 *   (until the next re-clustering it sits in the cluster of the kernel it was
 *   generated from); t_incumbent[b] = min(t_incumbent[b], t_new[b]) (the best
 *   runtime so far, Algorithm 1's return line); n_active[b] += 1.
 * appended [B] out, nullable: the row written, or -1.  A full frontier drops
 * the candidate and sets bit 0x008 of the device status word; parent[b] >=
 * n_active[b] sets 0x004 and appends nothing.
 *   verified [B], parent [B] in; x_new [B][D], t_new [B], flops_new [B],
 *   bytes_new [B], h_new [B][R] in; n_active [B] in/out;
 *   x [B][N_cap][D], t_cur, flops, bytes, dist2 [B][N_cap], h_cand
 *   [B][N_cap][R], labels [B][N_cap], pulls, reward_sum [B][N_cap][S] in/out;
 *   t_incumbent [B] in/out, nullable; dist2 nullable.
 * DEVICE memory.  One launch (one warp per instance), no workspace. */
kb_status kb_append_candidate(kb_ctx* ctx, int B, int N_cap, int D, int S, int R, const int32_t* verified,
                              const int32_t* parent, const float* x_new, const float* t_new,
                              const float* flops_new, const float* bytes_new, const float* h_new,
                              int32_t* n_active, float* x, float* t_cur, float* flops, float* bytes,
                              float* h_cand, int32_t* labels, float* dist2, int32_t* pulls, float* reward_sum,
                              float* t_incumbent, int32_t* appended);

/* Algorithm 1's test per search: due[b] = (t[b] mod tau == 0 and n_active[b]
 * >= 2K); any_due [1] out, nullable: 1 if any search is due, else 0 -- the one
 * word a host reads to decide whether to queue the re-clustering (which it may
 * also queue unconditionally with run_mask = due).  DEVICE memory; one launch. */
kb_status kb_recluster_due(kb_ctx* ctx, int B, int tau, int K, const int32_t* t, const int32_t* n_active,
                           int32_t* due, int32_t* any_due);

/* The signature of every cluster after a re-clustering (Algorithm 1: "profile
 * h_c^(i) <- NCU(k_c^(i))", the per-candidate signatures standing in for the
 * profiler): hsig[b][i][:] = h_cand[b][rep[b][i]][:], and +inf for an empty
 * cluster (rep -1), whose mask entry M_{i,s} = [h < theta_sat] is then 0, so
 * kb_select_pair never picks an empty cluster.  Instances with run_mask[b] ==
 * 0 (nullable: all run) keep their hsig.
 *   rep [B][K], h_cand [B][N][R], run_mask [B] in;  hsig [B][K][R] out.
 * DEVICE memory; one launch. */
kb_status kb_signatures_from_reps(kb_ctx* ctx, int B, int N, int K, int R, const int32_t* rep, const float* h_cand,
                                  const int32_t* run_mask, float* hsig);

/* The tail of the step alone: kb_prune (both masks and, when `bound` is given,
 * the gain bound) followed by kb_score_select, from labels and dist2 that the
 * CALLER provides (here `labels` and `dist2` of kb_step_args are INPUTS), with
 * the results those two calls give.  Reads B, N, K, S, R, theta_sat, score, the
 * pruning and scoring inputs, and writes keep, kept_count, bound (nullable),
 * the three cluster tables, arm_index (nullable) and the two selections; x,
 * init_rows, z, centroids, counts, inertia, rep, D and iters are ignored.
 * S in {4, 8, 16, 32} with 16-byte aligned per-arm arrays runs fused: the
 * pruning rides on the pass that gathers the cluster statistics, so a
 * candidate's label and keep word are touched once (Sec. 5's batched setting
 * scores millions of arms per step); three launches, or one for instances of
 * at most 1024 candidates.  Other shapes run the two calls one after the other.
 * Device pointers; needs the workspace of kb_workspace_bytes. */
kb_status kb_bandit_step_tail(kb_ctx* ctx, const kb_step_args* args);

/* The same step for a caller whose data lives in HOST memory: copies the
 * inputs to the device, runs the calls of kb_bandit_step, copies the requested
 * outputs back and synchronises the stream before returning.  The inputs that
 * only pruning and scoring read (work, traffic, runtimes, signatures, pulls,
 * rewards) travel on a second stream owned by the context while the clustering
 * runs on the caller's stream; the caller's stream waits for them before
 * kb_prune.  When bound is requested and holds a megabyte or more, the gain
 * bound, which depends on none of the clustering, is computed on a third stream
 * as soon as its six inputs are up and travels back while the clustering runs;
 * the values are the ones kb_prune gives.  The device
 * staging area is carved from the registered workspace, which must hold
 * kb_step_workspace_bytes(...) bytes.  Pinned host memory makes the copies
 * asynchronous; pageable memory works too.  Since this call synchronises
 * anyway, it also reads the device status word before returning: a timeout bit
 * gives KB_ERR_TIMEOUT, a contract bit (label, target or index out of range)
 * KB_ERR_INVALID_ARG; the outputs are then unspecified. */
kb_status kb_step_workspace_bytes(int B, int N, int D, int K, int S, int R, size_t* out);
kb_status kb_bandit_step_host(kb_ctx* ctx, const kb_step_args* host_args);

#ifdef __cplusplus
}
#endif
#endif /* KB_H_ */
