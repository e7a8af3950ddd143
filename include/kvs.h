/*
 * kvs.h - C ABI of the batched KV-memory-constrained schedule builder and evaluator (sm_100a).
 *
 * Problem statement (paper, Preliminaries / "Model and Objective"): an instance is a set of
 * jobs, job i having a prompt length s_i and a response length o_i; time proceeds in unit
 * rounds; a job that has received u rounds of processing holds s_i + u + 1 tokens of KV
 * memory in its next round; the tokens held by all active jobs must not exceed the budget M
 * in any round (Eq. Memory-Feasibility); the objective is the total flow time, the sum of
 * the completion rounds.
 *
 * A *run* is (job, start, len): the job is active in rounds start .. start+len-1.  A run
 * whose length equals o_i completes the job; a shorter run was killed and its progress lost.
 *
 * Conventions
 *   - Every entry point returns a kvs_status; nothing throws, aborts or traps on the device.
 *   - Pointers are marked HOST or DEVICE.  The library allocates no device memory: inputs,
 *     outputs and the workspace are caller-owned device buffers (for example PyTorch
 *     tensors) that must stay alive until the stream has finished the call.
 *   - All work is enqueued on the context's CUDA stream; calls do not synchronise the host
 *     unless stated.
 *   - Argument errors are found on the host before any launch.  Data errors (a job that
 *     cannot fit, an output range or capacity that is too small) are reported per
 *     evaluation in `status[]`; the kernels skip or clip the offending evaluation and
 *     finish normally.
 */
#ifndef KVS_H
#define KVS_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum kvs_status {
  KVS_OK = 0,
  KVS_E_ARG = -1,       /* null / inconsistent argument */
  KVS_E_CUDA = -2,      /* a CUDA runtime call failed; see kvs_last_error */
  KVS_E_CAPACITY = -3,  /* workspace too small */
  KVS_E_RANGE = -4,     /* a parameter is outside the supported range */
  KVS_E_STATE = -5      /* context not initialised / wrong device */
};

/* Schedule families.  GBA: Algorithm "Geometric Batching Algorithm"; GSA: Algorithm
 * "Geometric Slicing Algorithm"; SPS: Procedure "StaggeredPipelineSchedule" run once on the
 * whole instance; SIMS: the simultaneous schedule (Appendix "Lower Bounds for SimS"). */
enum kvs_family { KVS_GBA = 0, KVS_GSA = 1, KVS_SPS = 2, KVS_SIMS = 3,
                  /* GBA with dynamic refill (Numerical Experiments, "Dynamic Refill (GBA-D)"): the batching schedule is
                   * formed first; then, in its order, every job moves to the earliest round between the previous
                   * admission and its own start at which the whole plan - earlier jobs at their new starts, later
                   * ones still at their old ones - fits the budget in every round.  No job starts later than in the
                   * batching schedule.  Accepted by kvs_evaluate_built (which needs job_start, job_completion and a
                   * profile with the batching schedule's horizon as capacity: they are its working storage) and by
                   * kvs_build_schedule (which reports the batching schedule: its horizon sizes the profile); offline
                   * instances without estimates only. */
                  KVS_GBAD = 4,
                  /* GSA with speculative runs (Numerical Experiments, "Speculative Runs (GSA-Spec)"): the slicing
                   * schedule is formed first and kept; round by round, memory it leaves free starts further runs of
                   * jobs that are neither done nor running, lowest index first, as long as the first round of the
                   * next one fits; when the schedule's own runs need the memory the speculative run started last is
                   * killed; a job completed by a speculative run drops out of the schedule's later phases.  job_start and
                   * job_completion are those of the run that completed the job; job_steps and n_runs count every executed
                   * run, the rounds of killed speculative runs included; the profile holds both kinds of runs.  No job
                   * completes later than in the slicing schedule.  Accepted like KVS_GBAD (job_start, job_completion
                   * and a profile with the slicing schedule's horizon as capacity are the working storage;
                   * kvs_build_schedule reports the slicing schedule); offline instances without estimates, staggered
                   * subroutine, one prompt length for the parallelism. */
                  KVS_GSAS = 5 };

/* Bits of the per-evaluation status word. */
enum kvs_eval_status {
  KVS_EVAL_OK = 0,
  KVS_EVAL_INFEASIBLE = 1,  /* some o_i > M - s_bar, or no parallelism >= 1 fits: nothing was scheduled */
  KVS_EVAL_RANGE = 2,       /* a time does not fit the 32-bit outputs, or the memory bound exceeds 2^32 */
  KVS_EVAL_CAPACITY = 4,    /* runs or profile clipped at the caller's capacity */
  KVS_EVAL_BAD_INPUT = 8    /* instance has o_i < 1, s_i < 0, an estimate < 1, unsorted arrivals or too many jobs */
};

typedef struct kvs_ctx kvs_ctx; /* opaque; owned by the library (host object only) */

typedef struct {
  int32_t device;           /* CUDA device ordinal */
  void* stream;             /* cudaStream_t; NULL = the default stream */
  void* workspace;          /* DEVICE, caller-owned, 256-byte aligned */
  uint64_t workspace_bytes;
} kvs_init_params;

/* Creates a context bound to one device, one stream and one workspace.  Host-side only.
 * Fails with KVS_E_CUDA when no CUDA device is present: there is no CPU path. */
int kvs_init(const kvs_init_params* params, kvs_ctx** out);
int kvs_destroy(kvs_ctx* ctx);
/* Last error text of this context (valid until the next call on it). */
const char* kvs_last_error(const kvs_ctx* ctx);

/* Optional kernel timing: when enabled, the fused entry points bracket their two kernels with
 * CUDA events on the context's stream.  kvs_last_timing synchronises on those events and returns
 * the device time in milliseconds of the ordering kernel and of the builder/evaluator kernel of
 * the most recent fused call (0 if timing was off). */
int kvs_set_timing(kvs_ctx* ctx, int32_t enabled);
int kvs_last_timing(kvs_ctx* ctx, float* sort_ms, float* build_ms);
/* The same with the builder/evaluator stage split: the variant of the fast kernel for evaluations
 * that walk no rounds (`light_ms`) and everything after it - the full variant and the general
 * kernel, and the refill / speculative-run kernel of a call with such evaluations (`full_ms`).  A call
 * that took the general kernel alone reports it all as `full_ms`. */
int kvs_last_timing_split(kvs_ctx* ctx, float* sort_ms, float* light_ms, float* full_ms);

/* Checked build.  A library compiled with -DKVS_DEBUG tests every computed index of the fast fused kernel
 * (shared-memory ring, per-CTA scratch, the caller's profile and per-job outputs) and of the refill and
 * speculative-run kernels (profile rounds, per-job outputs, list, stack and scratch of a warp) against its bound
 * before the access; a violation is recorded in one device word (code << 56 | index, the first one wins), the
 * access is skipped and the kernel carries on - nothing traps.  This call returns that word for the
 * current device (0 = no violation; synchronises the device) and clears it if `reset` is nonzero;
 * *compiled_in = 1 for a checked build, 0 for a normal one (the word is then always 0).  Either pointer
 * may be NULL. */
int kvs_debug_check_word(uint64_t* word, int32_t* compiled_in, int32_t reset);

/* Workspace needed by any call whose sizes do not exceed the given ones.
 *   n_jobs_total           sum of jobs over all instances of a call
 *   n_instances            instances per call
 *   max_jobs_per_instance  largest instance
 *   n_evaluations          (instance, setting, family) evaluations per call
 *   generic_capacity       sum of profile capacities passed to kvs_evaluate_schedule (0 if unused)
 *   host_staging           nonzero if the *_host entry point will be used */
int kvs_workspace_bytes(int64_t n_jobs_total, int64_t n_instances, int64_t max_jobs_per_instance,
                        int64_t n_evaluations, int64_t generic_capacity, int32_t host_staging,
                        uint64_t* out);

/* Batched instances in CSR form.  Jobs of instance j are entries job_off[j] .. job_off[j+1]-1. */
typedef struct {
  int64_t n_instances;
  int64_t n_jobs_total;           /* = job_off[n_instances] (host copy, used for sizing) */
  int64_t max_jobs_per_instance;  /* upper bound on any instance's size (host copy) */
  const int64_t* job_off;         /* DEVICE [n_instances + 1] */
  const int32_t* s;               /* DEVICE [n_jobs_total], prompt lengths, >= 0 */
  const int32_t* o;               /* DEVICE [n_jobs_total], response lengths, >= 1 */
  const int32_t* o_est;           /* DEVICE [n_jobs_total] estimates (>= 1) used for ordering and class
                                     assignment, or NULL: the exact o is used */
  const int64_t* arrival;         /* DEVICE [n_jobs_total], nondecreasing per instance, or NULL (all 0) */
  int64_t window;                 /* W > 0: jobs are grouped by floor(arrival / W) and each group is
                                     scheduled as an offline instance released at (w+1)*W; 0: offline,
                                     `arrival` must be NULL */
} kvs_instances;

/* One evaluation = one instance under one parameter setting and one family. */
typedef struct {
  int64_t instance;
  int32_t family;               /* kvs_family */
  int32_t alpha_num, alpha_den; /* GBA/GSA scaling factor alpha = num/den > 1 (first line of both algorithms) */
  int32_t s_bar;                /* prompt length used for the ladder and k*; -1 = max_i s_i of the instance */
  int64_t M;                    /* KV-memory budget, 1 <= M < 2^31 */
  int64_t beta0;                /* 0: the paper's tau_hat_0 = (M - s_bar)/alpha^ell; > 0: tunable initial slice */
  int64_t tau;                  /* SPS/SIMS slice length; 0 = largest key of the (sub-)instance */
  int64_t k;                    /* SPS: parallelism, 0 = k*(tau, s_bar) (Eq. max-parallelism);
                                   SIMS: batch size, 0 = floor(M / (s_bar + tau)) */
  /* Variants inside the geometric classes (GBA / GSA only; both 0 = the paper's algorithms). */
  int32_t subroutine;           /* 0: every phase runs Procedure StaggeredPipelineSchedule; 1: every phase runs the
                                   simultaneous schedule instead - batches of floor(M / (s + tau_p)) jobs start together
                                   every tau_p rounds (Section "Subroutine: Staggered-Pipeline-Schedule", paragraph "The
                                   Simultaneous Batching Trap"; Appendix "Lower Bounds for SimS") */
  int32_t per_class_s;          /* 1: the prompt length that sizes a phase's parallelism (or batch) is the longest prompt
                                   among that phase's participants instead of s_bar; the ladder still ends at M - s_bar */
} kvs_setting;

/* Per-job and per-run outputs of the builder.  Any pointer may be NULL to skip that output. */
typedef struct {
  const int64_t* job_out_off;   /* DEVICE [P + 1]: evaluation e writes its n jobs at job_out_off[e] + i,
                                   i = the job's index inside its instance (original order) */
  int32_t* job_start;           /* DEVICE: start round of the job's completing run, -1 if never completed */
  int32_t* job_completion;      /* DEVICE: completion round = start + o_i, -1 if never completed */
  int64_t* job_start64;         /* DEVICE: 64-bit variants, for horizons >= 2^31 */
  int64_t* job_completion64;
  const int64_t* run_off;       /* DEVICE [P + 1]: capacity offsets of the explicit run list */
  int32_t* run_job;             /* DEVICE: runs in (window, phase, rank) order */
  int32_t* run_phase;
  int64_t* run_start;
  int32_t* run_len;
  int32_t* run_s;
  int64_t* n_runs;              /* DEVICE [P]: number of runs of the schedule (may exceed the capacity) */
} kvs_schedule_out;

/* Per-evaluation results.  Any pointer may be NULL. */
typedef struct {
  const int64_t* profile_off;   /* DEVICE [P + 1]: capacity offsets into `profile`; an evaluation with
                                   capacity 0 gets no profile (its peak is still computed) */
  int32_t* profile;             /* DEVICE, 16-byte aligned: tokens held in rounds 0 .. horizon-1 (clipped at the capacity);
                                   rounds between the horizon and the last slot end, if inside the
                                   capacity, are written as 0 */
  int64_t* peak;                /* DEVICE [P]: max over rounds of the profile (-1 if not computed) */
  int64_t* flow;                /* DEVICE [P]: sum over completed jobs of completion - arrival */
  int64_t* job_steps;           /* DEVICE [P]: sum of run lengths */
  int64_t* horizon;             /* DEVICE [P]: last run end */
  int64_t* n_unfinished;        /* DEVICE [P]: jobs that never complete (SPS/SIMS with o_i > tau) */
  uint8_t* feasible;            /* DEVICE [P]: 1 iff status is OK and peak <= M */
  int32_t* status;              /* DEVICE [P]: kvs_eval_status bits */
} kvs_eval_out;

/* Builds the schedules (start and completion round of every job, optional run list):
 * ordering by (estimated) response length, geometric class / slice assignment, ranks,
 * phase bases, start = base_p + floor(r * tau_p / k_p) (Procedure StaggeredPipelineSchedule),
 * completion = start + o_i.  `settings` is a HOST array of P entries; it is copied to the
 * workspace asynchronously (the caller must not modify it before the stream reaches the copy).
 * `ev` may be NULL; if given, only its scalar fields and status are filled (no profile, peak = -1). */
int kvs_build_schedule(kvs_ctx* ctx, const kvs_instances* inst, const kvs_setting* settings, int64_t P,
                       const kvs_schedule_out* out, const kvs_eval_out* ev);

/* Builder and evaluator fused: in addition to kvs_build_schedule, forms the per-round memory
 * profile of every schedule from two difference arrays (Eq. Memory-Feasibility: a run holds
 * s + u + 1 tokens in its round u), its peak, and the feasibility mask peak <= M.
 * `out` may be NULL when only the evaluation is wanted. */
int kvs_evaluate_built(kvs_ctx* ctx, const kvs_instances* inst, const kvs_setting* settings, int64_t P,
                       const kvs_schedule_out* out, const kvs_eval_out* ev);

/* Same as kvs_evaluate_built for HOST inputs and HOST scalar results: copies job_off, s, o
 * (and o_est, arrival) to the workspace, runs the fused path, and copies the per-evaluation
 * scalars back.  Every pointer of `inst` and of `ev` is a HOST pointer here (pinned memory
 * makes the copies asynchronous); `ev->profile` must be NULL.  The instances are worked off in up
 * to 16 chunks (of about a thousand evaluations or more, so small batches stay in one piece): the jobs of the next chunk are copied on a second stream while the kernels of the
 * current one run, so the settings may come in any order but are evaluated grouped by instance
 * (results are returned in the caller's order).  job_off is read on the host and must be
 * nondecreasing.  The call returns after the stream has been synchronised. */
int kvs_evaluate_built_host(kvs_ctx* ctx, const kvs_instances* inst, const kvs_setting* settings,
                            int64_t P, const kvs_eval_out* ev);

/* Explicit runs of P schedules (the builder's output or any user schedule). */
typedef struct {
  int64_t P;
  const int64_t* run_off;       /* DEVICE [P + 1] */
  const int64_t* run_start;     /* DEVICE [R], >= 0 */
  const int32_t* run_len;       /* DEVICE [R]; runs with len <= 0 are ignored */
  const int32_t* run_s;         /* DEVICE [R], prompt length of the run's job */
  const int64_t* run_flow;      /* DEVICE [R] or NULL: completion - arrival for completing runs, 0 for killed ones */
  const int64_t* M;             /* DEVICE [P] budgets for the feasibility mask, or NULL */
} kvs_runs;

/* Evaluates explicit runs by the definition (Eq. Memory-Feasibility): per-round memory,
 * peak, horizon, job-steps, flow (sum of run_flow) and the mask.  `ev->profile_off` is
 * required (capacities bound the dense arrays); runs reaching beyond the capacity set
 * KVS_EVAL_CAPACITY and are clipped.  `ev->n_unfinished` is not written.  Reads
 * profile_off[P] back to the host once (one small synchronous copy). */
int kvs_evaluate_schedule(kvs_ctx* ctx, const kvs_runs* runs, const kvs_eval_out* ev);

/* (No counterpart in the paper: a packaging variant of kvs_evaluate_schedule.)
 * For callers that must not allocate device memory at all - code that runs where cudaMalloc is
 * forbidden or unavailable, such as a plugin inside a serving process whose memory pool owns the
 * whole GPU, or a latency-critical loop that may not touch the allocator - and therefore cannot
 * provide a workspace.  The two difference arrays live in a fixed 12 MiB array inside the library
 * image (every GPU that loads the library holds it until the process exits).  No context is
 * needed; `device` and `stream` are given directly, `capacity_total` is the host copy of
 * profile_off[P].  Limit: capacity_total + P <= 1,048,576, otherwise KVS_E_CAPACITY and a message
 * in `err` (optional buffer of err_len bytes).  The call itself allocates nothing (no cudaMalloc,
 * no cudaFree, no allocating library routine).
 * The first call on each device looks up the array's device address; make that first call
 * before any stream capture (the look-up is safe against another host thread doing the same).
 * The work is issued with `device` current; the caller's current device is restored on return.
 * All calls on a device share the array: each call clears the part it uses, so results do not
 * depend on earlier calls, but calls that overlap on the GPU (two streams, two threads) race -
 * serialise them.  Outputs and status bits as kvs_evaluate_schedule.  The kernel trusts no host
 * copy: an evaluation whose DEVICE offsets profile_off[e], profile_off[e + 1] are not monotone or
 * reach beyond `capacity_total` is skipped with KVS_EVAL_CAPACITY | KVS_EVAL_BAD_INPUT in
 * status[e] (peak -1, other scalars 0) and nothing of it is written. */
int kvs_evaluate_schedule_noalloc(int32_t device, void* stream, const kvs_runs* runs,
                                  const kvs_eval_out* ev, int64_t capacity_total,
                                  char* err, uint64_t err_len);

/* Bounds that depend on an instance only through the sizes of its classes (class of a job = first
 * slice of the ladder that is at least its response length), per (instance, setting):
 *   upper_gba  UpperGBA, the sum of class-prefix and ladder terms (Lemma "GBA Upper Bound via Packing
 *              Efficiency"): the GBA schedule's total flow time is at most this;
 *   upper_gsa  the bound of Lemma "GSA Upper Bound via Packing Efficiency" (phase-prefix cost,
 *              phase spillover cost, ladder terms);
 *   lower_2m   2 * M * (WithinClass + BetweenClasses) of Lemma "Area-Based Lower Bound for OPT", an
 *              integer: the optimal total flow time is at least lower_2m / (2 M).  The memory-time
 *              area of class p is taken at the integer threshold x_p = tau_(p-1) (x_0 = 0) and at
 *              the prompt length s_bar of the setting, so the bound is the lemma's for instances
 *              with one prompt length and a valid, slightly weaker one otherwise when s_bar does
 *              not exceed any prompt length.
 * Each DEVICE array has P entries; any may be NULL.  status[] holds kvs_eval_status bits
 * (KVS_EVAL_RANGE: a value does not fit 63 bits); the three values are -1 unless status is 0. */
typedef struct {
  int64_t* upper_gba;
  int64_t* upper_gsa;
  int64_t* lower_2m;
  int32_t* status;
} kvs_bounds_out;

/* Uses instance, M, alpha_num/alpha_den, beta0 and s_bar of each setting (HOST array of P entries,
 * copied to the workspace asynchronously); the family, tau and k are ignored.  The instances must
 * be offline (window = 0); estimates, if present, are ignored: the bounds are statements about the
 * exact response lengths.  Asynchronous on the context's stream. */
int kvs_bounds(kvs_ctx* ctx, const kvs_instances* inst, const kvs_setting* settings, int64_t P,
               const kvs_bounds_out* out);

/* Parameter sweep on one instance: SPS or SIMS for every (tau, k) of a grid, scalars only. */
typedef struct {
  int64_t instance;
  int64_t M;                    /* budget for the feasibility mask */
  const int64_t* tau;           /* HOST [n_tau], each in [1, 2^31) */
  const int64_t* k;             /* HOST [n_k], each in [1, 2^31) */
  int32_t n_tau;
  int32_t n_k;                  /* n_tau * n_k <= 65536 */
  int32_t family;               /* KVS_SPS or KVS_SIMS: the (tau, k) grid; KVS_GBA or KVS_GSA: the beta0 grid below */
  /* Geometric families: the initial slice of the ladder is a tunable parameter (footnote to the overview of
   * the slicing algorithm; the experiments use 64 and 256).  One evaluation per entry of beta0 (0 = the
   * paper's (M - s_bar) / alpha^ell); tau, k, n_tau, n_k are ignored and every output has n_beta0 entries. */
  int32_t n_beta0;              /* <= 65536 */
  const int64_t* beta0;         /* HOST [n_beta0], each in [0, 2^31) */
  int32_t alpha_num, alpha_den;
  int32_t subroutine, per_class_s;   /* as in kvs_setting */
} kvs_sweep_params;

typedef struct {                /* DEVICE, each [n_tau * n_k], tau-major; any may be NULL */
  int64_t* peak;
  int64_t* flow;
  int64_t* n_completed;
  int64_t* horizon;
  int64_t* job_steps;
  uint8_t* feasible;            /* peak <= M */
} kvs_sweep_out;

/* Geometric families: for each beta0 the schedule of kvs_evaluate_built with s_bar = the longest prompt;
 * n_completed = jobs that complete (all of them unless the evaluation is infeasible: then peak = -1,
 * feasible = 0 and n_completed = 0).  The instances must be offline and carry no estimates.
 * For each (tau, k): job with rank r (stable order by exact response length) starts at
 * floor(r*tau/k) (SPS, Procedure StaggeredPipelineSchedule) or floor(r/k)*tau (SIMS), runs
 * min(o, tau) rounds and completes iff o <= tau; reports flow over completed jobs, their count,
 * the exact peak of the memory profile (Eq. Memory-Feasibility), horizon and job-steps.
 * No per-job or per-round output; horizons may exceed 2^32.  The instances must be offline
 * (window = 0) and carry no estimates (o_est = NULL).  Reads the instance's two offsets back
 * to the host once (one small synchronous copy). */
int kvs_sweep(kvs_ctx* ctx, const kvs_instances* inst, const kvs_sweep_params* params,
              const kvs_sweep_out* out);

#ifdef __cplusplus
}
#endif
#endif /* KVS_H */
