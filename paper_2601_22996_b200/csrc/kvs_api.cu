// C ABI: argument validation, workspace layout, launches.  Host code only.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "kvs_internal.cuh"

constexpr int KVS_HOST_CHUNKS = 16;   // the host entry point pipelines copies and kernels over this many chunks

struct kvs_ctx {
  int device = 0;
  cudaStream_t stream = nullptr;
  unsigned char* workspace = nullptr;
  uint64_t workspace_bytes = 0;
  int sm_count = 0;
  int build_ctas_per_sm = 1;
  int fused_ctas_per_sm = 1;
  int light_ctas_per_sm = 1;
  bool timing = false;
  bool timed = false;
  bool split_timed = false;   // the last timed call took the fast path (event between its two variants)
  cudaEvent_t ev[4] = {nullptr, nullptr, nullptr, nullptr};   // before the ordering kernel, after it, after the last kernel, after the light variant
  // host entry point: input copies run on a stream of their own, one event per chunk of instances
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t chunk_ev[KVS_HOST_CHUNKS + 1] = {};
  std::vector<kvs_setting> settings_tmp;   // a call's settings with the refill family mapped to the batching one
  std::string err;
};

namespace {

constexpr int64_t KVS_MAX_GRID = 1024;        // upper bound on CTAs of the fused kernel (sizes the carry lists)
constexpr int64_t KVS_TIME_LIMIT = 1ll << 31; // exclusive bound on M, tau, k

int fail(kvs_ctx* ctx, int code, const char* msg) {
  if (ctx) ctx->err = msg;
  return code;
}
int fail_cuda(kvs_ctx* ctx, cudaError_t e, const char* where) {
  if (ctx) ctx->err = std::string(where) + ": " + cudaGetErrorString(e);
  return KVS_E_CUDA;
}

size_t align_up(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

// Offsets of the scratch regions of the fused path inside the workspace.  Calls are ordered on
// one stream, so the entry points reuse the workspace from offset 0; the layout without staging
// is a prefix of the layout with staging.
struct Layout {
  size_t settings, stats, perm, perm_tmp, iperm, sorted_s, sorted_o, sorted_key, prefix_s, lists, fin_rank, counter, slow_list, walk_list, light_list;
  size_t refill_list;                                                    // evaluations whose batching schedule is refilled afterwards
  size_t sweep_unf, sweep_stat;                                         // unfinished counts and status words of a sweep over initial slices
  size_t st_off, st_s, st_o, st_key, st_arr;                            // host staging (inputs)
  size_t sc_peak, sc_flow, sc_steps, sc_hor, sc_unf, sc_feas, sc_stat;  // host staging (scalars)
  size_t total;
};

Layout make_layout(int64_t N, int64_t I, int64_t max_n, int64_t P, bool staging) {
  Layout L{};
  size_t at = 0;
  auto take = [&](size_t bytes) { size_t r = at; at += align_up(bytes); return r; };
  L.settings = take(static_cast<size_t>(P) * sizeof(kvs_setting));
  L.stats = take(static_cast<size_t>(I) * sizeof(InstStats));
  L.perm = take(static_cast<size_t>(N) * 4);
  L.perm_tmp = take(static_cast<size_t>(N) * 4);
  L.sorted_s = take(static_cast<size_t>(N) * 4);
  L.sorted_o = take(static_cast<size_t>(N) * 4);
  L.sorted_key = take(static_cast<size_t>(N) * 4);
  L.prefix_s = take(static_cast<size_t>(N + I) * 8);
  L.iperm = take(static_cast<size_t>(N) * 4);
  const int64_t grid = P < KVS_MAX_GRID ? P : KVS_MAX_GRID;
  L.lists = take(static_cast<size_t>(grid) * static_cast<size_t>(KVS_CTA_SCRATCH(max_n)));
  L.fin_rank = take(static_cast<size_t>(grid) * static_cast<size_t>(max_n) * 4);
  L.counter = take(256);  // work counters of the kernels, lengths of the evaluation lists
  L.slow_list = take(static_cast<size_t>(P) * 8);
  L.walk_list = take(static_cast<size_t>(P) * 8);
  L.light_list = take(static_cast<size_t>(P) * 8);
  L.refill_list = take(static_cast<size_t>(P) * 8);
  L.sweep_unf = take(static_cast<size_t>(P) * 8);
  L.sweep_stat = take(static_cast<size_t>(P) * 4);
  if (staging) {
    L.st_off = take(static_cast<size_t>(I + 1) * 8);
    L.st_s = take(static_cast<size_t>(N) * 4);
    L.st_o = take(static_cast<size_t>(N) * 4);
    L.st_key = take(static_cast<size_t>(N) * 4);
    L.st_arr = take(static_cast<size_t>(N) * 8);
    L.sc_peak = take(static_cast<size_t>(P) * 8);
    L.sc_flow = take(static_cast<size_t>(P) * 8);
    L.sc_steps = take(static_cast<size_t>(P) * 8);
    L.sc_hor = take(static_cast<size_t>(P) * 8);
    L.sc_unf = take(static_cast<size_t>(P) * 8);
    L.sc_feas = take(static_cast<size_t>(P));
    L.sc_stat = take(static_cast<size_t>(P) * 4);
  }
  L.total = at;
  return L;
}

// Generic evaluator: 64-bit constant terms and 32-bit slopes, capacity + one slot per evaluation.
size_t generic_bytes(int64_t cap_total, int64_t P, size_t* second) {
  const size_t a = align_up(static_cast<size_t>(cap_total + P) * 8);
  if (second) *second = a;
  return a + align_up(static_cast<size_t>(cap_total + P) * 4);
}

struct SweepLayout {
  size_t stats, perm, perm_tmp, sorted_s, sorted_o, prefix_s, prefix_o, tau, k, acc_peak, acc_flow, total;
};

SweepLayout make_sweep_layout(int64_t N, int64_t max_n) {
  SweepLayout L{};
  size_t at = 0;
  auto take = [&](size_t bytes) { size_t r = at; at += align_up(bytes); return r; };
  L.stats = take(sizeof(InstStats));
  L.perm = take(static_cast<size_t>(N) * 4);
  L.perm_tmp = take(static_cast<size_t>(N) * 4);
  L.sorted_s = take(static_cast<size_t>(N) * 4);
  L.sorted_o = take(static_cast<size_t>(N) * 4);
  L.prefix_s = take(static_cast<size_t>(max_n + 1) * 8);
  L.prefix_o = take(static_cast<size_t>(max_n + 1) * 8);
  L.tau = take(65536 * 8);
  L.k = take(65536 * 8);
  L.acc_peak = take(65536 * 8);
  L.acc_flow = take(65536 * 8);
  L.total = at;
  return L;
}

int check_instances(kvs_ctx* ctx, const kvs_instances* inst) {
  if (!inst) return fail(ctx, KVS_E_ARG, "instances: null");
  if (inst->n_instances < 0 || inst->n_jobs_total < 0 || inst->max_jobs_per_instance < 0)
    return fail(ctx, KVS_E_ARG, "instances: negative size");
  if (inst->max_jobs_per_instance >= (1ll << 31) - 1) return fail(ctx, KVS_E_RANGE, "instances: more than 2^31-2 jobs in one instance");
  if (!inst->job_off) return fail(ctx, KVS_E_ARG, "instances: job_off is null");
  if (inst->n_jobs_total > 0 && (!inst->s || !inst->o)) return fail(ctx, KVS_E_ARG, "instances: s or o is null");
  if (inst->window < 0) return fail(ctx, KVS_E_ARG, "instances: negative window");
  if (inst->window == 0 && inst->arrival) return fail(ctx, KVS_E_ARG, "instances: arrival given without a window (offline instances take arrival = NULL)");
  return KVS_OK;
}

// The ladder keeps a^j and X*b^j exactly in 128 bits.  With ell = floor(log_alpha X) the largest
// value formed is below a * X * b^(ell+1) (a^j <= X * b^j up to j = ell, one more factor for the
// test that ends the search); refuse parameters for which that might not fit, or that need more
// phases than the table holds.
bool ladder_fits(int64_t M, int a, int b) {
  const double la = std::log2(static_cast<double>(a)), lb = std::log2(static_cast<double>(b));
  const double lx = std::log2(static_cast<double>(M));
  const double ell = std::floor(lx / (la - lb)) + 1.0;   // one spare for rounding of the logarithms
  if (ell + 2.0 > KVS_MAX_PHASES) return false;
  return la + lx + (ell + 2.0) * lb < 125.0;             // also covers beta0 * a^p < a * X * b^p
}

int check_settings(kvs_ctx* ctx, const kvs_instances* inst, const kvs_setting* st, int64_t P) {
  if (P < 0) return fail(ctx, KVS_E_ARG, "settings: negative count");
  if (P > 0 && !st) return fail(ctx, KVS_E_ARG, "settings: null");
  for (int64_t e = 0; e < P; ++e) {
    const kvs_setting& s = st[e];
    if (s.instance < 0 || s.instance >= inst->n_instances) return fail(ctx, KVS_E_ARG, "settings: instance out of range");
    if (s.family < KVS_GBA || s.family > KVS_GSAS) return fail(ctx, KVS_E_ARG, "settings: unknown family");
    if (s.family == KVS_GSAS && (inst->o_est || inst->window != 0 || s.subroutine || s.per_class_s))
      return fail(ctx, KVS_E_ARG, "settings: speculative runs take offline instances without estimates and the plain slicing schedule");
    if (s.family == KVS_GBAD && (inst->o_est || inst->window != 0 || s.subroutine))
      return fail(ctx, KVS_E_ARG, "settings: the dynamic refill takes offline instances without estimates and the staggered subroutine");
    if (s.M < 1 || s.M >= KVS_TIME_LIMIT) return fail(ctx, KVS_E_RANGE, "settings: M outside [1, 2^31)");
    if (s.s_bar < -1) return fail(ctx, KVS_E_ARG, "settings: s_bar < -1");
    if (s.tau < 0 || s.tau >= KVS_TIME_LIMIT || s.k < 0 || s.k >= KVS_TIME_LIMIT)
      return fail(ctx, KVS_E_RANGE, "settings: tau or k outside [0, 2^31)");
    if (s.subroutine < 0 || s.subroutine > 1 || s.per_class_s < 0 || s.per_class_s > 1)
      return fail(ctx, KVS_E_ARG, "settings: subroutine and per_class_s are 0 or 1");
    if ((s.subroutine || s.per_class_s) && s.family != KVS_GBA && s.family != KVS_GSA && s.family != KVS_GBAD && s.family != KVS_GSAS)
      return fail(ctx, KVS_E_ARG, "settings: subroutine and per_class_s apply to the geometric families only");
    if (s.family == KVS_GBA || s.family == KVS_GSA || s.family == KVS_GBAD || s.family == KVS_GSAS) {
      if (s.alpha_den < 1 || s.alpha_num <= s.alpha_den) return fail(ctx, KVS_E_ARG, "settings: alpha must be > 1");
      if (s.beta0 < 0 || s.beta0 >= KVS_TIME_LIMIT) return fail(ctx, KVS_E_RANGE, "settings: beta0 outside [0, 2^31)");
      if (!(s.alpha_num == 2 && s.alpha_den == 1) && !ladder_fits(s.M, s.alpha_num, s.alpha_den))
        return fail(ctx, KVS_E_RANGE, "settings: ladder for this alpha and M needs more than 96 phases or 128-bit integers");
    }
  }
  return KVS_OK;
}

// A call on a sub-range of the instances (host entry point): the `P` settings all name instances in
// [i0, i1) and are evaluations e0 .. e0 + P - 1 of a batch of P_total; `ev` already points at e0.
struct FusedRange { int64_t i0, i1, e0, P_total; };

int run_fused(kvs_ctx* ctx, const kvs_instances* inst, const kvs_setting* settings, int64_t P,
              const kvs_schedule_out* out, const kvs_eval_out* ev, int do_profile, const FusedRange* rg = nullptr) {
  if (!ctx) return KVS_E_STATE;
  int rc = check_instances(ctx, inst);
  if (rc) return rc;
  rc = check_settings(ctx, inst, settings, P);
  if (rc) return rc;
  kvs_schedule_out o{};
  kvs_eval_out v{};
  if (out) o = *out;
  if (ev) v = *ev;
  const bool job_out = o.job_start || o.job_completion || o.job_start64 || o.job_completion64;
  if (job_out && !o.job_out_off) return fail(ctx, KVS_E_ARG, "schedule_out: job outputs need job_out_off");
  const bool run_out = o.run_job || o.run_phase || o.run_start || o.run_len || o.run_s;
  if (run_out && !o.run_off) return fail(ctx, KVS_E_ARG, "schedule_out: run outputs need run_off");
  if (v.profile && !v.profile_off) return fail(ctx, KVS_E_ARG, "eval_out: profile needs profile_off");
  if (reinterpret_cast<uintptr_t>(v.profile) & 15u) return fail(ctx, KVS_E_ARG, "eval_out: profile must be 16-byte aligned");
  if (!do_profile) v.profile = nullptr;
  if (P == 0) return KVS_OK;
  // Dynamic refill: the fused kernels form the batching schedule; a last kernel refills it in place.
  // Speculative runs: the same on top of the slicing schedule.
  std::vector<int64_t> refill, spec;
  for (int64_t e = 0; e < P; ++e) {
    if (settings[e].family == KVS_GBAD) refill.push_back(e);
    if (settings[e].family == KVS_GSAS) spec.push_back(e);
  }
  if (!refill.empty() || !spec.empty()) {
    if (rg) return fail(ctx, KVS_E_ARG, "the host entry point takes neither the dynamic refill nor speculative runs (they need per-job results and a profile on the device)");
    if (do_profile && (!o.job_start || !o.job_completion || !v.profile || o.job_start64 || o.job_completion64 || run_out))
      return fail(ctx, KVS_E_ARG, "the dynamic refill and speculative runs need job_start, job_completion and a profile (32-bit, no run list): they are their working storage");
    if (do_profile && (!v.horizon || !v.status))
      return fail(ctx, KVS_E_ARG, "the dynamic refill and speculative runs need the horizon and status outputs");
    ctx->settings_tmp.assign(settings, settings + P);
    for (int64_t e : refill) ctx->settings_tmp[static_cast<size_t>(e)].family = KVS_GBA;
    for (int64_t e : spec) ctx->settings_tmp[static_cast<size_t>(e)].family = KVS_GSA;
    settings = ctx->settings_tmp.data();
  }

  const int64_t N = inst->n_jobs_total, I = inst->n_instances, max_n = inst->max_jobs_per_instance;
  const Layout L = make_layout(N, I, max_n, rg ? rg->P_total : P, false);
  if (L.total > ctx->workspace_bytes)
    return fail(ctx, KVS_E_CAPACITY, "workspace too small for this call (see kvs_workspace_bytes)");
  cudaError_t ce = cudaSetDevice(ctx->device);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "cudaSetDevice");
  unsigned char* ws = ctx->workspace;
  const int64_t i0 = rg ? rg->i0 : 0, n_inst = rg ? rg->i1 - rg->i0 : I, e0 = rg ? rg->e0 : 0;
  unsigned char* const settings_dev = ws + L.settings + static_cast<size_t>(e0) * sizeof(kvs_setting);
  ce = cudaMemcpyAsync(settings_dev, settings, static_cast<size_t>(P) * sizeof(kvs_setting), cudaMemcpyHostToDevice, ctx->stream);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "copy of settings");

  bool need_order = inst->o_est != nullptr;
  for (int64_t e = 0; e < P && !need_order; ++e) need_order = settings[e].family != KVS_GSA;

  SortParams sp{};
  // the ordering kernel numbers its instances from 0: a sub-range shifts the per-instance arrays
  sp.job_off = inst->job_off + i0; sp.s = inst->s; sp.o = inst->o; sp.key = inst->o_est; sp.arrival = inst->arrival;
  sp.window = inst->window; sp.n_instances = n_inst; sp.max_jobs = max_n; sp.need_order = need_order ? 1 : 0;
  sp.stats = reinterpret_cast<InstStats*>(ws + L.stats) + i0;
  sp.perm = reinterpret_cast<int32_t*>(ws + L.perm);
  sp.perm_tmp = reinterpret_cast<int32_t*>(ws + L.perm_tmp);
  sp.iperm = reinterpret_cast<int32_t*>(ws + L.iperm);
  sp.sorted_s = reinterpret_cast<int32_t*>(ws + L.sorted_s);
  sp.sorted_o = reinterpret_cast<int32_t*>(ws + L.sorted_o);
  sp.sorted_key = reinterpret_cast<int32_t*>(ws + L.sorted_key);
  // SPS / SimS evaluations that ask for no profile take the peak from run ends instead of rounds;
  // that needs prefix sums of s in key order (exact keys only)
  bool event_form = false;
  if (do_profile && !inst->o_est)
    for (int64_t e = 0; e < P && !event_form; ++e) event_form = settings[e].family >= KVS_SPS;
  sp.prefix_s = event_form ? reinterpret_cast<i64*>(ws + L.prefix_s) + i0 : nullptr;   // instance j writes at job_off[j] + j
  const int64_t sort_cap = static_cast<int64_t>(ctx->sm_count) * 2;
  const int sort_grid = static_cast<int>(n_inst < sort_cap ? n_inst : sort_cap);
  if (ctx->timing && !rg) cudaEventRecord(ctx->ev[0], ctx->stream);
  ce = kvs_launch_sort(sp, sort_grid, ctx->stream);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "sort launch");
  if (ctx->timing && !rg) cudaEventRecord(ctx->ev[1], ctx->stream);

  BuildParams bp{};
  bp.job_off = inst->job_off; bp.s = inst->s; bp.o = inst->o; bp.key = inst->o_est; bp.arrival = inst->arrival;
  bp.window = inst->window; bp.n_instances = I; bp.max_jobs = max_n;
  bp.perm = sp.perm; bp.sorted_s = sp.sorted_s; bp.sorted_o = sp.sorted_o; bp.sorted_key = sp.sorted_key;
  bp.prefix_s = event_form ? reinterpret_cast<i64*>(ws + L.prefix_s) : nullptr;
  bp.iperm = sp.iperm;
  bp.fin_rank = reinterpret_cast<int32_t*>(ws + L.fin_rank);
  bp.stats = reinterpret_cast<InstStats*>(ws + L.stats);
  bp.settings = reinterpret_cast<const kvs_setting*>(settings_dev);
  bp.P = P; bp.out = o; bp.ev = v; bp.do_profile = do_profile;
  bp.lists = reinterpret_cast<int32_t*>(ws + L.lists);
  ull* const counters = reinterpret_cast<ull*>(ws + L.counter);
  auto grid_for = [&](int ctas_per_sm) {
    int64_t g = static_cast<int64_t>(ctx->sm_count) * ctas_per_sm;
    if (g > KVS_MAX_GRID) g = KVS_MAX_GRID;
    if (g > P) g = P;
    return static_cast<int>(g);
  };
  // The 32-bit fast kernel covers calls that want neither the explicit run list nor 64-bit job
  // results; evaluations it cannot finish (times of 2^31 or more, memory bound of 2^32 or more)
  // come back in a list that the general kernel works off.  Other calls go to the general kernel.
  const bool fast = !run_out && !o.job_start64 && !o.job_completion64;
  if (fast) {
    // Two variants of the fast kernel.  The light one (no ring, three CTAs per SM) takes the
    // evaluations that walk no rounds: all of them when no profile is formed, else the SPS / SimS
    // ones, of which it passes on those that turn out to want their profile.  The full one takes
    // the geometric evaluations, listed here on the host, and what the light one passed on.
    std::vector<int64_t> ids(static_cast<size_t>(P));
    int64_t n_full = 0, n_light = 0;
    for (int64_t e = 0; e < P; ++e)
      if (do_profile && settings[e].family <= KVS_GSA) ids[static_cast<size_t>(n_full++)] = e;
    for (int64_t e = 0; e < P; ++e)
      if (!(do_profile && settings[e].family <= KVS_GSA)) ids[static_cast<size_t>(n_full + n_light++)] = e;
    // Longest first: the rounds of a schedule grow as the budget shrinks and the slicing algorithm
    // visits more runs than the batching one, and the CTAs draw evaluations in list order, so this
    // order keeps the last CTAs from finishing a long evaluation alone.
    // Without estimates every family has its own instantiation of the kernel and its own part of the
    // list: in the full variant the slicing algorithm first, then the batching one.
    const bool split = inst->o_est == nullptr;
    std::stable_sort(ids.begin(), ids.begin() + n_full, [&](int64_t a, int64_t b) {
      if (split && settings[a].family != settings[b].family) return settings[a].family > settings[b].family;
      if (settings[a].M != settings[b].M) return settings[a].M < settings[b].M;
      return settings[a].family > settings[b].family;
    });
    if (split)
      std::stable_sort(ids.begin() + n_full, ids.end(), [&](int64_t a, int64_t b) { return settings[a].family < settings[b].family; });
    int64_t full_of[4] = {0, 0, 0, 0}, light_of[4] = {0, 0, 0, 0};
    if (split) {
      for (int64_t i = 0; i < n_full; ++i) ++full_of[settings[ids[static_cast<size_t>(i)]].family];
      for (int64_t i = n_full; i < P; ++i) ++light_of[settings[ids[static_cast<size_t>(i)]].family];
    }
    // [1] left-over count, [2] general work, [3] length of the full variant's list, [4] work of the full
    // variant for any family (starts behind the evaluations the family kernels take), [6] [7] work and
    // count of the light variant for any family, [8 + 2f] [9 + 2f] of the light kernel of family f,
    // [16 + 2f] [17 + 2f] of the full kernel of family f
    unsigned long long init[32] = {};
    init[3] = static_cast<unsigned long long>(n_full);
    init[4] = static_cast<unsigned long long>(split ? n_full : 0);
    init[7] = static_cast<unsigned long long>(split ? 0 : n_light);
    for (int f = 0; f < 4; ++f) {
      init[9 + 2 * f] = static_cast<unsigned long long>(light_of[f]);
      init[17 + 2 * f] = static_cast<unsigned long long>(full_of[f]);
    }
    if ((ce = cudaMemcpyAsync(counters, init, sizeof(init), cudaMemcpyHostToDevice, ctx->stream)) != cudaSuccess ||
        (n_full && (ce = cudaMemcpyAsync(ws + L.walk_list, ids.data(), static_cast<size_t>(n_full) * 8, cudaMemcpyHostToDevice, ctx->stream)) != cudaSuccess) ||
        (n_light && (ce = cudaMemcpyAsync(ws + L.light_list, ids.data() + n_full, static_cast<size_t>(n_light) * 8, cudaMemcpyHostToDevice, ctx->stream)) != cudaSuccess))
      return fail_cuda(ctx, ce, "copy of the evaluation lists");
    bp.slow_count = counters + 1;
    bp.slow_list = reinterpret_cast<i64*>(ws + L.slow_list);
    bp.walk_count = counters + 3;
    bp.walk_list = reinterpret_cast<i64*>(ws + L.walk_list);
    const i64* const light_list = reinterpret_cast<const i64*>(ws + L.light_list);
    if (split) {
      int64_t at = 0;
      for (int f = 0; f < 4; ++f) {
        if (light_of[f]) {
          bp.counter = counters + 8 + 2 * f;
          bp.eval_list = light_list + at;
          bp.eval_count = counters + 9 + 2 * f;
          ce = kvs_launch_fused(bp, grid_for(ctx->light_ctas_per_sm), 1, f, ctx->stream);
          if (ce != cudaSuccess) return fail_cuda(ctx, ce, "fused launch");
        }
        at += light_of[f];
      }
    } else if (n_light) {
      bp.counter = counters + 6;
      bp.eval_list = light_list;
      bp.eval_count = counters + 7;
      ce = kvs_launch_fused(bp, grid_for(ctx->light_ctas_per_sm), 1, KVS_FUSED_ANY, ctx->stream);
      if (ce != cudaSuccess) return fail_cuda(ctx, ce, "fused launch");
    }
    if (ctx->timing && !rg) cudaEventRecord(ctx->ev[3], ctx->stream);
    if (split) {
      int64_t at = 0;
      for (int f = KVS_GSA; f >= KVS_GBA; --f) {   // the order of the list
        if (full_of[f]) {
          bp.counter = counters + 16 + 2 * f;
          bp.eval_list = bp.walk_list + at;
          bp.eval_count = counters + 17 + 2 * f;
          ce = kvs_launch_fused(bp, grid_for(ctx->fused_ctas_per_sm), 0, f, ctx->stream);
          if (ce != cudaSuccess) return fail_cuda(ctx, ce, "fused launch");
        }
        at += full_of[f];
      }
    }
    if (n_light || (!split && n_full)) {
      // what the light variant passed on, and the geometric evaluations of a call with estimates
      bp.counter = counters + 4;
      bp.eval_list = bp.walk_list;
      bp.eval_count = bp.walk_count;
      ce = kvs_launch_fused(bp, grid_for(ctx->fused_ctas_per_sm), 0, KVS_FUSED_ANY, ctx->stream);
      if (ce != cudaSuccess) return fail_cuda(ctx, ce, "fused launch");
    }
    bp.eval_list = bp.slow_list;
    bp.eval_count = bp.slow_count;
  }
  bp.counter = counters + 2;
  ce = kvs_launch_build(bp, grid_for(ctx->build_ctas_per_sm), ctx->stream);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "build launch");
  if (do_profile && !refill.empty()) {
    ce = cudaMemcpyAsync(ws + L.refill_list, refill.data(), refill.size() * 8, cudaMemcpyHostToDevice, ctx->stream);
    if (ce != cudaSuccess) return fail_cuda(ctx, ce, "copy of the refill list");
    RefillParams rp{};
    rp.job_off = inst->job_off; rp.perm = sp.perm; rp.sorted_s = sp.sorted_s; rp.sorted_o = sp.sorted_o;
    rp.settings = reinterpret_cast<const kvs_setting*>(settings_dev);
    rp.eval_list = reinterpret_cast<const i64*>(ws + L.refill_list); rp.n_list = static_cast<i64>(refill.size());
    rp.job_out_off = o.job_out_off; rp.job_start = o.job_start; rp.job_completion = o.job_completion;
    rp.profile_off = v.profile_off; rp.profile = v.profile;
    rp.peak = v.peak; rp.flow = v.flow; rp.horizon = v.horizon; rp.feasible = v.feasible; rp.status = v.status;
    ce = kvs_launch_refill(rp, ctx->stream);
    if (ce != cudaSuccess) return fail_cuda(ctx, ce, "refill launch");
  }
  if (do_profile && !spec.empty()) {
    // the list shares the refill list's region (together at most P entries); the working storage is everything
    // the ordering and fused kernels (and the refill) kept between them - the orders, sorted copies, prefix sums
    // and per-CTA scratch, one contiguous stretch of the workspace - free once they have run
    unsigned char* const list_dev = ws + L.refill_list + refill.size() * 8;
    ce = cudaMemcpyAsync(list_dev, spec.data(), spec.size() * 8, cudaMemcpyHostToDevice, ctx->stream);
    if (ce != cudaSuccess) return fail_cuda(ctx, ce, "copy of the list of speculative evaluations");
    SpecParams q{};
    q.job_off = inst->job_off; q.s = inst->s; q.o = inst->o;
    q.stats = reinterpret_cast<const InstStats*>(ws + L.stats);
    q.settings = reinterpret_cast<const kvs_setting*>(settings_dev);
    q.eval_list = reinterpret_cast<const i64*>(list_dev); q.n_list = static_cast<i64>(spec.size());
    q.job_out_off = o.job_out_off; q.job_start = o.job_start; q.job_completion = o.job_completion;
    q.profile_off = v.profile_off; q.profile = v.profile;
    q.peak = v.peak; q.flow = v.flow; q.horizon = v.horizon; q.job_steps = v.job_steps; q.n_runs = o.n_runs;
    q.n_unfinished = v.n_unfinished; q.feasible = v.feasible; q.status = v.status;
    q.scratch = ws + L.perm; q.scratch_bytes = static_cast<i64>(L.counter - L.perm); q.max_jobs = max_n;
    const i64 room = static_cast<i64>(L.counter - L.perm) / kvs_spec_warp_bytes(max_n);
    const i64 want = static_cast<i64>(ctx->sm_count) * 32;
    q.n_warps = std::min<i64>(std::min<i64>(room, want), q.n_list);
    q.counter = counters + 24;
    ce = kvs_launch_spec(q, ctx->stream);
    if (ce != cudaSuccess) return fail_cuda(ctx, ce, "launch of the speculative runs");
  }
  if (ctx->timing && !rg) { cudaEventRecord(ctx->ev[2], ctx->stream); ctx->timed = true; ctx->split_timed = fast; }
  return KVS_OK;
}

}  // namespace

extern "C" {

int kvs_init(const kvs_init_params* params, kvs_ctx** out) {
  if (!params || !out) return KVS_E_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || count <= 0) return KVS_E_CUDA;  // no CPU fallback exists
  if (params->device < 0 || params->device >= count) return KVS_E_ARG;
  if (params->workspace_bytes > 0 && !params->workspace) return KVS_E_ARG;
  if (reinterpret_cast<uintptr_t>(params->workspace) & 255u) return KVS_E_ARG;
  kvs_ctx* ctx = new (std::nothrow) kvs_ctx();
  if (!ctx) return KVS_E_STATE;
  ctx->device = params->device;
  ctx->stream = static_cast<cudaStream_t>(params->stream);
  ctx->workspace = static_cast<unsigned char*>(params->workspace);
  ctx->workspace_bytes = params->workspace_bytes;
  cudaDeviceProp prop;
  if (cudaSetDevice(ctx->device) != cudaSuccess || cudaGetDeviceProperties(&prop, ctx->device) != cudaSuccess) {
    delete ctx;
    return KVS_E_CUDA;
  }
  ctx->sm_count = prop.multiProcessorCount;
  ctx->build_ctas_per_sm = kvs_build_ctas_per_sm();
  ctx->fused_ctas_per_sm = kvs_fused_ctas_per_sm(0);
  ctx->light_ctas_per_sm = kvs_fused_ctas_per_sm(1);
  *out = ctx;
  return KVS_OK;
}

int kvs_destroy(kvs_ctx* ctx) {
  if (ctx) {
    for (cudaEvent_t e : ctx->ev) if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : ctx->chunk_ev) if (e) cudaEventDestroy(e);
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  }
  delete ctx;
  return KVS_OK;
}

const char* kvs_last_error(const kvs_ctx* ctx) { return ctx ? ctx->err.c_str() : "no context"; }

int kvs_set_timing(kvs_ctx* ctx, int32_t enabled) {
  if (!ctx) return KVS_E_STATE;
  if (enabled && !ctx->ev[0]) {
    if (cudaSetDevice(ctx->device) != cudaSuccess) return fail(ctx, KVS_E_CUDA, "cudaSetDevice");
    for (cudaEvent_t& e : ctx->ev)
      if (cudaEventCreate(&e) != cudaSuccess) return fail(ctx, KVS_E_CUDA, "cudaEventCreate");
  }
  ctx->timing = enabled != 0;
  ctx->timed = false;
  return KVS_OK;
}

int kvs_last_timing(kvs_ctx* ctx, float* sort_ms, float* build_ms) {
  if (!ctx) return KVS_E_STATE;
  if (sort_ms) *sort_ms = 0.f;
  if (build_ms) *build_ms = 0.f;
  if (!ctx->timed) return KVS_OK;
  cudaError_t ce = cudaEventSynchronize(ctx->ev[2]);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "cudaEventSynchronize");
  if (sort_ms) cudaEventElapsedTime(sort_ms, ctx->ev[0], ctx->ev[1]);
  if (build_ms) cudaEventElapsedTime(build_ms, ctx->ev[1], ctx->ev[2]);
  return KVS_OK;
}

int kvs_last_timing_split(kvs_ctx* ctx, float* sort_ms, float* light_ms, float* full_ms) {
  if (!ctx) return KVS_E_STATE;
  if (sort_ms) *sort_ms = 0.f;
  if (light_ms) *light_ms = 0.f;
  if (full_ms) *full_ms = 0.f;
  if (!ctx->timed) return KVS_OK;
  cudaError_t ce = cudaEventSynchronize(ctx->ev[2]);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "cudaEventSynchronize");
  if (sort_ms) cudaEventElapsedTime(sort_ms, ctx->ev[0], ctx->ev[1]);
  // the event between the two variants exists only on the fast path
  if (cudaEventQuery(ctx->ev[3]) == cudaSuccess && ctx->split_timed) {
    if (light_ms) cudaEventElapsedTime(light_ms, ctx->ev[1], ctx->ev[3]);
    if (full_ms) cudaEventElapsedTime(full_ms, ctx->ev[3], ctx->ev[2]);
  } else if (full_ms) {
    cudaEventElapsedTime(full_ms, ctx->ev[1], ctx->ev[2]);
  }
  return KVS_OK;
}

int kvs_debug_check_word(uint64_t* word, int32_t* compiled_in, int32_t reset) {
  unsigned long long w = 0ull;
  int compiled = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return KVS_E_CUDA;
  if (kvs_fused_check_word(&w, &compiled, reset) != cudaSuccess) return KVS_E_CUDA;
  // the kernels of the sequential rules keep words of their own: the first violation found is reported
  unsigned long long w2 = 0ull, w3 = 0ull;
  if (kvs_refill_check_word(&w2, nullptr, reset) != cudaSuccess || kvs_spec_check_word(&w3, nullptr, reset) != cudaSuccess)
    return KVS_E_CUDA;
  if (w == 0ull) w = w2 ? w2 : w3;
  if (word) *word = w;
  if (compiled_in) *compiled_in = compiled;
  return KVS_OK;
}

int kvs_workspace_bytes(int64_t n_jobs_total, int64_t n_instances, int64_t max_jobs_per_instance,
                        int64_t n_evaluations, int64_t generic_capacity, int32_t host_staging, uint64_t* out) {
  if (!out || n_jobs_total < 0 || n_instances < 0 || max_jobs_per_instance < 0 || n_evaluations < 0 || generic_capacity < 0)
    return KVS_E_ARG;
  size_t need = make_layout(n_jobs_total, n_instances, max_jobs_per_instance, n_evaluations, host_staging != 0).total;
  if (generic_capacity > 0) {
    const size_t g = generic_bytes(generic_capacity, n_evaluations, nullptr);
    if (g > need) need = g;
  }
  const size_t w = make_sweep_layout(n_jobs_total, max_jobs_per_instance).total;
  if (w > need) need = w;
  *out = need;
  return KVS_OK;
}

int kvs_build_schedule(kvs_ctx* ctx, const kvs_instances* inst, const kvs_setting* settings, int64_t P,
                       const kvs_schedule_out* out, const kvs_eval_out* ev) {
  return run_fused(ctx, inst, settings, P, out, ev, 0);
}

int kvs_evaluate_built(kvs_ctx* ctx, const kvs_instances* inst, const kvs_setting* settings, int64_t P,
                       const kvs_schedule_out* out, const kvs_eval_out* ev) {
  return run_fused(ctx, inst, settings, P, out, ev, 1);
}

int kvs_evaluate_built_host(kvs_ctx* ctx, const kvs_instances* inst, const kvs_setting* settings, int64_t P,
                            const kvs_eval_out* ev) {
  if (!ctx) return KVS_E_STATE;
  int rc = check_instances(ctx, inst);
  if (rc) return rc;
  if (!ev) return fail(ctx, KVS_E_ARG, "eval_out: null");
  if (ev->profile) return fail(ctx, KVS_E_ARG, "host entry point returns scalars only (profile must be NULL)");
  rc = check_settings(ctx, inst, settings, P);
  if (rc) return rc;
  const int64_t N = inst->n_jobs_total, I = inst->n_instances;
  for (int64_t i = 0; i < I; ++i)
    if (inst->job_off[i] < 0 || inst->job_off[i + 1] < inst->job_off[i] || inst->job_off[i + 1] > N)
      return fail(ctx, KVS_E_ARG, "instances: job_off is not nondecreasing within [0, n_jobs_total]");
  const Layout L = make_layout(N, I, inst->max_jobs_per_instance, P, true);
  if (L.total > ctx->workspace_bytes) return fail(ctx, KVS_E_CAPACITY, "workspace too small for host staging (see kvs_workspace_bytes)");
  cudaError_t ce = cudaSetDevice(ctx->device);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "cudaSetDevice");
  if (!ctx->copy_stream) {
    if ((ce = cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking)) != cudaSuccess) return fail_cuda(ctx, ce, "cudaStreamCreate");
    for (cudaEvent_t& e : ctx->chunk_ev)
      if ((ce = cudaEventCreateWithFlags(&e, cudaEventDisableTiming)) != cudaSuccess) return fail_cuda(ctx, ce, "cudaEventCreate");
  }
  unsigned char* ws = ctx->workspace;

  // Evaluations are worked off chunk of instances by chunk of instances, so that the copy of the
  // next chunk's jobs overlaps the kernels of the current one: order them by instance (stable).
  std::vector<int64_t> order(static_cast<size_t>(P));
  for (int64_t e = 0; e < P; ++e) order[static_cast<size_t>(e)] = e;
  bool identity = true;
  for (int64_t e = 1; e < P && identity; ++e) identity = settings[e - 1].instance <= settings[e].instance;
  if (!identity)
    std::stable_sort(order.begin(), order.end(), [&](int64_t a, int64_t b) { return settings[a].instance < settings[b].instance; });
  std::vector<kvs_setting> sorted(static_cast<size_t>(P));
  for (int64_t r = 0; r < P; ++r) sorted[static_cast<size_t>(r)] = settings[order[static_cast<size_t>(r)]];

  kvs_instances dev = *inst;
  dev.job_off = reinterpret_cast<const int64_t*>(ws + L.st_off);
  dev.s = reinterpret_cast<const int32_t*>(ws + L.st_s);
  dev.o = reinterpret_cast<const int32_t*>(ws + L.st_o);
  dev.o_est = inst->o_est ? reinterpret_cast<const int32_t*>(ws + L.st_key) : nullptr;
  dev.arrival = inst->arrival ? reinterpret_cast<const int64_t*>(ws + L.st_arr) : nullptr;
  kvs_eval_out d{};
  d.peak = reinterpret_cast<int64_t*>(ws + L.sc_peak);
  d.flow = reinterpret_cast<int64_t*>(ws + L.sc_flow);
  d.job_steps = reinterpret_cast<int64_t*>(ws + L.sc_steps);
  d.horizon = reinterpret_cast<int64_t*>(ws + L.sc_hor);
  d.n_unfinished = reinterpret_cast<int64_t*>(ws + L.sc_unf);
  d.feasible = reinterpret_cast<uint8_t*>(ws + L.sc_feas);
  d.status = reinterpret_cast<int32_t*>(ws + L.sc_stat);

  // the staging areas may still be read by earlier work on the context's stream
  if ((ce = cudaEventRecord(ctx->chunk_ev[KVS_HOST_CHUNKS], ctx->stream)) != cudaSuccess ||
      (ce = cudaStreamWaitEvent(ctx->copy_stream, ctx->chunk_ev[KVS_HOST_CHUNKS], 0)) != cudaSuccess)
    return fail_cuda(ctx, ce, "stream ordering");
  ce = cudaMemcpyAsync(ws + L.st_off, inst->job_off, static_cast<size_t>(I + 1) * 8, cudaMemcpyHostToDevice, ctx->copy_stream);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "host-to-device copy of job_off");
  // a chunk should still fill the GPU: about a thousand evaluations each, at most KVS_HOST_CHUNKS chunks
  int64_t n_chunks = P / 1024;
  if (n_chunks > KVS_HOST_CHUNKS) n_chunks = KVS_HOST_CHUNKS;
  if (n_chunks > I) n_chunks = I;
  if (n_chunks < 1) n_chunks = 1;
  int64_t r0 = 0;
  for (int64_t c = 0; c < n_chunks; ++c) {
    const int64_t i0 = c * I / n_chunks, i1 = (c + 1) * I / n_chunks;
    const int64_t j0 = I ? inst->job_off[i0] : 0, j1 = I ? inst->job_off[i1] : 0;
    const size_t cnt = static_cast<size_t>(j1 - j0);
    auto h2d = [&](size_t off, const void* src, size_t elem) {
      return (src && cnt) ? cudaMemcpyAsync(ws + off + static_cast<size_t>(j0) * elem, static_cast<const unsigned char*>(src) + static_cast<size_t>(j0) * elem,
                                            cnt * elem, cudaMemcpyHostToDevice, ctx->copy_stream)
                          : cudaSuccess;
    };
    if ((ce = h2d(L.st_s, inst->s, 4)) != cudaSuccess || (ce = h2d(L.st_o, inst->o, 4)) != cudaSuccess ||
        (ce = h2d(L.st_key, inst->o_est, 4)) != cudaSuccess || (ce = h2d(L.st_arr, inst->arrival, 8)) != cudaSuccess)
      return fail_cuda(ctx, ce, "host-to-device copy of the instances");
    if ((ce = cudaEventRecord(ctx->chunk_ev[c], ctx->copy_stream)) != cudaSuccess ||
        (ce = cudaStreamWaitEvent(ctx->stream, ctx->chunk_ev[c], 0)) != cudaSuccess)
      return fail_cuda(ctx, ce, "stream ordering");
    int64_t r1 = r0;
    while (r1 < P && sorted[static_cast<size_t>(r1)].instance < i1) ++r1;
    if (r1 > r0) {
      kvs_eval_out dc = d;
      dc.peak += r0; dc.flow += r0; dc.job_steps += r0; dc.horizon += r0; dc.n_unfinished += r0; dc.feasible += r0; dc.status += r0;
      const FusedRange rg{i0, i1, r0, P};
      rc = run_fused(ctx, &dev, sorted.data() + r0, r1 - r0, nullptr, &dc, 1, &rg);
      if (rc) return rc;
    }
    r0 = r1;
  }

  // results come back in the order the evaluations were worked off
  const size_t p8 = static_cast<size_t>(P) * 8;
  std::vector<int64_t> t64;
  std::vector<int32_t> t32;
  std::vector<uint8_t> t8;
  auto fetch = [&](void* dst, size_t off, size_t elem) -> cudaError_t {
    if (!dst || P == 0) return cudaSuccess;
    if (identity) return cudaMemcpyAsync(dst, ws + off, static_cast<size_t>(P) * elem, cudaMemcpyDeviceToHost, ctx->stream);
    // scattered back through a temporary once the stream has finished
    return cudaSuccess;
  };
  if ((ce = fetch(ev->peak, L.sc_peak, 8)) != cudaSuccess || (ce = fetch(ev->flow, L.sc_flow, 8)) != cudaSuccess ||
      (ce = fetch(ev->job_steps, L.sc_steps, 8)) != cudaSuccess || (ce = fetch(ev->horizon, L.sc_hor, 8)) != cudaSuccess ||
      (ce = fetch(ev->n_unfinished, L.sc_unf, 8)) != cudaSuccess || (ce = fetch(ev->feasible, L.sc_feas, 1)) != cudaSuccess ||
      (ce = fetch(ev->status, L.sc_stat, 4)) != cudaSuccess)
    return fail_cuda(ctx, ce, "device-to-host copy of the results");
  ce = cudaStreamSynchronize(ctx->stream);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "stream synchronize");
  if (!identity && P > 0) {
    t64.resize(static_cast<size_t>(P)); t32.resize(static_cast<size_t>(P)); t8.resize(static_cast<size_t>(P));
    auto back64 = [&](int64_t* dst, size_t off) -> cudaError_t {
      if (!dst) return cudaSuccess;
      const cudaError_t e = cudaMemcpy(t64.data(), ws + off, p8, cudaMemcpyDeviceToHost);
      if (e == cudaSuccess) for (int64_t r = 0; r < P; ++r) dst[order[static_cast<size_t>(r)]] = t64[static_cast<size_t>(r)];
      return e;
    };
    if ((ce = back64(ev->peak, L.sc_peak)) != cudaSuccess || (ce = back64(ev->flow, L.sc_flow)) != cudaSuccess ||
        (ce = back64(ev->job_steps, L.sc_steps)) != cudaSuccess || (ce = back64(ev->horizon, L.sc_hor)) != cudaSuccess ||
        (ce = back64(ev->n_unfinished, L.sc_unf)) != cudaSuccess)
      return fail_cuda(ctx, ce, "device-to-host copy of the results");
    if (ev->feasible) {
      if ((ce = cudaMemcpy(t8.data(), ws + L.sc_feas, static_cast<size_t>(P), cudaMemcpyDeviceToHost)) != cudaSuccess) return fail_cuda(ctx, ce, "device-to-host copy of the results");
      for (int64_t r = 0; r < P; ++r) ev->feasible[order[static_cast<size_t>(r)]] = t8[static_cast<size_t>(r)];
    }
    if (ev->status) {
      if ((ce = cudaMemcpy(t32.data(), ws + L.sc_stat, static_cast<size_t>(P) * 4, cudaMemcpyDeviceToHost)) != cudaSuccess) return fail_cuda(ctx, ce, "device-to-host copy of the results");
      for (int64_t r = 0; r < P; ++r) ev->status[order[static_cast<size_t>(r)]] = t32[static_cast<size_t>(r)];
    }
  }
  return KVS_OK;
}

int kvs_evaluate_schedule(kvs_ctx* ctx, const kvs_runs* runs, const kvs_eval_out* ev) {
  if (!ctx) return KVS_E_STATE;
  if (!runs || !ev) return fail(ctx, KVS_E_ARG, "runs or eval_out is null");
  if (runs->P < 0) return fail(ctx, KVS_E_ARG, "runs: negative count");
  if (runs->P == 0) return KVS_OK;
  if (!runs->run_off || !runs->run_start || !runs->run_len || !runs->run_s) return fail(ctx, KVS_E_ARG, "runs: null array");
  if (!ev->profile_off) return fail(ctx, KVS_E_ARG, "eval_out: profile_off (capacities) is required");
  cudaError_t ce = cudaSetDevice(ctx->device);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "cudaSetDevice");
  // total capacity = profile_off[P]: one small synchronous read sizes the scratch arrays
  int64_t cap_total = 0;
  ce = cudaMemcpyAsync(&cap_total, ev->profile_off + runs->P, 8, cudaMemcpyDeviceToHost, ctx->stream);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(ctx->stream);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "read of profile_off");
  if (cap_total < 0) return fail(ctx, KVS_E_ARG, "eval_out: negative capacity");
  size_t need_a = 0;
  const size_t need = generic_bytes(cap_total, runs->P, &need_a);
  if (need > ctx->workspace_bytes) return fail(ctx, KVS_E_CAPACITY, "workspace too small for the generic evaluator");
  unsigned char* ws = ctx->workspace;
  GenericParams gp{};
  gp.runs = *runs; gp.ev = *ev;
  gp.dconst = reinterpret_cast<i64*>(ws);
  gp.dcount = reinterpret_cast<int32_t*>(ws + need_a);
  gp.slots = cap_total + runs->P;
  ce = cudaMemsetAsync(ws, 0, need, ctx->stream);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "memset");
  ce = kvs_launch_generic(gp, ctx->stream);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "generic launch");
  return KVS_OK;
}

int kvs_bounds(kvs_ctx* ctx, const kvs_instances* inst, const kvs_setting* settings, int64_t P, const kvs_bounds_out* out) {
  if (!ctx) return KVS_E_STATE;
  int rc = check_instances(ctx, inst);
  if (rc) return rc;
  if (!out) return fail(ctx, KVS_E_ARG, "bounds: out is null");
  if (inst->window != 0) return fail(ctx, KVS_E_ARG, "bounds: needs offline instances (window = 0)");
  // the family is not used: check the settings as geometric ones
  std::vector<kvs_setting> geo(settings, settings + (settings && P > 0 ? P : 0));
  for (kvs_setting& s : geo) { s.family = KVS_GBA; s.tau = 0; s.k = 0; }
  rc = check_settings(ctx, inst, P > 0 ? geo.data() : settings, P);
  if (rc) return rc;
  if (P == 0) return KVS_OK;
  const int64_t N = inst->n_jobs_total, I = inst->n_instances, max_n = inst->max_jobs_per_instance;
  const Layout L = make_layout(N, I, max_n, P, false);
  if (L.total > ctx->workspace_bytes) return fail(ctx, KVS_E_CAPACITY, "workspace too small for this call (see kvs_workspace_bytes)");
  cudaError_t ce = cudaSetDevice(ctx->device);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "cudaSetDevice");
  unsigned char* ws = ctx->workspace;
  ce = cudaMemcpyAsync(ws + L.settings, geo.data(), static_cast<size_t>(P) * sizeof(kvs_setting), cudaMemcpyHostToDevice, ctx->stream);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "copy of settings");
  // statistics and validation of the instances (largest prompt and response, input checks): the
  // ordering kernel without the ordering
  SortParams sp{};
  sp.job_off = inst->job_off; sp.s = inst->s; sp.o = inst->o; sp.key = nullptr; sp.arrival = nullptr;
  sp.window = 0; sp.n_instances = I; sp.max_jobs = max_n; sp.need_order = 0;
  sp.stats = reinterpret_cast<InstStats*>(ws + L.stats);
  const int64_t sort_cap = static_cast<int64_t>(ctx->sm_count) * 2;
  ce = kvs_launch_sort(sp, static_cast<int>(I < sort_cap ? I : sort_cap), ctx->stream);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "statistics launch");
  const int64_t cap = static_cast<int64_t>(ctx->sm_count) * 8;
  ce = kvs_launch_bounds(inst->job_off, inst->o, sp.stats, reinterpret_cast<const kvs_setting*>(ws + L.settings), P, *out,
                         static_cast<int>(P < cap ? P : cap), ctx->stream);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "bounds launch");
  return KVS_OK;
}

int kvs_sweep(kvs_ctx* ctx, const kvs_instances* inst, const kvs_sweep_params* params, const kvs_sweep_out* out) {
  if (!ctx) return KVS_E_STATE;
  int rc = check_instances(ctx, inst);
  if (rc) return rc;
  if (!params || !out) return fail(ctx, KVS_E_ARG, "sweep: params or out is null");
  if (inst->o_est || inst->window != 0) return fail(ctx, KVS_E_ARG, "sweep: needs offline instances ordered by the exact response length");
  if (params->instance < 0 || params->instance >= inst->n_instances) return fail(ctx, KVS_E_ARG, "sweep: instance out of range");
  if (params->family == KVS_GBA || params->family == KVS_GSA) {
    // one evaluation per initial slice, through the fused path, scalars only
    if (params->n_beta0 < 0 || params->n_beta0 > 65536) return fail(ctx, KVS_E_RANGE, "sweep: more than 65536 initial slices");
    if (params->n_beta0 == 0) return KVS_OK;
    if (!params->beta0) return fail(ctx, KVS_E_ARG, "sweep: null grid");
    const int64_t P = params->n_beta0;
    std::vector<kvs_setting> st(static_cast<size_t>(P));
    for (int64_t i = 0; i < P; ++i) {
      kvs_setting& s = st[static_cast<size_t>(i)];
      s = kvs_setting{};
      s.instance = params->instance; s.family = params->family; s.alpha_num = params->alpha_num; s.alpha_den = params->alpha_den;
      s.s_bar = -1; s.M = params->M; s.beta0 = params->beta0[i]; s.subroutine = params->subroutine; s.per_class_s = params->per_class_s;
    }
    const Layout L = make_layout(inst->n_jobs_total, inst->n_instances, inst->max_jobs_per_instance, P, false);
    if (L.total > ctx->workspace_bytes) return fail(ctx, KVS_E_CAPACITY, "workspace too small for the sweep (see kvs_workspace_bytes)");
    kvs_eval_out ev{};
    ev.peak = out->peak; ev.flow = out->flow; ev.horizon = out->horizon; ev.job_steps = out->job_steps; ev.feasible = out->feasible;
    ev.n_unfinished = reinterpret_cast<int64_t*>(ctx->workspace + L.sweep_unf);
    ev.status = reinterpret_cast<int32_t*>(ctx->workspace + L.sweep_stat);
    rc = run_fused(ctx, inst, st.data(), P, nullptr, &ev, 1);
    if (rc) return rc;
    if (out->n_completed) {
      const cudaError_t ce = kvs_launch_completed(inst->job_off + params->instance, ev.n_unfinished, ev.status, out->n_completed, P, ctx->stream);
      if (ce != cudaSuccess) return fail_cuda(ctx, ce, "sweep launch");
    }
    return KVS_OK;
  }
  if (params->family != KVS_SPS && params->family != KVS_SIMS) return fail(ctx, KVS_E_ARG, "sweep: unknown family");
  if (params->n_tau < 0 || params->n_k < 0 || static_cast<int64_t>(params->n_tau) * params->n_k > 65536)
    return fail(ctx, KVS_E_RANGE, "sweep: grid larger than 65536 settings");
  if (params->n_tau == 0 || params->n_k == 0) return KVS_OK;
  if (!params->tau || !params->k) return fail(ctx, KVS_E_ARG, "sweep: null grid");
  if (params->M < 1 || params->M >= KVS_TIME_LIMIT) return fail(ctx, KVS_E_RANGE, "sweep: M outside [1, 2^31)");
  for (int i = 0; i < params->n_tau; ++i)
    if (params->tau[i] < 1 || params->tau[i] >= KVS_TIME_LIMIT) return fail(ctx, KVS_E_RANGE, "sweep: tau outside [1, 2^31)");
  for (int i = 0; i < params->n_k; ++i)
    if (params->k[i] < 1 || params->k[i] >= KVS_TIME_LIMIT) return fail(ctx, KVS_E_RANGE, "sweep: k outside [1, 2^31)");
  const int64_t N = inst->n_jobs_total, max_n = inst->max_jobs_per_instance;
  const SweepLayout L = make_sweep_layout(N, max_n);
  if (L.total > ctx->workspace_bytes) return fail(ctx, KVS_E_CAPACITY, "workspace too small for the sweep (see kvs_workspace_bytes)");
  cudaError_t ce = cudaSetDevice(ctx->device);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "cudaSetDevice");
  unsigned char* ws = ctx->workspace;

  // order and statistics of the one instance: the sort kernel sees a batch of one
  SortParams sp{};
  sp.job_off = inst->job_off + params->instance; sp.s = inst->s; sp.o = inst->o; sp.key = nullptr; sp.arrival = nullptr;
  sp.window = 0; sp.n_instances = 1; sp.max_jobs = max_n; sp.need_order = 1;
  sp.stats = reinterpret_cast<InstStats*>(ws + L.stats);
  sp.perm = reinterpret_cast<int32_t*>(ws + L.perm);
  sp.perm_tmp = reinterpret_cast<int32_t*>(ws + L.perm_tmp);
  sp.sorted_s = reinterpret_cast<int32_t*>(ws + L.sorted_s);
  sp.sorted_o = reinterpret_cast<int32_t*>(ws + L.sorted_o);
  sp.sorted_key = nullptr;
  ce = kvs_launch_sort(sp, 1, ctx->stream);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "sort launch");
  // the instance's first job index and size are device values; read them once (16 bytes)
  int64_t range[2] = {0, 0};
  ce = cudaMemcpyAsync(range, inst->job_off + params->instance, 16, cudaMemcpyDeviceToHost, ctx->stream);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(ctx->stream);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "read of job_off");
  const int64_t lo = range[0], n = range[1] - range[0];
  if (lo < 0 || n < 0 || n > max_n || lo + n > N) return fail(ctx, KVS_E_ARG, "sweep: job_off inconsistent with the stated sizes");

  i64* ps = reinterpret_cast<i64*>(ws + L.prefix_s);
  i64* po = reinterpret_cast<i64*>(ws + L.prefix_o);
  ce = kvs_launch_prefix(sp.sorted_s + lo, sp.sorted_o + lo, n, ps, po, ctx->stream);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "prefix launch");
  ce = cudaMemcpyAsync(ws + L.tau, params->tau, static_cast<size_t>(params->n_tau) * 8, cudaMemcpyHostToDevice, ctx->stream);
  if (ce == cudaSuccess)
    ce = cudaMemcpyAsync(ws + L.k, params->k, static_cast<size_t>(params->n_k) * 8, cudaMemcpyHostToDevice, ctx->stream);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "copy of the grids");
  SweepParams wp{};
  wp.sorted_s = sp.sorted_s + lo; wp.sorted_o = sp.sorted_o + lo; wp.prefix_s = ps; wp.prefix_o = po;
  wp.n = n; wp.family = params->family; wp.M = params->M;
  wp.tau = reinterpret_cast<const i64*>(ws + L.tau); wp.k = reinterpret_cast<const i64*>(ws + L.k);
  wp.n_tau = params->n_tau; wp.n_k = params->n_k; wp.out = *out;
  ce = kvs_launch_sweep(wp, reinterpret_cast<i64*>(ws + L.acc_peak), reinterpret_cast<u64*>(ws + L.acc_flow), ctx->stream);
  if (ce != cudaSuccess) return fail_cuda(ctx, ce, "sweep launch");
  return KVS_OK;
}

}  // extern "C"
