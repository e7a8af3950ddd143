// Speculative runs on top of slicing schedules (Numerical Experiments, "Speculative Runs (GSA-Spec)"): memory
// that the pipeline leaves free runs unfinished jobs ahead of their turn; such runs are killed when the
// pipeline needs the memory, so the slicing schedule itself is kept; they start and are killed first come
// first served.
//
// The rule is a round-by-round simulation in which every decision depends on the rounds before it, so one
// warp simulates one evaluation and many evaluations run side by side.  The warp starts from what the fused
// kernels left - the per-round memory of the slicing schedule (the plan) in the caller's profile buffer -
// and forms the pipeline's runs again from the phase table: the participants of phase p are the jobs of class
// p or later in index order, rank r starts at base_p + floor(r tau_p / k_p) and holds its slot for tau_p rounds
// (Procedure StaggeredPipelineSchedule).  Round t:
//   (1) a speculative run that has received all its rounds completes its job;
//   (2) the pipeline's runs that start at t begin: a job that has completed is dropped from the plan (its ramp
//       is taken out of the profile), a job that is running speculatively loses that run;
//   (3) while pipeline and speculative runs together exceed M, the speculative run started last is killed;
//   (4) the jobs that are not done and not running are taken in index order: the lowest one starts a
//       speculative run if its first round fits (s + 1 tokens), then the next, until one does not fit;
//   (5) the round's memory, pipeline + speculative, is written over the plan's entry.
// The speculative runs hold A + t * count tokens in round t (a run started at t0 holds s + 1 - t0 + t).
// Per phase the participants are kept as a list in index order, so that rank r is entry r.  Two cursors walk
// it: one over the run starts, one over the slot ends start + tau (nondecreasing in the rank), which is when a
// killed job becomes free to speculate.  No entry before position `fpos` and none at or after `fhi` is free at the
// moment; the events that free a job (a slot end, a kill for memory) widen that range, a scan narrows it.
#include "kvs_check.cuh"
#include "kvs_ladder.cuh"

namespace {

constexpr int ST = 128;                 // threads per CTA: four warps, one evaluation each at a time
constexpr int SWARPS = ST / 32;
constexpr int MAXP = KVS_MAX_PHASES;
constexpr int NEVER = 0x7fffffff;
constexpr u32 NO_ROUND = 0xffffffffu;   // completion rounds are kept as 32-bit unsigned: t + o stays below 2^32

struct SpecShared {
  u128 pw_a[MAXP + 1];
  u128 pw_b[MAXP + 1];
  u32 tau[MAXP], k[MAXP], np[MAXP], hist[MAXP];
  i64 pbase[MAXP + 1];
  int n_phases;
};

// floor(r * tau / k) for r, tau, k below 2^31
__device__ __forceinline__ i64 slot_of(int r, u32 tau, u32 k) {
  const u64 x = static_cast<u64>(static_cast<u32>(r)) * tau;
  return (x >> 32) == 0 ? static_cast<i64>(static_cast<u32>(x) / k) : static_cast<i64>(x / k);
}

__device__ __forceinline__ u32 warp_min_u32(u32 v) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, d));
  return v;
}

// Number of ranks r < np with floor(r * tau / k) <= x: r * tau < (x + 1) * k, so ceil((x + 1) * k / tau) of them.
__device__ __forceinline__ int started(i64 x, u32 tau, u32 k, int np) {
  if (x < 0) return 0;
  const u64 v = (static_cast<u64>(x + 1) * k + tau - 1) / tau;
  return v < static_cast<u64>(np) ? static_cast<int>(v) : np;
}

// Bytes of one warp's working storage for instances of at most n jobs: five int arrays (position in the phase's
// list, start of the speculative run or -1, stack of speculative runs as job and completion round,
// participant list) and two byte arrays (class, done flag).
__host__ __device__ inline i64 spec_stride(i64 n) { return (22 * n + 255) & ~static_cast<i64>(255); }

__global__ void __launch_bounds__(ST) k_spec(SpecParams p) {
  __shared__ SpecShared shs[SWARPS];
  const int lane = lane_id(), warp = threadIdx.x >> 5;
  const unsigned lt_mask = (1u << lane) - 1u;
  SpecShared& sh = shs[warp];
  const i64 wslot = static_cast<i64>(blockIdx.x) * SWARPS + warp;
  if (wslot >= p.n_warps) return;
  const i64 cap = p.max_jobs;
  if (!KVS_OK_AT((wslot + 1) * spec_stride(cap) - 1, p.scratch_bytes, CHK_SP_SCRATCH)) return;
  unsigned char* const mine = p.scratch + wslot * spec_stride(cap);
  int* const pos_of = reinterpret_cast<int*>(mine);    // position of a job in the current phase's list
  int* const sst = pos_of + cap;
  int* const stk_job = sst + cap;
  int* const stk_fin = stk_job + cap;                    // round in which the entry's run would complete
  int* const list = stk_fin + cap;
  unsigned char* const cls = reinterpret_cast<unsigned char*>(list + cap);
  unsigned char* const done = cls + cap;

  for (;;) {
    ull slot = 0;
    if (lane == 0) slot = atomicAdd(p.counter, 1ull);
    slot = __shfl_sync(0xffffffffu, slot, 0);
    if (slot >= static_cast<ull>(p.n_list)) return;
    const i64 e = p.eval_list[slot];
    if (p.status[e] != 0) continue;                     // the slicing schedule was not formed or not stored in full
    const kvs_setting st = p.settings[e];
    const i64 lo = p.job_off[st.instance];
    const int n = static_cast<int>(p.job_off[st.instance + 1] - lo);
    const InstStats stats = p.stats[st.instance];
    const i64 M = st.M;
    const i64 s_bar = st.s_bar >= 0 ? st.s_bar : stats.s_max;
    const i64 X = M - s_bar;
    const int32_t* const S = p.s + lo;
    const int32_t* const O = p.o + lo;
    int32_t* const prof = p.profile + p.profile_off[e];
    int32_t* const js = p.job_start + p.job_out_off[e];
    int32_t* const jc = p.job_completion + p.job_out_off[e];
    const int H = static_cast<int>(p.horizon[e]);       // of the slicing schedule; within the profile's capacity (status 0)
    if (!KVS_OK_AT(H, p.profile_off[e + 1] - p.profile_off[e] + 1, CHK_SP_PROF) || !KVS_OK_AT(n, cap + 1, CHK_SP_JOB)) continue;
    if (n == 0) continue;

    // ---- phase table: ladder, classes, participants, first round of every phase ----
    ladder32(sh, X, st.alpha_num, st.alpha_den, st.beta0, static_cast<u32>(s_bar), static_cast<u32>(M));
    const int L = sh.n_phases;
    for (int q = lane; q < L; q += 32) sh.hist[q] = 0;
    __syncwarp();
    const bool pow2 = st.alpha_num == 2 && st.alpha_den == 1 && st.beta0 <= 0;
    for (int i = lane; i < n; i += 32) {
      const u32 oi = static_cast<u32>(O[i]);
      const int c = pow2 ? class_pow2(static_cast<u32>(X), oi) : class_of(sh.tau, L, oi);
      cls[i] = static_cast<unsigned char>(c);
      done[i] = 0; pos_of[i] = i; sst[i] = -1; list[i] = i;
      atomicAdd(&sh.hist[c], 1u);
    }
    __syncwarp();
    if (lane == 0) {
      u32 later = static_cast<u32>(n);
      i64 b = 0;
      for (int q = 0; q < L; ++q) {
        sh.np[q] = later;                               // jobs of class q or later take part in phase q
        sh.pbase[q] = b;
        if (later > 0) b += slot_of(static_cast<int>(later) - 1, sh.tau[q], sh.k[q]) + sh.tau[q];
        later -= sh.hist[q];
      }
      sh.pbase[L] = b;
    }
    __syncwarp();

    // ---- the simulation ----
    int ph = 0, np = n;                                 // phase that holds round t; its participants
    u32 tau_c = sh.tau[0], k_c = sh.k[0];
    i64 base_c = 0;
    int rs = 0, re = 0;                                 // ranks of the next run start and of the next slot end
    i64 ns = 0, ne = tau_c;                             // their rounds
    i64 A = 0;                                          // speculative runs hold A + t * cnt tokens in round t
    int cnt = 0, top = 0;                               // running speculative runs; entries on the stack (some stale)
    u32 next_comp = NO_ROUND;                           // no speculative run completes before this round
    int fpos = 0, fhi = n;
    int cj = -1, cs = 0;                                // the free job at fpos and its prompt length, while known (cj = -2: none is free)
    int left = n;
    i64 flow = 0, steps = 0, runs = 0, peak = 0;
    int hmax = 0;
    int Bw = 0;                                         // lane l holds the plan's memory of round (t & ~31) + l
    for (int t = 0; t <= H; ++t) {
      // (1) speculative completions
      const u32 tu = static_cast<u32>(t);
      if (tu == next_comp) {
        u32 nc = NO_ROUND;
        for (int g0 = 0; g0 < top; g0 += 128) {         // four chunks' completion rounds are loaded together
          u32 fq[4];
#pragma unroll
          for (int c = 0; c < 4; ++c) fq[c] = g0 + 32 * c + lane < top ? static_cast<u32>(stk_fin[g0 + 32 * c + lane]) : NO_ROUND;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const int q = g0 + 32 * c + lane;
            const u32 f = fq[c];
            if (f > tu) nc = min(nc, f);                // stale entries included: they cost one empty scan at most
            if (__ballot_sync(0xffffffffu, f == tu) == 0) continue;
            bool fin = false;
            int j = 0, s0 = 0;
            if (f == tu) {
              j = stk_job[q];
              if (!KVS_OK_AT(j, n, CHK_SP_JOB)) j = 0;
              s0 = t - O[j];
              fin = sst[j] == s0;                       // a live entry
            }
            const unsigned fm = __ballot_sync(0xffffffffu, fin);
            if (fm) {
              if (fin) { done[j] = 1; sst[j] = -1; js[j] = s0; jc[j] = t; }
              const i64 dA = warp_sum(fin ? static_cast<i64>(S[j]) + 1 - s0 : static_cast<i64>(0));
              const i64 dS = warp_sum(fin ? static_cast<i64>(O[j]) : static_cast<i64>(0));
              const int kf = __popc(fm);
              A -= dA; steps += dS; flow += static_cast<i64>(kf) * t;
              cnt -= kf; left -= kf; runs += kf;
              hmax = max(hmax, t);
            }
          }
        }
        next_comp = warp_min_u32(nc);
        __syncwarp();
      }
      // slots that have ended: a job killed at the end of its slot is free again.  The ranks whose slots end by
      // round t are [re, started(t - tau)); only those before fpos can lower it.
      if (ne <= t) {
        const int eend = started(static_cast<i64>(t) - tau_c - base_c, tau_c, k_c, np);
        // the ranks [re, eend) are free now unless done or running speculatively; those before fpos are looked at
        // here (the known candidate stays the lowest free job if none of them is), the others lie in the range
        const int lim = min(eend, fpos);
        for (int r0 = re; r0 < lim; r0 += 32) {
          const int r = r0 + lane;
          bool fr = false;
          if (r < lim && KVS_OK_AT(r, n, CHK_SP_LIST)) {
            const int j = list[r];
            if (KVS_OK_AT(j, n, CHK_SP_JOB)) fr = !done[j] && sst[j] < 0;
          }
          const unsigned hit = __ballot_sync(0xffffffffu, fr);
          if (hit) { fpos = r0 + __ffs(static_cast<int>(hit)) - 1; cj = -1; break; }
        }
        if (eend > fhi && (cj == -1 || eend > lim)) fhi = eend;
        re = eend;
        ne = re < np ? base_c + slot_of(re, tau_c, k_c) + tau_c : static_cast<i64>(NEVER) * 2;
      }
      // the next phase begins: its participants are the jobs of a later class, in index order
      if (rs >= np && ph + 1 < L && sh.np[ph + 1] > 0 && t == sh.pbase[ph + 1]) {
        ++ph;
        int w = 0;
        for (int q0 = 0; q0 < np; q0 += 32) {
          const int q = q0 + lane;
          bool keep = false;
          int j = 0;
          if (q < np) { j = list[q]; keep = cls[j] >= ph; }
          const unsigned m = __ballot_sync(0xffffffffu, keep);
          __syncwarp();
          if (keep) { const int d = w + __popc(m & lt_mask); list[d] = j; pos_of[j] = d; }
          w += __popc(m);
          __syncwarp();
        }
        np = w;
        tau_c = sh.tau[ph]; k_c = sh.k[ph]; base_c = sh.pbase[ph];
        rs = 0; re = 0; ns = base_c; ne = base_c + tau_c;
        fpos = 0; fhi = np; cj = -1;
      }
      // (2) pipeline runs that start now: ranks [rs, started(t)), 32 at a time (they concern different jobs)
      if (ns <= t) {
        const int rend = started(static_cast<i64>(t) - base_c, tau_c, k_c, np);
        bool cand_started = false;                      // a job that starts may be the known candidate
        for (int r0 = rs; r0 < rend; r0 += 32) {
          const int r = r0 + lane;
          bool act = r < rend && KVS_OK_AT(r, n, CHK_SP_LIST);
          int j = 0, oj = 0, sj = 0, s0 = -1;
          bool dn = false;
          if (act) { j = list[r]; act = KVS_OK_AT(j, n, CHK_SP_JOB); }
          if (act) { oj = O[j]; sj = S[j]; dn = done[j] != 0; s0 = sst[j]; }
          if (cj >= 0 && __ballot_sync(0xffffffffu, act && j == cj)) cand_started = true;
          const int len = oj < static_cast<int>(tau_c) ? oj : static_cast<int>(tau_c);
          const bool run = act && !dn, drop = act && dn;
          const bool kill = run && s0 >= 0;             // its speculative run is killed; the stack entry goes stale
          const bool comp = run && len == oj;
          const unsigned km = __ballot_sync(0xffffffffu, kill);
          if (km) {
            A -= warp_sum(kill ? static_cast<i64>(sj) + 1 - s0 : static_cast<i64>(0));
            steps += warp_sum(kill ? static_cast<i64>(t - s0) : static_cast<i64>(0));
            cnt -= __popc(km);
            runs += __popc(__ballot_sync(0xffffffffu, kill && t > s0));
          }
          const unsigned rm = __ballot_sync(0xffffffffu, run);
          if (rm) {
            steps += warp_sum(run ? static_cast<i64>(len) : static_cast<i64>(0));
            runs += __popc(rm);
            if (run) {
              sst[j] = -1;
              if (comp) { done[j] = 1; js[j] = t; jc[j] = t + len; }
            }
            const unsigned cm = __ballot_sync(0xffffffffu, comp);
            if (cm) {
              left -= __popc(cm);
              flow += warp_sum(comp ? static_cast<i64>(t + len) : static_cast<i64>(0));
              hmax = max(hmax, warp_max(comp ? t + len : 0));
            }
          }
          // dropped from the plan: short ramps lane by lane, long ones by the whole warp; the rounds of the
          // window held in registers are corrected there (the round of lane l is t - (t & 31) + l)
          unsigned dm = __ballot_sync(0xffffffffu, drop);
          if (dm) {
            if (drop && len <= 64)
              for (int u = 0; u < len; ++u)
                if (KVS_OK_AT(t + u, H, CHK_SP_DROP)) atomicSub(&prof[t + u], sj + u + 1);
            unsigned lm = __ballot_sync(0xffffffffu, drop && len > 64);
            while (lm) {
              const int src = __ffs(static_cast<int>(lm)) - 1;
              lm &= lm - 1u;
              const int ls = __shfl_sync(0xffffffffu, len, src), ss = __shfl_sync(0xffffffffu, sj, src);
              for (int u = lane; u < ls; u += 32)
                if (KVS_OK_AT(t + u, H, CHK_SP_DROP)) atomicSub(&prof[t + u], ss + u + 1);
            }
            if ((t & 31) != 0) {                        // at a window's first round the window is loaded afterwards
              const int u = lane - (t & 31);            // this lane's round, counted from t
              while (dm) {
                const int src = __ffs(static_cast<int>(dm)) - 1;
                dm &= dm - 1u;
                const int ls = __shfl_sync(0xffffffffu, len, src), ss = __shfl_sync(0xffffffffu, sj, src);
                if (u >= 0 && u < ls) Bw -= ss + u + 1;
              }
            }
          }
        }
        __syncwarp();
        if (cand_started) cj = -1;
        rs = rend;
        ns = rs < np ? base_c + slot_of(rs, tau_c, k_c) : static_cast<i64>(NEVER) * 2;
      }
      if (t == H) break;                                // nothing runs in round H; only completions were due
      if (left == 0) {
        // Every job is done, so every run the pipeline has yet to start is dropped: what is left of the plan are
        // the runs in progress, which are completing runs of ranks between the two cursors (a killed run in
        // progress would belong to an unfinished job).  Such a run's completion round lies beyond t and it began o earlier.
        __syncwarp();
        for (int u = t + lane; u < H; u += 32) prof[u] = 0;
        __syncwarp();
        for (int r = re; r < rs; ++r) {
          const int j = list[r];
          if (!KVS_OK_AT(j, n, CHK_SP_JOB)) continue;
          const int end = jc[j];                        // beyond t only for a completing run of the pipeline in progress
          if (end > t && KVS_OK_AT(end, H + 1, CHK_SP_PROF)) {
            const int first = end - O[j], sj = S[j];
            for (int u = t + lane; u < end; u += 32) prof[u] += sj + (u - first) + 1;
            __syncwarp();
          }
        }
        i64 pk = 0;
        for (int u = t + lane; u < hmax; u += 32) pk = max_i64(pk, __ldcg(prof + u));
        peak = max_i64(peak, warp_max(pk));
        break;
      }
      if ((t & 31) == 0) {                              // the plan's next 32 rounds, past the first-level cache: other lanes' atomics wrote them
        __syncwarp();
        const int u = t + lane;
        Bw = u < H ? __ldcg(prof + u) : 0;
      }
      const i64 B = __shfl_sync(0xffffffffu, Bw, t & 31);
      // (3) the pipeline comes first
      while (cnt > 0 && B + A + static_cast<i64>(t) * cnt > M) {
        int j = -1, s0 = 0;
        while (top > 0) {                               // the live entry nearest to the top
          --top;
          const int jj = stk_job[top];
          if (!KVS_OK_AT(jj, n, CHK_SP_JOB)) continue;
          s0 = static_cast<int>(static_cast<u32>(stk_fin[top]) - static_cast<u32>(O[jj]));
          if (sst[jj] == s0) { j = jj; break; }
        }
        if (j < 0) break;
        __syncwarp();
        A -= static_cast<i64>(S[j]) + 1 - s0;
        --cnt;
        steps += t - s0;
        runs += t > s0 ? 1 : 0;
        if (lane == 0) sst[j] = -1;
        __syncwarp();
        const int a = pos_of[j];                        // free again: it may come before the known candidate
        if (!KVS_OK_AT(a, np, CHK_SP_LIST)) break;
        if (a < fpos) { fpos = a; cj = -1; }
        if (a >= fhi) { fhi = a + 1; if (cj == -2) cj = -1; }
      }
      // (4) first come first served: the free jobs of a window of 32 list entries are admitted together as far as
      // their first rounds fit, in order; the first that does not fit ends the round's admissions
      for (;;) {
        const i64 room = M - (B + A + static_cast<i64>(t) * cnt);
        if (cj == -2 || (cj >= 0 && cs + 1 > room) || room <= 0) break;
        // the jobs in a pipeline run are the ranks whose slot has begun and not ended: [re, rs)
        if (fpos >= re && fpos < rs) fpos = rs;
        if (fpos >= fhi) { fpos = np; fhi = 0; cj = -2; break; }
        const int q = fpos + lane;
        bool fr = false;
        int j = 0, sj = 0;
        if (q < fhi && !(q >= re && q < rs) && KVS_OK_AT(q, n, CHK_SP_LIST)) {
          j = list[q];
          if (KVS_OK_AT(j, n, CHK_SP_JOB)) fr = !done[j] && sst[j] < 0; else j = 0;
        }
        const unsigned hit = __ballot_sync(0xffffffffu, fr);
        if (!hit) { fpos += 32; cj = -1; continue; }
        if (fr) sj = S[j];
        i64 need = fr ? static_cast<i64>(sj) + 1 : 0;   // inclusive prefix sums over the window, in list order
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const i64 y = __shfl_up_sync(0xffffffffu, need, d);
          if (lane >= d) need += y;
        }
        const bool ok = fr && need <= room;
        const unsigned okm = __ballot_sync(0xffffffffu, ok);
        const int m = __popc(okm);
        if (m) {
          if (top + 32 > static_cast<int>(cap) || top > 2 * cnt + 64) {   // mostly stale entries: keep the live ones, in order
            int w = 0;
            for (int q0 = 0; q0 < top; q0 += 32) {
              const int qq = q0 + lane;
              bool live = false;
              int jj = 0, ff = 0;
              if (qq < top) { jj = stk_job[qq]; ff = stk_fin[qq]; live = sst[jj] == static_cast<int>(static_cast<u32>(ff) - static_cast<u32>(O[jj])); }
              const unsigned lm = __ballot_sync(0xffffffffu, live);
              __syncwarp();
              if (live) { const int d = w + __popc(lm & lt_mask); stk_job[d] = jj; stk_fin[d] = ff; }
              w += __popc(lm);
              __syncwarp();
            }
            top = w;
          }
          const u32 fin = ok ? tu + static_cast<u32>(O[j]) : NO_ROUND;
          if (ok) {
            const int d = top + __popc(okm & lt_mask);
            if (KVS_OK_AT(d, cap, CHK_SP_STACK)) { sst[j] = t; stk_job[d] = j; stk_fin[d] = static_cast<int>(fin); }
          }
          __syncwarp();
          top += m;
          A += warp_sum(ok ? static_cast<i64>(sj) + 1 - t : static_cast<i64>(0));
          cnt += m;
          next_comp = min(next_comp, warp_min_u32(fin));
        }
        const unsigned failed = hit & ~okm;
        if (failed) {                                   // the first free job that does not fit is the candidate from now on
          const int src = __ffs(static_cast<int>(failed)) - 1;
          fpos += src;
          cj = __shfl_sync(0xffffffffu, j, src);
          cs = __shfl_sync(0xffffffffu, sj, src);
          break;
        }
        fpos += 32; cj = -1;
      }
      // (5) the round's memory
      const i64 mem = B + A + static_cast<i64>(t) * cnt;
      if (lane == 0 && KVS_OK_AT(t, H, CHK_SP_PROF)) prof[t] = static_cast<int32_t>(mem);
      peak = max_i64(peak, mem);
      if (cnt == 0) top = 0;                            // only stale entries are left
    }
    __syncwarp();
    if (lane == 0) {
      if (p.peak) p.peak[e] = peak;
      if (p.flow) p.flow[e] = flow;
      if (p.job_steps) p.job_steps[e] = steps;
      if (p.n_runs) p.n_runs[e] = runs;
      if (p.n_unfinished) p.n_unfinished[e] = left;
      p.horizon[e] = hmax;
      if (p.feasible) p.feasible[e] = peak <= M ? 1 : 0;
    }
    __syncwarp();
  }
}

}  // namespace

KVS_DEFINE_CHECK_WORD(kvs_spec_check_word)

i64 kvs_spec_warp_bytes(i64 max_jobs) { return spec_stride(max_jobs); }

cudaError_t kvs_launch_spec(const SpecParams& p, cudaStream_t stream) {
  if (p.n_list <= 0 || p.n_warps <= 0) return cudaSuccess;
  const cudaError_t err = cudaMemsetAsync(p.counter, 0, 8, stream);
  if (err != cudaSuccess) return err;
  k_spec<<<static_cast<unsigned>((p.n_warps + SWARPS - 1) / SWARPS), ST, 0, stream>>>(p);
  return cudaGetLastError();
}
