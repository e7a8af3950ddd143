// Exact peak of SPS / simultaneous schedules without forming the per-round profile.
//
// Jobs are in key order with key = exact response length; rank i starts at floor(i*tau/k)
// (Procedure StaggeredPipelineSchedule) or floor(i/k)*tau (simultaneous batches) and runs
// d_i = min(o_i, tau) rounds.  Starts and run lengths are both nondecreasing in i, hence so are the
// run ends, and the jobs active in round t are a contiguous index range [e, b).  Memory is
// piecewise linear and increasing between events, so its maximum is attained in the last round of
// some run, t = end_i - 1, where
//     memory(t) = sum_{j in [i, b)} (s_j + t - start_j + 1)
//               = PS_s[b] - PS_s[i] + (b - i)(t + 1) - sum_{j in [i, b)} start_j
// with b = #{j : start_j <= t} = min(n, ceil((t+1)k/tau))  (the count c(rho) in the proof of Lemma
// "Peak Memory Usage of SPS").  Using i instead of the first index with the same end can only drop
// non-negative terms, and that first index is itself a candidate, so the maximum is exact.
// A thread walks consecutive candidates, sliding the window sum of starts; long jumps of b use the
// closed form sum_{j<n} floor(j*tau/k) (Euclid-like floor sum).  Times are relative to the start
// of the schedule (the peak does not depend on a shift).
#pragma once

#include "kvs_internal.cuh"

#ifdef __CUDACC__

// sum_{j=0}^{n-1} floor((a*j + b) / m), arithmetic modulo 2^64
__device__ inline u64 floor_sum(u64 n, u64 m, u64 a, u64 b) {
  u64 ans = 0;
  for (;;) {
    if (a >= m) { ans += (n - 1) * n / 2 * (a / m); a %= m; }
    if (b >= m) { ans += n * (b / m); b %= m; }
    const u64 y = a * n + b;
    if (y < m) break;
    n = y / m;
    b = y % m;
    const u64 t = m; m = a; a = t;
  }
  return ans;
}

// Candidates i0 <= i < i1 of an SPS schedule of n jobs.  sorted_o[i] and prefix_s[i] (exclusive
// prefix sums of s, n + 1 entries) are indexed by rank.  Returns the largest candidate memory and
// adds start + o of the completing jobs to *flow.
__device__ inline i64 sps_range_peak(const int32_t* __restrict__ sorted_o, const i64* __restrict__ prefix_s, i64 n,
                                     i64 tau, i64 k, i64 i0, i64 i1, u64* flow) {
  i64 peak = 0;
  if (i0 >= i1) return peak;
  u64 qt_, rt_, q_, r_;
  divmod_u(static_cast<u64>(tau), static_cast<u64>(k), &qt_, &rt_);
  divmod_u(static_cast<u64>(i0) * static_cast<u64>(tau), static_cast<u64>(k), &q_, &r_);
  const i64 qt = static_cast<i64>(qt_), rt = static_cast<i64>(rt_);
  i64 qi = static_cast<i64>(q_), ri = static_cast<i64>(r_);
  i64 b = i0, qb = qi, rb = ri;   // b: first job not yet counted as started; (qb, rb): its start and remainder
  u64 W = 0;                      // sum of starts over [i, b)
  for (i64 i = i0; i < i1; ++i) {
    const i64 oi = sorted_o[i];
    const i64 d = oi < tau ? oi : tau;
    const i64 t = qi + d - 1;     // last round of run i
    if (oi <= tau) *flow += static_cast<u64>(qi + oi);
    int steps = 0;
    while (b < n && qb <= t) {
      if (steps == 32) {          // long jump: closed forms instead of stepping
        i64 bn = ceil_div_u(static_cast<u64>(t + 1) * static_cast<u64>(k), static_cast<u64>(tau));
        if (bn > n) bn = n;
        W += floor_sum(bn, k, tau, 0) - floor_sum(b, k, tau, 0);
        b = bn;
        divmod_u(static_cast<u64>(b) * static_cast<u64>(tau), static_cast<u64>(k), &q_, &r_);
        qb = static_cast<i64>(q_); rb = static_cast<i64>(r_);
        break;
      }
      W += static_cast<u64>(qb);
      ++b; rb += rt; qb += qt;
      if (rb >= k) { rb -= k; ++qb; }
      ++steps;
    }
    const i64 mem = (prefix_s[b] - prefix_s[i]) + (b - i) * (t + 1) - static_cast<i64>(W);
    peak = mem > peak ? mem : peak;
    W -= static_cast<u64>(qi);
    ri += rt; qi += qt;
    if (ri >= k) { ri -= k; ++qi; }
  }
  return peak;
}

// Same for simultaneous batches of k jobs every tau rounds: a batch is alone in its slot, and in
// round start + d_i - 1 the jobs i .. end of the batch are active with progress d_i - 1.
__device__ inline i64 sims_range_peak(const int32_t* __restrict__ sorted_o, const i64* __restrict__ prefix_s, i64 n,
                                      i64 tau, i64 k, i64 i0, i64 i1, u64* flow) {
  i64 peak = 0;
  if (i0 >= i1) return peak;
  u64 j_, rem_;
  divmod_u(static_cast<u64>(i0), static_cast<u64>(k), &j_, &rem_);
  i64 j = static_cast<i64>(j_), rem = static_cast<i64>(rem_);   // batch index and position inside the batch
  for (i64 i = i0; i < i1; ++i) {
    const i64 oi = sorted_o[i];
    const i64 d = oi < tau ? oi : tau;
    if (oi <= tau) *flow += static_cast<u64>(j * tau + oi);
    i64 bend = (j + 1) * k;
    if (bend > n) bend = n;
    const i64 mem = (prefix_s[bend] - prefix_s[i]) + (bend - i) * d;
    peak = mem > peak ? mem : peak;
    if (++rem == k) { rem = 0; ++j; }
  }
  return peak;
}

#endif  // __CUDACC__
