// Dynamic refill of batching schedules (Numerical Experiments, "Dynamic Refill (GBA-D)"): a job is admitted
// as soon as the pipeline can go on with it without violating memory feasibility, no job is delayed relative
// to the batching schedule, only idle time is filled.
//
// The rule is sequential - every admission changes the memory the next one sees - so one warp works on one
// evaluation and many evaluations run side by side.  The warp starts from what the fused kernels left: every
// job's start in the batching schedule and the per-round memory of that schedule (the plan).  Jobs are taken
// in the schedule's order (key order).  A job's ramp s + u + 1 is taken out of the plan, the earliest round t
// between the previous admission and the job's old start is found at which the ramp fits on top of the plan
// in every round, and the ramp is put back there.  With R(u) = plan(u) + u the ramp fits from t on iff
// max over u in [t, t + o) of R(u) <= M - s - 1 + t; if it does not, the maximising round u* rules out every
// start before min(max R - (M - s - 1), u* + 1), so the search jumps there instead of trying round by round.
// The plan's array is the caller's profile buffer, which ends up holding the refilled schedule's profile.
#include "kvs_check.cuh"

namespace {

constexpr int RT = 128;                 // threads per CTA: four warps, one evaluation each
constexpr int RWARPS = RT / 32;

__global__ void __launch_bounds__(RT) k_refill(RefillParams p) {
  const int lane = lane_id();
  const i64 slot = static_cast<i64>(blockIdx.x) * RWARPS + (threadIdx.x >> 5);
  if (slot >= p.n_list) return;
  const i64 e = p.eval_list[slot];
  if (p.status && p.status[e] != 0) return;            // the batching schedule was not formed or not stored in full
  const kvs_setting st = p.settings[e];
  const i64 lo = p.job_off[st.instance];
  const int n = static_cast<int>(p.job_off[st.instance + 1] - lo);
  const i64 M = st.M;
  int32_t* const prof = p.profile + p.profile_off[e];
  int32_t* const js = p.job_start + p.job_out_off[e];
  int32_t* const jc = p.job_completion + p.job_out_off[e];
  const i64 H = p.horizon[e];                           // of the batching schedule; within the profile's capacity (status 0)
  const i64 pcap = p.profile_off[e + 1] - p.profile_off[e];   // bound of every profile index below (checked build)
  (void)pcap;
  i64 flow = 0;
  int prev = 0, hmax = 0;
  for (int x = 0; x < n; ++x) {
    const int j = p.perm[lo + x];
    const int oj = p.sorted_o[lo + x], sj = p.sorted_s[lo + x];
    if (!KVS_OK_AT(j, n, CHK_RF_JOB)) continue;
    const int g = js[j];
    for (int u = lane; u < oj; u += 32)
      if (KVS_OK_AT(g + u, pcap, CHK_RF_PROF_OUT)) prof[g + u] -= sj + u + 1;
    __syncwarp();
    const i64 bound = M - sj - 1;
    int d = g, t = prev;
    while (t < g) {
      // max of plan(u) + u over the window, and the last round that attains it
      i64 best = -1;
      int arg = t;
      for (int u = t + lane; u < t + oj; u += 32) {
        if (!KVS_OK_AT(u, pcap, CHK_RF_PROF_WIN)) continue;
        const i64 r = static_cast<i64>(prof[u]) + u;
        if (r >= best) { best = r; arg = u; }
      }
#pragma unroll
      for (int dd = 16; dd > 0; dd >>= 1) {
        const i64 ob = __shfl_xor_sync(0xffffffffu, best, dd);
        const int oa = __shfl_xor_sync(0xffffffffu, arg, dd);
        if (ob > best || (ob == best && oa > arg)) { best = ob; arg = oa; }
      }
      if (best - t <= bound) { d = t; break; }
      const i64 need = best - bound;                    // no start before this round clears round `arg`
      t = static_cast<int>(min_i64(need, static_cast<i64>(arg) + 1));
    }
    for (int u = lane; u < oj; u += 32)
      if (KVS_OK_AT(d + u, pcap, CHK_RF_PROF_IN)) prof[d + u] += sj + u + 1;
    __syncwarp();
    if (lane == 0) { js[j] = d; jc[j] = d + oj; }
    flow += d + oj;
    hmax = max(hmax, d + oj);
    prev = d;
  }
  i64 peak = 0;
  for (i64 u = lane; u < H; u += 32) peak = max_i64(peak, prof[u]);
  peak = warp_max(peak);
  if (lane == 0) {
    if (p.peak) p.peak[e] = peak;
    if (p.flow) p.flow[e] = flow;
    p.horizon[e] = hmax;
    if (p.feasible) p.feasible[e] = peak <= M ? 1 : 0;
  }
}

}  // namespace

KVS_DEFINE_CHECK_WORD(kvs_refill_check_word)

cudaError_t kvs_launch_refill(const RefillParams& p, cudaStream_t stream) {
  if (p.n_list <= 0) return cudaSuccess;
  k_refill<<<static_cast<unsigned>((p.n_list + RWARPS - 1) / RWARPS), RT, 0, stream>>>(p);
  return cudaGetLastError();
}
