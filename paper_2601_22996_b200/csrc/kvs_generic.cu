// Generic evaluator for explicit runs (the builder's run list or any user schedule).
//
// A run (start, len, s) holds s + u + 1 tokens in round start + u (Eq. Memory-Feasibility),
// i.e. c + t tokens in round t with c = s + 1 - start.  Per evaluation, one CTA scatters
// (+c, +1) at `start` and (-c, -1) at `start + len` into two zero-initialised difference arrays
// in global memory (64-bit constant terms, 32-bit slopes), prefix-sums both tile by tile and
// forms memory(t) = A(t) + t * B(t), its maximum, and the scalar reductions.  Nothing is assumed
// about the order or overlap of the runs, so this path trades speed for generality.
#include "kvs_internal.cuh"

namespace {

constexpr int T = 512;
constexpr int ITEMS = 4;

__global__ void __launch_bounds__(T) k_generic_eval(GenericParams p) {
  __shared__ i64 red64[32];
  __shared__ int red32[32];
  __shared__ i64 scanA[32];
  __shared__ int scanB[32];
  const int tid = threadIdx.x;
  const kvs_runs& R = p.runs;
  for (i64 e = blockIdx.x; e < R.P; e += gridDim.x) {
    const i64 r0 = R.run_off[e], r1 = R.run_off[e + 1];
    const i64 pbase = p.ev.profile_off[e];
    const i64 cap = p.ev.profile_off[e + 1] - pbase;
    i64* const dA = p.dconst + pbase + e;      // cap + 1 entries
    int32_t* const dB = p.dcount + pbase + e;
    i64 steps = 0, hmax = 0, flow = 0;
    int bad = 0, clipped = 0;
    for (i64 r = r0 + tid; r < r1; r += T) {
      const i64 start = R.run_start[r];
      const i64 len = R.run_len[r];
      if (R.run_flow) flow += R.run_flow[r];
      if (len <= 0) continue;
      if (start < 0) { bad = 1; continue; }
      const i64 end = start + len;
      steps += len;
      hmax = max_i64(hmax, end);
      const i64 c = static_cast<i64>(R.run_s[r]) + 1 - start;
      if (end > cap) clipped = 1;
      if (start < cap) {
        atomicAdd(reinterpret_cast<ull*>(dA + start), static_cast<ull>(c));
        atomicAdd(dB + start, 1);
        if (end <= cap) {
          atomicAdd(reinterpret_cast<ull*>(dA + end), static_cast<ull>(-c));
          atomicAdd(dB + end, -1);
        }
      }
    }
    steps = block_sum(steps, red64);
    hmax = block_max(hmax, red64, static_cast<i64>(0));
    flow = block_sum(flow, red64);
    bad = block_max(bad, red32, 0);
    clipped = block_max(clipped, red32, 0);
    __threadfence();
    __syncthreads();

    const i64 t_end = hmax < cap ? hmax : cap;
    i64 A_run = 0, peak = 0;
    int B_run = 0, over = 0;
    for (i64 t0 = 0; t0 < t_end; t0 += T * ITEMS) {
      i64 a[ITEMS];
      int b[ITEMS];
      i64 sa = 0;
      int sb = 0;
#pragma unroll
      for (int i = 0; i < ITEMS; ++i) {
        const i64 t = t0 + tid * ITEMS + i;
        if (t < t_end) { sa += dA[t]; sb += dB[t]; }
        a[i] = sa; b[i] = sb;
      }
      i64 ia = sa;
      int ib = sb;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const i64 ya = __shfl_up_sync(0xffffffffu, ia, d);
        const int yb = __shfl_up_sync(0xffffffffu, ib, d);
        if (static_cast<int>(lane_id()) >= d) { ia += ya; ib += yb; }
      }
      __syncthreads();
      if (lane_id() == 31) { scanA[tid >> 5] = ia; scanB[tid >> 5] = ib; }
      __syncthreads();
      i64 wa = (lane_id() < T / 32) ? scanA[lane_id()] : 0;
      int wb = (lane_id() < T / 32) ? scanB[lane_id()] : 0;
      i64 wia = wa;
      int wib = wb;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const i64 ya = __shfl_up_sync(0xffffffffu, wia, d);
        const int yb = __shfl_up_sync(0xffffffffu, wib, d);
        if (static_cast<int>(lane_id()) >= d) { wia += ya; wib += yb; }
      }
      const i64 offA = A_run + __shfl_sync(0xffffffffu, wia - wa, tid >> 5) + (ia - sa);
      const int offB = B_run + __shfl_sync(0xffffffffu, wib - wb, tid >> 5) + (ib - sb);
      A_run += __shfl_sync(0xffffffffu, wia, 31);
      B_run += __shfl_sync(0xffffffffu, wib, 31);
#pragma unroll
      for (int i = 0; i < ITEMS; ++i) {
        const i64 t = t0 + tid * ITEMS + i;
        if (t < t_end) {
          const i64 mem = (offA + a[i]) + t * static_cast<i64>(offB + b[i]);
          peak = max_i64(peak, mem);
          if (mem > 0x7fffffffll) over = 1;
          if (p.ev.profile) p.ev.profile[pbase + t] = static_cast<int32_t>(mem > 0x7fffffffll ? 0x7fffffffll : mem);
        }
      }
    }
    peak = block_max(peak, red64, static_cast<i64>(0));
    over = block_max(over, red32, 0);
    if (tid == 0) {
      int status = 0;
      if (bad) status |= KVS_EVAL_BAD_INPUT;
      if (clipped) status |= KVS_EVAL_CAPACITY;
      if (over && p.ev.profile) status |= KVS_EVAL_RANGE;
      if (p.ev.peak) p.ev.peak[e] = peak;
      if (p.ev.flow) p.ev.flow[e] = flow;
      if (p.ev.job_steps) p.ev.job_steps[e] = steps;
      if (p.ev.horizon) p.ev.horizon[e] = hmax;
      if (p.ev.feasible) p.ev.feasible[e] = (!bad && !clipped && R.M && peak <= R.M[e]) ? 1 : 0;
      if (p.ev.status) p.ev.status[e] = status;
    }
    __syncthreads();
  }
}

}  // namespace

cudaError_t kvs_launch_generic(const GenericParams& p, cudaStream_t stream) {
  if (p.runs.P <= 0) return cudaSuccess;
  const int grid = static_cast<int>(p.runs.P < 4096 ? p.runs.P : 4096);
  k_generic_eval<<<grid, T, 0, stream>>>(p);
  return cudaGetLastError();
}
