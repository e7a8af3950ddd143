// Parameter sweep: SPS or the simultaneous schedule for every (tau, k) of a grid on one
// instance, scalars only.  Horizons reach billions of rounds, so nothing dense is formed: the
// peak comes from the candidate rounds described in kvs_events.cuh, one CTA per (setting, chunk
// of 8,192 ranks), each thread walking 64 consecutive ranks.
#include "kvs_events.cuh"

namespace {

constexpr int SW_THREADS = 128;
constexpr int SW_PER = 64;
constexpr int SW_CHUNK = SW_THREADS * SW_PER;

__global__ void __launch_bounds__(SW_THREADS) k_sweep(SweepParams p, i64 n_chunks, i64* acc_peak, u64* acc_flow) {
  __shared__ i64 red64[32];
  const i64 setting = blockIdx.x / n_chunks, chunk = blockIdx.x % n_chunks;
  const i64 tau = p.tau[setting / p.n_k], k = p.k[setting % p.n_k];
  const i64 n = p.n;
  const i64 i0 = chunk * SW_CHUNK + static_cast<i64>(threadIdx.x) * SW_PER;
  const i64 i1 = i0 + SW_PER < n ? i0 + SW_PER : n;
  u64 flow = 0;
  i64 peak = p.family == KVS_SPS ? sps_range_peak(p.sorted_o, p.prefix_s, n, tau, k, i0, i1, &flow)
                                 : sims_range_peak(p.sorted_o, p.prefix_s, n, tau, k, i0, i1, &flow);
  peak = block_max(peak, red64, static_cast<i64>(0));
  const i64 fsum = block_sum(static_cast<i64>(flow), red64);
  if (threadIdx.x == 0) {
    if (peak > 0) atomicMax(reinterpret_cast<long long*>(acc_peak + setting), static_cast<long long>(peak));
    if (fsum != 0) atomicAdd(reinterpret_cast<ull*>(acc_flow + setting), static_cast<ull>(fsum));
  }
}

__global__ void k_sweep_finish(SweepParams p, const i64* acc_peak, const u64* acc_flow) {
  const i64 setting = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (setting >= static_cast<i64>(p.n_tau) * p.n_k) return;
  const i64 tau = p.tau[setting / p.n_k], k = p.k[setting % p.n_k];
  const i64 n = p.n;
  i64 a = 0, b = n;                 // completed jobs = those with o <= tau: a prefix in key order
  while (a < b) { const i64 m = (a + b) >> 1; if (p.sorted_o[m] <= tau) a = m + 1; else b = m; }
  const i64 c = a;
  i64 horizon = 0;
  if (n > 0) {
    const i64 last = n - 1;
    const i64 start = p.family == KVS_SPS ? slot_offset(last, tau, k) : (last / k) * tau;
    const i64 ol = p.sorted_o[last];
    horizon = start + (ol < tau ? ol : tau);
  }
  if (p.out.peak) p.out.peak[setting] = acc_peak[setting];
  if (p.out.flow) p.out.flow[setting] = static_cast<i64>(acc_flow[setting]);
  if (p.out.n_completed) p.out.n_completed[setting] = c;
  if (p.out.horizon) p.out.horizon[setting] = horizon;
  if (p.out.job_steps) p.out.job_steps[setting] = p.prefix_o[c] + (n - c) * tau;
  if (p.out.feasible) p.out.feasible[setting] = acc_peak[setting] <= p.M ? 1 : 0;
}

// Exclusive prefix sums of s and o in key order (one CTA, tile after tile).
__global__ void __launch_bounds__(1024) k_prefix(const int32_t* s, const int32_t* o, i64 n, i64* ps, i64* po) {
  __shared__ i64 ws[32], wo[32];
  i64 run_s = 0, run_o = 0;
  const int tid = threadIdx.x;
  if (tid == 0) { ps[0] = 0; po[0] = 0; }
  for (i64 j0 = 0; j0 < n; j0 += 1024) {
    const i64 j = j0 + tid;
    const i64 vs = j < n ? s[j] : 0, vo = j < n ? o[j] : 0;
    i64 is = vs, io = vo;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const i64 ys = __shfl_up_sync(0xffffffffu, is, d), yo = __shfl_up_sync(0xffffffffu, io, d);
      if (static_cast<int>(lane_id()) >= d) { is += ys; io += yo; }
    }
    __syncthreads();
    if (lane_id() == 31) { ws[tid >> 5] = is; wo[tid >> 5] = io; }
    __syncthreads();
    i64 a = ws[lane_id()], b = wo[lane_id()];
    i64 ia = a, ib = b;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const i64 ya = __shfl_up_sync(0xffffffffu, ia, d), yb = __shfl_up_sync(0xffffffffu, ib, d);
      if (static_cast<int>(lane_id()) >= d) { ia += ya; ib += yb; }
    }
    const i64 off_s = run_s + __shfl_sync(0xffffffffu, ia - a, tid >> 5);
    const i64 off_o = run_o + __shfl_sync(0xffffffffu, ib - b, tid >> 5);
    if (j < n) { ps[j + 1] = off_s + is; po[j + 1] = off_o + io; }
    run_s += __shfl_sync(0xffffffffu, ia, 31);
    run_o += __shfl_sync(0xffffffffu, ib, 31);
  }
}

}  // namespace

cudaError_t kvs_launch_prefix(const int32_t* sorted_s, const int32_t* sorted_o, i64 n, i64* prefix_s,
                              i64* prefix_o, cudaStream_t stream) {
  k_prefix<<<1, 1024, 0, stream>>>(sorted_s, sorted_o, n, prefix_s, prefix_o);
  return cudaGetLastError();
}

cudaError_t kvs_launch_sweep(const SweepParams& p, i64* acc_peak, u64* acc_flow, cudaStream_t stream) {
  const i64 n_set = static_cast<i64>(p.n_tau) * p.n_k;
  if (n_set <= 0) return cudaSuccess;
  cudaError_t e = cudaMemsetAsync(acc_peak, 0, static_cast<size_t>(n_set) * 8, stream);
  if (e != cudaSuccess) return e;
  e = cudaMemsetAsync(acc_flow, 0, static_cast<size_t>(n_set) * 8, stream);
  if (e != cudaSuccess) return e;
  const i64 n_chunks = (p.n + SW_CHUNK - 1) / SW_CHUNK;
  if (n_chunks > 0) {
    const i64 blocks = n_set * n_chunks;
    if (blocks >= (static_cast<i64>(1) << 31)) return cudaErrorInvalidConfiguration;
    k_sweep<<<static_cast<unsigned>(blocks), SW_THREADS, 0, stream>>>(p, n_chunks, acc_peak, acc_flow);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  k_sweep_finish<<<static_cast<unsigned>((n_set + 255) / 256), 256, 0, stream>>>(p, acc_peak, acc_flow);
  return cudaGetLastError();
}

namespace {
__global__ void k_completed(const i64* job_off, const i64* n_unfinished, const int32_t* status, i64* n_completed, i64 P) {
  const i64 i = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= P) return;
  const bool skipped = (status[i] & (KVS_EVAL_INFEASIBLE | KVS_EVAL_BAD_INPUT)) != 0;
  n_completed[i] = skipped ? 0 : (job_off[1] - job_off[0]) - n_unfinished[i];
}
}  // namespace

cudaError_t kvs_launch_completed(const i64* job_off, const i64* n_unfinished, const int32_t* status, i64* n_completed, i64 P, cudaStream_t stream) {
  if (P <= 0) return cudaSuccess;
  k_completed<<<static_cast<unsigned>((P + 255) / 256), 256, 0, stream>>>(job_off, n_unfinished, status, n_completed, P);
  return cudaGetLastError();
}
