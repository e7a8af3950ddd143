// Generic evaluator for explicit runs (the builder's run list or any user schedule).
//
// A run (start, len, s) holds s + u + 1 tokens in round start + u (Eq. Memory-Feasibility),
// i.e. c + t tokens in round t with c = s + 1 - start.  Per evaluation, one CTA scatters
// (+c, +1) at `start` and (-c, -1) at `start + len` into two zero-initialised difference arrays
// in global memory (64-bit constant terms, 32-bit slopes), prefix-sums both tile by tile and
// forms memory(t) = A(t) + t * B(t), its maximum, and the scalar reductions.  Nothing is assumed
// about the order or overlap of the runs, so this path trades speed for generality.
#include <atomic>
#include <cstdio>

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
    // The difference arrays hold `slots` entries; evaluation e owns entries pbase + e .. pbase + e + cap.
    // Offsets on the device that do not fit (not monotone, or larger than the host said when the arrays
    // were sized) would send the atomics outside them: such an evaluation is reported and skipped.
    if (pbase < 0 || cap < 0 || pbase > p.slots || cap > p.slots - pbase || e + 1 > p.slots - pbase - cap) {
      if (tid == 0) {
        if (p.ev.peak) p.ev.peak[e] = -1;
        if (p.ev.flow) p.ev.flow[e] = 0;
        if (p.ev.job_steps) p.ev.job_steps[e] = 0;
        if (p.ev.horizon) p.ev.horizon[e] = 0;
        if (p.ev.feasible) p.ev.feasible[e] = 0;
        if (p.ev.status) p.ev.status[e] = KVS_EVAL_CAPACITY | KVS_EVAL_BAD_INPUT;
      }
      continue;
    }
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

// ---- variant without any caller- or library-allocated scratch -----------------------------------
//
// Same kernel, but the two difference arrays live in a fixed array that is part of the loaded
// library image on every GPU (12 MiB per device, held until the process exits).  The array is
// shared by all calls on a device and keeps what the previous call left, so each call clears the
// part it uses first; two calls that overlap on the GPU would race on it.

constexpr int64_t KVS_NOALLOC_SLOTS = int64_t(1) << 20;   // rounds + evaluations per call
static __device__ __align__(256) unsigned char kvs_noalloc_scratch[KVS_NOALLOC_SLOTS * 12];

namespace {
constexpr int KVS_NOALLOC_MAX_DEVICES = 64;
// Device address of the array, per device.  Atomic, so that two host threads making their first call on
// a device at the same time both end up with the same, fully written pointer.
std::atomic<void*> g_noalloc_ptr[KVS_NOALLOC_MAX_DEVICES] = {};
void put_msg(char* err, uint64_t len, const char* msg) {
  if (err && len) { snprintf(err, static_cast<size_t>(len), "%s", msg); }
}
}  // namespace

extern "C" int kvs_evaluate_schedule_noalloc(int32_t device, void* stream, const kvs_runs* runs,
                                             const kvs_eval_out* ev, int64_t capacity_total,
                                             char* err, uint64_t err_len) {
  if (!runs || !ev) { put_msg(err, err_len, "runs or eval_out is null"); return KVS_E_ARG; }
  if (runs->P < 0 || capacity_total < 0) { put_msg(err, err_len, "negative size"); return KVS_E_ARG; }
  if (device < 0 || device >= KVS_NOALLOC_MAX_DEVICES) { put_msg(err, err_len, "device ordinal out of range"); return KVS_E_ARG; }
  if (runs->P == 0) return KVS_OK;
  if (!runs->run_off || !runs->run_start || !runs->run_len || !runs->run_s || !ev->profile_off) {
    put_msg(err, err_len, "null run array or profile_off");
    return KVS_E_ARG;
  }
  if (runs->P > KVS_NOALLOC_SLOTS || capacity_total > KVS_NOALLOC_SLOTS - runs->P) {
    put_msg(err, err_len, "capacity_total + P exceeds the 1,048,576 slots of the built-in scratch array; "
                          "use kvs_evaluate_schedule with a workspace instead");
    return KVS_E_CAPACITY;
  }
  // The work is issued with `device` current; the caller's current device is put back before returning.
  int prev_device = -1;
  cudaError_t ce = cudaGetDevice(&prev_device);
  if (ce == cudaSuccess && prev_device != device) ce = cudaSetDevice(device);
  if (ce != cudaSuccess) { put_msg(err, err_len, cudaGetErrorString(ce)); return KVS_E_CUDA; }
  struct Restore {
    int prev, cur;
    ~Restore() { if (prev >= 0 && prev != cur) cudaSetDevice(prev); }
  } restore{prev_device, device};
  void* ptr = g_noalloc_ptr[device].load(std::memory_order_acquire);
  if (!ptr) {
    // In host code the array's name is only a handle; its device address has to be asked for,
    // once per device, with that device current.
    ce = cudaGetSymbolAddress(&ptr, kvs_noalloc_scratch);
    if (ce != cudaSuccess || !ptr) { put_msg(err, err_len, cudaGetErrorString(ce)); return KVS_E_CUDA; }
    g_noalloc_ptr[device].store(ptr, std::memory_order_release);
  }
  unsigned char* base = static_cast<unsigned char*>(ptr);
  const size_t slots = static_cast<size_t>(capacity_total + runs->P);
  const size_t bytes_a = (slots * 8 + 255) & ~static_cast<size_t>(255);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  ce = cudaMemsetAsync(base, 0, bytes_a + slots * 4, s);   // what must start at zero
  if (ce != cudaSuccess) { put_msg(err, err_len, cudaGetErrorString(ce)); return KVS_E_CUDA; }
  GenericParams gp{};
  gp.runs = *runs;
  gp.ev = *ev;
  gp.dconst = reinterpret_cast<i64*>(base);
  gp.dcount = reinterpret_cast<int32_t*>(base + bytes_a);
  gp.slots = static_cast<i64>(slots);
  ce = kvs_launch_generic(gp, s);
  if (ce != cudaSuccess) { put_msg(err, err_len, cudaGetErrorString(ce)); return KVS_E_CUDA; }
  return KVS_OK;
}
