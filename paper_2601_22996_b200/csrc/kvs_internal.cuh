// Internal declarations shared by the kernels and the C ABI (not part of the public interface).
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

#include "kvs.h"

typedef int64_t i64;
typedef uint64_t u64;
typedef unsigned long long ull;   // the type CUDA's 64-bit atomics are declared on
typedef unsigned int u32;

constexpr int KVS_MAX_PHASES = 96;      // slices of one geometric ladder
constexpr int KVS_SORT_THREADS = 1024;  // one CTA sorts one (instance, window) segment at a time
#ifndef KVS_EVAL_THREADS_CFG
#define KVS_EVAL_THREADS_CFG 512
#define KVS_EVAL_ITEMS_CFG 8
#define KVS_EVAL_MIN_CTAS_CFG 2
#endif
constexpr int KVS_EVAL_THREADS = KVS_EVAL_THREADS_CFG;    // one CTA per evaluation
constexpr int KVS_EVAL_ITEMS = KVS_EVAL_ITEMS_CFG;        // rounds per thread and tile
constexpr int KVS_EVAL_MIN_CTAS = KVS_EVAL_MIN_CTAS_CFG;  // CTAs per SM the register allocation aims at
constexpr int KVS_TILE = KVS_EVAL_THREADS * KVS_EVAL_ITEMS;  // rounds per shared-memory tile

// Scratch bytes of one CTA of the fused kernels (carry lists of the general kernel; class bytes, rank
// table - about 2.5 bytes per job - and two lists of (s, o) pairs of the fast kernel), for instances
// of at most max_jobs jobs.
// A multiple of 256 bytes, so that every CTA's block keeps the 16-byte alignment its vector accesses need.
#define KVS_CTA_SCRATCH(max_jobs) ((20 * static_cast<i64>(max_jobs) + 4096 + 255) & ~static_cast<i64>(255))

// Per-instance statistics produced by the first kernel.
struct InstStats {
  int32_t s_max;
  int32_t o_max;
  int32_t key_max;
  int32_t flags;  // KVS_EVAL_BAD_INPUT or 0
};

// Device view of one call of the fused builder/evaluator.
struct BuildParams {
  // instances
  const i64* job_off;
  const int32_t* s;
  const int32_t* o;
  const int32_t* key;       // estimates, or NULL when the exact o orders and classifies
  const i64* arrival;
  i64 window;
  i64 n_instances;
  i64 max_jobs;
  // order by key (per instance and window), produced by the sort kernel
  const int32_t* perm;      // position -> job index inside the instance
  const int32_t* sorted_s;
  const int32_t* sorted_o;
  const int32_t* sorted_key;
  const i64* prefix_s;      // see SortParams; NULL when no evaluation takes the event form of the peak
  const int32_t* iperm;     // job index inside the instance -> position in key order
  int32_t* fin_rank;        // per-CTA scratch, max_jobs entries each
  const InstStats* stats;
  // evaluations
  const kvs_setting* settings;
  i64 P;
  kvs_schedule_out out;
  kvs_eval_out ev;
  int do_profile;
  // per-CTA carry lists: 2 * max_jobs entries each
  int32_t* lists;
  ull* counter;             // next evaluation to hand out (zeroed before each launch)
  // The 32-bit fast kernel appends the evaluations it leaves to the general kernel here ...
  i64* slow_list;
  ull* slow_count;
  // ... and a kernel that is given a list works through eval_list[0 .. *eval_count)
  const i64* eval_list;
  const ull* eval_count;
  // evaluations the light variant of the fast kernel passes on to the full one
  i64* walk_list;
  ull* walk_count;
};

struct SortParams {
  const i64* job_off;
  const int32_t* s;
  const int32_t* o;
  const int32_t* key;       // NULL: sort by o
  const i64* arrival;
  i64 window;
  i64 n_instances;
  i64 max_jobs;
  int need_order;           // 0: statistics only
  InstStats* stats;
  int32_t* perm;
  int32_t* perm_tmp;
  int32_t* iperm;           // inverse of perm (job index -> position), or NULL
  int32_t* sorted_s;
  int32_t* sorted_o;
  int32_t* sorted_key;      // written only when key != NULL
  i64* prefix_s;            // NULL, or [n_jobs_total + n_instances]: instance j holds its n + 1 exclusive
                            // prefix sums of s in schedule order at job_off[j] + j
};

struct GenericParams {
  kvs_runs runs;
  kvs_eval_out ev;
  i64* dconst;              // [capacity_total + P] difference array of the constant terms
  int32_t* dcount;          // [capacity_total + P] difference array of the slopes
  i64 slots;                // entries of each array; the kernel skips an evaluation whose offsets reach beyond
};

// Dynamic refill of the batching schedules of the listed evaluations, in place (see kvs_refill.cu).
struct RefillParams {
  const i64* job_off;
  const int32_t* perm;         // key order -> job index, per instance
  const int32_t* sorted_s;     // prompt and response lengths in key order
  const int32_t* sorted_o;
  const kvs_setting* settings;
  const i64* eval_list;        // evaluations to refill
  i64 n_list;
  const i64* job_out_off;
  int32_t* job_start;          // in: starts of the batching schedule; out: refilled starts
  int32_t* job_completion;
  const i64* profile_off;
  int32_t* profile;            // in: memory of the batching schedule; out: of the refilled one
  i64* peak; i64* flow; i64* horizon; uint8_t* feasible;
  const int32_t* status;
};

// Speculative runs on top of the slicing schedules of the listed evaluations, in place (see kvs_spec.cu).
struct SpecParams {
  const i64* job_off;
  const int32_t* s;            // prompt and response lengths in index order
  const int32_t* o;
  const InstStats* stats;
  const kvs_setting* settings;
  const i64* eval_list;        // evaluations to work on
  i64 n_list;
  const i64* job_out_off;
  int32_t* job_start;          // in: of the slicing schedule; out: of the run that completed the job
  int32_t* job_completion;
  const i64* profile_off;
  int32_t* profile;            // in: memory of the slicing schedule; out: with the speculative runs
  i64* peak; i64* flow; i64* horizon; i64* job_steps; i64* n_runs; i64* n_unfinished; uint8_t* feasible;
  const int32_t* status;
  unsigned char* scratch;      // n_warps blocks of kvs_spec_warp_bytes(max_jobs) bytes
  i64 scratch_bytes;
  i64 max_jobs;
  i64 n_warps;                 // warps launched; each takes evaluations from the list until it is used up
  ull* counter;
};

struct SweepParams {
  const int32_t* sorted_s;  // the instance in key order
  const int32_t* sorted_o;
  const i64* prefix_s;      // [n + 1]
  const i64* prefix_o;      // [n + 1]
  i64 n;
  int family;
  i64 M;
  const i64* tau;           // DEVICE copies of the grids
  const i64* k;
  int n_tau, n_k;
  kvs_sweep_out out;
};

cudaError_t kvs_launch_sort(const SortParams& p, int grid, cudaStream_t stream);
cudaError_t kvs_launch_build(const BuildParams& p, int grid, cudaStream_t stream);
int kvs_build_ctas_per_sm();
enum { KVS_FUSED_ANY = -1 };   // instantiation of the fast kernel for any family; the others are named by the family id
cudaError_t kvs_launch_fused(const BuildParams& p, int grid, int light, int fam, cudaStream_t stream);
int kvs_fused_ctas_per_sm(int light);
cudaError_t kvs_fused_check_word(unsigned long long* word, int* compiled, int reset);
cudaError_t kvs_refill_check_word(unsigned long long* word, int* compiled, int reset);
cudaError_t kvs_spec_check_word(unsigned long long* word, int* compiled, int reset);
cudaError_t kvs_launch_generic(const GenericParams& p, cudaStream_t stream);
cudaError_t kvs_launch_refill(const RefillParams& p, cudaStream_t stream);
i64 kvs_spec_warp_bytes(i64 max_jobs);
cudaError_t kvs_launch_spec(const SpecParams& p, cudaStream_t stream);
cudaError_t kvs_launch_bounds(const i64* job_off, const int32_t* o, const InstStats* stats, const kvs_setting* settings,
                              i64 P, const kvs_bounds_out& out, int grid, cudaStream_t stream);
cudaError_t kvs_launch_prefix(const int32_t* sorted_s, const int32_t* sorted_o, i64 n, i64* prefix_s,
                              i64* prefix_o, cudaStream_t stream);
cudaError_t kvs_launch_sweep(const SweepParams& p, i64* acc_peak, u64* acc_flow, cudaStream_t stream);
// n_completed[i] = (job_off[1] - job_off[0]) - n_unfinished[i] where status[i] has neither the infeasible nor the bad-input bit, else 0
cudaError_t kvs_launch_completed(const i64* job_off, const i64* n_unfinished, const int32_t* status, i64* n_completed, i64 P, cudaStream_t stream);

// ---- small device helpers ---------------------------------------------------------------------
#ifdef __CUDACC__

__device__ __forceinline__ u32 lane_id() { return threadIdx.x & 31u; }
__device__ __forceinline__ u32 lanemask_lt() {
  u32 m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}

// floor(r * tau / k) for 0 <= r, tau < 2^31 and 1 <= k < 2^31.
__device__ __forceinline__ i64 slot_offset(i64 r, i64 tau, i64 k) {
  u64 x = static_cast<u64>(r) * static_cast<u64>(tau);
  if ((x >> 32) == 0) return static_cast<i64>(static_cast<u32>(x) / static_cast<u32>(k));
  return static_cast<i64>(x / static_cast<u64>(k));
}

// Quotient and remainder of non-negative 64-bit values.  64-bit division is emulated with well over
// a hundred instructions, so the common case of operands below 2^32 takes the 32-bit divider.
__device__ __forceinline__ void divmod_u(u64 x, u64 y, u64* q, u64* r) {
  if (((x | y) >> 32) == 0) {
    const u32 a = static_cast<u32>(x), b = static_cast<u32>(y);
    *q = a / b; *r = a % b;
  } else {
    *q = x / y; *r = x % y;
  }
}

__device__ __forceinline__ i64 ceil_div_u(u64 x, u64 y) {
  u64 q, r;
  divmod_u(x, y, &q, &r);
  return static_cast<i64>(q + (r != 0));
}
__device__ __forceinline__ i64 min_i64(i64 x, i64 y) { return x < y ? x : y; }
__device__ __forceinline__ i64 max_i64(i64 x, i64 y) { return x > y ? x : y; }

template <typename T>
__device__ __forceinline__ T warp_sum(T v) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
  return v;
}
template <typename T>
__device__ __forceinline__ T warp_max(T v) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    T w = __shfl_xor_sync(0xffffffffu, v, d);
    v = w > v ? w : v;
  }
  return v;
}

// Block-wide reductions; `scratch` has room for 32 values; result valid in every thread.
template <typename T>
__device__ __forceinline__ T block_sum(T v, T* scratch) {
  v = warp_sum(v);
  __syncthreads();
  if (lane_id() == 0) scratch[threadIdx.x >> 5] = v;
  __syncthreads();
  T r = 0;
  int nw = (blockDim.x + 31) >> 5;
  if (static_cast<int>(lane_id()) < nw) r = scratch[lane_id()];
  return warp_sum(r);
}
template <typename T>
__device__ __forceinline__ T block_max(T v, T* scratch, T lowest) {
  v = warp_max(v);
  __syncthreads();
  if (lane_id() == 0) scratch[threadIdx.x >> 5] = v;
  __syncthreads();
  T r = lowest;
  int nw = (blockDim.x + 31) >> 5;
  if (static_cast<int>(lane_id()) < nw) r = scratch[lane_id()];
  return warp_max(r);
}

#endif  // __CUDACC__
