// Per-instance statistics and the stable order of jobs by (estimated) response length.
//
// One CTA handles one instance at a time.  It first reduces the instance's statistics
// (largest prompt, response and key; input validation), then, window by window, sorts the
// job indices by key with a least-significant-digit radix sort (8-bit digits).  Stability
// (ties keep the original index order) is what makes the order unique, so that the per-job
// results agree bit for bit with a stable comparison sort.
//
// Each pass ranks one tile of 1024 jobs at a time: lanes with equal digits find each other with
// a warp match, per-warp digit counts go to shared memory, one column scan per digit turns them
// into offsets behind the running bucket position.  Only 4 bytes per job move per pass: the
// index, together with the key in the upper half of the word when both fit 16 bits; otherwise the
// next pass re-reads the key through the index.
#include "kvs_internal.cuh"

namespace {

constexpr int T = KVS_SORT_THREADS;
constexpr int WARPS = T / 32;

__device__ __forceinline__ int32_t key_at(const SortParams& p, i64 lo, int idx) {
  return p.key ? p.key[lo + idx] : p.o[lo + idx];
}

// Sort positions [seg_lo, seg_hi) of the instance starting at global job index lo.  The last pass
// holds every job's key when it places the job, so it also writes the keys in sorted order (one more
// scattered store that merges in L2 like the index, instead of a gather afterwards); returns
// whether it did.
// packed: indices and keys are below 2^16, so a pass that is not the last stores (key << 16 | index)
// and the next pass needs no look-up of the key through the index.
__device__ bool sort_segment(const SortParams& p, i64 lo, int seg_lo, int seg_hi, int passes, bool packed,
                             u32 (*warp_cnt)[256], u32 (*warp_off)[256], u32 (*hist)[256]) {
  const int tid = threadIdx.x, warp = tid >> 5;
  const int n = seg_hi - seg_lo;
  int32_t* const out = p.perm + lo + seg_lo;
  if (passes == 0 || n <= 1) {
    for (int j = tid; j < n; j += T) out[j] = seg_lo + j;
    __syncthreads();
    return false;
  }
  // digit histograms of all passes in one sweep
  for (int i = tid; i < 4 * 256; i += T) (&hist[0][0])[i] = 0;
  for (int i = tid; i < WARPS * 256; i += T) (&warp_cnt[0][0])[i] = 0;   // stays zero between tiles, see below
  __syncthreads();
  for (int j = tid; j < n; j += T) {
    u32 key = static_cast<u32>(key_at(p, lo, seg_lo + j));
    for (int d = 0; d < passes; ++d) atomicAdd(&hist[d][(key >> (8 * d)) & 255u], 1u);
  }
  __syncthreads();
  // exclusive scan of each histogram: warp d scans histogram d, 8 digits per lane
  if (warp < passes) {
    u32 v[8], sum = 0;
    for (int i = 0; i < 8; ++i) { v[i] = hist[warp][lane_id() * 8 + i]; sum += v[i]; }
    u32 incl = sum;
    for (int d = 1; d < 32; d <<= 1) {
      u32 y = __shfl_up_sync(0xffffffffu, incl, d);
      if (static_cast<int>(lane_id()) >= d) incl += y;
    }
    u32 run = incl - sum;
    for (int i = 0; i < 8; ++i) { hist[warp][lane_id() * 8 + i] = run; run += v[i]; }
  }
  __syncthreads();

  for (int pass = 0; pass < passes; ++pass) {
    // the last pass must land in perm: passes alternate between the two buffers
    const bool to_perm = ((passes - 1 - pass) & 1) == 0;
    int32_t* dst = (to_perm ? p.perm : p.perm_tmp) + lo + seg_lo;
    const int32_t* src = (to_perm ? p.perm_tmp : p.perm) + lo + seg_lo;
    int32_t* const key_dst = pass == passes - 1 ? (p.key ? p.sorted_key : p.sorted_o) + lo + seg_lo : nullptr;
    u32 bucket = tid < 256 ? hist[pass][tid] : 0u;   // thread d keeps the running position of digit d
    for (int j0 = 0; j0 < n; j0 += T) {
      // Two barriers per tile: the counts are written before the first and read before the second;
      // the offsets are written between them and read after the second (and not overwritten
      // before the first barrier of the next tile, which every thread reaches only after its store).
      // The lane that wrote a count clears it after the second barrier.
      const int j = j0 + tid;
      const bool valid = j < n;
      int idx = 0;
      u32 key = 0, digit = 256;  // sentinel for lanes past the end
      if (valid) {
        if (pass == 0) { idx = seg_lo + j; key = static_cast<u32>(key_at(p, lo, idx)); }
        else if (packed) { const u32 rec = static_cast<u32>(src[j]); idx = static_cast<int>(rec & 0xffffu); key = rec >> 16; }
        else { idx = src[j]; key = static_cast<u32>(key_at(p, lo, idx)); }
        digit = (key >> (8 * pass)) & 255u;
      }
      const u32 peers = __match_any_sync(0xffffffffu, digit);
      const u32 rank = __popc(peers & lanemask_lt());
      const bool leader = valid && rank == 0;
      if (leader) warp_cnt[warp][digit] = __popc(peers);
      __syncthreads();
      if (tid < 256) {
        u32 acc = bucket;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) {
          warp_off[w][tid] = acc;
          acc += warp_cnt[w][tid];
        }
        bucket = acc;
      }
      __syncthreads();
      if (valid) {
        const u32 pos = warp_off[warp][digit] + rank;
        dst[pos] = (packed && !key_dst) ? static_cast<int32_t>(key << 16 | static_cast<u32>(idx)) : idx;
        if (key_dst) key_dst[pos] = static_cast<int32_t>(key);
      }
      if (leader) warp_cnt[warp][digit] = 0;
      __syncwarp();
    }
    __syncthreads();   // the next pass reads what this one stored
  }
  return true;
}

__global__ void __launch_bounds__(KVS_SORT_THREADS) k_stats_sort(SortParams p) {
  extern __shared__ __align__(16) u32 dyn[];
  u32 (*const warp_cnt)[256] = reinterpret_cast<u32 (*)[256]>(dyn);
  u32 (*const warp_off)[256] = reinterpret_cast<u32 (*)[256]>(dyn + WARPS * 256);
  __shared__ u32 hist[4][256];
  __shared__ int red[32];
  __shared__ i64 wsum[32];
  __shared__ int seg_end;
  const int tid = threadIdx.x;

  for (i64 inst = blockIdx.x; inst < p.n_instances; inst += gridDim.x) {
    const i64 lo = p.job_off[inst], hi = p.job_off[inst + 1];
    int flags = 0;
    if (hi < lo || hi - lo > p.max_jobs) flags = KVS_EVAL_BAD_INPUT;
    const int n = flags ? 0 : static_cast<int>(hi - lo);
    int s_max = 0, o_max = 0, key_max = 0, bad = 0;
    for (int j = tid; j < n; j += T) {
      const int sv = p.s[lo + j], ov = p.o[lo + j], kv = key_at(p, lo, j);
      s_max = max(s_max, sv); o_max = max(o_max, ov); key_max = max(key_max, kv);
      bad |= (sv < 0) | (ov < 1) | (kv < 1);
      if (p.arrival) {
        const i64 a = p.arrival[lo + j];
        bad |= (a < 0) | (j > 0 && p.arrival[lo + j - 1] > a);
      }
    }
    s_max = block_max(s_max, red, 0);
    o_max = block_max(o_max, red, 0);
    key_max = block_max(key_max, red, 0);
    bad = block_max(bad, red, 0);
    if (bad) flags = KVS_EVAL_BAD_INPUT;
    if (tid == 0) p.stats[inst] = InstStats{s_max, o_max, key_max, flags};
    if (!p.need_order || flags) continue;  // uniform across the CTA

    const int passes = key_max > 0 ? (32 - __clz(key_max) + 7) / 8 : 0;
    int seg_lo = 0;
    while (seg_lo < n) {
      if (tid == 0) {
        int end = n;
        if (p.window > 0 && p.arrival) {  // first position whose arrival falls in a later window
          const i64 limit = (p.arrival[lo + seg_lo] / p.window + 1) * p.window;
          int a = seg_lo + 1, b = n;
          while (a < b) { int m = (a + b) >> 1; if (p.arrival[lo + m] < limit) a = m + 1; else b = m; }
          end = a;
        }
        seg_end = end;
      }
      __syncthreads();
      const int seg_hi = seg_end;
      const bool have_key = sort_segment(p, lo, seg_lo, seg_hi, passes, n <= 65536 && key_max < 65536, warp_cnt, warp_off, hist);
      __syncthreads();
      for (int j = seg_lo + tid; j < seg_hi; j += T) {
        const int idx = p.perm[lo + j];
        __stcs(&p.sorted_s[lo + j], p.s[lo + idx]);     // streaming stores: read back much later, by another kernel
        if (p.key) {
          __stcs(&p.sorted_o[lo + j], p.o[lo + idx]);
          if (!have_key) __stcs(&p.sorted_key[lo + j], p.key[lo + idx]);
        } else if (!have_key) {
          __stcs(&p.sorted_o[lo + j], p.o[lo + idx]);
        }
        if (p.iperm) p.iperm[lo + idx] = j;
      }
      __syncthreads();
      seg_lo = seg_hi;
    }
    if (p.prefix_s) {
      // exclusive prefix sums of s in schedule order (n + 1 entries per instance): the event form
      // of the peak reads the prompt tokens of any contiguous rank range as one difference
      i64* const ps = p.prefix_s + lo + inst;
      i64 run = 0;
      if (tid == 0) ps[0] = 0;
      for (int j0 = 0; j0 < n; j0 += T) {
        const int j = j0 + tid;
        const i64 v = j < n ? p.sorted_s[lo + j] : 0;
        i64 incl = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const i64 y = __shfl_up_sync(0xffffffffu, incl, d);
          if (static_cast<int>(lane_id()) >= d) incl += y;
        }
        __syncthreads();
        if (lane_id() == 31) wsum[tid >> 5] = incl;
        __syncthreads();
        const i64 w = static_cast<int>(lane_id()) < WARPS ? wsum[lane_id()] : 0;
        i64 wi = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const i64 y = __shfl_up_sync(0xffffffffu, wi, d);
          if (static_cast<int>(lane_id()) >= d) wi += y;
        }
        const i64 before = run + __shfl_sync(0xffffffffu, wi - w, tid >> 5);   // all lanes take part in the shuffle
        if (j < n) __stcs(&ps[j + 1], before + incl);
        run += __shfl_sync(0xffffffffu, wi, 31);
      }
    }
  }
}

}  // namespace

cudaError_t kvs_launch_sort(const SortParams& p, int grid, cudaStream_t stream) {
  if (p.n_instances <= 0) return cudaSuccess;
  constexpr size_t smem = 2 * WARPS * 256 * sizeof(u32);   // digit counts and offsets per warp
  const cudaError_t err = cudaFuncSetAttribute(k_stats_sort, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (err != cudaSuccess) return err;
  k_stats_sort<<<grid, KVS_SORT_THREADS, smem, stream>>>(p);
  return cudaGetLastError();
}
