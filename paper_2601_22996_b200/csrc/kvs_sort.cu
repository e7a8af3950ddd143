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
// into offsets behind the running bucket position.  What moves is an 8-byte record (key, job
// index), so the passes read contiguously and the keys are gathered only once.
#include "kvs_internal.cuh"

namespace {

constexpr int T = KVS_SORT_THREADS;
constexpr int WARPS = T / 32;

__device__ __forceinline__ int32_t key_at(const SortParams& p, i64 lo, int idx) {
  return p.key ? p.key[lo + idx] : p.o[lo + idx];
}

constexpr u32 COUNT_TAG = 0x80000000u;

// Lanes of the warp holding the same value (a digit, or 256 for lanes past the end).
__device__ __forceinline__ u32 match_digit(u32 digit) { return __match_any_sync(0xffffffffu, digit); }

// Sort positions [seg_lo, seg_hi) of the instance starting at global job index lo.
// cnt[digit][warp] (rows padded to 33 words: leaders of different digits and the column scans both
// hit distinct banks) must hold no tagged entry on entry; it holds none on return.
__device__ const u64* sort_segment(const SortParams& p, i64 lo, int seg_lo, int seg_hi, int passes,
                             u32 (*cnt)[WARPS + 1], u32* bucket, u32 (*hist)[256]) {
  const int tid = threadIdx.x, warp = tid >> 5;
  const int n = seg_hi - seg_lo;
  if (passes == 0 || n <= 1) {
    u64* const out = p.rec_a + lo + seg_lo;
    for (int j = tid; j < n; j += T)
      out[j] = (static_cast<u64>(static_cast<u32>(key_at(p, lo, seg_lo + j))) << 32) | static_cast<u32>(seg_lo + j);
    __syncthreads();
    return out;
  }
  // digit histograms of all passes in one sweep; lanes with equal digits add once per warp
  for (int i = tid; i < 4 * 256; i += T) (&hist[0][0])[i] = 0;
  __syncthreads();
  for (int j0 = 0; j0 < n; j0 += T) {
    const int j = j0 + tid;
    const u32 key = j < n ? static_cast<u32>(key_at(p, lo, seg_lo + j)) : 0u;
    for (int d = 0; d < passes; ++d) {
      const u32 digit = j < n ? (key >> (8 * d)) & 255u : 256u;
      const u32 peers = match_digit(digit);
      if (j < n && (peers & lanemask_lt()) == 0) atomicAdd(&hist[d][digit], static_cast<u32>(__popc(peers)));
    }
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

  // Records (key << 32 | job index) move between two buffers, so every pass reads contiguously and
  // never goes back to the keys; the record of the next tile is requested before this tile is
  // ranked, which hides the load latency behind the three barriers of a tile.
  for (int pass = 0; pass < passes; ++pass) {
    u64* dst = ((pass & 1) ? p.rec_b : p.rec_a) + lo + seg_lo;
    const u64* src = ((pass & 1) ? p.rec_a : p.rec_b) + lo + seg_lo;
    if (tid < 256) bucket[tid] = hist[pass][tid];
    __syncthreads();
    auto fetch = [&](int j) -> u64 {
      if (j >= n) return 0;
      if (pass > 0) return src[j];
      return (static_cast<u64>(static_cast<u32>(key_at(p, lo, seg_lo + j))) << 32) | static_cast<u32>(seg_lo + j);
    };
    u64 rec_next = fetch(tid);
    for (int j0 = 0; j0 < n; j0 += T) {
      const int j = j0 + tid;
      const bool valid = j < n;
      const u64 idx = rec_next;           // the whole record travels
      rec_next = fetch(j + T);
      const u32 digit = valid ? static_cast<u32>(idx >> (32 + 8 * pass)) & 255u : 256u;   // 256: lanes past the end
      const u32 peers = match_digit(digit);
      const u32 rank = __popc(peers & lanemask_lt());
      // count of this digit in this warp; the tag marks entries written for this tile (everything
      // else in the table is an offset left by the previous tile's scan, tag clear)
      if (valid && rank == 0) cnt[digit][warp] = static_cast<u32>(__popc(peers)) | COUNT_TAG;
      __syncthreads();
      // column scans: warp w turns the 32 per-warp counts of digits 8w .. 8w+7 into positions
      // behind the running bucket position, one lane per source warp
#pragma unroll
      for (int i = 0; i < 256 / WARPS; ++i) {
        const int dg = warp * (256 / WARPS) + i;
        const u32 raw = cnt[dg][lane_id()];
        const u32 v = (raw & COUNT_TAG) ? (raw & ~COUNT_TAG) : 0u;
        u32 incl = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const u32 y = __shfl_up_sync(0xffffffffu, incl, d);
          if (static_cast<int>(lane_id()) >= d) incl += y;
        }
        const u32 base = bucket[dg];
        cnt[dg][lane_id()] = base + incl - v;
        __syncwarp();
        if (lane_id() == 31) bucket[dg] = base + incl;
      }
      __syncthreads();
      if (valid) dst[cnt[digit][warp] + rank] = idx;
      __syncthreads();
    }
  }
  return (((passes - 1) & 1) ? p.rec_b : p.rec_a) + lo + seg_lo;
}

__global__ void __launch_bounds__(KVS_SORT_THREADS) k_stats_sort(SortParams p) {
  __shared__ u32 cnt[256][WARPS + 1];
  __shared__ u32 hist[4][256];
  __shared__ u32 bucket[256];
  __shared__ int red[32];
  __shared__ i64 wsum[32];
  __shared__ int seg_end;
  const int tid = threadIdx.x;
  for (int i = tid; i < 256 * (WARPS + 1); i += T) (&cnt[0][0])[i] = 0;
  __syncthreads();

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
      const u64* const sorted = sort_segment(p, lo, seg_lo, seg_hi, passes, cnt, bucket, hist);
      __syncthreads();
      for (int j = seg_lo + tid; j < seg_hi; j += T) {
        const u64 rec = sorted[j - seg_lo];
        const int idx = static_cast<int>(static_cast<u32>(rec));
        const int key = static_cast<int>(rec >> 32);
        p.perm[lo + j] = idx;
        p.sorted_s[lo + j] = p.s[lo + idx];
        p.sorted_o[lo + j] = p.key ? p.o[lo + idx] : key;
        if (p.key) p.sorted_key[lo + j] = key;
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
        const i64 w = wsum[lane_id()];
        i64 wi = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const i64 y = __shfl_up_sync(0xffffffffu, wi, d);
          if (static_cast<int>(lane_id()) >= d) wi += y;
        }
        const i64 before = run + __shfl_sync(0xffffffffu, wi - w, tid >> 5);   // all lanes take part in the shuffle
        if (j < n) ps[j + 1] = before + incl;
        run += __shfl_sync(0xffffffffu, wi, 31);
      }
    }
  }
}

}  // namespace

cudaError_t kvs_launch_sort(const SortParams& p, int grid, cudaStream_t stream) {
  if (p.n_instances <= 0) return cudaSuccess;
  k_stats_sort<<<grid, KVS_SORT_THREADS, 0, stream>>>(p);
  return cudaGetLastError();
}
