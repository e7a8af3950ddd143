// Fused schedule builder and evaluator: one CTA per (instance, setting, family) evaluation.
//
// For one evaluation the CTA
//   1. forms the phase table in shared memory: the geometric ladder tau_p and the largest
//      memory-feasible parallelism k_p (first line of the two geometric algorithms; Lemma
//      "Peak Memory Usage of SPS"; Eq. max-parallelism), or the single (tau, k) of SPS / SimS;
//   2. walks the phases in order.  The participants of a phase are the jobs carried over from
//      the previous phase (killed there) followed by the jobs whose class is this phase; in key
//      order the second group is a contiguous range found by binary search, the first is a
//      compacted list kept in an L2-resident scratch buffer.  Rank r starts at
//      base + floor(r*tau/k) (Procedure StaggeredPipelineSchedule) or base + floor(r/k)*tau
//      (simultaneous batches), runs min(o, tau) rounds, completes iff o <= tau;
//   3. builds the per-round memory of the phase tile by tile in shared memory from two
//      difference arrays - the constant term s+1-start and the slope 1 of every active run -
//      each prefix-summed once, memory(t) = A(t) + t*B(t) (Eq. Memory-Feasibility), reduces the
//      peak, and streams the profile out;
//   4. reduces flow time, job-steps, horizon and the number of unfinished jobs.
//
// The difference arrays and their sums are kept modulo 2^32.  Every intermediate may wrap, the
// final memory(t) is exact whenever it is below 2^32, which a per-phase bound guarantees
// (otherwise the evaluation reports KVS_EVAL_RANGE and skips the profile).
#include "kvs_internal.cuh"

namespace {

constexpr int T = KVS_EVAL_THREADS;
constexpr int ITEMS = KVS_EVAL_ITEMS;
constexpr int TILE = KVS_TILE;
constexpr int WARPS = T / 32;

typedef unsigned __int128 u128;

__device__ __forceinline__ i64 gcd_i64(i64 x, i64 y) {
  while (y) { i64 t = x % y; x = y; y = t; }
  return x;
}

// Largest k >= 1 with s*k + (tau*k + tau + k - gcd(tau, k))/2 <= M, given s + tau <= M.
// The condition reads k*(2s+tau+1) <= 2M - tau + gcd(tau,k); because 1 <= gcd <= tau the answer
// is k0 or k0 + 1 with k0 = floor((2M - tau + 1) / (2s + tau + 1)).
__device__ i64 max_parallelism(i64 tau, i64 s, i64 M) {
  const i64 D = 2 * s + tau + 1;
  const i64 k0 = (2 * M - tau + 1) / D;
  const i64 k1 = k0 + 1;
  return (k1 * D <= 2 * M - tau + gcd_i64(tau, k1)) ? k1 : k0;
}

struct Shared {
  u32 dA[TILE];             // difference array of constant terms, then the finished profile tile
  u32 dB[TILE];             // difference array of slopes
  i64 tau[KVS_MAX_PHASES];
  i64 k[KVS_MAX_PHASES];
  int ent[KVS_MAX_PHASES + 1];  // class boundaries in key order: entrants of phase p are [ent[p], ent[p+1])
  u128 pw_a[KVS_MAX_PHASES + 1];
  u128 pw_b[KVS_MAX_PHASES + 1];
  i64 red64[32];
  u32 redA[32], redB[32];
  int red32[32];
  int n_phases;
  int seg_end;
};

// Geometric ladder by warp 0.  Leaves the number of phases in sh.n_phases (0 = too many).
__device__ void build_ladder(Shared& sh, i64 X, int a, int b, i64 beta0, i64 s_bar, i64 M) {
  const int lane = lane_id();
  if (beta0 <= 0) {
    if (lane == 0) {
      // ell = largest j with a^j <= X * b^j, powers kept exactly in 128 bits
      u128 pa = 1, pb = 1;
      int ell = 0;
      sh.pw_a[0] = 1; sh.pw_b[0] = 1;
      while (ell + 1 < KVS_MAX_PHASES + 1) {
        const u128 na = pa * static_cast<u128>(a), nb = pb * static_cast<u128>(b);
        if (na > static_cast<u128>(X) * nb) break;
        pa = na; pb = nb; ++ell;
        sh.pw_a[ell] = pa; sh.pw_b[ell] = pb;
      }
      sh.n_phases = (ell + 1 <= KVS_MAX_PHASES) ? ell + 1 : 0;
    }
    __syncwarp();
    const int L = sh.n_phases;
    for (int p = lane; p < L; p += 32) {
      const int j = L - 1 - p;  // tau_p = floor(X * b^j / a^j)
      const i64 t = (a == 2 && b == 1) ? (X >> j) : static_cast<i64>(static_cast<u128>(X) * sh.pw_b[j] / sh.pw_a[j]);
      sh.tau[p] = t;
      sh.k[p] = max_parallelism(t, s_bar, M);
    }
  } else {
    if (lane == 0) {
      u128 pa = 1, pb = 1;
      int p = 0;
      for (;; ++p) {
        if (p >= KVS_MAX_PHASES) { p = -1; break; }
        // tau_p = min(floor(beta0 * a^p / b^p), X)
        const u128 num = static_cast<u128>(beta0) * pa;
        i64 t = (num >= static_cast<u128>(X) * pb) ? X : static_cast<i64>(num / pb);
        sh.tau[p] = t;
        sh.k[p] = max_parallelism(t, s_bar, M);
        if (t >= X) break;
        pa *= static_cast<u128>(a); pb *= static_cast<u128>(b);
      }
      sh.n_phases = p + 1;
    }
  }
  __syncwarp();
}

// Exclusive block scan of a 0/1 flag; returns this thread's offset, total in *total.
__device__ __forceinline__ int block_flag_scan(bool flag, int* red32, int* total) {
  const u32 ballot = __ballot_sync(0xffffffffu, flag);
  const int warp = threadIdx.x >> 5;
  __syncthreads();
  if (lane_id() == 0) red32[warp] = __popc(ballot);
  __syncthreads();
  int v = (lane_id() < WARPS) ? red32[lane_id()] : 0;
  int incl = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    int y = __shfl_up_sync(0xffffffffu, incl, d);
    if (static_cast<int>(lane_id()) >= d) incl += y;
  }
  const int warp_off = __shfl_sync(0xffffffffu, incl - v, warp);
  *total = __shfl_sync(0xffffffffu, incl, 31);
  return warp_off + __popc(ballot & lanemask_lt());
}

struct Acc {
  i64 flow = 0, steps = 0, hmax = 0;
  int unfinished = 0;
  u32 peak = 0;
};

__global__ void __launch_bounds__(KVS_EVAL_THREADS) k_build_eval(BuildParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Shared& sh = *reinterpret_cast<Shared*>(smem_raw);
  const int tid = threadIdx.x;
  int32_t* const list0 = p.lists + static_cast<i64>(blockIdx.x) * 2 * p.max_jobs;
  int32_t* const list1 = list0 + p.max_jobs;

  for (i64 e = blockIdx.x; e < p.P; e += gridDim.x) {
    const kvs_setting st = p.settings[e];
    const i64 lo = p.job_off[st.instance];
    const InstStats stats = p.stats[st.instance];
    const int n = stats.flags ? 0 : static_cast<int>(p.job_off[st.instance + 1] - lo);
    const i64 M = st.M;
    const i64 s_bar = st.s_bar >= 0 ? st.s_bar : stats.s_max;
    const i64 X = M - s_bar;
    const int family = st.family;
    const bool geometric = family == KVS_GBA || family == KVS_GSA;
    const bool simultaneous = family == KVS_SIMS;
    const bool keyed = !(family == KVS_GSA && p.key == nullptr);  // plain GSA keeps the index order
    const bool may_carry = geometric && (family == KVS_GSA || p.key != nullptr);
    const int32_t* const S = (keyed ? p.sorted_s : p.s) + lo;
    const int32_t* const O = (keyed ? p.sorted_o : p.o) + lo;
    const int32_t* const PERM = keyed ? p.perm + lo : nullptr;
    const int32_t* const KEY = p.key ? p.sorted_key + lo : O;

    int status = stats.flags;
    if (!status && (X < 1 || stats.o_max > X)) status = KVS_EVAL_INFEASIBLE;
    __syncthreads();  // previous evaluation done with shared memory
    if (!status && geometric) {
      if (tid < 32) build_ladder(sh, X, st.alpha_num, st.alpha_den, st.beta0, s_bar, M);
      __syncthreads();
      if (sh.n_phases == 0) status = KVS_EVAL_RANGE;
    }

    const i64 job_out = p.out.job_out_off ? p.out.job_out_off[e] : 0;
    const bool want32 = p.out.job_start || p.out.job_completion;
    const i64 run_base = p.out.run_off ? p.out.run_off[e] : 0;
    const i64 run_cap = p.out.run_off ? p.out.run_off[e + 1] - run_base : 0;
    const bool want_runs = p.out.run_off && (p.out.run_job || p.out.run_phase || p.out.run_start || p.out.run_len || p.out.run_s);
    const i64 prof_base = p.ev.profile_off ? p.ev.profile_off[e] : 0;
    const i64 prof_cap = (p.ev.profile && p.ev.profile_off) ? p.ev.profile_off[e + 1] - prof_base : 0;
    bool profile_on = p.do_profile != 0;

    Acc acc;
    i64 base = 0;          // first round of the next phase
    i64 written_to = 0;    // profile rounds [0, written_to) have been written
    i64 run_count = 0;

    int seg_lo = 0;
    while (!status && seg_lo < n) {
      // ---- window = offline sub-instance [seg_lo, seg_hi) ----
      if (tid == 0) {
        int end = n;
        if (p.window > 0 && p.arrival) {
          const i64 limit = (p.arrival[lo + seg_lo] / p.window + 1) * p.window;
          int a = seg_lo + 1, b = n;
          while (a < b) { int m = (a + b) >> 1; if (p.arrival[lo + m] < limit) a = m + 1; else b = m; }
          end = a;
        }
        sh.seg_end = end;
      }
      __syncthreads();
      const int seg_hi = sh.seg_end;
      const int nseg = seg_hi - seg_lo;
      if (p.window > 0 && p.arrival) {
        const i64 release = (p.arrival[lo + seg_lo] / p.window + 1) * p.window;
        base = max_i64(base, release);
      }

      int L = 1;
      if (geometric) {
        L = sh.n_phases;
        // class boundaries: entrants of phase p have clip(key) <= tau_p and > tau_(p-1)
        for (int q = tid; q <= L; q += T) {
          int v;
          if (q == 0) v = 0;
          else if (q == L || family == KVS_GSA) v = nseg;   // tau_(L-1) = X >= every clipped key
          else {
            const i64 t = sh.tau[q - 1];
            int a = 0, b = nseg;
            while (a < b) { int m = (a + b) >> 1; if (KEY[seg_lo + m] <= t) a = m + 1; else b = m; }
            v = a;
          }
          sh.ent[q] = v;
        }
      } else if (tid == 0) {
        i64 tau = st.tau > 0 ? st.tau : static_cast<i64>(KEY[seg_hi - 1]);  // largest key of the segment
        i64 k = st.k;
        if (k <= 0) k = simultaneous ? M / (s_bar + tau) : (s_bar + tau <= M ? max_parallelism(tau, s_bar, M) : 0);
        sh.tau[0] = tau; sh.k[0] = k;
        sh.ent[0] = 0; sh.ent[1] = nseg;
      }
      __syncthreads();
      if (!geometric && sh.k[0] < 1) { status = KVS_EVAL_INFEASIBLE; break; }

      int C = 0;                       // jobs carried over from the previous phase
      int32_t* cur = list0;
      int32_t* nxt = list1;
      for (int ph = 0; ph < L; ++ph) {
        const int ent_lo = sh.ent[ph], ent_hi = sh.ent[ph + 1];
        const int N = C + (ent_hi - ent_lo);
        if (N == 0) continue;          // an empty class takes no time
        const i64 tau = sh.tau[ph], k = sh.k[ph];
        const i64 len = (simultaneous ? ((N - 1) / k) * tau : slot_offset(N - 1, tau, k)) + tau;

        // ---- pass A: starts, completions, carry list ----
        int C_next = 0;
        for (int r0 = 0; r0 < N; r0 += T) {
          const int r = r0 + tid;
          bool carry = false;
          int pos = 0;
          if (r < N) {
            pos = r < C ? cur[r] : ent_lo + (r - C);
            const int oi = O[seg_lo + pos], si = S[seg_lo + pos];
            const i64 start = base + (simultaneous ? (r / k) * tau : slot_offset(r, tau, k));
            const i64 d = oi < tau ? oi : tau;
            const bool fin = oi <= tau;
            acc.steps += d;
            acc.hmax = max_i64(acc.hmax, start + d);
            const int orig = PERM ? PERM[seg_lo + pos] : seg_lo + pos;
            if (fin) {
              const i64 done = start + oi;
              acc.flow += done - (p.arrival ? p.arrival[lo + orig] : 0);
              if (p.out.job_start) p.out.job_start[job_out + orig] = static_cast<int32_t>(start);
              if (p.out.job_completion) p.out.job_completion[job_out + orig] = static_cast<int32_t>(done);
              if (p.out.job_start64) p.out.job_start64[job_out + orig] = start;
              if (p.out.job_completion64) p.out.job_completion64[job_out + orig] = done;
            } else if (!geometric) {
              ++acc.unfinished;
              if (p.out.job_start) p.out.job_start[job_out + orig] = -1;
              if (p.out.job_completion) p.out.job_completion[job_out + orig] = -1;
              if (p.out.job_start64) p.out.job_start64[job_out + orig] = -1;
              if (p.out.job_completion64) p.out.job_completion64[job_out + orig] = -1;
            } else {
              carry = true;
            }
            if (want_runs && run_count + r < run_cap) {
              const i64 w = run_base + run_count + r;
              if (p.out.run_job) p.out.run_job[w] = orig;
              if (p.out.run_phase) p.out.run_phase[w] = ph;
              if (p.out.run_start) p.out.run_start[w] = start;
              if (p.out.run_len) p.out.run_len[w] = static_cast<int32_t>(d);
              if (p.out.run_s) p.out.run_s[w] = si;
            }
          }
          if (may_carry) {
            int total;
            const int off = block_flag_scan(carry, sh.red32, &total);
            if (carry) nxt[C_next + off] = pos;
            C_next += total;
          }
        }
        run_count += N;

        // ---- pass B: per-round memory of rounds [base, base + len) ----
        if (profile_on) {
          const i64 active = min_i64(N, k + 1);
          if (active * (static_cast<i64>(stats.s_max) + tau) >= (static_cast<i64>(1) << 32)) {
            profile_on = false;
            status |= KVS_EVAL_RANGE;
          }
        }
        if (profile_on) {
          // idle rounds before this phase (window release) hold nothing
          if (prof_cap > 0)
            for (i64 t = written_to + tid; t < base && t < prof_cap; t += T) p.ev.profile[prof_base + t] = 0;
          u32 A_run = 0, B_run = 0;
          const i64 t_end = base + len;
          for (i64 t0 = base; t0 < t_end; t0 += TILE) {
            __syncthreads();
#pragma unroll
            for (int i = 0; i < ITEMS; ++i) { sh.dA[tid + i * T] = 0; sh.dB[tid + i * T] = 0; }
            __syncthreads();
            const i64 u0 = t0 - base;
            const int wlen = static_cast<int>(min_i64(TILE, t_end - t0));
            const i64 v0 = u0 > tau ? u0 - tau : 0;   // runs ending in this tile started at or after v0
            i64 r_lo, r_hi;
            if (simultaneous) {
              r_lo = ceil_div_u(v0, tau) * k;
              r_hi = ceil_div_u(u0 + wlen, tau) * k;
            } else {
              r_lo = ceil_div_u(static_cast<u64>(v0) * k, tau);
              r_hi = ceil_div_u(static_cast<u64>(u0 + wlen) * k, tau);
            }
            if (r_hi > N) r_hi = N;
            for (i64 r = r_lo + tid; r < r_hi; r += T) {
              const int pos = r < C ? cur[r] : ent_lo + static_cast<int>(r - C);
              const int oi = O[seg_lo + pos], si = S[seg_lo + pos];
              const i64 start = base + (simultaneous ? (r / k) * tau : slot_offset(r, tau, k));
              const i64 d = oi < tau ? oi : tau;
              const u32 c = static_cast<u32>(si + 1) - static_cast<u32>(start);  // tokens(t) = c + t while active
              const i64 srel = start - t0, erel = srel + d;
              if (srel >= 0) { atomicAdd(&sh.dA[srel], c); atomicAdd(&sh.dB[srel], 1u); }
              if (erel >= 0 && erel < wlen) { atomicAdd(&sh.dA[erel], 0u - c); atomicAdd(&sh.dB[erel], 0xffffffffu); }
            }
            __syncthreads();
            // prefix sums of both arrays: thread owns ITEMS consecutive rounds
            u32 a[ITEMS], b[ITEMS];
            u32 sa = 0, sb = 0;
#pragma unroll
            for (int i = 0; i < ITEMS; ++i) {
              sa += sh.dA[tid * ITEMS + i]; sb += sh.dB[tid * ITEMS + i];
              a[i] = sa; b[i] = sb;
            }
            u32 ia = sa, ib = sb;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
              const u32 ya = __shfl_up_sync(0xffffffffu, ia, d), yb = __shfl_up_sync(0xffffffffu, ib, d);
              if (static_cast<int>(lane_id()) >= d) { ia += ya; ib += yb; }
            }
            if (lane_id() == 31) { sh.redA[tid >> 5] = ia; sh.redB[tid >> 5] = ib; }
            __syncthreads();
            u32 wa = (lane_id() < WARPS) ? sh.redA[lane_id()] : 0, wb = (lane_id() < WARPS) ? sh.redB[lane_id()] : 0;
            u32 wia = wa, wib = wb;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
              const u32 ya = __shfl_up_sync(0xffffffffu, wia, d), yb = __shfl_up_sync(0xffffffffu, wib, d);
              if (static_cast<int>(lane_id()) >= d) { wia += ya; wib += yb; }
            }
            const u32 offA = A_run + __shfl_sync(0xffffffffu, wia - wa, tid >> 5) + (ia - sa);
            const u32 offB = B_run + __shfl_sync(0xffffffffu, wib - wb, tid >> 5) + (ib - sb);
            A_run += __shfl_sync(0xffffffffu, wia, 31);
            B_run += __shfl_sync(0xffffffffu, wib, 31);
            const u32 tt = static_cast<u32>(t0) + static_cast<u32>(tid * ITEMS);
#pragma unroll
            for (int i = 0; i < ITEMS; ++i) {
              const u32 mem = (offA + a[i]) + (tt + i) * (offB + b[i]);
              if (tid * ITEMS + i < wlen) acc.peak = max(acc.peak, mem);
              sh.dA[tid * ITEMS + i] = mem;
            }
            __syncthreads();
            if (prof_cap > 0)
              for (int i = tid; i < wlen; i += T) {
                const i64 t = t0 + i;
                if (t < prof_cap) p.ev.profile[prof_base + t] = static_cast<int32_t>(sh.dA[i]);
              }
          }
          written_to = t_end;
        }

        base += len;
        __syncthreads();               // carry list complete before it is read as `cur`
        int32_t* tmp = cur; cur = nxt; nxt = tmp;
        C = C_next;
        if (C == 0 && ent_hi == nseg) break;   // nothing left in this window
      }
      seg_lo = seg_hi;
    }

    // ---- scalars ----
    const i64 flow = block_sum(acc.flow, sh.red64);
    const i64 steps = block_sum(acc.steps, sh.red64);
    const i64 hmax = block_max(acc.hmax, sh.red64, static_cast<i64>(0));
    const int unfinished = block_sum(acc.unfinished, sh.red32);
    const u32 peak = block_max(acc.peak, sh.redA, 0u);
    if (tid == 0) {
      const bool skipped = (status & (KVS_EVAL_INFEASIBLE | KVS_EVAL_BAD_INPUT)) != 0;
      if (!skipped) {
        if (want32 && hmax > 0x7fffffffll) status |= KVS_EVAL_RANGE;
        if (want_runs && run_count > run_cap) status |= KVS_EVAL_CAPACITY;
        if (prof_cap > 0 && hmax > prof_cap) status |= KVS_EVAL_CAPACITY;   // capacity 0 = profile not wanted
      }
      const bool have_peak = p.do_profile && profile_on && !skipped;
      if (p.ev.peak) p.ev.peak[e] = have_peak ? static_cast<i64>(peak) : -1;
      if (p.ev.flow) p.ev.flow[e] = flow;
      if (p.ev.job_steps) p.ev.job_steps[e] = steps;
      if (p.ev.horizon) p.ev.horizon[e] = hmax;
      if (p.ev.n_unfinished) p.ev.n_unfinished[e] = unfinished;
      if (p.ev.feasible) p.ev.feasible[e] = (have_peak && !(status & KVS_EVAL_RANGE) && static_cast<i64>(peak) <= M) ? 1 : 0;
      if (p.ev.status) p.ev.status[e] = status;
      if (p.out.n_runs) p.out.n_runs[e] = run_count;
    }
  }
}

}  // namespace

static size_t build_smem_bytes() { return sizeof(Shared); }

int kvs_build_ctas_per_sm() {
  int n = 0;
  cudaFuncSetAttribute(k_build_eval, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(build_smem_bytes()));
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k_build_eval, KVS_EVAL_THREADS, build_smem_bytes()) != cudaSuccess) n = 1;
  return n < 1 ? 1 : n;
}

cudaError_t kvs_launch_build(const BuildParams& p, int grid, cudaStream_t stream) {
  if (p.P <= 0) return cudaSuccess;
  cudaError_t err = cudaFuncSetAttribute(k_build_eval, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(build_smem_bytes()));
  if (err != cudaSuccess) return err;
  k_build_eval<<<grid, KVS_EVAL_THREADS, build_smem_bytes(), stream>>>(p);
  return cudaGetLastError();
}
