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
//   3. walks the rounds of the phase tile by tile.  Ranks start in nondecreasing rounds, so the
//      runs that start inside a tile are a contiguous rank range and every run is visited exactly
//      once: its start and completion are written, it is appended to the carry list if killed, and
//      its two events go into the difference arrays - the constant term s+1-start and the slope 1 -
//      of the current tile or of the next one (a two-tile ring in shared memory; only slices longer
//      than a tile need a second look for ends that land further ahead).  Each array is
//      prefix-summed once, memory(t) = A(t) + t*B(t) (Eq. Memory-Feasibility), the peak is reduced
//      and the profile is stored straight from registers, 16 bytes at a time;
//   4. reduces flow time, job-steps, horizon and the number of unfinished jobs.
//
// The difference arrays and their sums are kept modulo 2^32.  Every intermediate may wrap, the
// final memory(t) is exact whenever it is below 2^32, which a per-phase bound guarantees
// (otherwise the evaluation reports KVS_EVAL_RANGE and skips the profile).
#include "kvs_events.cuh"
#include "kvs_ladder.cuh"

namespace {

constexpr int T = KVS_EVAL_THREADS;
constexpr int ITEMS = KVS_EVAL_ITEMS;      // 8 rounds per thread and tile: two 16-byte vectors
constexpr int TILE = KVS_TILE;
constexpr int WARPS = T / 32;
constexpr int RPT = 4;                     // consecutive ranks per thread in the run loop
constexpr int CHUNK = T * RPT;
constexpr int VEC = ITEMS / 4;              // 16-byte vectors per thread and tile
static_assert(ITEMS % 4 == 0 && (ITEMS & (ITEMS - 1)) == 0, "rounds per thread: a power of two, whole vectors");

// Shared-memory word of round e of a tile.  Thread t owns rounds ITEMS*t .. ITEMS*t + ITEMS-1 as VEC
// 4-word vectors; vector c of thread t sits at vector index c*T + t, so a warp's vector access is
// contiguous.
__device__ __forceinline__ int slot(int e) { return ((((e >> 2) % VEC) * T + e / ITEMS) << 2) + (e & 3); }

struct Shared {
  uint4 dA[2][TILE / 4];    // two-tile ring: difference arrays of the constant terms
  uint4 dB[2][TILE / 4];    //                and of the slopes
  i64 tau[KVS_MAX_PHASES];
  i64 k[KVS_MAX_PHASES];
  i64 pbase[KVS_MAX_PHASES];    // first round of each phase of the current window
  int ent[KVS_MAX_PHASES + 1];  // class boundaries in key order: entrants of phase p are [ent[p], ent[p+1])
  u128 pw_a[KVS_MAX_PHASES + 1];
  u128 pw_b[KVS_MAX_PHASES + 1];
  i64 red64[32];
  u32 redA[32], redB[32];
  int red32[32];
  int n_phases;
  int seg_end;
  i64 next_eval;
};

// Adds (c, one) at word idx for every lane with idx >= 0.  With `combine`, lanes of a warp that
// target the same word (runs that start or end in the same round - thousands of them in a short
// slice with high parallelism) are summed first, so the word receives one atomic per warp.
__device__ __forceinline__ void add_event(u32* dA, u32* dB, int idx, u32 c, u32 one, bool combine) {
  if (combine) {
    const u32 peers = __match_any_sync(0xffffffffu, idx);
    if (idx >= 0) {
      const u32 csum = __reduce_add_sync(peers, c);
      if ((peers & lanemask_lt()) == 0) {
        atomicAdd(&dA[idx], csum);
        atomicAdd(&dB[idx], one * static_cast<u32>(__popc(peers)));
      }
    }
  } else if (idx >= 0) {
    atomicAdd(&dA[idx], c);
    atomicAdd(&dB[idx], one);
  }
}

// Geometric ladder by warp 0.  Leaves the number of phases in sh.n_phases (0 = too many).
// Parallelism of a phase: the largest memory-feasible one of Procedure StaggeredPipelineSchedule (Eq.
// max-parallelism), or the batch size of the simultaneous schedule; 0 if not even one job fits.
__device__ __forceinline__ i64 phase_parallelism(i64 tau, i64 s, i64 M, bool batches) {
  if (s + tau > M) return 0;
  return batches ? M / (s + tau) : max_parallelism64(tau, s, M);
}

__device__ void build_ladder(Shared& sh, i64 X, int a, int b, i64 beta0, i64 s_bar, i64 M, bool batches) {
  ladder_phases(sh, X, a, b, beta0, [=](i64 t) { return phase_parallelism(t, s_bar, M, batches); });
}

// Exclusive block scan of a small per-thread count; returns this thread's offset, total in *total.
__device__ __forceinline__ int block_count_scan(int v, int* red32, int* total) {
  int incl = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, incl, d);
    if (static_cast<int>(lane_id()) >= d) incl += y;
  }
  const int warp = threadIdx.x >> 5;
  __syncthreads();
  if (lane_id() == 31) red32[warp] = incl;
  __syncthreads();
  const int w = (lane_id() < WARPS) ? red32[lane_id()] : 0;
  int wi = w;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, wi, d);
    if (static_cast<int>(lane_id()) >= d) wi += y;
  }
  *total = __shfl_sync(0xffffffffu, wi, 31);
  return __shfl_sync(0xffffffffu, wi - w, warp) + (incl - v);
}

struct Acc {
  i64 flow = 0, steps = 0, hmax = 0;
  int unfinished = 0;
  u32 peak = 0;             // from the profile tiles
  i64 peak64 = 0;           // from the event form
};

// Everything one phase needs that does not change while it runs.
struct Phase {
  i64 base, tau, k, t_end;
  i64 qt, rt;               // tau = qt * k + rt: the start offset advances by qt (+1 on carry) per rank
  int N, C, ent_lo, ph, seg_lo;
  bool simultaneous, geometric, may_carry, profile_on, combine;
  bool dense;               // several runs start per round and tau < TILE: events are combined per round
};

// Per-evaluation pointers and output windows.
struct EvalCtx {
  const int32_t* S;       // prompt lengths in schedule order (of the instance)
  const int32_t* O;       // response lengths in schedule order
  const int32_t* PERM;    // schedule order -> job index inside the instance, or NULL (identity)
  const i64* ARR;         // arrivals of the instance, or NULL
  const int32_t* O_JOB;   // response lengths in original job order
  const int32_t* KEY_JOB; // estimates in original job order, or NULL (exact keys)
  const int32_t* IPERM;   // job index -> position in schedule order, or NULL (identity)
  int32_t* fin_rank;      // scratch of this CTA: rank of a job in the phase that completes it
  i64 job_out;            // offset of the evaluation's per-job block
  i64 run_base, run_cap, run_count;
  i64 prof_base, prof_cap;
  bool want_runs;
};

// Visits ranks [ra, rb) of a phase once: outputs, carry list, and (if the profile is on) the two
// events of every run.  All of these runs start inside the tile with origin t0; `buf` is the ring
// half of that tile.  Returns the new length of the carry list.
template <bool WIDE> struct OffsetType { typedef int type; };
template <> struct OffsetType<true> { typedef i64 type; };

// SIM, CARRY, EVENTS, RUNS: simultaneous starts, carried jobs possible, events wanted, explicit run
// list wanted.  WIDE: the phase is 2^30 rounds or longer, offsets inside it need 64 bits; otherwise
// all per-run arithmetic is 32-bit (ranks, slice lengths and parallelism are below 2^31).
template <bool SIM, bool CARRY, bool EVENTS, bool RUNS, bool WIDE>
__device__ __forceinline__ int process_runs_t(const BuildParams& p, Shared& sh, const EvalCtx& ec, const Phase& P,
                                              const int32_t* cur, int32_t* nxt, int C_next, int ra, int rb,
                                              i64 t0, int buf, Acc& acc) {
  typedef typename OffsetType<WIDE>::type off_t;
  const int tid = threadIdx.x;
  u32* const dA = reinterpret_cast<u32*>(sh.dA);
  u32* const dB = reinterpret_cast<u32*>(sh.dB);
  const u32 tau = static_cast<u32>(P.tau), k = static_cast<u32>(P.k);
  const u32 qt = static_cast<u32>(P.qt), rt = static_cast<u32>(P.rt);
  const off_t trel = static_cast<off_t>(t0 - P.base);        // tile origin relative to the phase
  const off_t len = static_cast<off_t>(P.t_end - P.base);
  const u32 cbase = static_cast<u32>(P.base);
  off_t far = 0;                                             // largest run end seen, relative to the phase
  for (int c0 = ra; c0 < rb;) {
    // short ranges are spread one run per thread; long ones give each thread consecutive ranks
    const int left = rb - c0;
    const int rpt = left > 2 * T ? RPT : (left > T ? 2 : 1);
    const int r_first = c0 + tid * rpt;
    c0 += T * rpt;
    int cpos[RPT];
    u32 cmask = 0;
    if (r_first - static_cast<int>(lane_id()) * rpt < rb) {   // warps past the end of the range skip the visit
      // gather first, all loads of a stage in flight together: position -> (o, s) -> job index
      int pos_[RPT], o_[RPT], s_[RPT], orig_[RPT];
#pragma unroll
      for (int j = 0; j < RPT; ++j) {
        const int r = r_first + j;
        pos_[j] = (j < rpt && r < rb) ? (r < P.C ? cur[r] : P.ent_lo + (r - P.C)) : -1;
      }
#pragma unroll
      for (int j = 0; j < RPT; ++j) {
        o_[j] = pos_[j] >= 0 ? __ldg(ec.O + P.seg_lo + pos_[j]) : 0;
        s_[j] = pos_[j] >= 0 ? __ldg(ec.S + P.seg_lo + pos_[j]) : 0;
      }
      if (RUNS) {
#pragma unroll
        for (int j = 0; j < RPT; ++j)   // only the explicit run list names the job
          orig_[j] = pos_[j] >= 0 ? (ec.PERM ? __ldg(ec.PERM + P.seg_lo + pos_[j]) : P.seg_lo + pos_[j]) : 0;
      }
      off_t q = 0;      // start offset of the current rank inside the phase
      u32 rem = 0;      // and the remainder that advances it
      if (r_first < rb) {
        if (SIM) {
          const u32 b = static_cast<u32>(r_first) / k;
          q = static_cast<off_t>(b) * static_cast<off_t>(tau);
          rem = static_cast<u32>(r_first) - b * k;
        } else {
          u64 dq_, dr_;
          divmod_u(static_cast<u64>(r_first) * tau, k, &dq_, &dr_);
          q = static_cast<off_t>(dq_);
          rem = static_cast<u32>(dr_);
        }
      }
      u32 steps = 0;
      // Dense phases (several runs start per round): the runs of a lane that start in the round of
      // its first run are summed in registers, then equal rounds - contiguous lanes, because
      // consecutive ranks start in nondecreasing rounds - are summed across the warp with a
      // segmented scan, and one lane per round issues the atomics.  Runs that hold their whole
      // slot end together (start + tau), so their end events are combined the same way.
      const bool dense = EVENTS && !SIM && P.dense;
      int seg = 0x7fffffff;                 // round (relative to the tile) of the lane's segment
      u32 seg_all = 0, seg_full = 0;        // sums of c over the segment: all runs / runs holding the whole slot
      u32 seg_cnt = 0;                      // counts: all | full << 16
#pragma unroll
      for (int j = 0; j < RPT; ++j) {
        int sidx = -1, eidx = -1;
        u32 c = 0;
        cpos[j] = 0;
        if (pos_[j] >= 0) {
          const int r = r_first + j;
          const u32 oi = static_cast<u32>(o_[j]);
          const u32 d = oi < tau ? oi : tau;
          const bool fin = oi <= tau;
          const off_t end = q + static_cast<off_t>(d);
          if (CARRY) {   // without carried jobs there is one run per job, accounted in write_jobs
            steps += d;
            far = end > far ? end : far;
          }
          // Per-job results are written later, in original job order (write_jobs); a job that
          // completes among carried ones leaves its rank for that pass.
          if (CARRY && fin) ec.fin_rank[P.seg_lo + pos_[j]] = r;
          if (RUNS && ec.run_count + r < ec.run_cap) {
            const i64 w = ec.run_base + ec.run_count + r;
            if (p.out.run_job) p.out.run_job[w] = orig_[j];
            if (p.out.run_phase) p.out.run_phase[w] = P.ph;
            if (p.out.run_start) p.out.run_start[w] = P.base + q;
            if (p.out.run_len) p.out.run_len[w] = static_cast<int32_t>(d);
            if (p.out.run_s) p.out.run_s[w] = s_[j];
          }
          if (CARRY && !fin) { cpos[j] = pos_[j]; cmask |= 1u << j; }
          if (EVENTS) {
            c = static_cast<u32>(s_[j] + 1) - cbase - static_cast<u32>(q);   // tokens(t) = c + t while active
            const int srel = static_cast<int>(q - trel);
            sidx = buf * TILE + slot(srel);
            if (end < len) {                                   // an end at the phase end is never read
              const u32 erel = static_cast<u32>(srel) + d;
              if (erel < TILE) eidx = buf * TILE + slot(static_cast<int>(erel));
              else if (erel < 2 * TILE) eidx = (buf ^ 1) * TILE + slot(static_cast<int>(erel - TILE));
            }
            if (dense) {
              if (seg == 0x7fffffff) seg = srel;
              if (srel == seg) {
                seg_all += c; seg_cnt += 1u;
                sidx = -1;
                if (d == tau) { seg_full += c; seg_cnt += 1u << 16; eidx = -1; }
              }
            }
          }
          if (SIM) { if (++rem == k) { rem = 0; q += static_cast<off_t>(tau); } }
          else { rem += rt; q += static_cast<off_t>(qt); if (rem >= k) { rem -= k; ++q; } }
        }
        if (EVENTS) {
          add_event(dA, dB, sidx, c, 1u, P.combine);
          add_event(dA, dB, eidx, 0u - c, 0xffffffffu, P.combine);
        }
      }
      if (dense) {
        int key = seg;
        u32 va = seg_all, vf = seg_full, vn = seg_cnt;
#pragma unroll
        for (int dd = 1; dd < 32; dd <<= 1) {
          const int kk = __shfl_up_sync(0xffffffffu, key, dd);
          const u32 ya = __shfl_up_sync(0xffffffffu, va, dd), yf = __shfl_up_sync(0xffffffffu, vf, dd);
          const u32 yn = __shfl_up_sync(0xffffffffu, vn, dd);
          if (static_cast<int>(lane_id()) >= dd && kk == key) { va += ya; vf += yf; vn += yn; }
        }
        const int next_key = __shfl_down_sync(0xffffffffu, key, 1);
        if (key != 0x7fffffff && (lane_id() == 31 || next_key != key)) {   // last lane of its round
          const int si = buf * TILE + slot(key);
          atomicAdd(&dA[si], va);
          atomicAdd(&dB[si], vn & 0xffffu);
          const u32 n_full = vn >> 16;
          if (n_full && static_cast<off_t>(key) + trel + static_cast<off_t>(tau) < len) {
            const u32 erel = static_cast<u32>(key) + tau;      // tau < TILE in dense phases
            const int ei = erel < TILE ? buf * TILE + slot(static_cast<int>(erel))
                                       : (buf ^ 1) * TILE + slot(static_cast<int>(erel - TILE));
            atomicAdd(&dA[ei], 0u - vf);
            atomicAdd(&dB[ei], 0u - n_full);
          }
        }
      }
      acc.steps += steps;
    }
    if (CARRY) {
      int total;
      int off = C_next + block_count_scan(__popc(cmask), sh.red32, &total);
#pragma unroll
      for (int j = 0; j < RPT; ++j)
        if (cmask >> j & 1u) nxt[off++] = cpos[j];
      C_next += total;
    }
  }
  acc.hmax = max_i64(acc.hmax, P.base + static_cast<i64>(far));
  return C_next;
}

// Picks the specialisation: each variant carries only the registers and branches it needs.
template <bool EVENTS, bool WIDE>
__device__ __forceinline__ int process_runs_w(const BuildParams& p, Shared& sh, const EvalCtx& ec, const Phase& P,
                                              const int32_t* cur, int32_t* nxt, int C_next, int ra, int rb,
                                              i64 t0, int buf, Acc& acc) {
  if (P.simultaneous && P.may_carry) {   // simultaneous batches inside the phases of a geometric algorithm with carried jobs
    if (ec.want_runs) return process_runs_t<true, true, EVENTS, true, WIDE>(p, sh, ec, P, cur, nxt, C_next, ra, rb, t0, buf, acc);
    return process_runs_t<true, true, EVENTS, false, WIDE>(p, sh, ec, P, cur, nxt, C_next, ra, rb, t0, buf, acc);
  }
  if (ec.want_runs) {
    if (P.simultaneous) return process_runs_t<true, false, EVENTS, true, WIDE>(p, sh, ec, P, cur, nxt, C_next, ra, rb, t0, buf, acc);
    if (P.may_carry) return process_runs_t<false, true, EVENTS, true, WIDE>(p, sh, ec, P, cur, nxt, C_next, ra, rb, t0, buf, acc);
    return process_runs_t<false, false, EVENTS, true, WIDE>(p, sh, ec, P, cur, nxt, C_next, ra, rb, t0, buf, acc);
  }
  if (P.simultaneous) return process_runs_t<true, false, EVENTS, false, WIDE>(p, sh, ec, P, cur, nxt, C_next, ra, rb, t0, buf, acc);
  if (P.may_carry) return process_runs_t<false, true, EVENTS, false, WIDE>(p, sh, ec, P, cur, nxt, C_next, ra, rb, t0, buf, acc);
  return process_runs_t<false, false, EVENTS, false, WIDE>(p, sh, ec, P, cur, nxt, C_next, ra, rb, t0, buf, acc);
}

template <bool EVENTS>
__device__ __forceinline__ int process_runs(const BuildParams& p, Shared& sh, const EvalCtx& ec, const Phase& P,
                                            const int32_t* cur, int32_t* nxt, int C_next, i64 ra, i64 rb,
                                            i64 t0, int buf, Acc& acc) {
  const int a = static_cast<int>(ra), b = static_cast<int>(rb);
  if (P.t_end - P.base >= (static_cast<i64>(1) << 30))
    return process_runs_w<EVENTS, true>(p, sh, ec, P, cur, nxt, C_next, a, b, t0, buf, acc);
  return process_runs_w<EVENTS, false>(p, sh, ec, P, cur, nxt, C_next, a, b, t0, buf, acc);
}

// Prefix-sums one tile of the ring, turns it into memory(t), reduces the peak, stores the profile
// and leaves the tile zeroed for its next use.  Contains one __syncthreads.
__device__ __forceinline__ void scan_tile(Shared& sh, int buf, i64 t0, int wlen, i64 first_round,
                                          u32& A_run, u32& B_run, Acc& acc, const EvalCtx& ec, int32_t* profile) {
  const int tid = threadIdx.x;
  const uint4 zero = make_uint4(0, 0, 0, 0);
  u32 a[ITEMS], b[ITEMS];
#pragma unroll
  for (int v = 0; v < VEC; ++v) {
    const uint4 x = sh.dA[buf][v * T + tid], y = sh.dB[buf][v * T + tid];
    sh.dA[buf][v * T + tid] = zero;
    sh.dB[buf][v * T + tid] = zero;
    a[4 * v] = x.x; a[4 * v + 1] = x.y; a[4 * v + 2] = x.z; a[4 * v + 3] = x.w;
    b[4 * v] = y.x; b[4 * v + 1] = y.y; b[4 * v + 2] = y.z; b[4 * v + 3] = y.w;
  }
#pragma unroll
  for (int i = 1; i < ITEMS; ++i) { a[i] += a[i - 1]; b[i] += b[i - 1]; }
  const u32 sa = a[ITEMS - 1], sb = b[ITEMS - 1];
  u32 ia = sa, ib = sb;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const u32 ya = __shfl_up_sync(0xffffffffu, ia, d), yb = __shfl_up_sync(0xffffffffu, ib, d);
    if (static_cast<int>(lane_id()) >= d) { ia += ya; ib += yb; }
  }
  if (lane_id() == 31) { sh.redA[tid >> 5] = ia; sh.redB[tid >> 5] = ib; }
  __syncthreads();
  const u32 wa = (lane_id() < WARPS) ? sh.redA[lane_id()] : 0, wb = (lane_id() < WARPS) ? sh.redB[lane_id()] : 0;
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
  const int e0 = tid * ITEMS;
  const u32 tt = static_cast<u32>(t0) + static_cast<u32>(e0);
  u32 mem[ITEMS];
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) {
    mem[i] = (offA + a[i]) + (tt + i) * (offB + b[i]);
    if (e0 + i < wlen) acc.peak = max(acc.peak, mem[i]);
  }
  if (ec.prof_cap > 0) {
    // rounds [lo, hi) of this tile belong to the phase and fit the caller's capacity
    const i64 lo = first_round, hi = min_i64(t0 + wlen, ec.prof_cap);
#pragma unroll
    for (int v = 0; v < VEC; ++v) {
      const i64 rs = t0 + e0 + 4 * v;
      int32_t* dst = profile + ec.prof_base + rs;
      if (rs >= lo && rs + 4 <= hi) {
        *reinterpret_cast<int4*>(dst) = make_int4(static_cast<int>(mem[4 * v]), static_cast<int>(mem[4 * v + 1]),
                                                  static_cast<int>(mem[4 * v + 2]), static_cast<int>(mem[4 * v + 3]));
      } else if (rs + 4 > lo && rs < hi) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (rs + i >= lo && rs + i < hi) dst[i] = static_cast<int>(mem[4 * v + i]);
      }
    }
  }
}

// Slices longer than a tile: ends that land two or more tiles after the run's start were not
// inserted when the run was visited; pick them up when their tile comes.
__device__ __forceinline__ void insert_far_ends(Shared& sh, const EvalCtx& ec, const Phase& P, const int32_t* cur,
                                                i64 t0_first, i64 t0, int wlen, int buf) {
  const i64 u0 = t0 - P.base;
  if (u0 <= TILE) return;
  const i64 lo = u0 > P.tau ? u0 - P.tau : 0, hi = u0 - TILE;   // start offsets of the candidates: [lo, hi)
  i64 r_lo, r_hi;
  if (P.simultaneous) { r_lo = ceil_div_u(lo, P.tau) * P.k; r_hi = ceil_div_u(hi, P.tau) * P.k; }
  else { r_lo = ceil_div_u(static_cast<u64>(lo) * P.k, P.tau); r_hi = ceil_div_u(static_cast<u64>(hi) * P.k, P.tau); }
  if (r_hi > P.N) r_hi = P.N;
  u32* const dA = reinterpret_cast<u32*>(sh.dA);
  u32* const dB = reinterpret_cast<u32*>(sh.dB);
  for (i64 r0 = r_lo; r0 < r_hi; r0 += T) {
    const i64 r = r0 + threadIdx.x;
    int eidx = -1;
    u32 c = 0;
    if (r < r_hi) {
      const int pos = r < P.C ? cur[r] : P.ent_lo + static_cast<int>(r - P.C);
      const int oi = ec.O[P.seg_lo + pos], si = ec.S[P.seg_lo + pos];
      const i64 start = P.base + (P.simultaneous ? (r / P.k) * P.tau : slot_offset(r, P.tau, P.k));
      const i64 end = start + (oi < P.tau ? oi : P.tau);
      const i64 ts = t0_first + ((start - t0_first) / TILE) * TILE;   // origin of the tile the run started in
      if (end >= ts + 2 * TILE && end >= t0 && end < t0 + wlen && end < P.t_end) {
        c = static_cast<u32>(si + 1) - static_cast<u32>(start);
        eidx = buf * TILE + slot(static_cast<int>(end - t0));
      }
    }
    add_event(dA, dB, eidx, 0u - c, 0xffffffffu, false);
  }
}

// Per-job results of one window, written in original job order so that the stores are contiguous.
// The phase that completes job j is the later of its key's class and the class of o_j
// (class(x) = first p with tau_p >= x); its rank there is its position inside the class when no
// jobs are carried, else the rank noted when it completed.  Also accumulates the flow time.
__device__ __forceinline__ void write_jobs(const BuildParams& p, const Shared& sh, const EvalCtx& ec, int family, bool simultaneous,
                                           int L, i64 X, int seg_lo, int seg_hi, bool may_carry, Acc& acc) {
  const bool geometric = family == KVS_GBA || family == KVS_GSA;
  for (int j = seg_lo + threadIdx.x; j < seg_hi; j += T) {
    const int oj = __ldg(ec.O_JOB + j);
    const int pos = ec.IPERM ? __ldg(ec.IPERM + j) : j;
    int ph = 0;
    bool fin = true;
    if (geometric) {
      i64 x = oj;
      if (family == KVS_GBA && ec.KEY_JOB) {          // class of the estimate, clipped to [1, X]
        i64 kj = __ldg(ec.KEY_JOB + j);
        kj = kj < 1 ? 1 : (kj > X ? X : kj);
        x = kj > x ? kj : x;                          // classes are monotone: max of classes = class of max
      }
      int a = 0, b = L - 1;                           // tau_(L-1) = X >= x
      while (a < b) { const int m = (a + b) >> 1; if (sh.tau[m] >= x) b = m; else a = m + 1; }
      ph = a;
    } else {
      fin = oj <= sh.tau[0];
    }
    i64 start = -1, done = -1;
    {
      const i64 rank = may_carry ? static_cast<i64>(ec.fin_rank[pos]) : static_cast<i64>(pos - seg_lo - sh.ent[ph]);
      const i64 tau = sh.tau[ph], k = sh.k[ph];
      const i64 st = sh.pbase[ph] + (simultaneous ? (rank / k) * tau : slot_offset(rank, tau, k));
      if (!may_carry) {   // exactly one run per job: its length and end are accounted here, not in the visit
        const i64 d = fin ? oj : tau;
        acc.steps += d;
        acc.hmax = max_i64(acc.hmax, st + d);
      }
      if (fin) {
        start = st;
        done = st + oj;
        acc.flow += done - (ec.ARR ? __ldg(ec.ARR + j) : 0);
      } else {
        ++acc.unfinished;
      }
    }
    if (p.out.job_start) p.out.job_start[ec.job_out + j] = static_cast<int32_t>(start);
    if (p.out.job_completion) p.out.job_completion[ec.job_out + j] = static_cast<int32_t>(done);
    if (p.out.job_start64) p.out.job_start64[ec.job_out + j] = start;
    if (p.out.job_completion64) p.out.job_completion64[ec.job_out + j] = done;
  }
}

__global__ void __launch_bounds__(KVS_EVAL_THREADS, KVS_EVAL_MIN_CTAS) k_build_eval(BuildParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Shared& sh = *reinterpret_cast<Shared*>(smem_raw);
  const int tid = threadIdx.x;
  int32_t* const list0 = p.lists + static_cast<i64>(blockIdx.x) * 2 * p.max_jobs;
  int32_t* const list1 = list0 + p.max_jobs;
  {  // the ring starts zeroed and every tile leaves its half zeroed
    const uint4 zero = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < 2 * (TILE / 4); i += T) { (&sh.dA[0][0])[i] = zero; (&sh.dB[0][0])[i] = zero; }
  }

  for (;;) {
    __syncthreads();  // previous evaluation done with shared memory
    if (tid == 0) sh.next_eval = static_cast<i64>(atomicAdd(reinterpret_cast<ull*>(p.counter), 1ull));
    __syncthreads();
    const i64 slot_no = sh.next_eval;
    if (slot_no >= (p.eval_list ? static_cast<i64>(*p.eval_count) : p.P)) break;
    const i64 e = p.eval_list ? p.eval_list[slot_no] : slot_no;
    const kvs_setting st = p.settings[e];
    const i64 lo = p.job_off[st.instance];
    const InstStats stats = p.stats[st.instance];
    const int n = stats.flags ? 0 : static_cast<int>(p.job_off[st.instance + 1] - lo);
    const i64 M = st.M;
    const i64 s_bar = st.s_bar >= 0 ? st.s_bar : stats.s_max;
    const i64 X = M - s_bar;
    const int family = st.family;
    const bool geometric = family == KVS_GBA || family == KVS_GSA;
    // variants inside the geometric classes: simultaneous batches as the subroutine of every phase; the
    // parallelism of a phase sized by the longest prompt among its participants
    const bool simultaneous = family == KVS_SIMS || (geometric && st.subroutine == 1);
    const bool per_class = geometric && st.per_class_s == 1;
    const bool keyed = !(family == KVS_GSA && p.key == nullptr);  // plain GSA keeps the index order
    const int32_t* const KEY = p.key ? p.sorted_key + lo : p.sorted_o + lo;

    EvalCtx ec;
    ec.S = (keyed ? p.sorted_s : p.s) + lo;
    ec.O = (keyed ? p.sorted_o : p.o) + lo;
    ec.PERM = keyed ? p.perm + lo : nullptr;
    ec.ARR = p.arrival ? p.arrival + lo : nullptr;
    ec.O_JOB = p.o + lo;
    ec.KEY_JOB = p.key ? p.key + lo : nullptr;
    ec.IPERM = keyed ? p.iperm + lo : nullptr;
    ec.fin_rank = p.fin_rank + static_cast<i64>(blockIdx.x) * p.max_jobs;
    ec.job_out = p.out.job_out_off ? p.out.job_out_off[e] : 0;
    ec.run_base = p.out.run_off ? p.out.run_off[e] : 0;
    ec.run_cap = p.out.run_off ? p.out.run_off[e + 1] - ec.run_base : 0;
    ec.want_runs = p.out.run_off && (p.out.run_job || p.out.run_phase || p.out.run_start || p.out.run_len || p.out.run_s);
    ec.prof_base = p.ev.profile_off ? p.ev.profile_off[e] : 0;
    ec.prof_cap = (p.ev.profile && p.ev.profile_off) ? p.ev.profile_off[e + 1] - ec.prof_base : 0;
    ec.run_count = 0;
    const bool want32 = p.out.job_start || p.out.job_completion;

    int status = stats.flags;
    if (!status && (X < 1 || stats.o_max > X)) status = KVS_EVAL_INFEASIBLE;
    if (!status && geometric) {
      if (tid < 32) build_ladder(sh, X, st.alpha_num, st.alpha_den, st.beta0, s_bar, M, simultaneous);
      __syncthreads();
      if (sh.n_phases == 0) status = KVS_EVAL_RANGE;
    }
    bool profile_on = p.do_profile != 0;

    Acc acc;
    i64 base = 0;          // first round of the next phase
    i64 written_to = 0;    // profile rounds [0, written_to) have been written

    int seg_lo = 0;
    while (!status && seg_lo < n) {
      // ---- window = offline sub-instance [seg_lo, seg_hi) ----
      if (tid == 0) {
        int end = n;
        if (p.window > 0 && p.arrival) {
          const i64 limit = (ec.ARR[seg_lo] / p.window + 1) * p.window;
          int a = seg_lo + 1, b = n;
          while (a < b) { int m = (a + b) >> 1; if (ec.ARR[m] < limit) a = m + 1; else b = m; }
          end = a;
        }
        sh.seg_end = end;
      }
      __syncthreads();
      const int seg_hi = sh.seg_end;
      const int nseg = seg_hi - seg_lo;
      if (p.window > 0 && p.arrival) base = max_i64(base, (ec.ARR[seg_lo] / p.window + 1) * p.window);

      int L = 1;
      if (geometric) {
        L = sh.n_phases;
        // class boundaries: entrants of phase q-1 have clip(key) <= tau_(q-1) and > tau_(q-2)
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
        if (k <= 0) k = simultaneous ? M / (s_bar + tau) : (s_bar + tau <= M ? max_parallelism64(tau, s_bar, M) : 0);
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
        Phase P;
        if (tid == 0) sh.pbase[ph] = base;   // read by write_jobs after the window's last barrier
        P.base = base; P.tau = sh.tau[ph]; P.k = sh.k[ph];
        if (per_class) {
          // longest prompt among this phase's participants: the carried jobs and the entrants
          i64 s_p = 0;
          for (int r = tid; r < N; r += T) {
            const int pos = r < C ? cur[r] : ent_lo + (r - C);
            s_p = max_i64(s_p, __ldg(ec.S + seg_lo + pos));
          }
          s_p = block_max(s_p, sh.red64, static_cast<i64>(0));
          P.k = phase_parallelism(P.tau, s_p, M, simultaneous);
          __syncthreads();                   // every thread has read the old entry
          if (tid == 0) sh.k[ph] = P.k;      // read by write_jobs after the window's last barrier
        }
        if (P.k < 1) { status = KVS_EVAL_INFEASIBLE; break; }
        P.N = N; P.C = C; P.ent_lo = ent_lo; P.ph = ph; P.seg_lo = seg_lo;
        P.simultaneous = simultaneous; P.geometric = geometric;
        P.may_carry = geometric && (family == KVS_GSA || p.key != nullptr);
        // Combining equal targets inside a warp (match + reduce) costs more than the serialised
        // shared-memory atomics it saves unless a whole warp hits one word: only whole simultaneous
        // batches do that.
        P.combine = simultaneous && P.k >= 32;
        P.dense = !simultaneous && P.tau < TILE && P.k >= 4 * P.tau;
        {
          u64 a_, b_;
          divmod_u(static_cast<u64>(P.tau), static_cast<u64>(P.k), &a_, &b_);
          P.qt = static_cast<i64>(a_); P.rt = static_cast<i64>(b_);
        }
        const i64 len = (simultaneous ? static_cast<i64>(ceil_div_u(N, P.k) - 1) * P.tau : slot_offset(N - 1, P.tau, P.k)) + P.tau;
        P.t_end = base + len;
        // SPS / SimS in exact key order with no profile wanted: the peak comes from the run ends
        // (kvs_events.cuh), no rounds are walked
        const bool event_form = profile_on && !geometric && p.prefix_s != nullptr && ec.prof_cap == 0;
        if (profile_on && !event_form &&
            min_i64(N, P.k + 1) * (static_cast<i64>(stats.s_max) + P.tau) >= (static_cast<i64>(1) << 32)) {
          profile_on = false;
          status |= KVS_EVAL_RANGE;
        }
        P.profile_on = profile_on && !event_form;

        int C_next = 0;
        if (!P.profile_on) {
          if (P.may_carry || ec.want_runs)   // otherwise write_jobs does everything a run needs
            C_next = process_runs<false>(p, sh, ec, P, cur, nxt, 0, 0, N, 0, 0, acc);
          if (event_form) {
            const i64* const ps = p.prefix_s + lo + st.instance + seg_lo;
            const i64 per = (static_cast<i64>(N) + T - 1) / T;
            const i64 i0 = min_i64(N, tid * per), i1 = min_i64(N, i0 + per);
            u64 unused_flow = 0;
            const i64 pk = simultaneous ? sims_range_peak(ec.O + seg_lo, ps, N, P.tau, P.k, i0, i1, &unused_flow)
                                        : sps_range_peak(ec.O + seg_lo, ps, N, P.tau, P.k, i0, i1, &unused_flow);
            acc.peak64 = max_i64(acc.peak64, pk);
          }
        } else {
          // idle rounds before this phase (window release) hold nothing
          if (ec.prof_cap > 0)
            for (i64 t = written_to + tid; t < base && t < ec.prof_cap; t += T) p.ev.profile[ec.prof_base + t] = 0;
          // tile origins keep the profile stores 16-byte aligned
          const i64 t0_first = base - ((ec.prof_base + base) & 3);
          u32 A_run = 0, B_run = 0;
          i64 r_next = 0;
          int buf = 0;
          // Ranks that start before offset u: ceil(u*k/tau) (SPS) or ceil(u/tau)*k (SimS).  The tile
          // ends advance by TILE, so the quotient and remainder of u*mult/tau are stepped, with one
          // division pair per phase instead of one per tile.
          const u64 mult = simultaneous ? 1 : static_cast<u64>(P.k);
          const u64 utau = static_cast<u64>(P.tau);
          const u64 v1 = static_cast<u64>(t0_first + TILE - base) * mult, dv = static_cast<u64>(TILE) * mult;
          u64 cq, cr, dq, dr;
          divmod_u(v1, utau, &cq, &cr);
          divmod_u(dv, utau, &dq, &dr);
          for (i64 t0 = t0_first; t0 < P.t_end; t0 += TILE) {
            const int wlen = static_cast<int>(min_i64(TILE, P.t_end - t0));
            i64 r_b = N;                         // the last tile takes every remaining rank
            if (t0 + TILE < P.t_end) {
              r_b = static_cast<i64>(cq + (cr > 0)) * (simultaneous ? P.k : 1);
              if (r_b > N) r_b = N;
            }
            cq += dq; cr += dr;
            if (cr >= utau) { cr -= utau; ++cq; }
            C_next = process_runs<true>(p, sh, ec, P, cur, nxt, C_next, r_next, r_b, t0, buf, acc);
            r_next = r_b;
            if (P.tau > TILE) insert_far_ends(sh, ec, P, cur, t0_first, t0, wlen, buf);
            __syncthreads();
            scan_tile(sh, buf, t0, wlen, base, A_run, B_run, acc, ec, p.ev.profile);
            buf ^= 1;
          }
          written_to = P.t_end;
        }
        ec.run_count += N;
        base += len;
        __syncthreads();               // carry list complete before it is read as `cur`
        int32_t* tmp = cur; cur = nxt; nxt = tmp;
        C = C_next;
        if (C == 0 && ent_hi == nseg) break;   // nothing left in this window
      }
      if (status & KVS_EVAL_INFEASIBLE) break;
      write_jobs(p, sh, ec, family, simultaneous, L, X, seg_lo, seg_hi, geometric && (family == KVS_GSA || p.key != nullptr), acc);
      seg_lo = seg_hi;
    }

    // ---- scalars ----
    const i64 flow = block_sum(acc.flow, sh.red64);
    const i64 steps = block_sum(acc.steps, sh.red64);
    const i64 hmax = block_max(acc.hmax, sh.red64, static_cast<i64>(0));
    const int unfinished = block_sum(acc.unfinished, sh.red32);
    const u32 peak32 = block_max(acc.peak, sh.redA, 0u);
    const i64 peak = max_i64(static_cast<i64>(peak32), block_max(acc.peak64, sh.red64, static_cast<i64>(0)));
    if (tid == 0) {
      const bool skipped = (status & (KVS_EVAL_INFEASIBLE | KVS_EVAL_BAD_INPUT)) != 0;
      if (!skipped) {
        if (want32 && hmax > 0x7fffffffll) status |= KVS_EVAL_RANGE;
        if (ec.want_runs && ec.run_count > ec.run_cap) status |= KVS_EVAL_CAPACITY;
        if (ec.prof_cap > 0 && hmax > ec.prof_cap) status |= KVS_EVAL_CAPACITY;   // capacity 0 = profile not wanted
      }
      const bool have_peak = p.do_profile && profile_on && !skipped;
      if (p.ev.peak) p.ev.peak[e] = have_peak ? peak : -1;
      if (p.ev.flow) p.ev.flow[e] = flow;
      if (p.ev.job_steps) p.ev.job_steps[e] = steps;
      if (p.ev.horizon) p.ev.horizon[e] = hmax;
      if (p.ev.n_unfinished) p.ev.n_unfinished[e] = unfinished;
      if (p.ev.feasible) p.ev.feasible[e] = (have_peak && !(status & KVS_EVAL_RANGE) && peak <= M) ? 1 : 0;
      if (p.ev.status) p.ev.status[e] = status;
      if (p.out.n_runs) p.out.n_runs[e] = ec.run_count;
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
  err = cudaMemsetAsync(p.counter, 0, 8, stream);   // work counter: CTAs draw evaluations from it
  if (err != cudaSuccess) return err;
  k_build_eval<<<grid, KVS_EVAL_THREADS, build_smem_bytes(), stream>>>(p);
  return cudaGetLastError();
}
