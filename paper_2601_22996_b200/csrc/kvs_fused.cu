// Fused schedule builder and evaluator, 32-bit fast path: one CTA per (instance, setting, family)
// evaluation, times below 2^31.
//
// For one evaluation (and one arrival window at a time) the CTA
//   1. forms the phase table: the geometric ladder tau_p with the largest memory-feasible
//      parallelism k_p (first line of the two geometric algorithms; Lemma "Peak Memory Usage of
//      SPS"; Eq. max-parallelism), or the single (tau, k) of SPS / SimS;
//   2. plans the phases without touching a run: a job enters at the class f of its key and leaves
//      at the class l of the larger of key and response length, so phase p has
//      N_p = #{f <= p} - #{l < p} participants; that fixes every phase's length
//      floor((N_p - 1) tau_p / k_p) + tau_p and first round;
//   3. writes every job's start and completion: the job's rank in the phase that completes it is
//      the number of earlier positions (in schedule order) that leave in that phase or later; for
//      exact keys that is the position inside the class, otherwise it is counted with one warp
//      ballot per phase over 32 positions at a time, behind per-warp class histograms.
//      start = base_p + floor(r*tau_p/k_p) (Procedure StaggeredPipelineSchedule) or
//      base + floor(r/k)*tau (simultaneous batches), completion = start + o;
//   4. if the memory profile is wanted, walks the phases tile by tile as the general kernel does:
//      the runs that start inside a tile are a contiguous rank range, every run adds (c, 1) at its
//      first round and (-c, -1) after its last one to two shared-memory difference arrays
//      (c = s + 1 - start), one scan per array gives memory(t) = A(t) + t*B(t)
//      (Eq. Memory-Feasibility), the peak is reduced and the profile stored 16 bytes at a time.
//      Jobs killed at the end of their slot are carried to the next phase as (s, o) pairs, so a
//      phase reads its participants as one contiguous stream.
//
// An evaluation whose times reach 2^31 or whose memory bound reaches 2^32 is not finished here: its
// index is appended to a list that the general kernel works off afterwards.
#include <cstddef>

#include "kvs_events.cuh"
#include "kvs_ladder.cuh"

namespace {

constexpr int T = KVS_EVAL_THREADS;
constexpr int ITEMS = KVS_EVAL_ITEMS;
constexpr int TILE = KVS_TILE;
constexpr int WARPS = T / 32;
constexpr int VEC = ITEMS / 4;
constexpr int RPT = 4;                       // consecutive ranks per thread in the run visit
constexpr int MAXP = KVS_MAX_PHASES;
constexpr int RINGW = 2 * TILE + (2 * TILE) / 8;
constexpr int GCOL = 2049;
static_assert((TILE & (TILE - 1)) == 0 && ITEMS % 4 == 0 && ITEMS <= 32 && 32 % ITEMS == 0, "tile layout");
constexpr u32 TIME_LIMIT = 0x7fffffffu - 4u * TILE;   // phase ends stay below this

// Checked build (-DKVS_DEBUG): every computed index into the ring, the per-CTA scratch (class bytes, rank
// table, lists, start rounds, prefix sums) and the caller's profile and per-job outputs is tested against
// its bound before the access.  A violation records (code << 56 | index) in one device word - the first
// one wins - and the access is skipped; nothing traps.  The host reads the word with
// kvs_debug_check_word.  In the normal build KVS_IN is the constant true and costs nothing.
#ifdef KVS_DEBUG
__device__ unsigned long long g_check_word = 0ull;
__device__ __forceinline__ bool kvs_in_range(i64 idx, i64 limit, int code) {
  if (idx >= 0 && idx < limit) return true;
  atomicCAS(&g_check_word, 0ull, (static_cast<ull>(code) << 56) | (static_cast<ull>(idx) & 0x00ffffffffffffffull));
  return false;
}
#define KVS_IN(idx, limit, code) kvs_in_range(static_cast<i64>(idx), static_cast<i64>(limit), (code))
#else
#define KVS_IN(idx, limit, code) true
#endif
enum { CHK_GCOL = 1, CHK_G = 2, CHK_CLS = 3, CHK_RING = 4, CHK_LIST = 5, CHK_LIST_OUT = 6, CHK_PS = 7, CHK_PROFILE = 8,
       CHK_JOB_OUT = 11, CHK_FIN = 12, CHK_Z = 13 };

struct FShared {
  u128 pw_a[MAXP + 1];
  u128 pw_b[MAXP + 1];
  u64 taupre[MAXP + 1];       // sum of tau_q over q < p
  u64 kinv[MAXP];             // floor(2^64 / k_p) + 1, see slot_mul
  i64 plen[MAXP];
  i64 red64[32];
  i64 next_eval;
  i64 base_next;
  i64 n_runs;
  u32 tau[MAXP], k[MAXP], pbase[MAXP], np[MAXP];
  u32 cnt[WARPS][MAXP];       // per-warp class counts, then ranks before each warp's segment
  u32 gcol[GCOL];             // the current phase's column of the rank table (windows of up to (GCOL-1)*256 jobs)
  u32 redA[32], redB[32];
  int red32[32];
  int ent[MAXP + 1];          // class boundaries in key order
  int n_phases, seg_end, fallback;
  // two-tile ring of difference arrays: constant terms and slopes.  Round e of the ring (0 <= e <
  // 2*TILE) lives at word e + 4*(e/32): four spare words after every 32 keep the 16-byte loads of
  // the scan (a thread owns ITEMS consecutive rounds) free of bank conflicts while the index of an
  // event stays a shift and an add.  Last in the struct: the kernel for evaluations that walk no
  // rounds is launched without this part.
  alignas(16) u32 dA[RINGW];
  alignas(16) u32 dB[RINGW];
};

// floor(r * tau / k) for r, tau, k below 2^31 with a result below 2^31
__device__ __forceinline__ u32 slot32(u32 r, u32 tau, u32 k) {
  const u64 x = static_cast<u64>(r) * tau;
  if ((x >> 32) == 0) return static_cast<u32>(x) / k;
  return static_cast<u32>(x / k);
}

// The same with the division replaced by a multiplication: kinv = floor(2^64 / k) + 1 (k >= 2).
// For x = r * tau below 2^32, x * kinv / 2^64 = x/k + x*e/(k*2^64) with 0 < e <= k; the excess is
// below 2^-32 while the fractional part of x/k stays at least 1/k > 2^-31 short of the next integer,
// so the high word of the product is exactly floor(x / k).
__device__ __forceinline__ u32 slot_mul(u32 r, u32 tau, u32 k, u64 kinv) {
  const u64 x = static_cast<u64>(r) * tau;
  if ((x >> 32) == 0) return k == 1 ? static_cast<u32>(x) : static_cast<u32>(__umul64hi(x, kinv));
  return static_cast<u32>(x / k);
}

// Word of the round `rel` rounds after the origin of ring half `buf`, 0 <= rel < 2*TILE.
__device__ __forceinline__ int ring(int buf, int rel) {
  if (!KVS_IN(rel, 2 * TILE, CHK_RING)) rel = 0;
  const int e = (buf * TILE + rel) & (2 * TILE - 1);
  return e + ((e >> 5) << 2);
}

// One phase as the run visit sees it.  Positions are relative to the window, in schedule order.
// Exact keys: the participants are the positions [x_lo, x_hi) and the rank is the offset from x_lo.
// Carried jobs (FILTER): position x < x_hi takes part iff its leaving class cls[x] >= ph, and the
// rank table G[seg * L + ph] holds the number of such positions before segment `seg` (SEG positions
// each), so a warp can start at any segment without looking at the ones before it.
struct PhaseView {
  const int32_t* S;
  const int32_t* O;
  const unsigned char* cls;
  const u32* G;
  const u32* gcol;        // column ph of G in shared memory, or NULL
  int L, ph, nsegs;
  int cls_cap, g_cap;     // bytes of cls and words of G in this CTA's scratch
  int n_src;              // positions of the window (S and O may be read below this index)
  int x_lo, x_hi;
  u32 tau, k, qt, rt;     // tau = qt*k + rt
  u32 len;                // rounds of the phase
  u32 base;               // its first round
};

constexpr int SEG = 256;  // positions per warp step: 8 consecutive positions per lane

// participants of the phase before segment `seg`
__device__ __forceinline__ int rank_before(const PhaseView& P, int seg) {
  if (P.gcol) return KVS_IN(seg, GCOL, CHK_GCOL) ? static_cast<int>(P.gcol[seg]) : 0;
  return KVS_IN(seg * P.L + P.ph, P.g_cap, CHK_G) ? static_cast<int>(P.G[seg * P.L + P.ph]) : 0;
}

// The 8 positions of one lane in segment `seg`: bit j of `bits` is set if position xb + j takes part,
// and those positions have the consecutive ranks r_first, r_first + 1, ...
// With FILTER, `fbits` marks the participants whose leaving class is this phase (they complete here;
// the others are killed at the end of their slot and their response length is not needed).
struct LaneGroup { u32 bits; u32 fbits; int r_first; int xb; };

// Bit j of the result is set iff byte j of `w` is >= (ge) or == the byte replicated in `p4`.
__device__ __forceinline__ u32 byte_mask4(u32 w, u32 p4, bool ge) {
  const u32 m = (ge ? __vcmpgeu4(w, p4) : __vcmpeq4(w, p4)) & 0x08040201u;
  return (m | (m >> 8) | (m >> 16) | (m >> 24)) & 15u;
}

template <bool FILTER>
__device__ __forceinline__ LaneGroup lane_group(const PhaseView& P, int seg) {
  LaneGroup g;
  const int lane = lane_id();
  if (FILTER) {
    g.xb = seg * SEG + 8 * lane;
    const uint2 cw = KVS_IN(g.xb + 7, P.cls_cap, CHK_CLS) ? *reinterpret_cast<const uint2*>(P.cls + g.xb) : make_uint2(0, 0);
    const int room = P.x_hi - g.xb;                        // positions of this lane below x_hi
    const u32 lim = room >= 8 ? 0xffu : (room > 0 ? (1u << room) - 1u : 0u);
    const u32 p4 = static_cast<u32>(P.ph) * 0x01010101u;
    g.bits = (byte_mask4(cw.x, p4, true) | byte_mask4(cw.y, p4, true) << 4) & lim;
    g.fbits = (byte_mask4(cw.x, p4, false) | byte_mask4(cw.y, p4, false) << 4) & lim;
    int incl = __popc(g.bits);
    const int cnt = incl;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += y;
    }
    g.r_first = rank_before(P, seg) + incl - cnt;
  } else {
    g.r_first = seg * SEG + 8 * lane;
    g.xb = P.x_lo + g.r_first;
    const int room = P.x_hi - g.xb;
    g.bits = room >= 8 ? 0xffu : (room > 0 ? (1u << room) - 1u : 0u);
    g.fbits = g.bits;
  }
  return g;
}

// Segments that hold the ranks [ra, rb) of the phase.
template <bool FILTER>
__device__ __forceinline__ void segment_range(const PhaseView& P, int ra, int rb, int* seg_a, int* seg_b) {
  if (FILTER) {
    // G[.][ph] is nondecreasing over the nsegs + 1 rows; last row = number of participants
    int a = 0, b = P.nsegs;               // largest seg with G[seg] <= ra
    while (a < b) { const int m = (a + b + 1) >> 1; if (rank_before(P, m) <= ra) a = m; else b = m - 1; }
    *seg_a = a;
    a = 0; b = P.nsegs;                   // smallest seg with G[seg] >= rb
    while (a < b) { const int m = (a + b) >> 1; if (rank_before(P, m) >= rb) b = m; else a = m + 1; }
    *seg_b = a;
  } else {
    *seg_a = ra / SEG;
    *seg_b = (rb + SEG - 1) / SEG;
  }
}

// Visits ranks [ra, rb), all of which start inside the tile whose origin is `trel` rounds after
// the phase's first round (trel may be slightly negative) and whose ring half is `buf`: adds the
// two events of every run.  Warps take segments in turn; nothing is written to global memory and
// no block-wide barrier is needed.
template <bool SIM, bool FILTER>
__device__ __forceinline__ void visit_runs(FShared& sh, const PhaseView& P, int ra, int rb, int trel, int buf,
                                           bool dense, bool combine) {
  if (ra >= rb) return;
  u32* const dA = sh.dA;
  u32* const dB = sh.dB;
  const u32 tau = P.tau, k = P.k;
  const int warp = threadIdx.x >> 5;
  // 16-byte loads need aligned rows; without the filter a lane's first position is x_lo + 8*(...)
  const bool vec = ((reinterpret_cast<uintptr_t>(P.S) | reinterpret_cast<uintptr_t>(P.O)) & 15u) == 0 && (FILTER || (P.x_lo & 3) == 0);
  int seg_a, seg_b;
  segment_range<FILTER>(P, ra, rb, &seg_a, &seg_b);
  for (int seg = seg_a + warp; seg < seg_b; seg += WARPS) {
    // The prompt lengths of the lane's eight positions do not depend on which of them take part:
    // where all eight exist and the rows are 16-byte aligned they are requested first, as two
    // 16-byte loads, so that they travel together with the class bytes instead of after them.
    const int xb0 = (FILTER ? 0 : P.x_lo) + seg * SEG + 8 * static_cast<int>(lane_id());
    const bool vload = vec && xb0 + 8 <= P.n_src;
    uint4 a0 = make_uint4(0, 0, 0, 0), a1 = a0;
    if (vload) {
      a0 = __ldg(reinterpret_cast<const uint4*>(P.S + xb0));
      a1 = __ldg(reinterpret_cast<const uint4*>(P.S + xb0) + 1);
    }
    const LaneGroup g = lane_group<FILTER>(P, seg);
    // of this lane's participants, entries [skip, skip + take) have ranks inside [ra, rb)
    const int cnt = __popc(g.bits);
    const int skip = max(0, ra - g.r_first);
    const int take = min(cnt, rb - g.r_first) - skip;
    if (__ballot_sync(0xffffffffu, take > 0) == 0) continue;
    u32 s_[8], o_[8];
    // a killed run lasts tau rounds whatever its response length: only completing jobs load it
    const u32 need_o = take > 0 ? g.fbits : 0u;
    if (vload) {
      s_[0] = a0.x; s_[1] = a0.y; s_[2] = a0.z; s_[3] = a0.w; s_[4] = a1.x; s_[5] = a1.y; s_[6] = a1.z; s_[7] = a1.w;
      if (FILTER) {
#pragma unroll
        for (int j = 0; j < 8; ++j) o_[j] = (need_o >> j & 1u) ? static_cast<u32>(__ldg(P.O + g.xb + j)) : 0xffffffffu;
      } else {
        const uint4 b0 = take > 0 ? __ldg(reinterpret_cast<const uint4*>(P.O + g.xb)) : make_uint4(0, 0, 0, 0);
        const uint4 b1 = take > 0 ? __ldg(reinterpret_cast<const uint4*>(P.O + g.xb) + 1) : make_uint4(0, 0, 0, 0);
        o_[0] = b0.x; o_[1] = b0.y; o_[2] = b0.z; o_[3] = b0.w; o_[4] = b1.x; o_[5] = b1.y; o_[6] = b1.z; o_[7] = b1.w;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        s_[j] = 0; o_[j] = 0xffffffffu;
        if (take > 0 && (g.bits >> j & 1u)) s_[j] = static_cast<u32>(__ldg(P.S + g.xb + j));
        if (need_o >> j & 1u) o_[j] = static_cast<u32>(__ldg(P.O + g.xb + j));
      }
    }
    u32 q = 0, rem = 0;      // start offset of the current rank inside the phase and its remainder
    if (take > 0) {
      const u32 r0 = static_cast<u32>(g.r_first + skip);
      if (SIM) {
        const u32 b = r0 / k;
        q = b * tau;
        rem = r0 - b * k;
      } else {
        u64 dq_, dr_;
        divmod_u(static_cast<u64>(r0) * tau, k, &dq_, &dr_);
        q = static_cast<u32>(dq_);
        rem = static_cast<u32>(dr_);
      }
    }
    // Dense phases (several runs start per round): the runs of a lane that start in the round of
    // its first run are summed in registers, then equal rounds - contiguous lanes, because
    // consecutive ranks start in nondecreasing rounds - are summed across the warp with a
    // segmented scan, and one lane per round issues the atomics.  Runs that hold their whole
    // slot end together (start + tau), so their end events are combined the same way.
    const bool dn = !SIM && dense;
    int seg_key = 0x7fffffff;
    u32 seg_all = 0, seg_full = 0, seg_cnt = 0;
    int idx = 0;             // index among this lane's participants
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      int sidx = -1, eidx = -1;
      u32 c = 0;
      const bool part = (g.bits >> j & 1u) != 0;
      const bool on = part && idx >= skip && idx < skip + take;
      if (part) ++idx;
      if (on) {
        const u32 oi = o_[j];
        const u32 d = oi < tau ? oi : tau;
        c = s_[j] + 1u - P.base - q;                          // tokens(t) = c + t while active
        const int srel = static_cast<int>(q) - trel;
        sidx = ring(buf, srel);
        if (q + d < P.len) {                                   // an end at the phase end is never read
          const u32 erel = static_cast<u32>(srel) + d;
          if (erel < 2u * TILE) eidx = ring(buf, static_cast<int>(erel));
        }
        if (dn) {
          if (seg_key == 0x7fffffff) seg_key = srel;
          if (srel == seg_key) {
            seg_all += c; seg_cnt += 1u;
            sidx = -1;
            if (d == tau) { seg_full += c; seg_cnt += 1u << 16; eidx = -1; }
          }
        }
        if (SIM) { if (++rem == k) { rem = 0; q += tau; } }
        else { rem += P.rt; q += P.qt; if (rem >= k) { rem -= k; ++q; } }
      }
      if (SIM && combine) {
        // whole simultaneous batches hit one word: sum equal targets inside the warp first
        const u32 ps = __match_any_sync(0xffffffffu, sidx);
        if (sidx >= 0) {
          const u32 cs = __reduce_add_sync(ps, c);
          if ((ps & lanemask_lt()) == 0) { atomicAdd(&dA[sidx], cs); atomicAdd(&dB[sidx], static_cast<u32>(__popc(ps))); }
        }
        const u32 pe = __match_any_sync(0xffffffffu, eidx);
        if (eidx >= 0) {
          const u32 ce = __reduce_add_sync(pe, c);
          if ((pe & lanemask_lt()) == 0) { atomicAdd(&dA[eidx], 0u - ce); atomicAdd(&dB[eidx], 0u - static_cast<u32>(__popc(pe))); }
        }
      } else {
        if (sidx >= 0) { atomicAdd(&dA[sidx], c); atomicAdd(&dB[sidx], 1u); }
        if (eidx >= 0) { atomicAdd(&dA[eidx], 0u - c); atomicAdd(&dB[eidx], 0xffffffffu); }
      }
    }
    if (dn) {
      // a lane without runs takes the round of the nearest lane before it that has some, so that
      // equal rounds stay contiguous for the segmented scan
      const u32 has = __ballot_sync(0xffffffffu, seg_key != 0x7fffffff);
      const u32 before = has & lanemask_lt();
      const int src = (seg_key == 0x7fffffff && before) ? 31 - __clz(before) : static_cast<int>(lane_id());
      int key = __shfl_sync(0xffffffffu, seg_key, src);
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
        const int si = ring(buf, key);
        atomicAdd(&dA[si], va);
        atomicAdd(&dB[si], vn & 0xffffu);
        const u32 n_full = vn >> 16;
        // start offset of this round inside the phase: key + trel
        if (n_full && static_cast<u32>(key + trel) + tau < P.len) {
          const int ei = ring(buf, key + static_cast<int>(tau));          // tau < TILE in dense phases
          atomicAdd(&dA[ei], 0u - vf);
          atomicAdd(&dB[ei], 0u - n_full);
        }
      }
    }
  }
}

// The run visit of a phase with carried jobs in which at least eight runs start per round (and the
// slice is shorter than a tile).  A lane's up to eight participants then start in one round or in
// two consecutive ones, so the lane first treats all of them as killed at the end of their slot:
// one start event and one end event per round, from sums over its participants, without a loop
// over runs.  Afterwards each participant that completes before the end of its slot moves its own
// end event from start + tau to start + o.  Same events in total as visit_runs<false, true>.
__device__ __forceinline__ void visit_runs_sliced(FShared& sh, const PhaseView& P, int ra, int rb, int trel, int buf, u64 kinv) {
  if (ra >= rb) return;
  u32* const dA = sh.dA;
  u32* const dB = sh.dB;
  const u32 tau = P.tau, k = P.k;
  const int warp = threadIdx.x >> 5;
  const bool vec = (reinterpret_cast<uintptr_t>(P.S) & 15u) == 0;
  int seg_a, seg_b;
  segment_range<true>(P, ra, rb, &seg_a, &seg_b);
  for (int seg = seg_a + warp; seg < seg_b; seg += WARPS) {
    const int xb0 = seg * SEG + 8 * static_cast<int>(lane_id());
    const bool vload = vec && xb0 + 8 <= P.n_src;
    uint4 a0 = make_uint4(0, 0, 0, 0), a1 = a0;
    if (vload) {
      a0 = __ldg(reinterpret_cast<const uint4*>(P.S + xb0));
      a1 = __ldg(reinterpret_cast<const uint4*>(P.S + xb0) + 1);
    }
    const LaneGroup g = lane_group<true>(P, seg);
    const int cnt = __popc(g.bits);
    const int skip = max(0, ra - g.r_first);
    const int take = min(cnt, rb - g.r_first) - skip;
    if (__ballot_sync(0xffffffffu, take > 0) == 0) continue;
    if (take <= 0) continue;
    // the lane's participants with ranks inside [ra, rb)
    u32 bits = g.bits;
    for (int i = 0; i < skip; ++i) bits &= bits - 1u;
    for (int extra = __popc(bits) - take; extra > 0; --extra) bits &= ~(0x80000000u >> __clz(bits));
    u32 s_[8];
    if (vload) {
      s_[0] = a0.x; s_[1] = a0.y; s_[2] = a0.z; s_[3] = a0.w; s_[4] = a1.x; s_[5] = a1.y; s_[6] = a1.z; s_[7] = a1.w;
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) s_[j] = (bits >> j & 1u) ? static_cast<u32>(__ldg(P.S + g.xb + j)) : 0u;
    }
    const u32 n = static_cast<u32>(take);
    const u32 r0 = static_cast<u32>(g.r_first + skip);
    const u32 q0 = slot_mul(r0, tau, k, kinv);
    // rank r0 + j starts in round q0 + floor((rem + j tau) / k): the first m stay in round q0
    const u32 rem = static_cast<u32>(static_cast<u64>(r0) * tau - static_cast<u64>(q0) * k);
    u32 m = 1;
#pragma unroll
    for (u32 j = 1; j < 8; ++j) m += (rem + j * tau < k) ? 1u : 0u;
    m = min(m, n);
    u32 sumA = 0, sumB = 0, idx = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (bits >> j & 1u) {
        const u32 v = s_[j] + 1u;
        if (idx < m) sumA += v; else sumB += v;
        ++idx;
      }
    }
    const int srel = static_cast<int>(q0) - trel;
    {
      const u32 c = sumA - m * (P.base + q0);
      const int si = ring(buf, srel);
      atomicAdd(&dA[si], c);
      atomicAdd(&dB[si], m);
      if (q0 + tau < P.len) {
        const int ei = ring(buf, srel + static_cast<int>(tau));
        atomicAdd(&dA[ei], 0u - c);
        atomicAdd(&dB[ei], 0u - m);
      }
    }
    if (n > m) {
      const u32 c = sumB - (n - m) * (P.base + q0 + 1u);
      const int si = ring(buf, srel + 1);
      atomicAdd(&dA[si], c);
      atomicAdd(&dB[si], n - m);
      if (q0 + 1u + tau < P.len) {
        const int ei = ring(buf, srel + 1 + static_cast<int>(tau));
        atomicAdd(&dA[ei], 0u - c);
        atomicAdd(&dB[ei], 0u - (n - m));
      }
    }
    // completing jobs: the end moves from start + tau to start + o
    u32 fb = g.fbits & bits;
    while (fb) {
      const int j = __ffs(static_cast<int>(fb)) - 1;
      fb &= fb - 1u;
      const u32 oi = static_cast<u32>(__ldg(P.O + g.xb + j));
      if (oi < tau) {
        const u32 before = static_cast<u32>(__popc(bits & ((1u << j) - 1u)));
        const u32 q = q0 + (before >= m ? 1u : 0u);
        const u32 c = static_cast<u32>(__ldg(P.S + g.xb + j)) + 1u - P.base - q;
        const int sr = static_cast<int>(q) - trel;
        if (q + oi < P.len) {
          const int ei = ring(buf, sr + static_cast<int>(oi));
          atomicAdd(&dA[ei], 0u - c);
          atomicAdd(&dB[ei], 0xffffffffu);
        }
        if (q + tau < P.len) {
          const int ki = ring(buf, sr + static_cast<int>(tau));
          atomicAdd(&dA[ki], c);
          atomicAdd(&dB[ki], 1u);
        }
      }
    }
  }
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

// Participants of a phase as a list (used once fewer than half of a window's positions still take
// part): rank r < C is the (s, o) pair cur[r], rank r >= C is position src + (r - C) of the
// window (jobs that enter in this phase).
struct ListView {
  const uint2* cur;
  int C;
  int src;
  int cap;                // entries of either list in this CTA's scratch
};

// Run visit over a list: ranks [ra, rb), one to four consecutive ranks per thread, so that a tile
// with few runs is spread over the whole block instead of a few warps.  Adds the two events of
// every run and appends the killed jobs to `nxt`; returns the new length of `nxt`.  Block-wide
// (two barriers per 2048 ranks for the positions of the survivors).
__device__ __forceinline__ int visit_list(FShared& sh, const PhaseView& P, const ListView& V, uint2* nxt, int C_next,
                                          int ra, int rb, int trel, int buf, bool dense) {
  const int tid = threadIdx.x, lane = lane_id();
  u32* const dA = sh.dA;
  u32* const dB = sh.dB;
  const u32 tau = P.tau, k = P.k;
  for (int c0 = ra; c0 < rb;) {
    const int left = rb - c0;
    const int rpt = left > 2 * T ? RPT : (left > T ? 2 : 1);
    const int r_first = c0 + tid * rpt;
    c0 += T * rpt;
    uint2 keep[RPT];
    u32 cmask = 0;
    if (r_first - lane * rpt < rb) {   // warps past the end of the range skip the visit
      u32 s_[RPT], o_[RPT];
      bool on[RPT];
#pragma unroll
      for (int j = 0; j < RPT; ++j) {
        const int r = r_first + j;
        on[j] = j < rpt && r < rb;
        s_[j] = 0; o_[j] = 0;
        if (on[j]) {
          if (r < V.C) { if (KVS_IN(r, V.cap, CHK_LIST)) { const uint2 e = V.cur[r]; s_[j] = e.x; o_[j] = e.y; } }
          else { s_[j] = static_cast<u32>(__ldg(P.S + V.src + (r - V.C))); o_[j] = static_cast<u32>(__ldg(P.O + V.src + (r - V.C))); }
        }
      }
      u32 q = 0, rem = 0;
      if (on[0]) {
        u64 dq_, dr_;
        divmod_u(static_cast<u64>(r_first) * tau, k, &dq_, &dr_);
        q = static_cast<u32>(dq_);
        rem = static_cast<u32>(dr_);
      }
      int seg_key = 0x7fffffff;
      u32 seg_all = 0, seg_full = 0, seg_cnt = 0;
#pragma unroll
      for (int j = 0; j < RPT; ++j) {
        if (on[j]) {
          const u32 oi = o_[j];
          const u32 d = oi < tau ? oi : tau;
          if (oi > tau) { keep[j] = make_uint2(s_[j], oi); cmask |= 1u << j; }
          const u32 c = s_[j] + 1u - P.base - q;
          const int srel = static_cast<int>(q) - trel;
          int sidx = ring(buf, srel), eidx = -1;
          if (q + d < P.len) {
            const u32 erel = static_cast<u32>(srel) + d;
            if (erel < 2u * TILE) eidx = ring(buf, static_cast<int>(erel));
          }
          if (dense) {
            if (seg_key == 0x7fffffff) seg_key = srel;
            if (srel == seg_key) {
              seg_all += c; seg_cnt += 1u;
              sidx = -1;
              if (d == tau) { seg_full += c; seg_cnt += 1u << 16; eidx = -1; }
            }
          }
          if (sidx >= 0) { atomicAdd(&dA[sidx], c); atomicAdd(&dB[sidx], 1u); }
          if (eidx >= 0) { atomicAdd(&dA[eidx], 0u - c); atomicAdd(&dB[eidx], 0xffffffffu); }
          rem += P.rt; q += P.qt;
          if (rem >= k) { rem -= k; ++q; }
        }
      }
      if (dense) {
        const u32 has = __ballot_sync(0xffffffffu, seg_key != 0x7fffffff);
        const u32 before = has & lanemask_lt();
        const int src = (seg_key == 0x7fffffff && before) ? 31 - __clz(before) : lane;
        const int key = __shfl_sync(0xffffffffu, seg_key, src);
        u32 va = seg_all, vf = seg_full, vn = seg_cnt;
#pragma unroll
        for (int dd = 1; dd < 32; dd <<= 1) {
          const int kk = __shfl_up_sync(0xffffffffu, key, dd);
          const u32 ya = __shfl_up_sync(0xffffffffu, va, dd), yf = __shfl_up_sync(0xffffffffu, vf, dd);
          const u32 yn = __shfl_up_sync(0xffffffffu, vn, dd);
          if (lane >= dd && kk == key) { va += ya; vf += yf; vn += yn; }
        }
        const int next_key = __shfl_down_sync(0xffffffffu, key, 1);
        if (key != 0x7fffffff && (lane == 31 || next_key != key)) {
          const int si = ring(buf, key);
          atomicAdd(&dA[si], va);
          atomicAdd(&dB[si], vn & 0xffffu);
          const u32 n_full = vn >> 16;
          if (n_full && static_cast<u32>(key + trel) + tau < P.len) {
            const int ei = ring(buf, key + static_cast<int>(tau));
            atomicAdd(&dA[ei], 0u - vf);
            atomicAdd(&dB[ei], 0u - n_full);
          }
        }
      }
    }
    int total;
    int off = C_next + block_count_scan(__popc(cmask), sh.red32, &total);
#pragma unroll
    for (int j = 0; j < RPT; ++j)
      if (cmask >> j & 1u) { if (KVS_IN(off, V.cap, CHK_LIST_OUT)) nxt[off] = keep[j]; ++off; }
    C_next += total;
  }
  return C_next;
}

// insert_far_ends for a list: slices longer than a tile only.
__device__ __forceinline__ void insert_far_ends_list(FShared& sh, const PhaseView& P, const ListView& V, int N, int a0,
                                                     int u0, int wlen, int buf) {
  if (u0 <= TILE) return;
  const u32 lo = static_cast<u32>(u0) > P.tau ? static_cast<u32>(u0) - P.tau : 0u, hi = static_cast<u32>(u0 - TILE);
  i64 r_lo = ceil_div_u(static_cast<u64>(lo) * P.k, P.tau), r_hi = ceil_div_u(static_cast<u64>(hi) * P.k, P.tau);
  if (r_hi > N) r_hi = N;
  for (i64 r0 = r_lo; r0 < r_hi; r0 += T) {
    const i64 rr = r0 + threadIdx.x;
    if (rr < r_hi) {
      const int r = static_cast<int>(rr);
      u32 si, oi;
      if (r < V.C) { uint2 e = make_uint2(0, 1); if (KVS_IN(r, V.cap, CHK_LIST)) e = V.cur[r]; si = e.x; oi = e.y; }
      else { si = static_cast<u32>(__ldg(P.S + V.src + (r - V.C))); oi = static_cast<u32>(__ldg(P.O + V.src + (r - V.C))); }
      const u32 q = slot32(static_cast<u32>(r), P.tau, P.k);
      const u32 end = q + (oi < P.tau ? oi : P.tau);
      const int ts = a0 + ((static_cast<int>(q) - a0) / TILE) * TILE;
      if (static_cast<int>(end) >= ts + 2 * TILE && static_cast<int>(end) >= u0 && static_cast<int>(end) < u0 + wlen && end < P.len) {
        const u32 c = si + 1u - P.base - q;
        const int ei = ring(buf, static_cast<int>(end) - u0);
        atomicAdd(&sh.dA[ei], 0u - c);
        atomicAdd(&sh.dB[ei], 0xffffffffu);
      }
    }
  }
}

// A phase in which every position of the window takes part and none completes (index order, all
// response lengths beyond the slice: the early phases of the slicing algorithm) needs no visit of
// its runs.  Rank = position, every run lasts tau rounds, so the events of a round are sums over
// position ranges: with PS[x] = sum of (s + 1) over positions below x and B(u) = number of ranks that
// start in round u or earlier = min(N, ceil((u + 1) k / tau)), the runs that start in round u add
// (PS[B(u)] - PS[B(u-1)] - cnt (base + u), cnt) there and the opposite tau rounds later.  Each thread
// forms the events of its own ITEMS rounds of the tile - starts at u and ends of the runs started
// at u - tau - and adds them to its own words of the ring: no atomics, no dependence on the number
// of runs.  u0 = offset of the tile's origin inside the phase.
__device__ __forceinline__ void pure_phase_events(FShared& sh, const PhaseView& P, const u32* __restrict__ PS, int ps_cap, int N, int u0, int buf) {
  (void)ps_cap;
  const int e0 = ITEMS * static_cast<int>(threadIdx.x);
  const int w0 = ring(buf, e0);
  const u32 tau = P.tau, k = P.k;
  const u32 kq = k / tau, kr = k - kq * tau;          // k = kq * tau + kr
#pragma unroll
  for (int stream = 0; stream < 2; ++stream) {
    // stream 0: runs that start in the thread's rounds; stream 1: runs that end there (started tau earlier)
    const i64 ufirst = static_cast<i64>(u0) + e0 - (stream ? static_cast<i64>(tau) : 0);   // start round of the first event
    // B(ufirst - 1) by one division, then stepped: (u + 1) k = Q tau + R
    u64 Q = 0, R = 0;
    i64 u = ufirst - 1;
    if (u >= 0) divmod_u(static_cast<u64>(u + 1) * k, tau, &Q, &R);
    u32 b_prev = u >= 0 ? static_cast<u32>(min(static_cast<u64>(N), Q + (R > 0))) : 0u;
    u32 ps_prev = KVS_IN(b_prev, ps_cap, CHK_PS) ? PS[b_prev] : 0u;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
      ++u;
      if (u == 0) { Q = kq; R = kr; }                  // (0 + 1) k
      else if (u > 0) { Q += kq; R += kr; if (R >= tau) { R -= tau; ++Q; } }
      const i64 land = u + (stream ? static_cast<i64>(tau) : 0);          // round the event lands in
      if (u >= 0 && land < static_cast<i64>(P.len)) {
        const u32 b = static_cast<u32>(min(static_cast<u64>(N), Q + (R > 0)));
        if (b != b_prev) {
          const u32 ps = KVS_IN(b, ps_cap, CHK_PS) ? PS[b] : 0u;
          const u32 cnt = b - b_prev;
          const u32 c = (ps - ps_prev) - cnt * (P.base + static_cast<u32>(u));
          if (stream == 0) { sh.dA[w0 + i] += c; sh.dB[w0 + i] += cnt; }
          else { sh.dA[w0 + i] -= c; sh.dB[w0 + i] -= cnt; }
          b_prev = b; ps_prev = ps;
        }
      }
    }
  }
}

// Slices longer than a tile: ends that land two or more tiles after the run's start were not
// inserted when the run was visited; pick them up when their tile comes.  u0 = offset of this
// tile's origin inside the phase, a0 = the same for the phase's first tile (0 or slightly negative).
template <bool FILTER>
__device__ __forceinline__ void insert_far_ends(FShared& sh, const PhaseView& P, bool sim, int N, int a0, int u0,
                                                int wlen, int buf) {
  if (u0 <= TILE) return;
  const u32 lo = static_cast<u32>(u0) > P.tau ? static_cast<u32>(u0) - P.tau : 0u, hi = static_cast<u32>(u0 - TILE);
  i64 r_lo, r_hi;   // ranks whose start offset lies in [lo, hi)
  if (sim) { r_lo = ceil_div_u(lo, P.tau) * P.k; r_hi = ceil_div_u(hi, P.tau) * P.k; }
  else { r_lo = ceil_div_u(static_cast<u64>(lo) * P.k, P.tau); r_hi = ceil_div_u(static_cast<u64>(hi) * P.k, P.tau); }
  if (r_hi > N) r_hi = N;
  if (r_lo >= r_hi) return;
  const int ra = static_cast<int>(r_lo), rb = static_cast<int>(r_hi);
  u32* const dA = sh.dA;
  u32* const dB = sh.dB;
  const int warp = threadIdx.x >> 5;
  int seg_a, seg_b;
  segment_range<FILTER>(P, ra, rb, &seg_a, &seg_b);
  for (int seg = seg_a + warp; seg < seg_b; seg += WARPS) {
    const LaneGroup g = lane_group<FILTER>(P, seg);
    int r = g.r_first;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (!(g.bits >> j & 1u)) continue;
      const int rr = r++;
      if (rr < ra || rr >= rb) continue;
      const u32 si = static_cast<u32>(__ldg(P.S + g.xb + j)), oi = static_cast<u32>(__ldg(P.O + g.xb + j));
      const u32 q = sim ? (static_cast<u32>(rr) / P.k) * P.tau : slot32(static_cast<u32>(rr), P.tau, P.k);
      const u32 end = q + (oi < P.tau ? oi : P.tau);
      const int ts = a0 + ((static_cast<int>(q) - a0) / TILE) * TILE;   // origin of the tile the run started in
      if (static_cast<int>(end) >= ts + 2 * TILE && static_cast<int>(end) >= u0 && static_cast<int>(end) < u0 + wlen && end < P.len) {
        const u32 c = si + 1u - P.base - q;
        const int ei = ring(buf, static_cast<int>(end) - u0);
        atomicAdd(&dA[ei], 0u - c);
        atomicAdd(&dB[ei], 0xffffffffu);
      }
    }
  }
}

// inclusive suffix sum across the lanes of a warp
__device__ __forceinline__ u32 warp_suffix(u32 v) {
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const u32 y = __shfl_down_sync(0xffffffffu, v, d);
    if (static_cast<int>(lane_id()) + d < 32) v += y;
  }
  return v;
}

// Prefix-sums one tile of the ring, turns it into memory(t), reduces the peak, stores the profile
// and leaves the tile zeroed for its next use.  Contains one __syncthreads.  t0 = absolute round
// of the tile's origin; rounds [first_round, t0 + wlen) below prof_cap are stored.
__device__ __forceinline__ void scan_tile(FShared& sh, int buf, i64 t0, int wlen, u32 first_round,
                                          u32& A_run, u32& B_run, u32& peak, int32_t* prof, i64 prof_cap) {
  const int tid = threadIdx.x;
  const uint4 zero = make_uint4(0, 0, 0, 0);
  u32 a[ITEMS], b[ITEMS];
  const int w0 = ring(buf, ITEMS * tid);       // the thread's ITEMS rounds are consecutive words
#pragma unroll
  for (int v = 0; v < VEC; ++v) {
    uint4* const pa = reinterpret_cast<uint4*>(&sh.dA[w0 + 4 * v]);
    uint4* const pb = reinterpret_cast<uint4*>(&sh.dB[w0 + 4 * v]);
    const uint4 x = *pa, y = *pb;
    *pa = zero;
    *pb = zero;
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
  for (int i = 0; i < ITEMS; ++i) mem[i] = (offA + a[i]) + (tt + i) * (offB + b[i]);
  // a tile that lies inside the phase and inside the caller's capacity needs no per-round tests
  const bool whole = wlen == TILE && (prof_cap <= 0 || (t0 >= static_cast<i64>(first_round) && t0 + TILE <= prof_cap));
  if (whole) {
    u32 m = mem[0];
#pragma unroll
    for (int i = 1; i < ITEMS; ++i) m = max(m, mem[i]);
    peak = max(peak, m);
    if (prof_cap > 0 && KVS_IN(t0 + e0, prof_cap - (ITEMS - 1), CHK_PROFILE)) {
      int4* dst = reinterpret_cast<int4*>(prof + t0 + e0);
#pragma unroll
      for (int v = 0; v < VEC; ++v)
        __stcs(&dst[v], make_int4(static_cast<int>(mem[4 * v]), static_cast<int>(mem[4 * v + 1]),
                                  static_cast<int>(mem[4 * v + 2]), static_cast<int>(mem[4 * v + 3])));   // written once, never re-read: streaming
    }
    return;
  }
#pragma unroll
  for (int i = 0; i < ITEMS; ++i)
    if (e0 + i < wlen) peak = max(peak, mem[i]);
  if (prof_cap > 0) {
    const i64 lo = first_round, hi = min_i64(t0 + wlen, prof_cap);
#pragma unroll
    for (int v = 0; v < VEC; ++v) {
      const i64 rs = t0 + e0 + 4 * v;
      int32_t* dst = prof + rs;
      if (rs >= lo && rs + 4 <= hi && KVS_IN(rs, prof_cap - 3, CHK_PROFILE)) {
        *reinterpret_cast<int4*>(dst) = make_int4(static_cast<int>(mem[4 * v]), static_cast<int>(mem[4 * v + 1]),
                                                  static_cast<int>(mem[4 * v + 2]), static_cast<int>(mem[4 * v + 3]));
      } else if (rs + 4 > lo && rs < hi) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (rs + i >= lo && rs + i < hi && KVS_IN(rs + i, prof_cap, CHK_PROFILE)) dst[i] = static_cast<int>(mem[4 * v + i]);
      }
    }
  }
}

struct FAcc {
  u64 flow = 0, steps = 0;
  u32 hmax = 0;
  int unfinished = 0;
  u32 peak = 0;
  i64 peak64 = 0;
};

// LIGHT: the variant for evaluations that walk no rounds (schedule only, or SPS / SimS whose peak
// comes from the run ends): no ring in shared memory and fewer registers, so that three CTAs fit an
// SM; an evaluation that needs its rounds walked is passed on to the full variant through a list.
// FAM: KVS_FUSED_ANY takes any evaluation; a family id (KVS_GBA .. KVS_SIMS) gives the kernel compiled
// for that family on exact response lengths only (the caller lists nothing else for it), so that
// each keeps just its own paths and gets its own register allocation.
template <bool LIGHT, int FAM>
__global__ void __launch_bounds__(KVS_EVAL_THREADS, LIGHT ? KVS_EVAL_MIN_CTAS + 1 : KVS_EVAL_MIN_CTAS) k_fused_eval(BuildParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  FShared& sh = *reinterpret_cast<FShared*>(smem_raw);
  const int tid = threadIdx.x, lane = lane_id(), warp = tid >> 5;
  // per-CTA scratch: class bytes of the current window (padded to whole segments), then the rank table
  unsigned char* const cls = reinterpret_cast<unsigned char*>(p.lists) + static_cast<i64>(blockIdx.x) * KVS_CTA_SCRATCH(p.max_jobs);
  u32* const G = reinterpret_cast<u32*>(cls + ((p.max_jobs + SEG + 15) & ~static_cast<i64>(15)));
  // two lists of (s, o) pairs for windows of which fewer than half of the positions still take part
  uint2* const list0 = reinterpret_cast<uint2*>(reinterpret_cast<unsigned char*>(G) + ((static_cast<size_t>(p.max_jobs) / SEG + 2) * MAXP * 4));
  uint2* const list1 = list0 + (p.max_jobs + 1);
  u32* const fin_start = reinterpret_cast<u32*>(p.fin_rank) + static_cast<i64>(blockIdx.x) * p.max_jobs;
  // bounds of the scratch parts, for the checked build
  const int cls_cap = static_cast<int>((p.max_jobs + SEG + 15) & ~static_cast<i64>(15));       // bytes
  const int g_cap = static_cast<int>((static_cast<size_t>(p.max_jobs) / SEG + 2) * MAXP);       // words
  const int list_cap = static_cast<int>(p.max_jobs + 1);                                        // (s, o) pairs per list
  const int z_cap = static_cast<int>(KVS_CTA_SCRATCH(p.max_jobs) / 4);                          // words of the whole block
  (void)cls_cap; (void)g_cap; (void)list_cap; (void)z_cap;
  if (!LIGHT) {
    for (int i = tid; i < RINGW; i += T) { sh.dA[i] = 0; sh.dB[i] = 0; }
  }

  for (;;) {
    __syncthreads();
    if (tid == 0) {
      sh.next_eval = static_cast<i64>(atomicAdd(p.counter, 1ull));
      sh.fallback = 0;
      sh.n_runs = 0;
    }
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
    const int family = FAM == KVS_FUSED_ANY ? st.family : FAM;
    const bool geometric = family == KVS_GBA || family == KVS_GSA;
    const bool sim = family == KVS_SIMS;
    const bool est = FAM == KVS_FUSED_ANY && p.key != nullptr;
    const bool keyed = !(family == KVS_GSA && !est);          // plain GSA keeps the index order
    const bool carry = geometric && (family == KVS_GSA || est);
    const bool est_class = est && family == KVS_GBA;          // classes by the clipped estimate
    const bool pow2 = geometric && st.alpha_num == 2 && st.alpha_den == 1 && st.beta0 <= 0;
    if (geometric && (st.subroutine | st.per_class_s)) {
      // the variants inside the geometric classes are the general kernel's
      if (tid == 0) p.slow_list[atomicAdd(p.slow_count, 1ull)] = e;
      continue;
    }
    // arrays in schedule order (of the instance)
    const int32_t* const S_ord = (keyed ? p.sorted_s : p.s) + lo;
    const int32_t* const O_ord = (keyed ? p.sorted_o : p.o) + lo;
    const int32_t* const K_ord = est ? p.sorted_key + lo : O_ord;
    const int32_t* const IPERM = keyed ? p.iperm + lo : nullptr;
    const int32_t* const O_JOB = p.o + lo;
    const i64* const ARR = p.arrival ? p.arrival + lo : nullptr;
    const i64 job_out = p.out.job_out_off ? p.out.job_out_off[e] : 0;
    int32_t* const out_start = p.out.job_start ? p.out.job_start + job_out : nullptr;
    int32_t* const out_done = p.out.job_completion ? p.out.job_completion + job_out : nullptr;
    const i64 prof_base = p.ev.profile_off ? p.ev.profile_off[e] : 0;
    const i64 prof_cap = (p.ev.profile && p.ev.profile_off) ? p.ev.profile_off[e + 1] - prof_base : 0;
    int32_t* const prof = p.ev.profile ? p.ev.profile + prof_base : nullptr;
    const bool want32 = p.out.job_start || p.out.job_completion;
    const bool event_form = p.do_profile && !geometric && p.prefix_s != nullptr && prof_cap == 0;
    const bool walk = p.do_profile && !event_form;            // rounds are walked tile by tile
    if (LIGHT && walk) {
      if (tid == 0) p.walk_list[atomicAdd(p.walk_count, 1ull)] = e;
      continue;
    }

    int status = stats.flags;
    if (!status && (X < 1 || stats.o_max > X)) status = KVS_EVAL_INFEASIBLE;
    if (!status && geometric) {
      if (tid < 32) ladder32(sh, X, st.alpha_num, st.alpha_den, st.beta0, static_cast<u32>(s_bar), static_cast<u32>(M));
      __syncthreads();
      if (sh.n_phases == 0) status = KVS_EVAL_RANGE;
    }

    FAcc acc;
    i64 base = 0;          // first round of the next phase
    i64 written_to = 0;    // profile rounds [0, written_to) have been written
    bool give_up = false;

    int seg_lo = 0;
    while (!status && !give_up && seg_lo < n) {
      // ---- window = offline sub-instance [seg_lo, seg_hi) ----
      if (tid == 0) {
        int end = n;
        if (p.window > 0 && ARR) {
          const i64 limit = (ARR[seg_lo] / p.window + 1) * p.window;
          int a = seg_lo + 1, b = n;
          while (a < b) { const int m = (a + b) >> 1; if (ARR[m] < limit) a = m + 1; else b = m; }
          end = a;
        }
        sh.seg_end = end;
      }
      __syncthreads();
      const int seg_hi = sh.seg_end;
      const int nseg = seg_hi - seg_lo;
      if (p.window > 0 && ARR) base = max_i64(base, (ARR[seg_lo] / p.window + 1) * p.window);

      int L = 1;
      if (geometric) {
        L = sh.n_phases;
        for (int q = tid; q <= L; q += T) {
          int v;
          if (q == 0) v = 0;
          else if (q == L || family == KVS_GSA) v = nseg;
          else {
            const i64 t = sh.tau[q - 1];
            int a = 0, b = nseg;
            while (a < b) { const int m = (a + b) >> 1; if (K_ord[seg_lo + m] <= t) a = m + 1; else b = m; }
            v = a;
          }
          sh.ent[q] = v;
        }
      } else if (tid == 0) {
        const i64 tau = st.tau > 0 ? st.tau : static_cast<i64>(K_ord[seg_hi - 1]);   // largest key of the segment
        i64 k = st.k;
        if (k <= 0) k = sim ? M / (s_bar + tau) : (s_bar + tau <= M ? static_cast<i64>(max_parallelism32(static_cast<u32>(tau), static_cast<u32>(s_bar), static_cast<u32>(M))) : 0);
        sh.tau[0] = static_cast<u32>(tau);
        sh.k[0] = k < 1 ? 0u : static_cast<u32>(k);
        sh.ent[0] = 0; sh.ent[1] = nseg;
      }
      if (carry) for (int i = tid; i < WARPS * MAXP; i += T) (&sh.cnt[0][0])[i] = 0;
      __syncthreads();
      if (!geometric && sh.k[0] < 1) { status = KVS_EVAL_INFEASIBLE; break; }

      // ---- plan: participants, length and first round of every phase ----
      const u32 Xc = static_cast<u32>(X);
      const int nsegs = (nseg + SEG - 1) / SEG;
      if (carry) {
        // leaving class of every position, and per segment the number of positions that leave in
        // phase q or later (row `seg` of the table, not yet summed over the segments before it)
        for (int seg = warp; seg < nsegs; seg += WARPS) {
          const int xb = seg * SEG + 8 * lane;
          u32 w0 = 0, w1 = 0;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int x = xb + j;
            u32 c = 0;
            if (x < nseg) {
              u32 v = static_cast<u32>(__ldg(O_ord + seg_lo + x));
              if (est_class) { const u32 kc = min(static_cast<u32>(__ldg(K_ord + seg_lo + x)), Xc); v = max(v, kc); }
              c = static_cast<u32>(pow2 ? class_pow2(Xc, v) : class_of(sh.tau, L, v));
              atomicAdd(&sh.cnt[warp][c], 1u);
            }
            if (j < 4) w0 |= c << (8 * j); else w1 |= c << (8 * (j - 4));
          }
          if (KVS_IN(xb + 7, cls_cap, CHK_CLS)) *reinterpret_cast<uint2*>(cls + xb) = make_uint2(w0, w1);
          __syncwarp();
          u32 h0 = lane < L ? sh.cnt[warp][lane] : 0u;
          u32 h1 = lane + 32 < L ? sh.cnt[warp][lane + 32] : 0u;
          u32 h2 = lane + 64 < L ? sh.cnt[warp][lane + 64] : 0u;
          if (lane < L) sh.cnt[warp][lane] = 0;
          if (lane + 32 < L) sh.cnt[warp][lane + 32] = 0;
          if (lane + 64 < L) sh.cnt[warp][lane + 64] = 0;
          h2 = warp_suffix(h2);
          h1 = warp_suffix(h1) + __shfl_sync(0xffffffffu, h2, 0);
          h0 = warp_suffix(h0) + __shfl_sync(0xffffffffu, h1, 0);
          if (KVS_IN(seg * L + L - 1, g_cap, CHK_G)) {
            if (lane < L) G[seg * L + lane] = h0;
            if (lane + 32 < L) G[seg * L + lane + 32] = h1;
            if (lane + 64 < L) G[seg * L + lane + 64] = h2;
          }
          __syncwarp();
        }
        __syncthreads();
        // exclusive sums over the segments; row nsegs = totals
        const int rpw = (nsegs + WARPS - 1) / WARPS;
        const int sa = min(nsegs, warp * rpw), sb = KVS_IN(nsegs * L + L - 1, g_cap, CHK_G) ? min(nsegs, sa + rpw) : sa;
        u32 a0 = 0, a1 = 0, a2 = 0;
        for (int seg = sa; seg < sb; ++seg) {
          if (lane < L) a0 += G[seg * L + lane];
          if (lane + 32 < L) a1 += G[seg * L + lane + 32];
          if (lane + 64 < L) a2 += G[seg * L + lane + 64];
        }
        sh.cnt[warp][lane] = a0; sh.cnt[warp][lane + 32] = a1; sh.cnt[warp][lane + 64] = a2;
        __syncthreads();
        u32 r0 = 0, r1 = 0, r2 = 0;
        for (int w = 0; w < warp; ++w) { r0 += sh.cnt[w][lane]; r1 += sh.cnt[w][lane + 32]; r2 += sh.cnt[w][lane + 64]; }
        for (int seg = sa; seg < sb; ++seg) {
          if (lane < L) { const u32 t = G[seg * L + lane]; G[seg * L + lane] = r0; r0 += t; }
          if (lane + 32 < L) { const u32 t = G[seg * L + lane + 32]; G[seg * L + lane + 32] = r1; r1 += t; }
          if (lane + 64 < L) { const u32 t = G[seg * L + lane + 64]; G[seg * L + lane + 64] = r2; r2 += t; }
        }
        if (warp == WARPS - 1 && KVS_IN(nsegs * L + L - 1, g_cap, CHK_G)) {
          // positions that leave in phase q or later: all of them take part in q once they have entered
          if (lane < L) { G[nsegs * L + lane] = r0; sh.np[lane] = r0; }
          if (lane + 32 < L) { G[nsegs * L + lane + 32] = r1; sh.np[lane + 32] = r1; }
          if (lane + 64 < L) { G[nsegs * L + lane + 64] = r2; sh.np[lane + 64] = r2; }
        }
        __syncthreads();
        for (int i = tid; i < WARPS * MAXP; i += T) (&sh.cnt[0][0])[i] = 0;
      }
      if (tid < L) {
        // entered by phase tid: positions below ent[tid + 1]; of those, the ones that leave in tid or later
        const u32 N = carry ? static_cast<u32>(sh.ent[tid + 1]) - static_cast<u32>(nseg) + sh.np[tid]
                            : static_cast<u32>(sh.ent[tid + 1] - sh.ent[tid]);
        sh.np[tid] = N;
        const u32 tau = sh.tau[tid], k = sh.k[tid];
        i64 len = 0;
        if (N > 0) len = (sim ? static_cast<i64>(ceil_div_u(N, k) - 1) * tau : static_cast<i64>(static_cast<u64>(N - 1) * tau / k)) + tau;
        sh.plen[tid] = len;
        sh.kinv[tid] = k >= 2 ? ~0ull / k + 1ull : 0ull;
        // memory is kept modulo 2^32: the general kernel reports evaluations whose bound reaches that
        if ((walk || event_form) && N > 0 && min_i64(N, static_cast<i64>(k) + 1) * (static_cast<i64>(stats.s_max) + tau) >= (static_cast<i64>(1) << 32))
          sh.fallback = 1;
      }
      __syncthreads();
      if (tid == 0) {
        i64 b = base, runs = sh.n_runs;
        u64 tp = 0;
        for (int q = 0; q < L; ++q) {
          sh.taupre[q] = tp;
          tp += sh.tau[q];
          sh.pbase[q] = static_cast<u32>(b);
          b += sh.plen[q];
          runs += sh.np[q];
          if (b >= TIME_LIMIT) { sh.fallback = 1; break; }
        }
        sh.taupre[L] = tp;
        sh.base_next = b;
        sh.n_runs = runs;
      }
      __syncthreads();
      if (sh.fallback) { give_up = true; break; }

      // ---- per-job results ----
      if (!carry) {
        // exactly one run per job; the rank is the position inside the class.  Four jobs per thread
        // and step, loads first, so that enough memory requests are in flight.
        const u32 tau0 = sh.tau[0];
        constexpr int JU = 4;
        for (int j0 = seg_lo + tid; j0 < seg_hi; j0 += JU * T) {
          u32 oj_[JU];
          int pos_[JU];
#pragma unroll
          for (int u = 0; u < JU; ++u) {
            const int j = j0 + u * T;
            oj_[u] = 0; pos_[u] = 0;
            if (j < seg_hi) {
              oj_[u] = static_cast<u32>(__ldg(O_JOB + j));
              pos_[u] = IPERM ? __ldg(IPERM + j) : j;
            }
          }
#pragma unroll
          for (int u = 0; u < JU; ++u) {
            const int j = j0 + u * T;
            if (j >= seg_hi) break;
            const u32 oj = oj_[u];
            int ph = 0;
            bool fin = true;
            if (geometric) ph = pow2 ? class_pow2(Xc, oj) : class_of(sh.tau, L, oj);
            else fin = oj <= tau0;
            const u32 rank = static_cast<u32>(pos_[u] - seg_lo - sh.ent[ph]);
            const u32 tau = sh.tau[ph], k = sh.k[ph];
            const u32 stt = sh.pbase[ph] + (sim ? (rank / k) * tau : slot_mul(rank, tau, k, sh.kinv[ph]));
            const u32 d = fin ? oj : tau;
            acc.steps += d;
            acc.hmax = max(acc.hmax, stt + d);
            int32_t start = -1, done = -1;
            if (fin) {
              start = static_cast<int32_t>(stt);
              done = static_cast<int32_t>(stt + oj);
              acc.flow += static_cast<u64>(static_cast<i64>(done) - (ARR ? __ldg(ARR + j) : 0));
            } else {
              ++acc.unfinished;
            }
            if (!KVS_IN(j, n, CHK_JOB_OUT)) continue;
            if (out_start) __stcs(&out_start[j], start);
            if (out_done) __stcs(&out_done[j], done);
          }
        }
      } else {
        // The rank of a job in the phase that completes it = positions before it that leave in that
        // phase or later: the table gives the count before the segment; inside the segment a lane
        // holds the classes of eight consecutive positions, and for every class q present one byte
        // compare per lane and one warp scan count the positions with class >= q before each lane.
        const bool vec_o = (reinterpret_cast<uintptr_t>(O_ord + seg_lo) & 15u) == 0;
        for (int seg = warp; seg < nsegs; seg += WARPS) {
          const int xb = seg * SEG + 8 * lane;
          const int room = nseg - xb;
          const u32 lim = room >= 8 ? 0xffu : (room > 0 ? (1u << room) - 1u : 0u);
          u32 ov_[8];
          if (vec_o && room >= 8) {
            const uint4 b0 = __ldg(reinterpret_cast<const uint4*>(O_ord + seg_lo + xb));
            const uint4 b1 = __ldg(reinterpret_cast<const uint4*>(O_ord + seg_lo + xb) + 1);
            ov_[0] = b0.x; ov_[1] = b0.y; ov_[2] = b0.z; ov_[3] = b0.w; ov_[4] = b1.x; ov_[5] = b1.y; ov_[6] = b1.z; ov_[7] = b1.w;
          } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) ov_[j] = (lim >> j & 1u) ? static_cast<u32>(__ldg(O_ord + seg_lo + xb + j)) : 0u;
          }
          const uint2 cw = KVS_IN(xb + 7, cls_cap, CHK_CLS) ? *reinterpret_cast<const uint2*>(cls + xb) : make_uint2(0, 0);
          // smallest and largest class among the warp's valid positions
          u32 lo4 = 0xffu, hi4 = 0u;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const u32 c = ((j < 4 ? cw.x : cw.y) >> (8 * (j & 3))) & 0xffu;
            if (lim >> j & 1u) { lo4 = min(lo4, c); hi4 = max(hi4, c); }
          }
          const int pmin = static_cast<int>(__reduce_min_sync(0xffffffffu, lo4));
          const int pmax = static_cast<int>(__reduce_max_sync(0xffffffffu, hi4));
          u32 rk_[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) rk_[j] = 0;
          for (int q = pmin; q <= pmax; ++q) {
            const u32 p4 = static_cast<u32>(q) * 0x01010101u;
            const u32 ge = (byte_mask4(cw.x, p4, true) | byte_mask4(cw.y, p4, true) << 4) & lim;
            const u32 eq = (byte_mask4(cw.x, p4, false) | byte_mask4(cw.y, p4, false) << 4) & lim;
            const u32 cnt = static_cast<u32>(__popc(ge));
            u32 incl = cnt;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
              const u32 y = __shfl_up_sync(0xffffffffu, incl, d);
              if (lane >= d) incl += y;
            }
            if (eq) {
              const u32 before = (KVS_IN(seg * L + q, g_cap, CHK_G) ? G[seg * L + q] : 0u) + incl - cnt;
#pragma unroll
              for (int j = 0; j < 8; ++j)
                if (eq >> j & 1u) rk_[j] = before + static_cast<u32>(__popc(ge & ((1u << j) - 1u)));
            }
          }
          u32 st_[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            st_[j] = 0;
            if (lim >> j & 1u) {
              const int l = static_cast<int>(((j < 4 ? cw.x : cw.y) >> (8 * (j & 3))) & 0xffu);
              int f = 0;
              if (est_class) {
                const u32 kc = min(static_cast<u32>(__ldg(K_ord + seg_lo + xb + j)), Xc);
                f = pow2 ? class_pow2(Xc, kc) : class_of(sh.tau, L, kc);
              }
              const u32 tau = sh.tau[l], k = sh.k[l];
              st_[j] = sh.pbase[l] + slot_mul(rk_[j], tau, k, sh.kinv[l]);
              acc.steps += ov_[j] + (sh.taupre[l] - sh.taupre[f]);
            }
          }
          if (keyed) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if ((lim >> j & 1u) && KVS_IN(seg_lo + xb + j, p.max_jobs, CHK_FIN)) fin_start[seg_lo + xb + j] = st_[j];
          } else {
            if (room > 0 && !KVS_IN(seg_lo + xb + min(room, 8) - 1, n, CHK_JOB_OUT)) continue;
            const bool vec_out = room >= 8 && ((seg_lo + xb) & 3) == 0 &&
                                 ((reinterpret_cast<uintptr_t>(out_start) | reinterpret_cast<uintptr_t>(out_done)) & 15u) == 0;
            u32 dn_[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              dn_[j] = st_[j] + ov_[j];
              if (lim >> j & 1u) {
                acc.hmax = max(acc.hmax, dn_[j]);
                acc.flow += static_cast<u64>(static_cast<i64>(dn_[j]) - (ARR ? __ldg(ARR + seg_lo + xb + j) : 0));
              }
            }
            if (vec_out) {
              if (out_start) {
                int4* const d = reinterpret_cast<int4*>(out_start + seg_lo + xb);
                __stcs(d, make_int4(static_cast<int>(st_[0]), static_cast<int>(st_[1]), static_cast<int>(st_[2]), static_cast<int>(st_[3])));
                __stcs(d + 1, make_int4(static_cast<int>(st_[4]), static_cast<int>(st_[5]), static_cast<int>(st_[6]), static_cast<int>(st_[7])));
              }
              if (out_done) {
                int4* const d = reinterpret_cast<int4*>(out_done + seg_lo + xb);
                __stcs(d, make_int4(static_cast<int>(dn_[0]), static_cast<int>(dn_[1]), static_cast<int>(dn_[2]), static_cast<int>(dn_[3])));
                __stcs(d + 1, make_int4(static_cast<int>(dn_[4]), static_cast<int>(dn_[5]), static_cast<int>(dn_[6]), static_cast<int>(dn_[7])));
              }
            } else {
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                if (lim >> j & 1u) {
                  if (out_start) __stcs(&out_start[seg_lo + xb + j], static_cast<int32_t>(st_[j]));
                  if (out_done) __stcs(&out_done[seg_lo + xb + j], static_cast<int32_t>(dn_[j]));
                }
              }
            }
          }
        }
        if (keyed) {
          __syncthreads();
          for (int j = seg_lo + tid; j < seg_hi; j += T) {
            const u32 oj = static_cast<u32>(__ldg(O_JOB + j));
            const int ip = __ldg(IPERM + j);
            if (!KVS_IN(ip, p.max_jobs, CHK_FIN) || !KVS_IN(j, n, CHK_JOB_OUT)) continue;
            const u32 stt = fin_start[ip];
            const u32 done = stt + oj;
            acc.hmax = max(acc.hmax, done);
            acc.flow += static_cast<u64>(static_cast<i64>(done) - (ARR ? __ldg(ARR + j) : 0));
            if (out_start) __stcs(&out_start[j], static_cast<int32_t>(stt));
            if (out_done) __stcs(&out_done[j], static_cast<int32_t>(done));
          }
        }
      }

      // ---- memory profile ----
      if (event_form) {
        // SPS / SimS in exact key order with no profile wanted: the peak comes from the run ends
        // (see kvs_events.cuh for why the last round of every run is enough), here in 32-bit
        // arithmetic, which the bound checked by the plan makes exact.
        const u32* const ps32 = reinterpret_cast<const u32*>(p.prefix_s + lo + st.instance + seg_lo);   // low words
        const u32 tau = sh.tau[0], k = sh.k[0];
        const u32 N = static_cast<u32>(nseg);
        const int32_t* const Ow = O_ord + seg_lo;
        if (sim) {
          // a batch is alone in its slot: in the last round of run i the jobs i .. end of the batch
          // are active with progress d_i - 1
          for (u32 i0 = tid; i0 < N; i0 += 4 * T) {
            u32 o_[4], p_[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const u32 i = i0 + u * T;
              o_[u] = i < N ? static_cast<u32>(__ldg(Ow + i)) : 0u;
              p_[u] = i < N ? ps32[2 * static_cast<size_t>(i)] : 0u;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const u32 i = i0 + u * T;
              if (i < N) {
                const u32 bend = min(N, (i / k + 1u) * k);
                const u32 d = min(o_[u], tau);
                acc.peak = max(acc.peak, ps32[2 * static_cast<size_t>(bend)] - p_[u] + (bend - i) * d);
              }
            }
          }
        } else {
          // Z[m] = sum over ranks j < m of (s_j - start_j): the jobs [i, b) active in round t hold
          // Z[b] - Z[i] + (b - i)(t + 1) tokens.  First Z for every rank, then one candidate per run.
          // four ranks per thread and step: shorter dependent chains than the ring's rounds per thread
          constexpr int EVI = 4;
          u32* const Z = reinterpret_cast<u32*>(cls);      // N + 1 words of this CTA's scratch
          const u32 qt = tau / k, rt = tau - qt * k;
          u32 F_run = 0;
          for (u32 c0 = 0; c0 <= N; c0 += (T * EVI)) {
            const u32 r = c0 + EVI * tid;
            u32 q = 0, rem = 0;
            if (r <= N) { u64 dq_, dr_; divmod_u(static_cast<u64>(r) * tau, k, &dq_, &dr_); q = static_cast<u32>(dq_); rem = static_cast<u32>(dr_); }
            u32 f[EVI], tot = 0;
#pragma unroll
            for (int j = 0; j < EVI; ++j) {
              f[j] = tot;
              if (r + j < N) tot += q;
              rem += rt; q += qt;
              if (rem >= k) { rem -= k; ++q; }
            }
            u32 incl = tot;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
              const u32 y = __shfl_up_sync(0xffffffffu, incl, d);
              if (lane >= d) incl += y;
            }
            __syncthreads();
            if (lane == 31) sh.redA[warp] = incl;
            __syncthreads();
            const u32 w = lane < WARPS ? sh.redA[lane] : 0u;
            u32 wi = w;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
              const u32 y = __shfl_up_sync(0xffffffffu, wi, d);
              if (lane >= d) wi += y;
            }
            const u32 off = F_run + __shfl_sync(0xffffffffu, wi - w, warp) + (incl - tot);
            F_run += __shfl_sync(0xffffffffu, wi, 31);
#pragma unroll
            for (int j = 0; j < EVI; ++j)
              if (r + j <= N && KVS_IN(r + j, z_cap, CHK_Z)) Z[r + j] = ps32[2 * static_cast<size_t>(r + j)] - (off + f[j]);
          }
          __syncthreads();
          for (u32 c0 = 0; c0 < N; c0 += (T * EVI)) {
            const u32 r = c0 + EVI * tid;
            if (r >= N) continue;
            u64 dq_, dr_;
            divmod_u(static_cast<u64>(r) * tau, k, &dq_, &dr_);
            u32 q = static_cast<u32>(dq_), rem = static_cast<u32>(dr_);
            u32 o_[EVI], z_[EVI];
#pragma unroll
            for (int j = 0; j < EVI; ++j) {
              o_[j] = r + j < N ? static_cast<u32>(__ldg(Ow + r + j)) : 0u;
              z_[j] = (r + j < N && KVS_IN(r + j, z_cap, CHK_Z)) ? Z[r + j] : 0u;
            }
#pragma unroll
            for (int j = 0; j < EVI; ++j) {
              if (r + j < N) {
                const u32 t1 = q + min(o_[j], tau);                       // last round of the run, plus one
                const u64 x = static_cast<u64>(t1) * k + (tau - 1u);      // b = ranks that start before t1
                const u32 b = (x >> 32) ? static_cast<u32>(min(static_cast<u64>(N), x / tau)) : min(N, static_cast<u32>(x) / tau);
                if (KVS_IN(b, z_cap, CHK_Z)) acc.peak = max(acc.peak, Z[b] - z_[j] + (b - (r + j)) * t1);
              }
              rem += rt; q += qt;
              if (rem >= k) { rem -= k; ++q; }
            }
          }
          __syncthreads();     // Z is scratch of the next window too
        }
      } else if (!LIGHT && walk) {
        bool list_mode = false;
        uint2* cur = list0;
        uint2* nxt = list1;
        int C = 0;
        // index order without estimates: the phases before the first class that holds a job are
        // walked from prefix sums of s + 1 over the positions (see pure_phase_events)
        int n_pure = 0;
        u32* const PS = reinterpret_cast<u32*>(list1);
        if (carry && !est) {
          while (n_pure + 1 < L && KVS_IN(nsegs * L + n_pure + 1, g_cap, CHK_G) && static_cast<int>(G[nsegs * L + n_pure + 1]) == nseg) ++n_pure;
          if (n_pure > 0) {
            u32 run = 0;
            for (int x0 = 0; x0 <= nseg; x0 += T * 4) {
              const int x = x0 + 4 * tid;
              u32 v[4], tot = 0;
#pragma unroll
              for (int j = 0; j < 4; ++j) { v[j] = tot; if (x + j < nseg) tot += static_cast<u32>(__ldg(S_ord + seg_lo + x + j)) + 1u; }
              u32 incl = tot;
#pragma unroll
              for (int d = 1; d < 32; d <<= 1) {
                const u32 y = __shfl_up_sync(0xffffffffu, incl, d);
                if (lane >= d) incl += y;
              }
              __syncthreads();
              if (lane == 31) sh.redA[warp] = incl;
              __syncthreads();
              const u32 w = lane < WARPS ? sh.redA[lane] : 0u;
              u32 wi = w;
#pragma unroll
              for (int d = 1; d < 32; d <<= 1) {
                const u32 y = __shfl_up_sync(0xffffffffu, wi, d);
                if (lane >= d) wi += y;
              }
              const u32 off = run + __shfl_sync(0xffffffffu, wi - w, warp) + (incl - tot);
              run += __shfl_sync(0xffffffffu, wi, 31);
#pragma unroll
              for (int j = 0; j < 4; ++j) if (x + j <= nseg && KVS_IN(x + j, 2 * list_cap, CHK_PS)) PS[x + j] = off + v[j];
            }
            __syncthreads();
          }
        }
        for (int ph = 0; ph < L; ++ph) {
          const int N = static_cast<int>(sh.np[ph]);
          if (N == 0) continue;
          PhaseView P;
          P.S = S_ord + seg_lo; P.O = O_ord + seg_lo;
          P.cls = cls; P.G = G; P.L = L; P.ph = ph; P.nsegs = nsegs;
          P.cls_cap = cls_cap; P.g_cap = g_cap;
          P.gcol = nullptr;
          if (carry && nsegs < GCOL) {
            for (int seg = tid; seg <= nsegs; seg += T)
              if (KVS_IN(seg * L + ph, g_cap, CHK_G)) sh.gcol[seg] = G[seg * L + ph];
            P.gcol = sh.gcol;
            __syncthreads();
          }
          P.n_src = nseg;
          P.x_lo = carry ? 0 : sh.ent[ph];
          P.x_hi = sh.ent[ph + 1];
          P.tau = sh.tau[ph]; P.k = sh.k[ph];
          P.qt = P.tau / P.k; P.rt = P.tau - P.qt * P.k;
          P.len = static_cast<u32>(sh.plen[ph]);
          P.base = sh.pbase[ph];
          const bool combine = sim && P.k >= 32;
          const bool dense = !sim && P.tau < TILE && P.k >= 4 * P.tau;
          ListView V;
          V.cur = cur; V.C = C; V.src = sh.ent[ph]; V.cap = list_cap;
          if (carry && !list_mode && 2 * N <= nseg) {
            // from here on the participants are kept as a list in rank order: first this phase's
            for (int seg = warp; seg < nsegs; seg += WARPS) {
              const LaneGroup g = lane_group<true>(P, seg);
              int r = g.r_first;
#pragma unroll
              for (int j = 0; j < 8; ++j)
                if (g.bits >> j & 1u) {
                  if (KVS_IN(r, list_cap, CHK_LIST_OUT)) cur[r] = make_uint2(static_cast<u32>(__ldg(P.S + g.xb + j)), static_cast<u32>(__ldg(P.O + g.xb + j)));
                  ++r;
                }
            }
            list_mode = true;
            V.C = N;
            __syncthreads();
          }
          int C_next = 0;
          // idle rounds before this phase (window release) hold nothing
          if (prof_cap > 0)
            for (i64 t = written_to + tid; t < P.base && t < prof_cap; t += T) prof[t] = 0;
          // tile origins keep the profile stores 16-byte aligned
          const int a0 = -static_cast<int>((prof_base + P.base) & 3);
          u32 A_run = 0, B_run = 0;
          int r_next = 0, buf = 0;
          // ranks that start before offset u: ceil(u*k/tau) (SPS) or ceil(u/tau)*k (SimS); the tile
          // ends advance by TILE, so quotient and remainder are stepped
          const u64 mult = sim ? 1 : static_cast<u64>(P.k);
          const u64 utau = P.tau;
          u64 cq, cr, dq, dr;
          divmod_u(static_cast<u64>(a0 + TILE) * mult, utau, &cq, &cr);
          divmod_u(static_cast<u64>(TILE) * mult, utau, &dq, &dr);
          for (int u0 = a0; u0 < static_cast<int>(P.len); u0 += TILE) {
            const int wlen = min(TILE, static_cast<int>(P.len) - u0);
            int r_b = N;                          // the last tile takes every remaining rank
            if (u0 + TILE < static_cast<int>(P.len)) {
              const u64 rb64 = (cq + (cr > 0)) * (sim ? static_cast<u64>(P.k) : 1ull);
              if (rb64 < static_cast<u64>(N)) r_b = static_cast<int>(rb64);
            }
            cq += dq; cr += dr;
            if (cr >= utau) { cr -= utau; ++cq; }
            if (ph < n_pure) pure_phase_events(sh, P, PS, 2 * list_cap, N, u0, buf);
            else if (sim) visit_runs<true, false>(sh, P, r_next, r_b, u0, buf, dense, combine);
            else if (list_mode) C_next = visit_list(sh, P, V, nxt, C_next, r_next, r_b, u0, buf, dense);
            else if (carry && P.tau < static_cast<u32>(TILE) && P.k >= 8u * P.tau) visit_runs_sliced(sh, P, r_next, r_b, u0, buf, sh.kinv[ph]);
            else if (carry) visit_runs<false, true>(sh, P, r_next, r_b, u0, buf, dense, combine);
            else visit_runs<false, false>(sh, P, r_next, r_b, u0, buf, dense, combine);
            r_next = r_b;
            if (P.tau > TILE && ph >= n_pure) {
              if (list_mode) insert_far_ends_list(sh, P, V, N, a0, u0, wlen, buf);
              else if (carry) insert_far_ends<true>(sh, P, sim, N, a0, u0, wlen, buf);
              else insert_far_ends<false>(sh, P, sim, N, a0, u0, wlen, buf);
            }
            __syncthreads();
            scan_tile(sh, buf, static_cast<i64>(P.base) + u0, wlen, P.base, A_run, B_run, acc.peak, prof, prof_cap);
            buf ^= 1;
          }
          written_to = static_cast<i64>(P.base) + P.len;
          if (list_mode) {
            __syncthreads();               // the list of killed jobs is complete before it is read
            uint2* const tmp = cur; cur = nxt; nxt = tmp;
            C = C_next;
          }
        }
      }
      base = sh.base_next;
      seg_lo = seg_hi;
    }

    if (give_up) {
      // left to the general kernel, which writes every output of this evaluation
      if (tid == 0) p.slow_list[atomicAdd(p.slow_count, 1ull)] = e;
      continue;
    }

    // ---- scalars ----
    const i64 flow = static_cast<i64>(block_sum(acc.flow, reinterpret_cast<u64*>(sh.red64)));
    const i64 steps = static_cast<i64>(block_sum(acc.steps, reinterpret_cast<u64*>(sh.red64)));
    const i64 hmax = block_max(acc.hmax, sh.redA, 0u);
    const int unfinished = block_sum(acc.unfinished, sh.red32);
    const u32 peak32 = block_max(acc.peak, sh.redA, 0u);
    const i64 peak = max_i64(static_cast<i64>(peak32), block_max(acc.peak64, sh.red64, static_cast<i64>(0)));
    if (tid == 0) {
      const bool skipped = (status & (KVS_EVAL_INFEASIBLE | KVS_EVAL_BAD_INPUT)) != 0;
      if (!skipped && prof_cap > 0 && hmax > prof_cap) status |= KVS_EVAL_CAPACITY;   // capacity 0 = profile not wanted
      const bool have_peak = p.do_profile && !skipped;
      if (p.ev.peak) p.ev.peak[e] = have_peak ? peak : -1;
      if (p.ev.flow) p.ev.flow[e] = flow;
      if (p.ev.job_steps) p.ev.job_steps[e] = steps;
      if (p.ev.horizon) p.ev.horizon[e] = hmax;
      if (p.ev.n_unfinished) p.ev.n_unfinished[e] = unfinished;
      if (p.ev.feasible) p.ev.feasible[e] = (have_peak && !(status & KVS_EVAL_RANGE) && peak <= M) ? 1 : 0;
      if (p.ev.status) p.ev.status[e] = status;
      if (p.out.n_runs) p.out.n_runs[e] = sh.n_runs;
    }
    (void)want32;
  }
}

}  // namespace

static size_t fused_smem_bytes(bool light) { return light ? offsetof(FShared, dA) : sizeof(FShared); }

template <bool LIGHT, int FAM>
static int ctas_per_sm() {
  int n = 0;
  cudaFuncSetAttribute(k_fused_eval<LIGHT, FAM>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(fused_smem_bytes(LIGHT)));
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k_fused_eval<LIGHT, FAM>, KVS_EVAL_THREADS, fused_smem_bytes(LIGHT)) != cudaSuccess) n = 1;
  return n < 1 ? 1 : n;
}

// CTAs per SM that every instantiation used for this kind of launch reaches.
int kvs_fused_ctas_per_sm(int light) {
  int n;
  if (light) {
    n = ctas_per_sm<true, KVS_FUSED_ANY>();
    n = min(n, min(min(ctas_per_sm<true, KVS_GBA>(), ctas_per_sm<true, KVS_GSA>()), min(ctas_per_sm<true, KVS_SPS>(), ctas_per_sm<true, KVS_SIMS>())));
  } else {
    n = min(ctas_per_sm<false, KVS_FUSED_ANY>(), min(ctas_per_sm<false, KVS_GBA>(), ctas_per_sm<false, KVS_GSA>()));
  }
  return n;
}

template <bool LIGHT, int FAM>
static cudaError_t launch(const BuildParams& p, int grid, cudaStream_t stream) {
  const cudaError_t err = cudaFuncSetAttribute(k_fused_eval<LIGHT, FAM>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(fused_smem_bytes(LIGHT)));
  if (err != cudaSuccess) return err;
  k_fused_eval<LIGHT, FAM><<<grid, KVS_EVAL_THREADS, fused_smem_bytes(LIGHT), stream>>>(p);
  return cudaGetLastError();
}

// The caller zeroes the counters.  light: the variant without the ring (see k_fused_eval); fam:
// KVS_FUSED_ANY, or a family id for a list of that family alone in a call without estimates (the
// full variant has such kernels for the two geometric families, the light one for all four).
cudaError_t kvs_launch_fused(const BuildParams& p, int grid, int light, int fam, cudaStream_t stream) {
  if (p.P <= 0) return cudaSuccess;
  if (light) {
    switch (fam) {
      case KVS_GBA: return launch<true, KVS_GBA>(p, grid, stream);
      case KVS_GSA: return launch<true, KVS_GSA>(p, grid, stream);
      case KVS_SPS: return launch<true, KVS_SPS>(p, grid, stream);
      case KVS_SIMS: return launch<true, KVS_SIMS>(p, grid, stream);
      default: return launch<true, KVS_FUSED_ANY>(p, grid, stream);
    }
  }
  if (fam == KVS_GBA) return launch<false, KVS_GBA>(p, grid, stream);
  if (fam == KVS_GSA) return launch<false, KVS_GSA>(p, grid, stream);
  return launch<false, KVS_FUSED_ANY>(p, grid, stream);
}

// First violation recorded by the checked build (0 = none); `compiled` = 1 if this library was built with
// -DKVS_DEBUG.  `reset` clears the word after reading it.
cudaError_t kvs_fused_check_word(unsigned long long* word, int* compiled, int reset) {
#ifdef KVS_DEBUG
  if (compiled) *compiled = 1;
  cudaError_t e = cudaMemcpyFromSymbol(word, g_check_word, sizeof(unsigned long long));
  if (e == cudaSuccess && reset) { const unsigned long long z = 0ull; e = cudaMemcpyToSymbol(g_check_word, &z, sizeof(z)); }
  return e;
#else
  if (compiled) *compiled = 0;
  *word = 0ull;
  (void)reset;
  return cudaSuccess;
#endif
}
