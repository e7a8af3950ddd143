// Geometric ladder of slice lengths and the largest memory-feasible parallelism of each slice (first
// line of the two geometric algorithms; Lemma "Peak Memory Usage of SPS"; Eq. max-parallelism), and
// the class of a response length.  Shared by the fused kernels, the bound kernel and the speculative-run kernel.
#pragma once

#include "kvs_internal.cuh"

#ifdef __CUDACC__

typedef unsigned __int128 u128;

__device__ __forceinline__ u32 gcd_u32(u32 x, u32 y) {
  while (y) { const u32 t = x % y; x = y; y = t; }
  return x;
}

// Largest k >= 1 with s*k + (tau*k + tau + k - gcd(tau, k))/2 <= M, given s + tau <= M: the
// condition reads k*(2s+tau+1) <= 2M - tau + gcd(tau,k), and 1 <= gcd <= tau leaves k0 or k0 + 1
// with k0 = floor((2M - tau + 1) / (2s + tau + 1)).
__device__ inline u32 max_parallelism32(u32 tau, u32 s, u32 M) {
  const u64 D = 2ull * s + tau + 1ull;
  const u64 num = 2ull * M - tau + 1ull;
  u64 k0, r;
  divmod_u(num, D, &k0, &r);
  const u64 k1 = k0 + 1;
  if (k1 >> 31) return static_cast<u32>(k0);
  return (k1 * D <= 2ull * M - tau + gcd_u32(tau, static_cast<u32>(k1))) ? static_cast<u32>(k1) : static_cast<u32>(k0);
}

// The same in 64-bit arithmetic (the general kernel: budgets and slices up to 2^31, carried in int64).
__device__ __forceinline__ i64 gcd_i64(i64 x, i64 y) {
  while (y) { const i64 t = x % y; x = y; y = t; }
  return x;
}
__device__ inline i64 max_parallelism64(i64 tau, i64 s, i64 M) {
  const i64 D = 2 * s + tau + 1;
  const i64 k0 = (2 * M - tau + 1) / D;
  const i64 k1 = k0 + 1;
  return (k1 * D <= 2 * M - tau + gcd_i64(tau, k1)) ? k1 : k0;
}

// The ladder tau_0 .. tau_(L-1) of one evaluation and, through `par(tau)`, the parallelism of every slice.
// `sh` provides pw_a, pw_b (u128 [MAXP + 1]), tau, k ([MAXP], 32- or 64-bit) and n_phases (0 = the ladder
// needs more than MAXP slices); called by one warp.
template <class Sh, class Par>
__device__ __forceinline__ void ladder_phases(Sh& sh, i64 X, int a, int b, i64 beta0, Par par) {
  constexpr int MAXP = KVS_MAX_PHASES;
  typedef decltype(sh.tau[0] + 0) V;                      // value type of the tables
  const int lane = lane_id();
  if (beta0 <= 0) {
    if (lane == 0) {
      // ell = largest j with a^j <= X * b^j, powers kept exactly in 128 bits
      u128 pa = 1, pb = 1;
      int ell = 0;
      sh.pw_a[0] = 1; sh.pw_b[0] = 1;
      while (ell + 1 < MAXP + 1) {
        const u128 na = pa * static_cast<u128>(a), nb = pb * static_cast<u128>(b);
        if (na > static_cast<u128>(X) * nb) break;
        pa = na; pb = nb; ++ell;
        sh.pw_a[ell] = pa; sh.pw_b[ell] = pb;
      }
      sh.n_phases = (ell + 1 <= MAXP) ? ell + 1 : 0;
    }
    __syncwarp();
    const int L = sh.n_phases;
    for (int p = lane; p < L; p += 32) {
      const int j = L - 1 - p;  // tau_p = floor(X * b^j / a^j)
      const V t = (a == 2 && b == 1) ? static_cast<V>(X >> j)
                                     : static_cast<V>(static_cast<u128>(X) * sh.pw_b[j] / sh.pw_a[j]);
      sh.tau[p] = t;
      sh.k[p] = par(t);
    }
  } else {
    if (lane == 0) {
      u128 pa = 1, pb = 1;
      int p = 0;
      for (;; ++p) {
        if (p >= MAXP) { p = -1; break; }
        const u128 num = static_cast<u128>(beta0) * pa;   // tau_p = min(floor(beta0 * a^p / b^p), X)
        const V t = (num >= static_cast<u128>(X) * pb) ? static_cast<V>(X) : static_cast<V>(num / pb);
        sh.tau[p] = t;
        sh.k[p] = par(t);
        if (static_cast<i64>(t) >= X) break;
        pa *= static_cast<u128>(a); pb *= static_cast<u128>(b);
      }
      sh.n_phases = p + 1;
    }
  }
  __syncwarp();
}

// 32-bit tables with the largest memory-feasible parallelism of the staggered pipeline.
template <class Sh>
__device__ __forceinline__ void ladder32(Sh& sh, i64 X, int a, int b, i64 beta0, u32 s_bar, u32 M) {
  ladder_phases(sh, X, a, b, beta0, [=](u32 t) { return max_parallelism32(t, s_bar, M); });
}

// class(v) = first p with tau_p >= v (tau is nondecreasing and tau_(L-1) >= v)
__device__ __forceinline__ int class_of(const u32* tau, int L, u32 v) {
  int a = 0, b = L - 1;
  while (a < b) { const int m = (a + b) >> 1; if (tau[m] >= v) b = m; else a = m + 1; }
  return a;
}

// The same for the ladder of alpha = 2, tau_p = X >> (ell - p) with ell = floor(log2 X): the largest
// shift j with (X >> j) >= v is the difference of the bit lengths, or one less.  1 <= v <= X.
__device__ __forceinline__ int class_pow2(u32 X, u32 v) {
  const int j0 = __clz(v) - __clz(X);
  const int j = (X >> j0) >= v ? j0 : j0 - 1;
  return (31 - __clz(X)) - j;
}

#endif  // __CUDACC__
