// Bounds on total flow time that depend on an instance only through its class sizes
// (Lemma "Area-Based Lower Bound for OPT", Lemma "GBA Upper Bound via Packing Efficiency",
// Lemma "GSA Upper Bound via Packing Efficiency").
//
// One CTA per (instance, setting): the ladder tau_p with k_p = k*(tau_p, s_bar), a histogram of
// the classes of the response lengths (class = first p with tau_p >= o), then one thread adds up,
// phase by phase in exact 128-bit integers,
//   ladder term        Q_p = n_p tau_p + sum_{i < n_p} floor(i tau_p / k_p)   (closed form: floor sum)
//   class-prefix term  S_p = sum_{q < p} (floor(n_q tau_q / k_q) + tau_q)
//   UpperGBA           = sum_p (n_p S_p + Q_p)
//   spillover cost     D_p = ceil(n_{>p} tau_p / k_p)
//   phase-prefix cost  T_p = sum_{q < p} (floor(n_{>=q} tau_q / k_q) + tau_q)
//   GSA bound          = sum_p n_p (T_p + D_p) + sum_p Q_p
//   2 M * lower bound  = sum_p 2 Area(x_p, s_bar) (n_p (n_p + 1) / 2 + n_{>p} n_p),
//                        Area(x, s) = s x + x (x + 1) / 2, x_0 = 0 and x_p = tau_(p-1): every job of
//                        class p is longer than x_p (the integer part of the paper's real threshold).
#include "kvs_ladder.cuh"

namespace {

constexpr int BT = 256;
constexpr int MAXP = KVS_MAX_PHASES;

struct BShared {
  u128 pw_a[MAXP + 1];
  u128 pw_b[MAXP + 1];
  u32 tau[MAXP], k[MAXP];
  u32 cnt[MAXP];
  int n_phases;
};

// sum_{i=0}^{n-1} floor(i * a / m), exact in 128 bits (n, a, m below 2^31): the Euclid-like
// recursion on (a mod m, m) with the quotient parts taken out in closed form.
__device__ u128 floor_sum128(u64 n, u64 m, u64 a) {
  u128 ans = 0;
  u64 b = 0;
  for (;;) {
    if (a >= m) { ans += static_cast<u128>(n - 1) * n / 2 * (a / m); a %= m; }
    if (b >= m) { ans += static_cast<u128>(n) * (b / m); b %= m; }
    const u64 y = a * n + b;            // below 2^31 * 2^31 + 2^31
    if (y < m) break;
    n = y / m;
    b = y % m;
    const u64 t = m; m = a; a = t;
  }
  return ans;
}

__global__ void __launch_bounds__(BT) k_bounds(const i64* __restrict__ job_off, const int32_t* __restrict__ o,
                                               const InstStats* __restrict__ stats, const kvs_setting* __restrict__ settings,
                                               i64 P, kvs_bounds_out out) {
  __shared__ BShared sh;
  const int tid = threadIdx.x;
  for (i64 e = blockIdx.x; e < P; e += gridDim.x) {
    __syncthreads();
    const kvs_setting st = settings[e];
    const i64 lo = job_off[st.instance];
    const InstStats is = stats[st.instance];
    const int n = is.flags ? 0 : static_cast<int>(job_off[st.instance + 1] - lo);
    const i64 M = st.M;
    const i64 s_bar = st.s_bar >= 0 ? st.s_bar : is.s_max;
    const i64 X = M - s_bar;
    int status = is.flags;
    if (!status && (X < 1 || is.o_max > X)) status = KVS_EVAL_INFEASIBLE;
    if (!status) {
      if (tid < 32) ladder32(sh, X, st.alpha_num, st.alpha_den, st.beta0, static_cast<u32>(s_bar), static_cast<u32>(M));
      for (int i = tid; i < MAXP; i += BT) sh.cnt[i] = 0;
      __syncthreads();
      if (sh.n_phases == 0) status = KVS_EVAL_RANGE;
    }
    u128 upper_gba = 0, gsa = 0, lower = 0;
    if (!status) {
      const int L = sh.n_phases;
      const bool pow2 = st.alpha_num == 2 && st.alpha_den == 1 && st.beta0 <= 0;
      const u32 Xc = static_cast<u32>(X);
      for (int j = tid; j < n; j += BT) {
        const u32 v = static_cast<u32>(__ldg(o + lo + j));
        atomicAdd(&sh.cnt[pow2 ? class_pow2(Xc, v) : class_of(sh.tau, L, v)], 1u);
      }
      __syncthreads();
      if (tid == 0) {
        const u128 LIMIT = (static_cast<u128>(1) << 63) - 1;
        u128 class_prefix = 0, phase_prefix = 0;
        u64 later = static_cast<u64>(n);      // jobs in this class or a later one
        for (int p = 0; p < L; ++p) {
          const u64 np = sh.cnt[p], t = sh.tau[p], kk = sh.k[p];
          const u64 n_ge = later, n_gt = later - np;
          const u128 Q = static_cast<u128>(np) * t + (np ? floor_sum128(np, kk, t) : 0);
          upper_gba += static_cast<u128>(np) * class_prefix + Q;
          const u128 D = (static_cast<u128>(n_gt) * t + kk - 1) / kk;
          gsa += static_cast<u128>(np) * (phase_prefix + D) + Q;
          const u128 x = p == 0 ? 0 : sh.tau[p - 1];
          const u128 area2 = 2 * static_cast<u128>(s_bar) * x + x * (x + 1);
          lower += area2 * (static_cast<u128>(np) * (np + 1) / 2 + static_cast<u128>(n_gt) * np);
          class_prefix += static_cast<u128>(np) * t / kk + t;
          phase_prefix += static_cast<u128>(n_ge) * t / kk + t;
          later -= np;
          if (upper_gba > LIMIT || gsa > LIMIT || lower > LIMIT) { status = KVS_EVAL_RANGE; break; }
        }
      }
    }
    if (tid == 0) {
      const bool ok = status == 0;
      if (out.upper_gba) out.upper_gba[e] = ok ? static_cast<i64>(upper_gba) : -1;
      if (out.upper_gsa) out.upper_gsa[e] = ok ? static_cast<i64>(gsa) : -1;
      if (out.lower_2m) out.lower_2m[e] = ok ? static_cast<i64>(lower) : -1;
      if (out.status) out.status[e] = status;
    }
  }
}

}  // namespace

cudaError_t kvs_launch_bounds(const i64* job_off, const int32_t* o, const InstStats* stats, const kvs_setting* settings,
                              i64 P, const kvs_bounds_out& out, int grid, cudaStream_t stream) {
  if (P <= 0) return cudaSuccess;
  k_bounds<<<grid, BT, 0, stream>>>(job_off, o, stats, settings, P, out);
  return cudaGetLastError();
}
