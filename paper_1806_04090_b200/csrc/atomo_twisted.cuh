// Eigenvector of a symmetric tridiagonal matrix for a given eigenvalue: twisted factorisation (device code shared by
// the two vector kernels of the tridiagonal routes; the work vectors may sit in shared or in global memory).
#pragma once
#include "atomo_common.cuh"

namespace atomo {

__device__ __forceinline__ bool finite64(double x) { return fabs(x) <= 1.7e308; }
constexpr double kPivMin = 1.0e-280;

// Twisted factorisation of T - lambda I: forward pivots D+_i = p_i / p_{i-1} from the leading principal minors
// p_i = (d_i - lambda) p_{i-1} - e_{i-1}^2 p_{i-2} (lane 0), backward pivots D- from the trailing ones (lane 1, the same
// instructions on mirrored indices).  The recurrences carry no division: numerator and denominator of every pivot
// are stored as a pair (the running pair is rescaled by a power of two every 8 steps, after it was stored) and the
// quotients are taken by all lanes afterwards.  Twist index at the smallest |gamma_k| = |D+_k + D-_k - (d_k - lambda)|,
// z_k = 1, z_i = -(e_i / D+_i) z_{i+1} above and z_{i+1} = -(e_i / D-_{i+1}) z_i below.  Returns gamma_k / z^T z, the
// Rayleigh-quotient correction of lambda.  wa, wb, wc, wd, z: r doubles each, in shared or global memory.
static __device__ __noinline__ double twisted_vector(const double* __restrict__ d, const double* __restrict__ e, int r, double lambda,
                                 double* wa, double* wb, double* wc, double* wd, double* z, int lane, int skip,
                                 double* znorm2) {
  if (lane < 2) {
    const bool back = lane == 1;
    double* N = back ? wb : wa;                               // numerators
    double* Q = back ? wd : wc;                               // denominators
    int cur = back ? r - 1 : 0;
    double pm = 1.0, p = d[cur] - lambda;
    N[cur] = p; Q[cur] = pm;
    double ee = r > 1 ? e[back ? r - 2 : 0] : 0.0;
    double dn = r > 1 ? d[back ? r - 2 : 1] : 0.0;
    for (int t = 0; t + 1 < r; ++t) {
      const int nxt = back ? cur - 1 : cur + 1;
      const int ie2 = back ? max(r - 3 - t, 0) : min(t + 1, r - 2);      // next step's off-diagonal and diagonal
      const int in2 = back ? max(nxt - 1, 0) : min(nxt + 1, r - 1);
      const double ee2 = e[ie2], dn2 = d[in2];
      const double pn = fma(dn - lambda, p, -(ee * ee) * pm);
      N[nxt] = pn; Q[nxt] = p;
      pm = p; p = pn;
      if ((t & 7) == 7) {
        const int ex = ((__double2hiint(fabs(p) + fabs(pm)) >> 20) & 0x7ff) - 1023;
        const double sc = __hiloint2double((1023 - max(min(ex, 1022), -1022)) << 20, 0);
        p *= sc; pm *= sc;
      }
      cur = nxt; ee = ee2; dn = dn2;
    }
  }
  __syncwarp();
  // pivots: wa <- D+, wb <- D- (a zero or non-finite quotient is replaced, as a perturbed pivot would be)
  for (int i = lane; i < r; i += 32) {
    double dp = wa[i] / wc[i], dm = wb[i] / wd[i];
    if (!(fabs(dp) >= kPivMin)) dp = kPivMin;
    if (!(fabs(dm) >= kPivMin)) dm = kPivMin;
    if (!finite64(dp)) dp = 1.0e300;
    if (!finite64(dm)) dm = 1.0e300;
    wa[i] = dp; wb[i] = dm;
  }
  __syncwarp();
  // twist index: the (skip+1)-th smallest |gamma| (lowest index on ties).  skip > 0 for the later members of a group
  // of kept atoms with coinciding eigenvalues: z = gamma_k (T - lambda I)^{-1} e_k, so another k is another start
  // vector of inverse iteration and gives another vector of the invariant subspace.
  double best = -1.0; int bk = -1;
  for (int pick = 0; pick <= skip; ++pick) {
    const double pb = best; const int pk = bk;
    double cb = 1.0e300; int ck = 0x7fffffff;
    for (int i = lane; i < r; i += 32) {
      const double gam = fabs(wa[i] + wb[i] - (d[i] - lambda));
      const bool after = gam > pb || (gam == pb && i > pk);   // not picked yet
      if (after && (gam < cb || (gam == cb && i < ck))) { cb = gam; ck = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double ob = __shfl_xor_sync(0xffffffffu, cb, o);
      const int ok = __shfl_xor_sync(0xffffffffu, ck, o);
      if (ob < cb || (ob == cb && ok < ck)) { cb = ob; ck = ok; }
    }
    if (ck == 0x7fffffff) break;                              // fewer candidates than skip (non-finite input)
    best = cb; bk = ck;
  }
  if (bk < 0) bk = 0;
  const double gamma = wa[bk] + wb[bk] - (d[bk] - lambda);
  __syncwarp();
  // multipliers in place: wa[i] <- e_i / D+_i (i < r-1), wb[i] <- e_i / D-_{i+1}
  for (int i0 = 0; i0 < r; i0 += 32) {
    const int i = i0 + lane;
    double l = 0.0, u = 0.0;
    if (i + 1 < r) { l = e[i] / wa[i]; u = e[i] / wb[i + 1]; }
    __syncwarp();
    if (i < r) { wa[i] = l; wb[i] = u; }
    __syncwarp();
  }
  if (lane == 0) z[bk] = 1.0;
  __syncwarp();
  if (lane < 2) {
    const bool down = lane == 1;
    double zz = 1.0;
    const int n = down ? r - 1 - bk : bk;
    for (int t = 0; t < n; ++t) {
      const int i = down ? bk + t : bk - 1 - t;               // multiplier index
      zz = -(down ? wb[i] : wa[i]) * zz;
      z[down ? i + 1 : i] = zz;
    }
  }
  __syncwarp();
  double n2 = 0.0;
  for (int i = lane; i < r; i += 32) n2 = fma(z[i], z[i], n2);
  n2 = warp_sum(n2);
  *znorm2 = n2;
  return gamma / n2;
}


}  // namespace atomo
