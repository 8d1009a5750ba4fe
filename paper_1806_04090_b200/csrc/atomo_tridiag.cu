// Spectral atoms by the tridiagonal route (Section 5 of the paper asks for the SVD of every layer gradient; only
// the singular VALUES of all atoms enter the probabilities of Eq. 3 / Algorithm 1, and only the few KEPT atoms of
// Eq. 2 need their vectors).  For layers with a short side of at most 512:
//
//   sp_tridiag_cluster_kernel : Householder reduction of the scaled Gram matrix A (r x r) to a symmetric
//                               tridiagonal T = Q^T A Q, in fp64.  A layer's rows are dealt cyclically to rp/32 CTAs
//                               of a 16-CTA cluster and stay in shared memory; per step the pivot column and the
//                               product A v travel through distributed shared memory (two cluster barriers per
//                               step).  The reflectors go to global memory for the back-transformation.
//   sp_bisect_kernel          : all eigenvalues of T, one warp per eigenvalue: 8 rounds of 33-section on Sturm
//                               counts (division-free three-term recurrence with power-of-two rescaling).
//   (sp_finalize_sample_kernel sorts, solves Algorithm 1 and draws, as for the other routes)
//   sp_eigvec_kernel          : for the kept atoms only: eigenvector of T by a twisted factorisation with one
//                               Rayleigh-quotient correction, back-transformation u = Q z with the reflectors
//                               (four at a time), normalised short-side vector into the payload; kept atoms with
//                               nearly equal eigenvalues are orthogonalised against each other at the end.
//
// Work per layer: about 2 r^3 fp64 flops for the reduction (full symmetric storage: matrix-vector product and
// rank-two update of the trailing block), r^2 * 8 * 33 recurrence steps for the eigenvalues, O(r^2) per kept atom.
#include <cooperative_groups.h>

#include "atomo_kernels.cuh"

namespace cg = cooperative_groups;

namespace atomo {

namespace {

constexpr int kTriCtas = 16;          // CTAs per cluster
constexpr int kTriThreads = 512;
constexpr int kTriWarps = kTriThreads / 32;
constexpr int kTriRows = 32;          // rows of A per CTA
constexpr int kTriMaxRp = 512;        // largest padded short side
constexpr int kTriCols = kTriMaxRp / 32;   // columns per lane

__device__ __forceinline__ bool finite64(double x) { return fabs(x) <= 1.7e308; }

}  // namespace

// ---- Householder tridiagonalisation ------------------------------------------------------------------------
// Step k (k = 0 .. r-3) with x = A[k+1.., k]:  alpha = -sign(x_0) ||x||,  v = x - alpha e_1,  beta = 2 / v^T v,
// H = I - beta v v^T;  p = beta A22 v,  K = beta/2 p^T v,  w = p - K v,  A22 -= v w^T + w v^T;  d_k = A[k][k],
// e_k = alpha.  Row i of a layer lives in the CTA with group rank i mod nc at local row i / nc.
__global__ void __launch_bounds__(kTriThreads, 1) sp_tridiag_cluster_kernel(const SpLayer* __restrict__ layers,
                                                                            const ClusterCta* __restrict__ ctas) {
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ __align__(16) unsigned char tri_smem[];
  double* As = reinterpret_cast<double*>(tri_smem);          // [32][rp]
  __shared__ double s_v[2][kTriMaxRp];                        // pivot column of step k in s_v[k & 1] (written by the row owners)
  __shared__ double s_p[kTriMaxRp];                           // beta A22 v (written by the row owners)
  const ClusterCta me = ctas[blockIdx.x];
  const int tid = threadIdx.x, lane = tid % 32, w = tid / 32;
  // every CTA of the cluster keeps the same number of barriers: the longest reduction among the cluster's layers
  int steps = 0;
  {
    const int c0 = blockIdx.x / kTriCtas * kTriCtas;
    for (int c = 0; c < kTriCtas; ++c) { const int l = ctas[c0 + c].layer; if (l >= 0) steps = max(steps, layers[l].r - 2); }
  }
  cluster.sync();                                             // every CTA of the cluster runs: remote stores may start
  if (me.layer < 0) {
    for (int k = 0; k < steps; ++k) { cluster.sync(); cluster.sync(); }
    cluster.sync();
    return;
  }
  const SpLayer& L = layers[me.layer];
  const int r = L.r, rp = L.rp, nc = me.pad, g = me.slot, base = me.base_rank;
  const int ncol = rp / 32;                                   // columns per lane: j = lane + 32 m
  for (int li = w; li < kTriRows; li += kTriWarps) {
    const int i = li * nc + g;
    for (int j = lane; j < rp; j += 32) As[li * rp + j] = (i < r && j < r) ? (double)L.A[(int64_t)i * L.lda + j] : 0.0;
  }
  __syncthreads();
  const int my_steps = max(r - 2, 0);
  for (int k = 0; k < steps; ++k) {
    const bool active = k < my_steps;
    const int par = k & 1;
    if (active) {
      // pivot column: every owned entry below the diagonal goes to all CTAs of the layer
      const int li = tid % kTriRows, dest = tid / kTriRows;
      const int i = li * nc + g;
      if (dest < nc && i > k && i < r) cluster.map_shared_rank(&s_v[0][0], base + dest)[par * kTriMaxRp + i] = As[li * rp + k];
      if (tid == 0 && k % nc == g) L.td_d[k] = As[(k / nc) * rp + k];
    }
    cluster.sync();
    double v[kTriCols];
    double beta = 0.0, v0 = 0.0;
    if (active) {
      // every warp forms v and beta from the same values in the same order (no broadcast needed)
      double nx2 = 0.0;
#pragma unroll
      for (int m = 0; m < kTriCols; ++m) {
        const int j = lane + 32 * m;
        v[m] = (m < ncol && j > k && j < r) ? s_v[par][j] : 0.0;
        nx2 = fma(v[m], v[m], nx2);
      }
      nx2 = warp_sum(nx2);
      const double x0 = s_v[par][k + 1];
      double alpha = 0.0;
      if (nx2 > 0.0) {
        alpha = -copysign(sqrt(nx2), x0);
        v0 = x0 - alpha;
        const double den = alpha * (alpha - x0);              // = v^T v / 2 > 0
        beta = den > 0.0 ? 1.0 / den : 0.0;
      }
      // v = x with its first entry replaced (a zero column leaves H = I)
#pragma unroll
      for (int m = 0; m < kTriCols; ++m) {
        if (!(nx2 > 0.0)) v[m] = 0.0;
        else if (lane + 32 * m == k + 1) v[m] = v0;
      }
      if (k % nc == g) {                                      // one CTA of the layer files the step's results
        if (tid == 0) { L.td_e[k] = alpha; L.td_tau[k] = beta; }
        if (w == 1) {
#pragma unroll
          for (int m = 0; m < kTriCols; ++m) if (m < ncol && lane + 32 * m < r) L.td_V[(int64_t)k * r + lane + 32 * m] = v[m];
        }
      }
      // p_i = beta sum_j A_ij v_j for the owned rows below the pivot
      for (int li = w; li < kTriRows; li += kTriWarps) {
        const int i = li * nc + g;
        if (i > k && i < r) {
          const double* row = As + li * rp;
          double acc = 0.0;
#pragma unroll
          for (int m = 0; m < kTriCols; ++m) if (m < ncol) acc = fma(row[lane + 32 * m], v[m], acc);
          acc = warp_sum(acc) * beta;
          if (lane < nc) cluster.map_shared_rank(&s_p[0], base + lane)[i] = acc;
        }
      }
    }
    cluster.sync();
    if (active) {
      double wv[kTriCols];
      double pv = 0.0;
#pragma unroll
      for (int m = 0; m < kTriCols; ++m) {
        const int j = lane + 32 * m;
        wv[m] = (m < ncol && j > k && j < r) ? s_p[j] : 0.0;
        pv = fma(wv[m], v[m], pv);
      }
      pv = warp_sum(pv);
      const double K = 0.5 * beta * pv;
#pragma unroll
      for (int m = 0; m < kTriCols; ++m) wv[m] = fma(-K, v[m], wv[m]);
      for (int li = w; li < kTriRows; li += kTriWarps) {
        const int i = li * nc + g;
        if (i > k && i < r) {
          // v_i and w_i of this row, from the same shared arrays every warp read its columns from
          const double vi = beta == 0.0 ? 0.0 : (i == k + 1 ? v0 : s_v[par][i]);
          const double wi = fma(-K, vi, s_p[i]);
          double* row = As + li * rp;
#pragma unroll
          for (int m = 0; m < kTriCols; ++m)
            if (m < ncol) row[lane + 32 * m] -= fma(vi, wv[m], wi * v[m]);
        }
      }
    }
    __syncthreads();                                          // the next pivot column is read with another thread mapping
  }
  // the last 2 x 2 block (r >= 2) or the single entry (r = 1)
  if (tid == 0) {
    if (r >= 2) {
      if ((r - 2) % nc == g) L.td_d[r - 2] = As[((r - 2) / nc) * rp + (r - 2)];
      if ((r - 1) % nc == g) { L.td_d[r - 1] = As[((r - 1) / nc) * rp + (r - 1)]; L.td_e[r - 2] = As[((r - 1) / nc) * rp + (r - 2)]; }
    } else if (g == 0) {
      L.td_d[0] = As[0];
    }
  }
  cluster.sync();                                             // nobody leaves while a peer may still write here
}

// ---- eigenvalues of T: Sturm counts -------------------------------------------------------------------------
// count(x) = number of eigenvalues below x = sign changes of p_0 = 1, p_1 = d_0 - x, p_{i+1} = (d_i - x) p_i -
// e_{i-1}^2 p_{i-1}.  The pair (p_i, p_{i-1}) is rescaled by a power of two every 8 steps (ratios and signs keep).
__device__ __forceinline__ int sturm_count(const double* __restrict__ d, const double* __restrict__ e2, int r, double x) {
  double pm = 1.0, p = d[0] - x;
  int cnt = p < 0.0 ? 1 : 0;
  for (int i = 1; i < r; ++i) {
    const double pn = fma(d[i] - x, p, -e2[i - 1] * pm);
    cnt += ((pn < 0.0) != (p < 0.0)) ? 1 : 0;
    pm = p; p = pn;
    if ((i & 7) == 0) {
      const int ex = ((__double2hiint(fabs(p) + fabs(pm)) >> 20) & 0x7ff) - 1023;
      const double sc = __hiloint2double((1023 - max(min(ex, 1022), -1022)) << 20, 0);
      p *= sc; pm *= sc;
    }
  }
  return cnt;
}

constexpr int kBisThreads = 256;
constexpr int kBisRounds = 8;         // 33^8 = 1.4e12: interval width below 1e-12 of the spectrum's extent

__global__ void __launch_bounds__(kBisThreads) sp_bisect_kernel(const SpLayer* __restrict__ layers) {
  const SpLayer& L = layers[blockIdx.y];
  const int r = L.r;
  const int tid = threadIdx.x, lane = tid % 32, w = tid / 32;
  if ((int)blockIdx.x * (kBisThreads / 32) >= r) return;
  __shared__ double s_d[kTriMaxRp], s_e2[kTriMaxRp];
  for (int i = tid; i < r; i += kBisThreads) {
    s_d[i] = L.td_d[i];
    const double e = i + 1 < r ? L.td_e[i] : 0.0;
    s_e2[i] = e * e;
  }
  __syncthreads();
  // Gershgorin interval (every warp the same), widened a little; a NaN or Inf anywhere poisons the result
  double gl = 1.0e300, gu = -1.0e300;
  bool bad = false;
  for (int i = lane; i < r; i += 32) {
    const double el = i > 0 ? sqrt(s_e2[i - 1]) : 0.0, er = sqrt(s_e2[i]);
    gl = fmin(gl, s_d[i] - el - er); gu = fmax(gu, s_d[i] + el + er);
    bad |= !finite64(s_d[i]) || !finite64(s_e2[i]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { gl = fmin(gl, __shfl_xor_sync(0xffffffffu, gl, o)); gu = fmax(gu, __shfl_xor_sync(0xffffffffu, gu, o)); }
  bad = __any_sync(0xffffffffu, bad);
  const int j = blockIdx.x * (kBisThreads / 32) + w;          // this warp's eigenvalue, ascending order
  if (j >= r) return;
  if (bad) {
    if (lane == 0) { L.lam64[j] = __longlong_as_double(0x7ff8000000000000ll); L.lam[j] = __int_as_float(0x7fc00000); }
    return;
  }
  const double pad = 1.0e-14 * fmax(fabs(gl), fabs(gu)) + 1.0e-300;
  double lo = gl - pad, hi = gu + pad;
  for (int it = 0; it < kBisRounds; ++it) {
    const double h = (hi - lo) * (1.0 / 33.0);
    const double x = fma((double)(lane + 1), h, lo);
    const int cnt = sturm_count(s_d, s_e2, r, x);
    const int nle = __popc(__ballot_sync(0xffffffffu, cnt <= j));   // points not above lambda_j
    const double nlo = fma((double)nle, h, lo);
    hi = fmin(hi, fma((double)(nle + 1), h, lo));
    lo = nlo;
  }
  if (lane == 0) { const double lam = 0.5 * (lo + hi); L.lam64[j] = lam; L.lam[j] = (float)lam; }
}

// ---- vectors of the kept atoms --------------------------------------------------------------------------------
constexpr int kVecThreads = 256;
constexpr int kVecWarps = kVecThreads / 32;
constexpr int kVecCtasPerLayer = 4;
constexpr int kVecGroup = 4;          // reflectors applied together in the back-transformation
constexpr double kPivMin = 1.0e-280;
constexpr double kSameEig = 1.0e-9;   // scaled units (largest eigenvalue below 1): eigenvalues this close share a subspace

// Twisted factorisation of T - lambda I (forward pivots D+ in lane 0, backward pivots D- in lane 1, the same
// instructions on mirrored indices), twist index at the smallest |gamma_k| = |D+_k + D-_k - (d_k - lambda)|,
// z_k = 1, z_i = -(e_i / D+_i) z_{i+1} above and z_{i+1} = -(e_i / D-_{i+1}) z_i below.  Returns gamma_k / z^T z, the
// Rayleigh-quotient correction of lambda.  wa, wb, z: r doubles each in shared memory.
__device__ double twisted_vector(const double* __restrict__ d, const double* __restrict__ e, int r, double lambda,
                                 double* wa, double* wb, double* z, int lane, int skip, double* znorm2) {
  if (lane < 2) {
    const bool back = lane == 1;
    double* D = back ? wb : wa;
    int cur = back ? r - 1 : 0;
    double piv = d[cur] - lambda;
    if (fabs(piv) < kPivMin) piv = kPivMin;
    D[cur] = piv;
    for (int t = 0; t + 1 < r; ++t) {
      const int ie = back ? r - 2 - t : t;                    // the off-diagonal between cur and next
      const int nxt = back ? cur - 1 : cur + 1;
      const double ee = e[ie];
      piv = fma(-(ee / piv), ee, d[nxt] - lambda);
      if (fabs(piv) < kPivMin) piv = kPivMin;
      D[nxt] = piv;
      cur = nxt;
    }
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

__global__ void __launch_bounds__(kVecThreads, 1) sp_eigvec_kernel(const SpLayer* __restrict__ layers) {
  const SpLayer& L = layers[blockIdx.x];
  extern __shared__ __align__(16) unsigned char vec_smem[];
  const int r = L.r, rp = L.rp;
  double* s_d = reinterpret_cast<double*>(vec_smem);          // [rp]
  double* s_e = s_d + rp;                                     // [rp]
  double* s_ref = s_e + rp;                                   // [2][kVecGroup][rp] reflectors of the current / next group
  double* s_work = s_ref + 2 * kVecGroup * rp;                // [warps][3][rp]
  __shared__ double s_beta[2][kVecGroup];
  __shared__ uint32_t s_last;
  const int tid = threadIdx.x, lane = tid % 32, w = tid / 32;
  const uint32_t k = L.hdr->k;
  const int nref = max(r - 2, 0);
  const int ngroups = (nref + kVecGroup - 1) / kVecGroup;
  for (int i = tid; i < r; i += kVecThreads) { s_d[i] = L.td_d[i]; s_e[i] = i + 1 < r ? L.td_e[i] : 0.0; }
  __syncthreads();
  double* wa = s_work + (size_t)w * 3 * rp;
  double* wb = wa + rp;
  double* z = wb + rp;
  constexpr int kCols = kTriCols;
  for (uint32_t a0 = blockIdx.y * kVecWarps; a0 < k; a0 += kVecCtasPerLayer * kVecWarps) {
    const uint32_t a = a0 + w;
    const bool have = a < k;
    double zr[kCols];                                         // z[lane + 32 m]
#pragma unroll
    for (int m = 0; m < kCols; ++m) zr[m] = 0.0;
    if (have) {
      const int ei = L.perm[L.idx[a]];                        // index of the atom's eigenvalue (ascending order)
      double lambda = L.lam64[ei];
      // earlier kept atoms with the same eigenvalue (to the accuracy of the bisection): each takes another twist index
      int skip = 0;
      for (uint32_t b = lane; b < a; b += 32) skip += fabs(L.lam64[L.perm[L.idx[b]]] - lambda) <= kSameEig ? 1 : 0;
      skip = (int)warp_sum((uint32_t)skip);
      double n2 = 1.0;
      const double corr = twisted_vector(s_d, s_e, r, lambda, wa, wb, z, lane, skip, &n2);
      if (finite64(corr) && skip == 0) {                      // one Rayleigh-quotient step, then the vector again
        lambda += corr;
        __syncwarp();
        twisted_vector(s_d, s_e, r, lambda, wa, wb, z, lane, 0, &n2);
      }
      const double inv = n2 > 0.0 ? rsqrt(n2) : 0.0;
#pragma unroll
      for (int m = 0; m < kCols; ++m) { const int i = lane + 32 * m; zr[m] = i < r ? z[i] * inv : 0.0; }
    }
    // u = H_0 H_1 ... H_{r-3} z: the reflectors from the last to the first, kVecGroup at a time.  For a group applied in
    // the order 0, 1, 2, 3:  s_0 = beta_0 v_0.z,  s_i = beta_i (v_i.z - sum_{j<i} s_j v_i.v_j),  z -= sum s_i v_i.
    __syncthreads();
    // group gi holds the reflectors kk = nref-1 - 4 gi - q, q = 0..3 in the order of application; a thread stages
    // kPre entries of the next group in registers while the current one is applied
    constexpr int kPre = kVecGroup * kTriMaxRp / kVecThreads;
    double pre[kPre];
    auto fetch_group = [&](int gi) {
#pragma unroll
      for (int t = 0; t < kPre; ++t) {
        const int el = tid + kVecThreads * t;
        const int q = el / rp, i = el - q * rp;
        const int kk = nref - 1 - kVecGroup * gi - q;
        pre[t] = (el < kVecGroup * rp && kk >= 0 && i < r) ? L.td_V[(int64_t)kk * r + i] : 0.0;
      }
    };
    auto store_group = [&](int gi, int buf) {
#pragma unroll
      for (int t = 0; t < kPre; ++t) {
        const int el = tid + kVecThreads * t;
        if (el < kVecGroup * rp) s_ref[(size_t)buf * kVecGroup * rp + el] = pre[t];
      }
      if (tid < kVecGroup) { const int kk = nref - 1 - kVecGroup * gi - tid; s_beta[buf][tid] = kk >= 0 ? L.td_tau[kk] : 0.0; }
    };
    if (ngroups > 0) { fetch_group(0); store_group(0, 0); }
    __syncthreads();
    for (int gi = 0; gi < ngroups; ++gi) {
      const int buf = gi & 1;
      if (gi + 1 < ngroups) fetch_group(gi + 1);
      if (have) {
        const double* v0 = s_ref + ((size_t)buf * kVecGroup + 0) * rp;
        const double* v1 = v0 + rp; const double* v2 = v1 + rp; const double* v3 = v2 + rp;
        double z0 = 0, z1 = 0, z2 = 0, z3 = 0, g10 = 0, g20 = 0, g21 = 0, g30 = 0, g31 = 0, g32 = 0;
#pragma unroll
        for (int m = 0; m < kCols; ++m) {
          if (32 * m < rp) {
            const int i = lane + 32 * m;
            const double a0v = v0[i], a1v = v1[i], a2v = v2[i], a3v = v3[i], zz = zr[m];
            z0 = fma(a0v, zz, z0); z1 = fma(a1v, zz, z1); z2 = fma(a2v, zz, z2); z3 = fma(a3v, zz, z3);
            g10 = fma(a1v, a0v, g10); g20 = fma(a2v, a0v, g20); g21 = fma(a2v, a1v, g21);
            g30 = fma(a3v, a0v, g30); g31 = fma(a3v, a1v, g31); g32 = fma(a3v, a2v, g32);
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          z0 += __shfl_xor_sync(0xffffffffu, z0, o); z1 += __shfl_xor_sync(0xffffffffu, z1, o);
          z2 += __shfl_xor_sync(0xffffffffu, z2, o); z3 += __shfl_xor_sync(0xffffffffu, z3, o);
          g10 += __shfl_xor_sync(0xffffffffu, g10, o); g20 += __shfl_xor_sync(0xffffffffu, g20, o);
          g21 += __shfl_xor_sync(0xffffffffu, g21, o); g30 += __shfl_xor_sync(0xffffffffu, g30, o);
          g31 += __shfl_xor_sync(0xffffffffu, g31, o); g32 += __shfl_xor_sync(0xffffffffu, g32, o);
        }
        const double c0 = s_beta[buf][0] * z0;
        const double c1 = s_beta[buf][1] * (z1 - c0 * g10);
        const double c2 = s_beta[buf][2] * (z2 - c0 * g20 - c1 * g21);
        const double c3 = s_beta[buf][3] * (z3 - c0 * g30 - c1 * g31 - c2 * g32);
#pragma unroll
        for (int m = 0; m < kCols; ++m) {
          if (32 * m < rp) {
            const int i = lane + 32 * m;
            zr[m] -= fma(c0, v0[i], fma(c1, v1[i], fma(c2, v2[i], c3 * v3[i])));
          }
        }
      }
      if (gi + 1 < ngroups) store_group(gi + 1, buf ^ 1);
      __syncthreads();
    }
    if (have) {
      double n2 = 0.0;
#pragma unroll
      for (int m = 0; m < kCols; ++m) n2 = fma(zr[m], zr[m], n2);
      n2 = warp_sum(n2);
      const double inv = n2 > 0.0 ? rsqrt(n2) : 0.0;
#pragma unroll
      for (int m = 0; m < kCols; ++m) { const int i = lane + 32 * m; if (i < r) L.shortv[(int64_t)a * r + i] = (float)(zr[m] * inv); }
    }
  }
  // the last CTA of the layer orthogonalises kept atoms whose eigenvalues nearly coincide (their vectors are
  // determined only as a subspace): modified Gram-Schmidt in payload order, one warp
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = atomicAdd(L.vec_ticket, 1u) == (uint32_t)(kVecCtasPerLayer - 1) ? 1u : 0u;
  __syncthreads();
  if (!s_last || w != 0 || k < 2) return;
  __threadfence();
  for (uint32_t a = 1; a < k; ++a) {
    const double la = L.lam64[L.perm[L.idx[a]]];
    bool changed = false;
    for (uint32_t b = 0; b < a; ++b) {
      const double lb = L.lam64[L.perm[L.idx[b]]];
      if (fabs(la - lb) > kSameEig) continue;
      volatile float* va = L.shortv + (int64_t)a * r;
      const volatile float* vb = L.shortv + (int64_t)b * r;
      double dot = 0.0;
      for (int i = lane; i < r; i += 32) dot = fma((double)va[i], (double)vb[i], dot);
      dot = warp_sum(dot);
      for (int i = lane; i < r; i += 32) va[i] = (float)((double)va[i] - dot * (double)vb[i]);
      __syncwarp();
      changed = true;
    }
    if (changed) {
      volatile float* va = L.shortv + (int64_t)a * r;
      double n2 = 0.0;
      for (int i = lane; i < r; i += 32) n2 = fma((double)va[i], (double)va[i], n2);
      n2 = warp_sum(n2);
      const double inv = n2 > 0.0 ? rsqrt(n2) : 0.0;
      for (int i = lane; i < r; i += 32) va[i] = (float)((double)va[i] * inv);
      __syncwarp();
    }
  }
}

// ---- host side ---------------------------------------------------------------------------------------------------
static size_t tri_smem_bytes(int rp_max) { return (size_t)kTriRows * rp_max * sizeof(double); }
static size_t vec_smem_bytes(int rp_max) { return (size_t)(2 + 2 * kVecGroup + 3 * kVecWarps) * rp_max * sizeof(double); }

int sp_tridiag_max_rp() { return kTriMaxRp; }
int sp_tridiag_cluster_ctas() { return kTriCtas; }
int sp_tridiag_ctas_of(int rp) { return rp / kTriRows < 1 ? 1 : rp / kTriRows; }

int sp_configure_tridiag() {
  // optional route: a GPU that refuses the cluster size or the shared memory simply reports it as unavailable
  if (cudaFuncSetAttribute(sp_tridiag_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tri_smem_bytes(kTriMaxRp)) != cudaSuccess ||
      cudaFuncSetAttribute(sp_tridiag_cluster_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess ||
      cudaFuncSetAttribute(sp_eigvec_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)vec_smem_bytes(kTriMaxRp)) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kTriCtas); cfg.blockDim = dim3(kTriThreads); cfg.dynamicSmemBytes = tri_smem_bytes(kTriMaxRp);
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = kTriCtas; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, sp_tridiag_cluster_kernel, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
  return n;
}

int launch_sp_tridiag(const SpLayer* d_layers, const ClusterCta* d_ctas, int n_clusters, int rp_max, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_clusters * kTriCtas); cfg.blockDim = dim3(kTriThreads);
  cfg.dynamicSmemBytes = tri_smem_bytes(rp_max); cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = kTriCtas; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return (int)cudaLaunchKernelEx(&cfg, sp_tridiag_cluster_kernel, d_layers, d_ctas);
}

void launch_sp_bisect(const SpLayer* d_layers, int n_layers, int r_max, cudaStream_t st) {
  const int per = kBisThreads / 32;
  sp_bisect_kernel<<<dim3((r_max + per - 1) / per, n_layers), kBisThreads, 0, st>>>(d_layers);
}

void launch_sp_eigvec(const SpLayer* d_layers, int n_layers, int rp_max, cudaStream_t st) {
  sp_eigvec_kernel<<<dim3(n_layers, kVecCtasPerLayer), kVecThreads, vec_smem_bytes(rp_max), st>>>(d_layers);
}

}  // namespace atomo
