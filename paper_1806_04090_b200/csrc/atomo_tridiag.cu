// Spectral atoms by the tridiagonal route (Section 5 of the paper asks for the SVD of every layer gradient; only
// the singular VALUES of all atoms enter the probabilities of Eq. 3 / Algorithm 1, and only the few KEPT atoms of
// Eq. 2 need their vectors).  For layers with a short side of at most 512:
//
//   sp_tridiag_cluster_kernel : Householder reduction of the scaled Gram matrix A (r x r) to a symmetric
//                               tridiagonal T = Q^T A Q, in fp64.  A layer's rows sit in blocks of 32 on rp/32 CTAs
//                               of a 16-CTA cluster and stay in registers; per step the product A v, the next
//                               pivot column's ingredients and the parts of p^T v travel through distributed
//                               shared memory (one cluster barrier per step).  The reflectors go to global memory
//                               as fp32 unit vectors for the back-transformation.
//   sp_bisect_kernel          : all eigenvalues of T, eight lanes per eigenvalue: 13 rounds of 9-section on Sturm
//                               counts (division-free three-term recurrence with power-of-two rescaling).
//   (sp_finalize_sample_kernel sorts, solves Algorithm 1 and draws, as for the other routes)
//   sp_eigvec_kernel          : for the kept atoms only: eigenvector of T by a twisted factorisation with one
//                               Rayleigh-quotient correction, back-transformation u = Q z with the reflectors
//                               (four at a time, fp32), normalised short-side vector into the payload; kept atoms with
//                               nearly equal eigenvalues are orthogonalised against each other at the end.
//
// Work per layer: about 2 r^3 fp64 flops for the reduction (full symmetric storage: matrix-vector product and
// rank-two update of the trailing block), r^2 * 13 * 8 recurrence steps for the eigenvalues, O(r^2) per kept atom.
#include <type_traits>

#include <cooperative_groups.h>

#include "atomo_kernels.cuh"
#include "atomo_twisted.cuh"

namespace cg = cooperative_groups;

namespace atomo {

namespace {

constexpr int kTriCtas = 16;          // CTAs per cluster
constexpr int kTriThreads = 512;
constexpr int kTriWarps = kTriThreads / 32;
constexpr int kTriRows = 32;          // rows of A per CTA
constexpr int kTriMaxRp = 512;        // largest padded short side
constexpr int kTriCols = kTriMaxRp / 32;   // columns per lane

}  // namespace

// ---- Householder tridiagonalisation ------------------------------------------------------------------------
// Step k (k = 0 .. r-3) with x = A[k+1.., k]:  alpha = -sign(x_0) ||x||,  v = x - alpha e_1,  beta = 2 / v^T v,
// H = I - beta v v^T;  p = beta A22 v,  K = beta/2 p^T v,  w = p - K v,  A22 -= v w^T + w v^T;  d_k = A[k][k],
// e_k = alpha.
// Layout: CTA g of a layer's nc = rp / 32 CTAs holds the rows 32 g .. 32 g + 31, two per warp, in registers for the
// whole reduction; a lane holds the columns j = lane + 32 m.  The 32 entries of a vector that a CTA produces are
// contiguous: one warp sends them to a peer as one 256-byte store into the peer's shared memory.  The trailing
// block shrinks from the top left: column slots m < (k+1)/32 are dead and skipped, so a step costs in proportion
// to the columns that are left (the CTAs of the dead rows only keep the barriers).
// One cluster barrier per step: with p_i the owners also send c_i = A[i][k+1] as it is after update k-1, from which
// every CTA forms the next pivot column x_i = c_i - v_i w_{k+1} - w_i v_{k+1} itself, hence v_{k+1}; the update of
// step k and the product A v_{k+1} then share one pass over the rows.
__device__ __forceinline__ double tri_block_sum(double x, double* s_red, int lane, int w) {
  x = warp_sum(x);
  if (lane == 0) s_red[w] = x;
  __syncthreads();
  double t = s_red[lane & (kTriWarps - 1)];
#pragma unroll
  for (int o = kTriWarps / 2; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  return t;                                                   // the same bits in every thread of the CTA
}

// alpha, beta and the first entry of v from ||x||^2 and x_0.  The square root comes from the reciprocal square root
// and beta from a reciprocal: two short dependent sequences instead of a square root and a division (the chain sits
// on the critical path of every step); v^T v / 2 = alpha (alpha - x_0) = ||x||^2 + |x_0| ||x||.
__device__ __forceinline__ void tri_reflector(double nx2, double x0, double& alpha, double& beta, double& v0) {
  alpha = 0.0; beta = 0.0; v0 = 0.0;
  if (nx2 > 1.0e-290) {                                       // below: treated as a zero column (H = I)
    const double nx = nx2 * rsqrt(nx2);
    alpha = -copysign(nx, x0);
    v0 = x0 - alpha;
    const double den = fma(fabs(x0), nx, nx2);
    beta = __drcp_rn(den);
  }
}

// one entry of each of the two register rows, slot chosen at run time (uniform over the warp): a jump, not 16 selects
#define TRI_PICK(slot, out0, out1)                                                                       \
  switch (slot) {                                                                                        \
    case 0: out0 = row0[0]; out1 = row1[0]; break;    case 1: out0 = row0[1]; out1 = row1[1]; break;     \
    case 2: out0 = row0[2]; out1 = row1[2]; break;    case 3: out0 = row0[3]; out1 = row1[3]; break;     \
    case 4: out0 = row0[4]; out1 = row1[4]; break;    case 5: out0 = row0[5]; out1 = row1[5]; break;     \
    case 6: out0 = row0[6]; out1 = row1[6]; break;    case 7: out0 = row0[7]; out1 = row1[7]; break;     \
    case 8: out0 = row0[8]; out1 = row1[8]; break;    case 9: out0 = row0[9]; out1 = row1[9]; break;     \
    case 10: out0 = row0[10]; out1 = row1[10]; break; case 11: out0 = row0[11]; out1 = row1[11]; break;  \
    case 12: out0 = row0[12]; out1 = row1[12]; break; case 13: out0 = row0[13]; out1 = row1[13]; break;  \
    case 14: out0 = row0[14]; out1 = row1[14]; break; default: out0 = row0[15]; out1 = row1[15]; break;  \
  }

__global__ void __launch_bounds__(kTriThreads, 1) sp_tridiag_cluster_kernel(const SpLayer* __restrict__ layers,
                                                                            const ClusterCta* __restrict__ ctas) {
  static_assert(kTriCols == 16, "TRI_PICK lists 16 slots");
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ double s_p[2][kTriMaxRp];                        // beta A22 v of step k in s_p[k & 1] (written by the row owners)
  __shared__ double s_c[2][kTriMaxRp];                        // column k+1 after update k-1, likewise
  __shared__ double s_v[2][kTriMaxRp];                        // v of step k in s_v[k & 1]
  __shared__ double s_w[kTriMaxRp];
  __shared__ double s_stage[2][kTriRows];                     // this CTA's 32 entries of p and c on their way out
  __shared__ double s_pk[2][kTriCtas];                        // the CTAs' parts of p^T v, sent along with p (same parity)
  __shared__ double s_red2[kTriWarps];
  __shared__ double s_x0, s_scal[3];                          // first entry of the next pivot column; alpha, beta, v_0 of the next reflector
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
    for (int k = 0; k <= steps; ++k) cluster.sync();
    cluster.sync();
    return;
  }
  const SpLayer& L = layers[me.layer];
  const int r = L.r, nc = me.pad, g = me.slot, base = me.base_rank;
  // the layer's pointers in registers: a field read through `layers` inside a loop would be a global load each time
  double* const td_d = L.td_d; double* const td_e = L.td_e; double* const td_tau = L.td_tau; float* const td_V = L.td_V;
  const float* const gA = L.A; const int64_t lda = L.lda; const int ldv = L.td_ldv;
  const int my_steps = max(r - 2, 0);
  const int li0 = w, li1 = w + kTriWarps;                     // this warp's two rows
  const int i0 = 32 * g + li0, i1 = 32 * g + li1;
  double row0[kTriCols], row1[kTriCols];
#pragma unroll
  for (int m = 0; m < kTriCols; ++m) {
    const int j = lane + 32 * m;
    const bool in = m < nc && j < r;
    row0[m] = (in && i0 < r) ? (double)gA[(int64_t)i0 * lda + j] : 0.0;
    row1[m] = (in && i1 < r) ? (double)gA[(int64_t)i1 * lda + j] : 0.0;
  }
  const int sq = w * 32 + lane;                               // this thread's entry of the vectors (warps < nc)
  const int sj = sq;                                          // its index
  const bool slice = w < nc;
  // ---- the first reflector and A v_0 ----
  double beta = 0.0, v0 = 0.0;
  if (my_steps > 0) {
    const double xq = (slice && sj > 0 && sj < r) ? (double)gA[sj] : 0.0;   // column 0 = row 0 (symmetric)
    if (slice) s_v[0][sq] = xq;
    const double nx2 = tri_block_sum(xq * xq, s_red2, lane, w);
    const int q1 = 1;
    if (tid == 0) {
      double alpha;
      tri_reflector(nx2, (double)gA[1], alpha, beta, v0);
      s_scal[0] = alpha; s_scal[1] = beta; s_scal[2] = v0;
      s_v[0][q1] = v0;
      if (g == 0) { td_d[0] = (double)gA[0]; td_e[0] = alpha; td_tau[0] = beta; }
    }
    __syncthreads();
    beta = s_scal[1]; v0 = s_scal[2];
    {
      // reflectors are filed as unit vectors (H = I - 2 u u^T, u = v sqrt(beta / 2)): no range trouble in fp32
      const double un = sqrt(0.5 * beta);
      if (g == 0) for (int j = tid; j < r; j += kTriThreads) td_V[j] = (float)(s_v[0][j] * un);   // row 0
    }
    double a0 = 0.0, a1 = 0.0;
#pragma unroll
    for (int m = 0; m < kTriCols; ++m) {
      if (m < nc) {
        const double vq = s_v[0][lane + 32 * m];
        a0 = fma(row0[m], vq, a0); a1 = fma(row1[m], vq, a1);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { a0 += __shfl_xor_sync(0xffffffffu, a0, o); a1 += __shfl_xor_sync(0xffffffffu, a1, o); }
    double c0 = 0.0, c1 = 0.0;
    TRI_PICK(q1 >> 5, c0, c1);
    if (lane == (q1 & 31)) { s_stage[1][li0] = c0; s_stage[1][li1] = c1; }
    if (lane == 0) {
      s_stage[0][li0] = (i0 > 0 && i0 < r) ? a0 * beta : 0.0;
      s_stage[0][li1] = (i1 > 0 && i1 < r) ? a1 * beta : 0.0;
    }
  }
  __syncthreads();
  if (my_steps > 0 && w < nc) {                               // warp w carries this CTA's 32 entries to peer w
    const double pl = s_stage[0][lane];
    cluster.map_shared_rank(&s_p[0][0], base + w)[g * 32 + lane] = pl;
    cluster.map_shared_rank(&s_c[0][0], base + w)[g * 32 + lane] = s_stage[1][lane];
    // ... and this CTA's part of p^T v (its 32 rows), from which every CTA forms K without a reduction of its own
    const double part = warp_sum(pl * s_v[0][g * 32 + lane]);
    if (lane == 0) cluster.map_shared_rank(&s_pk[0][0], base + w)[g] = part;
  }
  cluster.sync();
  // warp w < nc talks to peer w: that CTA's copies of the three arrays, mapped once
  const int peer = base + min(w, nc - 1);
  double* const peer_p = cluster.map_shared_rank(&s_p[0][0], peer);
  double* const peer_c = cluster.map_shared_rank(&s_c[0][0], peer);
  double* const peer_pk = cluster.map_shared_rank(&s_pk[0][0], peer);
  // A layer that fills its cluster finishes alone: once every live row sits in the CTA of the last rows, that CTA runs
  // the remaining steps (at most 31) by itself, with stores into its own shared memory and __syncthreads in place of
  // the cluster barrier, and the other CTAs leave the loop.
  const int g_last = (max(r, 1) - 1) >> 5;
  const int k_tail = nc == kTriCtas ? 32 * g_last - 1 : 0x7fffffff;
  // instances: with the cluster (a layer that fills it, or a smaller one) and alone; for the layers that fill the
  // cluster also one per first live column slot, so that the pass over the rows is straight-line code
  auto step = [&](auto solo_tag, auto full_tag, auto mlo_tag, const int k) {
    constexpr bool solo = decltype(solo_tag)::value;
    constexpr int kMlo = decltype(mlo_tag)::value;            // first live column slot, or -1: taken from k at run time
    constexpr bool full = decltype(full_tag)::value;          // the layer has all kTriCtas CTAs: loop bounds known at compile time
    const int ncc = full ? kTriCtas : nc;
    const bool active = k < my_steps;
    const bool last = k + 1 == my_steps;                      // no reflector follows
    const int par = k & 1, nxt = par ^ 1;
    const int q1 = k + 1, q2 = k + 2;
    const int m_lo = kMlo >= 0 ? kMlo : (k + 1) >> 5;         // first column slot that is still alive
    double beta_n = 0.0, v0_n = 0.0;
    if (active) {
      // K = beta/2 p^T v: the CTAs' parts arrived with p; every thread adds them in the same order
      const double vq = slice ? s_v[par][sq] : 0.0;
      const double pq = slice ? s_p[par][sq] : 0.0;
      const int kc = lane & (kTriCtas - 1);                   // (alone, only this CTA's part is there)
      double ksum = (solo ? kc == g : kc < ncc) ? s_pk[par][kc] : 0.0;
#pragma unroll
      for (int o = kTriCtas / 2; o > 0; o >>= 1) ksum += __shfl_xor_sync(0xffffffffu, ksum, o);
      const double K = 0.5 * beta * ksum;
      const double w1 = fma(-K, v0, s_p[par][q1]);            // w_{k+1}
      // w, and the next pivot column x_j = c_j - v_j w_{k+1} - w_j v_{k+1} for j > k+1
      const double wq = fma(-K, vq, pq);
      double xn = 0.0;
      if (slice) {
        s_w[sq] = wq;
        if (sj > k + 1 && sj < r && !last) xn = s_c[par][sq] - fma(vq, w1, wq * v0);
        s_v[nxt][sq] = xn;
        if (sq == q2) s_x0 = xn;
      }
      const double nx2 = tri_block_sum(xn * xn, s_red2, lane, w);
      if (tid == 0) {                                         // one thread forms the reflector; a zero column gives v = 0
        double alpha_n;
        tri_reflector(nx2, s_x0, alpha_n, beta_n, v0_n);
        s_scal[0] = alpha_n; s_scal[1] = beta_n; s_scal[2] = v0_n;
        if (!last) s_v[nxt][q2] = v0_n;
      }
      __syncthreads();
      beta_n = s_scal[1]; v0_n = s_scal[2];
      // update of the two rows with (v, w), fused with their products with the next v
      const double vi0 = s_v[par][g * 32 + li0], vi1 = s_v[par][g * 32 + li1];
      const double wi0 = s_w[g * 32 + li0], wi1 = s_w[g * 32 + li1];
      const double* __restrict__ pv = &s_v[par][lane];
      const double* __restrict__ pn = &s_v[nxt][lane];
      const double* __restrict__ pw = &s_w[lane];
      double a0 = 0.0, a1 = 0.0;
#pragma unroll
      for (int m = 0; m < kTriCols; ++m) {
        if (m >= m_lo && m < ncc) {
          const double vq2 = pv[32 * m], wq2 = pw[32 * m], vn = pn[32 * m];
          row0[m] = fma(-vi0, wq2, fma(-wi0, vq2, row0[m]));
          row1[m] = fma(-vi1, wq2, fma(-wi1, vq2, row1[m]));
          a0 = fma(row0[m], vn, a0); a1 = fma(row1[m], vn, a1);
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) { a0 += __shfl_xor_sync(0xffffffffu, a0, o); a1 += __shfl_xor_sync(0xffffffffu, a1, o); }
      // column k+2 of the two rows goes out with the products; column k+1 holds the entries of T that are final now
      double c20 = 0.0, c21 = 0.0;
      TRI_PICK(q2 >> 5, c20, c21);
      if (lane == (q2 & 31)) {
        s_stage[1][li0] = c20; s_stage[1][li1] = c21;
        if (last) { if (i0 == r - 1) td_d[r - 1] = c20; if (i1 == r - 1) td_d[r - 1] = c21; }
      }
      if (i0 == k + 1 || i1 == k + 1 || (last && (i0 == r - 1 || i1 == r - 1))) {
        double c10 = 0.0, c11 = 0.0;
        TRI_PICK(q1 >> 5, c10, c11);
        if (lane == (q1 & 31)) {
          if (i0 == k + 1) td_d[k + 1] = c10;
          if (i1 == k + 1) td_d[k + 1] = c11;
          if (last) { if (i0 == r - 1) td_e[r - 2] = c10; if (i1 == r - 1) td_e[r - 2] = c11; }
        }
      }
      if (lane == 0) {
        s_stage[0][li0] = (i0 > k + 1 && i0 < r) ? a0 * beta_n : 0.0;
        s_stage[0][li1] = (i1 > k + 1 && i1 < r) ? a1 * beta_n : 0.0;
      }
    }
    __syncthreads();
    if (active && !last && (solo ? w == 0 : w < ncc)) {        // alone: the same entries into this CTA's own arrays
      double* const to_p = solo ? &s_p[0][0] : peer_p;
      double* const to_c = solo ? &s_c[0][0] : peer_c;
      double* const to_pk = solo ? &s_pk[0][0] : peer_pk;
      const double pl = s_stage[0][lane];
      to_p[nxt * kTriMaxRp + g * 32 + lane] = pl;
      to_c[nxt * kTriMaxRp + g * 32 + lane] = s_stage[1][lane];
      const double part = warp_sum(pl * s_v[nxt][g * 32 + lane]);
      if (lane == 0) to_pk[nxt * kTriCtas + g] = part;
    }
    if (!solo) cluster.barrier_arrive();                      // (release) the entries above are on their way
    if (active && !last && (solo || g == 0)) {                // meanwhile the CTA of the first rows (dead after 31 steps) files the reflector
      if (tid == 0) { td_e[k + 1] = s_scal[0]; td_tau[k + 1] = beta_n; }
      const double un = sqrt(0.5 * beta_n);                   // filed as a unit vector: H = I - 2 u u^T
      for (int j = tid; j < r; j += kTriThreads) td_V[(int64_t)(k + 1) * ldv + j] = (float)(s_v[nxt][j] * un);
    }
    beta = beta_n; v0 = v0_n;
    if (solo) __syncthreads(); else cluster.barrier_wait();
  };
  const int k_mid = min(steps, k_tail);
  using Dyn = std::integral_constant<int, -1>;
  if (nc == kTriCtas) {
#define TRI_SLOT(M) case M: step(std::false_type{}, std::true_type{}, std::integral_constant<int, M>{}, k); break;
    for (int k = 0; k < k_mid; ++k) {
      switch ((k + 1) >> 5) {
        TRI_SLOT(0) TRI_SLOT(1) TRI_SLOT(2) TRI_SLOT(3) TRI_SLOT(4) TRI_SLOT(5) TRI_SLOT(6) TRI_SLOT(7)
        TRI_SLOT(8) TRI_SLOT(9) TRI_SLOT(10) TRI_SLOT(11) TRI_SLOT(12) TRI_SLOT(13) TRI_SLOT(14)
        default: step(std::false_type{}, std::true_type{}, std::integral_constant<int, 15>{}, k); break;
      }
    }
#undef TRI_SLOT
    if (g == g_last) for (int k = k_mid; k < steps; ++k) step(std::true_type{}, std::true_type{}, Dyn{}, k);
  } else {
    for (int k = 0; k < steps; ++k) step(std::false_type{}, std::false_type{}, Dyn{}, k);
  }
  // matrices of order 1 and 2 are tridiagonal as they are
  if (my_steps == 0 && g == 0 && tid == 0) {
    td_d[0] = (double)gA[0];
    if (r == 2) { td_d[1] = (double)gA[lda + 1]; td_e[0] = (double)gA[lda]; }
  }
  cluster.sync();                                             // nobody leaves while a peer may still write here
}
#undef TRI_PICK

// ---- eigenvalues of T: Sturm counts -------------------------------------------------------------------------
// count(x) = number of eigenvalues below x = sign changes of p_0 = 1, p_1 = d_0 - x, p_{i+1} = (d_i - x) p_i -
// e_{i-1}^2 p_{i-1}.  The pair (p_i, p_{i-1}) is rescaled by a power of two every 8 steps (ratios and signs keep).
__device__ __forceinline__ int sturm_count(const double* __restrict__ d, const double* __restrict__ e2, int r, double x) {
  double pm = 1.0, p = d[0] - x;
  int neg = __double2hiint(p);                                // sign bit of the previous term
  int cnt = (uint32_t)neg >> 31;
  // eight steps at a time: their operands are fetched together, so that only the multiply-add chain is serial.
  // The caller pads d with kSturmPad (far above every eigenvalue) and e2 with 0 up to a multiple of 8 past the end:
  // there the step is p <- (pad - x) p, which keeps the sign.
  for (int i0 = 1; i0 < r; i0 += 8) {
    double dd[8], ee[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) { dd[u] = d[i0 + u] - x; ee[u] = e2[i0 + u - 1]; }   // padded arrays: no bounds test
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const double pn = fma(dd[u], p, -ee[u] * pm);
      const int hn = __double2hiint(pn);
      cnt += (uint32_t)(hn ^ neg) >> 31;
      neg = hn;
      pm = p; p = pn;
    }
    const int ex = ((__double2hiint(fabs(p) + fabs(pm)) >> 20) & 0x7ff) - 1023;
    const double sc = __hiloint2double((1023 - max(min(ex, 1022), -1022)) << 20, 0);
    p *= sc; pm *= sc;
  }
  return cnt;
}

constexpr double kSturmPad = 1.0e6;    // diagonal entries past the end (the matrices are scaled to trace <= 1)
constexpr int kBisThreads = 64;           // small CTAs: the warps of a large layer spread over all SMs (the recurrences are latency-bound)
// Points per round and eigenvalue (kBisLanes lanes work on one eigenvalue: the interval shrinks kBisLanes + 1 times per
// round) and rounds, chosen so that the final interval is below 1e-12 of the spectrum's extent: 8 lanes and 13 rounds
// (9^13 = 2.5e12) where the batch has few eigenvalues and the chain of rounds is what takes the time; 2 lanes and 26
// rounds (3^26 = 2.5e12) where it has many: half the Sturm counts per eigenvalue, and enough eigenvalues to fill the GPU.
template <int kBisLanes, int kBisRounds>
__global__ void __launch_bounds__(kBisThreads) sp_bisect_kernel(const SpLayer* __restrict__ layers, int bis_stride) {
  constexpr int kBisPerCta = kBisThreads / kBisLanes;
  const SpLayer& L = layers[blockIdx.y];
  if (!L.tri) return;
  const int r = L.r;
  const int tid = threadIdx.x, lane = tid % 32;
  if ((int)blockIdx.x * kBisPerCta >= r) return;
  extern __shared__ __align__(16) double bis_smem[];           // d and e^2, r_max + 8 entries each
  double* const s_d = bis_smem;
  double* const s_e2 = bis_smem + bis_stride;
  for (int i = tid; i < r + 8; i += kBisThreads) {
    s_d[i] = i < r ? L.td_d[i] : kSturmPad;
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
  const int grp = lane / kBisLanes, t = lane % kBisLanes;     // 4 eigenvalues per warp, 8 lanes each
  const int j = blockIdx.x * kBisPerCta + (tid / 32) * (32 / kBisLanes) + grp;   // ascending order
  const int jj = min(j, r - 1);                               // lanes past the end follow the last eigenvalue
  if (bad) {
    if (t == 0 && j < r) { L.lam64[j] = __longlong_as_double(0x7ff8000000000000ll); L.lam[j] = __int_as_float(0x7fc00000); }
    return;
  }
  const double pad = 1.0e-14 * fmax(fabs(gl), fabs(gu)) + 1.0e-300;
  double lo = gl - pad, hi = gu + pad;
  for (int it = 0; it < kBisRounds; ++it) {
    const double h = (hi - lo) * (1.0 / (kBisLanes + 1));
    const double x = fma((double)(t + 1), h, lo);
    const int cnt = sturm_count(s_d, s_e2, r, x);
    const uint32_t le = __ballot_sync(0xffffffffu, cnt <= jj);              // points not above lambda_j
    const int nle = __popc((le >> (grp * kBisLanes)) & ((1u << kBisLanes) - 1u));
    const double nlo = fma((double)nle, h, lo);
    hi = fmin(hi, fma((double)(nle + 1), h, lo));
    lo = nlo;
  }
  if (t == 0 && j < r) { const double lam = 0.5 * (lo + hi); L.lam64[j] = lam; L.lam[j] = (float)lam; }
}

// ---- vectors of the kept atoms --------------------------------------------------------------------------------
constexpr int kVecThreads = 256;
constexpr int kVecWarps = kVecThreads / 32;
constexpr int kVecCtasPerLayer = 4;
constexpr int kVecGroup = 4;          // reflectors applied together in the back-transformation
constexpr int kVecStages = 4;         // groups in flight between global and shared memory
constexpr int kVecWork = 5;           // work vectors of the twisted factorisation per warp
constexpr double kSameEig = 1.0e-9;   // scaled units (largest eigenvalue below 1): eigenvalues this close share a subspace

__global__ void __launch_bounds__(kVecThreads, 1) sp_eigvec_kernel(const SpLayer* __restrict__ layers) {
  const SpLayer& L = layers[blockIdx.x];
  if (L.tri != 1) return;                                     // larger layers: sp_eigvec_big_kernel
  extern __shared__ __align__(16) unsigned char vec_smem[];
  const int r = L.r, rp = L.rp;
  double* s_d = reinterpret_cast<double*>(vec_smem);          // [rp]
  double* s_e = s_d + rp;                                     // [rp]
  double* s_work = s_e + rp;                                  // [warps][kVecWork][rp]
  float* s_ref = reinterpret_cast<float*>(s_work + (size_t)kVecWarps * kVecWork * rp);   // [kVecStages][kVecGroup][rp] ring of reflector groups
  __shared__ float s_beta[kVecStages][kVecGroup];
  __shared__ uint32_t s_last;
  const int tid = threadIdx.x, lane = tid % 32, w = tid / 32;
  const uint32_t k = L.hdr->k;
  // the layer's pointers in registers (a field read through `layers` inside a loop is a global load each time)
  const float* const gV = L.td_V; const int ldv = L.td_ldv; const double* const gLam = L.lam64;
  const int* const gPerm = L.perm; const uint32_t* const gIdx = L.idx; float* const gShort = L.shortv;
  const int nref = max(r - 2, 0);
  const int ngroups = (nref + kVecGroup - 1) / kVecGroup;
  for (int i = tid; i < r; i += kVecThreads) { s_d[i] = L.td_d[i]; s_e[i] = i + 1 < r ? L.td_e[i] : 0.0; }
  __syncthreads();
  double* wa = s_work + (size_t)w * kVecWork * rp;
  double* wb = wa + rp;
  double* wc = wb + rp;
  double* wd = wc + rp;
  double* z = wd + rp;
  constexpr int kCols = kTriCols;
  for (uint32_t a0 = blockIdx.y * kVecWarps; a0 < k; a0 += kVecCtasPerLayer * kVecWarps) {
    const uint32_t a = a0 + w;
    const bool have = a < k;
    float zr[kCols];                                          // z[lane + 32 m]
#pragma unroll
    for (int m = 0; m < kCols; ++m) zr[m] = 0.0f;
    if (have) {
      const int ei = gPerm[gIdx[a]];                          // index of the atom's eigenvalue (ascending order)
      double lambda = gLam[ei];
      // earlier kept atoms with the same eigenvalue (to the accuracy of the bisection): each takes another twist index
      int skip = 0;
      for (uint32_t b = lane; b < a; b += 32) skip += fabs(gLam[gPerm[gIdx[b]]] - lambda) <= kSameEig ? 1 : 0;
      skip = (int)warp_sum((uint32_t)skip);
      double n2 = 1.0;
      const double corr = twisted_vector(s_d, s_e, r, lambda, wa, wb, wc, wd, z, lane, skip, &n2);
      // the vector's error is about |correction| / gap to the nearest other eigenvalue: well-separated atoms are done
      double gap = 1.0e300;
      if (ei > 0) gap = fmin(gap, fabs(lambda - gLam[ei - 1]));
      if (ei + 1 < r) gap = fmin(gap, fabs(gLam[ei + 1] - lambda));
      if (finite64(corr) && skip == 0 && !(fabs(corr) <= 1.0e-9 * gap)) {   // one Rayleigh-quotient step, then the vector again
        lambda += corr;
        __syncwarp();
        twisted_vector(s_d, s_e, r, lambda, wa, wb, wc, wd, z, lane, 0, &n2);
      }
      const double inv = n2 > 0.0 ? rsqrt(n2) : 0.0;
#pragma unroll
      for (int m = 0; m < kCols; ++m) { const int i = lane + 32 * m; zr[m] = i < r ? (float)(z[i] * inv) : 0.0f; }
    }
    // u = H_0 H_1 ... H_{r-3} z: the reflectors from the last to the first, kVecGroup at a time, in fp32 (an orthogonal
    // map of a unit vector whose result is stored in fp32 anyway).  For a group applied in the order 0, 1, 2, 3:
    // s_0 = beta_0 v_0.z,  s_i = beta_i (v_i.z - sum_{j<i} s_j v_i.v_j),  z -= sum s_i v_i.
    __syncthreads();
    // group gi holds the reflectors kk = nref-1 - 4 gi - q, q = 0..3 in the order of application.  The groups stream
    // through a ring of kVecStages buffers filled by asynchronous copies, kVecStages - 1 groups ahead of use; warp w
    // copies half of row q = w mod 4.
    auto issue_group = [&](int gi) {
      if (gi < ngroups) {
        const int buf = gi % kVecStages;
        const int q = w & (kVecGroup - 1);
        const int kk = nref - 1 - kVecGroup * gi - q;
        const float* srow = gV + (int64_t)max(kk, 0) * ldv;   // rows start on 16-byte boundaries (ldv is a multiple of 4)
        float* drow = s_ref + ((size_t)buf * kVecGroup + q) * rp;
        for (int i = 4 * ((w / kVecGroup) * 32 + lane); i < rp; i += 4 * 32 * (kVecWarps / kVecGroup)) {
          const int bytes = kk >= 0 ? 4 * max(0, min(4, r - i)) : 0;   // the rest of the 16 bytes is filled with zeros
          const uint32_t dst = (uint32_t)__cvta_generic_to_shared(drow + i);
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(bytes ? srow + i : gV), "r"(bytes) : "memory");
        }
        if (tid < kVecGroup) { const int kq = nref - 1 - kVecGroup * gi - tid; s_beta[buf][tid] = kq >= 0 ? 2.0f : 0.0f; }   // unit reflectors
      }
      asm volatile("cp.async.commit_group;" ::: "memory");    // one group per call, empty or not: the counting stays uniform
    };
    for (int st = 0; st < kVecStages - 1; ++st) issue_group(st);
    for (int gi = 0; gi < ngroups; ++gi) {
      const int buf = gi % kVecStages;
      asm volatile("cp.async.wait_group %0;" ::"n"(kVecStages - 2) : "memory");
      __syncthreads();                                        // group gi has landed for everybody; the buffer of gi-1 is free
      issue_group(gi + kVecStages - 1);
      if (have) {
        const float* v0 = s_ref + ((size_t)buf * kVecGroup + 0) * rp;
        const float* v1 = v0 + rp; const float* v2 = v1 + rp; const float* v3 = v2 + rp;
        // the group's four reflectors into registers first (64 loads in flight), then the arithmetic
        float r0[kCols], r1[kCols], r2[kCols], r3[kCols];
#pragma unroll
        for (int m = 0; m < kCols; ++m) {
          const int i = lane + 32 * m;
          const bool in = 32 * m < rp;
          r0[m] = in ? v0[i] : 0.0f; r1[m] = in ? v1[i] : 0.0f; r2[m] = in ? v2[i] : 0.0f; r3[m] = in ? v3[i] : 0.0f;
        }
        float z0 = 0, z1 = 0, z2 = 0, z3 = 0, g10 = 0, g20 = 0, g21 = 0, g30 = 0, g31 = 0, g32 = 0;
#pragma unroll
        for (int m = 0; m < kCols; ++m) {
          const float zz = zr[m];
          z0 = fmaf(r0[m], zz, z0); z1 = fmaf(r1[m], zz, z1); z2 = fmaf(r2[m], zz, z2); z3 = fmaf(r3[m], zz, z3);
          g10 = fmaf(r1[m], r0[m], g10); g20 = fmaf(r2[m], r0[m], g20); g21 = fmaf(r2[m], r1[m], g21);
          g30 = fmaf(r3[m], r0[m], g30); g31 = fmaf(r3[m], r1[m], g31); g32 = fmaf(r3[m], r2[m], g32);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          z0 += __shfl_xor_sync(0xffffffffu, z0, o); z1 += __shfl_xor_sync(0xffffffffu, z1, o);
          z2 += __shfl_xor_sync(0xffffffffu, z2, o); z3 += __shfl_xor_sync(0xffffffffu, z3, o);
          g10 += __shfl_xor_sync(0xffffffffu, g10, o); g20 += __shfl_xor_sync(0xffffffffu, g20, o);
          g21 += __shfl_xor_sync(0xffffffffu, g21, o); g30 += __shfl_xor_sync(0xffffffffu, g30, o);
          g31 += __shfl_xor_sync(0xffffffffu, g31, o); g32 += __shfl_xor_sync(0xffffffffu, g32, o);
        }
        const float c0 = s_beta[buf][0] * z0;
        const float c1 = s_beta[buf][1] * (z1 - c0 * g10);
        const float c2 = s_beta[buf][2] * (z2 - c0 * g20 - c1 * g21);
        const float c3 = s_beta[buf][3] * (z3 - c0 * g30 - c1 * g31 - c2 * g32);
#pragma unroll
        for (int m = 0; m < kCols; ++m) zr[m] -= fmaf(c0, r0[m], fmaf(c1, r1[m], fmaf(c2, r2[m], c3 * r3[m])));
      }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (have) {
      float n2 = 0.0f;
#pragma unroll
      for (int m = 0; m < kCols; ++m) n2 = fmaf(zr[m], zr[m], n2);
      n2 = warp_sum(n2);
      const float inv = n2 > 0.0f ? rsqrtf(n2) : 0.0f;
#pragma unroll
      for (int m = 0; m < kCols; ++m) { const int i = lane + 32 * m; if (i < r) gShort[(int64_t)a * r + i] = zr[m] * inv; }
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
    const double la = gLam[gPerm[gIdx[a]]];
    bool changed = false;
    for (uint32_t b = 0; b < a; ++b) {
      const double lb = gLam[gPerm[gIdx[b]]];
      if (fabs(la - lb) > kSameEig) continue;
      volatile float* va = gShort + (int64_t)a * r;
      const volatile float* vb = gShort + (int64_t)b * r;
      double dot = 0.0;
      for (int i = lane; i < r; i += 32) dot = fma((double)va[i], (double)vb[i], dot);
      dot = warp_sum(dot);
      for (int i = lane; i < r; i += 32) va[i] = (float)((double)va[i] - dot * (double)vb[i]);
      __syncwarp();
      changed = true;
    }
    if (changed) {
      volatile float* va = gShort + (int64_t)a * r;
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
static size_t tri_smem_bytes(int) { return 0; }             // rows in registers, vectors in static shared memory
static size_t vec_smem_bytes(int rp_max) {
  return (size_t)(2 + kVecWork * kVecWarps) * rp_max * sizeof(double) + (size_t)kVecStages * kVecGroup * rp_max * sizeof(float);
}

int sp_tridiag_max_rp() { return kTriMaxRp; }
int sp_tridiag_cluster_ctas() { return kTriCtas; }
int sp_tridiag_ctas_of(int rp) { return rp / kTriRows < 1 ? 1 : rp / kTriRows; }

// the eigenvalue kernel keeps d and e^2 of a layer in shared memory: more than the default 48 KB above a short side of
// about 3000.  Both tridiagonal routes need this (a batch may hold large layers only).  0 if it went through.
int sp_configure_bisect() {
  const int bytes = (int)(2 * (kMaxShort + 10) * sizeof(double));
  if (cudaFuncSetAttribute(sp_bisect_kernel<1, 41>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess ||
      cudaFuncSetAttribute(sp_bisect_kernel<8, 13>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess ||
      cudaFuncSetAttribute(sp_bisect_kernel<2, 26>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) {
    cudaGetLastError();
    return 1;
  }
  return 0;
}

int sp_configure_tridiag() {
  // optional route: a GPU that refuses the cluster size or the shared memory simply reports it as unavailable
  if (cudaFuncSetAttribute(sp_tridiag_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tri_smem_bytes(kTriMaxRp)) != cudaSuccess ||
      cudaFuncSetAttribute(sp_tridiag_cluster_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess ||
      cudaFuncSetAttribute(sp_eigvec_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)vec_smem_bytes(kTriMaxRp)) != cudaSuccess ||
      sp_configure_bisect() != 0) {
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

void launch_sp_bisect(const SpLayer* d_layers, int n_layers, int r_max, int64_t n_eigenvalues, cudaStream_t st) {
  const int stride = (r_max + 8 + 1) & ~1;
  const size_t smem = 2 * (size_t)stride * sizeof(double);
  if (n_eigenvalues >= 65536) {
    // enough eigenvalues to fill the fp64 pipes with one lane each: plain bisection gets one bit per Sturm count
    // (3-section 0.79, 9-section 0.40), 41 rounds for the same final width as the other forms
    constexpr int per = kBisThreads;
    sp_bisect_kernel<1, 41><<<dim3((r_max + per - 1) / per, n_layers), kBisThreads, smem, st>>>(d_layers, stride);
  } else if (n_eigenvalues >= 16384) {
    constexpr int per = kBisThreads / 2;
    sp_bisect_kernel<2, 26><<<dim3((r_max + per - 1) / per, n_layers), kBisThreads, smem, st>>>(d_layers, stride);
  } else {
    constexpr int per = kBisThreads / 8;
    sp_bisect_kernel<8, 13><<<dim3((r_max + per - 1) / per, n_layers), kBisThreads, smem, st>>>(d_layers, stride);
  }
}

void launch_sp_eigvec(const SpLayer* d_layers, int n_layers, int rp_max, cudaStream_t st) {
  sp_eigvec_kernel<<<dim3(n_layers, kVecCtasPerLayer), kVecThreads, vec_smem_bytes(rp_max), st>>>(d_layers);
}

}  // namespace atomo
