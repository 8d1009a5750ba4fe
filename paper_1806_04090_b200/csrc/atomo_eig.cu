// Eigen-solver of the spectral path: eigenvalues and eigenvectors of the short-side Gram matrix
// A = G G^T (or G^T G), i.e. sigma_i^2 and the short-side singular vectors of Section 5's SVD.
//
// Two routes share one Jacobi kernel:
//   mode 1 (default)  sp_cholesky : A = L L^T (fp32, pivots below a noise floor are set to zero), then
//                     one-sided (Hestenes) Jacobi on the rows of L^T.  Orthogonal row rotations J keep
//                     (J L^T)^T (J L^T) = A; at convergence the rows are mutually orthogonal:
//                     row i = sigma_i w_i^T, so A = sum_i sigma_i^2 w_i w_i^T.  No eigenvector accumulation.
//   mode 0            one-sided Jacobi on the rows of X = [A | I]: row i is (x_i | v_i), x_i = v_i^T A; at
//                     convergence x_i = lambda_i v_i^T.  Twice the row length and about twice the sweeps
//                     (the rows of A start nearly parallel), kept as a cross-check.
//
// Blocks of 16 rows are paired by a recursive-halving schedule (step_plan); a CTA holds one block pair in shared
// memory, one warp per rotation; inside a block the pairs follow a round-robin tournament, once per sweep.  Row
// norms are tracked (alpha' = alpha - t gamma, beta' = beta + t gamma) and refreshed when they cancel; rotations
// are applied in the scaled ("fast Givens") form, one FMA per element, with the cosines collected in a per-row
// factor that is folded back when a block is stored or handed over.
//
// Three launch forms around the same rotation code (rotate_pair):
//   sp_jacobi_cluster_kernel     layers of up to 16 block pairs: a layer's CTAs in one 16-CTA cluster for the whole
//                                solve, blocks handed over through distributed shared memory, cluster barrier per step
//   sp_jacobi_persistent_kernel  cooperative launch over groups of whole layers, blocks through global memory (L2),
//                                a barrier among the CTAs of a layer per step
//   sp_jacobi_step_kernel        one launch per step, the host reads a convergence flag once per sweep
// and, before them, the Cholesky factorisation (clusters of 8 CTAs per layer; a cooperative kernel above 1024 rows).
#include <algorithm>

#include <cooperative_groups.h>

#include "atomo_kernels.cuh"

namespace cg = cooperative_groups;

namespace atomo {

// round-robin tournament over n (even) players: pair `slot` of round `round`
__device__ __forceinline__ void rr_pair(int n, int round, int slot, int& p, int& q) {
  const int m = n - 1;
  if (slot == 0) { p = n - 1; q = round % m; }
  else { p = (round + slot) % m; q = (round - slot + m) % m; }
}

// Which two blocks a CTA pairs at step `local` of a sweep (nb blocks, a power of two; nb / 2 CTAs; nb - 1 steps).
// Recursive halving: at level l the blocks form groups of g = nb >> l; inside a group, CTA k keeps block k of
// the first half for the g / 2 steps of the level while the blocks of the second half pass by, one per step
// ((k + t) mod g/2 at step t); the next level treats each half as a group of its own.  Every pair of blocks
// meets exactly once in nb/2 + nb/4 + ... + 1 = nb - 1 steps, and only half of the blocks move at a step.
struct StepPlan { int bi, bj; bool first_in_level, last_in_level; };
struct StepLevel { int lg, t; };                       // group size 2^lg, step t inside the level
__device__ __forceinline__ StepLevel step_level(int nb, int local) {
  int lg = 31 - __clz(nb), base = 0;
  while (local - base >= (1 << (lg - 1))) { base += 1 << (lg - 1); --lg; }
  return {lg, local - base};
}
__device__ __forceinline__ StepPlan step_plan(int nb, int local, int slot) {
  const StepLevel lv = step_level(nb, local);
  const int m = 1 << (lv.lg - 1);
  const int grp = slot >> (lv.lg - 1), k = slot & (m - 1);
  return {(grp << lv.lg) + k, (grp << lv.lg) + m + ((k + lv.t) & (m - 1)), lv.t == 0, lv.t == m - 1};
}
// the inverse: which CTA pairs block `blk` at step `local`, and as what (0 = resident, 1 = moving)
__device__ __forceinline__ void find_holder(int nb, int local, int blk, int& slot, int& role) {
  const StepLevel lv = step_level(nb, local);
  const int m = 1 << (lv.lg - 1);
  const int grp = blk >> lv.lg, pos = blk & ((1 << lv.lg) - 1);
  role = pos >= m;
  slot = grp * m + (role ? ((pos - m - lv.t) & (m - 1)) : pos);
}

// A is scaled to trace 1, so a squared row norm below this is an eigenvalue of A below 1e-12 (mode 0)
// or a singular value of L below 1e-12 (mode 1): rounding noise of the fp32 Gram matrix, not signal.
constexpr float kRowFloor = 1e-24f;
constexpr int kJB = 16;                 // rows per block

// One row held by a warp: lane l keeps float4 number l + 32 t (t < T4).
template <int T4>
struct RowRegs { float4 v[T4]; };

template <int T4>
__device__ __forceinline__ void load_row(RowRegs<T4>& x, const float* row, int lane, int V4) {
#pragma unroll
  for (int t = 0; t < T4; ++t)
    x.v[t] = (lane + 32 * t < V4) ? reinterpret_cast<const float4*>(row)[lane + 32 * t] : make_float4(0.f, 0.f, 0.f, 0.f);
}
template <int T4>
__device__ __forceinline__ void store_row(const RowRegs<T4>& x, float* row, int lane, int V4, float scale = 1.0f) {
#pragma unroll
  for (int t = 0; t < T4; ++t)
    if (lane + 32 * t < V4) {
      const float4 a = x.v[t];
      reinterpret_cast<float4*>(row)[lane + 32 * t] = make_float4(a.x * scale, a.y * scale, a.z * scale, a.w * scale);
    }
}
template <int T4>
__device__ __forceinline__ float row_norm2_partial(const RowRegs<T4>& x, int lane, int A4) {
  float n = 0.f;
#pragma unroll
  for (int t = 0; t < T4; ++t)
    if (lane + 32 * t < A4) {
      const float4 a = x.v[t];
      n = fmaf(a.x, a.x, fmaf(a.y, a.y, fmaf(a.z, a.z, fmaf(a.w, a.w, n))));
    }
  return n;
}

// Sum of one value per lane over a whole row.  A row is held by WPR warps (one segment each): the warp
// sums are exchanged through shared memory under a named barrier of the WPR warps that share the pair,
// and added in a fixed order, so every warp of the pair gets the same bits and takes the same branches.
template <int WPR>
struct RowSum {
  float* slots;      // [2][WPR] for this pair (double-buffered)
  int bar_id, seg, lane, phase;
  __device__ __forceinline__ float operator()(float v) {
    v = warp_sum(v);
    if constexpr (WPR == 1) return v;
    float* slot = slots + (phase & 1) * WPR;
    if (lane == 0) slot[seg] = v;
    asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(32 * WPR) : "memory");
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < WPR; ++i) t += slot[i];
    ++phase;
    return t;
  }
};

// single-instruction approximations (about 2 ulp); their inputs here are never subnormal
__device__ __forceinline__ float rcp_approx(float v) { float r; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v)); return r; }
__device__ __forceinline__ float rsqrt_approx(float v) { float r; asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v)); return r; }

// One plane rotation of the stored rows (xp, xq); true rows are dp * xp and dq * xq, with tracked squared
// norms np2, nq2 of their first A4 float4 (the part that is orthogonalised).  All lanes take the same branch.
//   Rotate while the cosine of the angle between the rows exceeds tol.
//   tan(2 theta) = 2 gamma / (beta - alpha), |theta| <= pi/4, from normalised quantities (no overflow for
//   norm ratios up to 1e24): with g = gamma / (||x_p|| ||x_q||), tau = (beta - alpha) / (||x_p|| ||x_q||),
//   h = sqrt(tau^2 + 4 g^2):  t = tan(theta) = 2 g sign(tau) / (h + |tau|).  Approximate rsqrt / reciprocal
//   (about 2 ulp) are enough for t: an error there leaves a residual cosine of that relative size, far
//   below tol.  The cosine c is then derived from t itself with a Newton step, so the applied
//   transformation is orthogonal to 1 ulp.
//   The cosine g when one warp holds the rows: each lane scales its part of the dot product by
//   d_p d_q / (||x_p|| ||x_q||) (known before the products), so that the parts add up to at most 1 in
//   magnitude, converts to fixed point with 29 fractional bits and the warp adds the integers in one
//   instruction: an absolute error below 3e-8 in g (a tenth of the smallest tol in use), exact and
//   order-free integer addition, a fifth of the latency of a shuffle tree.
//   Scaled ("fast Givens") update, one FMA per element:  x_p' = c (x_p - t x_q),  x_q' = c (x_q + t x_p)
//   becomes v_p += a v_q, v_q += b v_p(old) with a = -t d_q/d_p, b = t d_p/d_q, and d_p, d_q *= c.
//   `store` is called as soon as the rows are updated; cosine, factors and norms follow it.
//   Norms are tracked: alpha' = alpha - t gamma, beta' = beta + t gamma; the shrinking one loses digits by
//   cancellation and is recomputed from the row when it dropped by 1000x.  (A stale norm can only waste or
//   postpone a rotation: a sweep that rotates nothing changes no norm, so the convergence test always sees
//   norms computed from the rows.)
template <int T4, int WPR, typename Store>
__device__ __forceinline__ bool rotate_pair(RowRegs<T4>& xp, RowRegs<T4>& xq, float& np2, float& nq2, float& dp,
                                            float& dq, int lane, int A4, float tol, RowSum<WPR>& row_sum, Store&& store) {
  // dot product and update in packed fp32 pairs (one instruction per two elements)
  uint64_t gA = 0ull, gB = 0ull;
#pragma unroll
  for (int t = 0; t < T4; ++t) {
    if (lane + 32 * t < A4) {
      const float4 a = xp.v[t], b = xq.v[t];
      gA = fma2(pack2(a.x, a.y), pack2(b.x, b.y), gA);
      gB = fma2(pack2(a.z, a.w), pack2(b.z, b.w), gB);
    }
  }
  float g0, g1, g2, g3;
  unpack2(gA, g0, g2); unpack2(gB, g1, g3);
  g0 += g2; g1 += g3;
  // everything that does not need the dot product
  const float al = np2, be = nq2;
  const float m = rsqrt_approx(al) * rsqrt_approx(be);
  const float dpq = dp * dq;
  const float ratio_qp = dq * rcp_approx(dp), ratio_pq = dp * rcp_approx(dq);
  const float tau = (be - al) * m;
  const float tau2 = tau * tau, atau = fabsf(tau);
  const bool valid = al >= kRowFloor && be >= kRowFloor;
  float gn, ga;                                              // cosine between the rows, dot product of the true rows
  if constexpr (WPR == 1) {
    const int part = __float2int_rn((g0 + g1) * (dpq * m * 536870912.0f));       // 2^29; NaN -> 0, saturating
    gn = (float)__reduce_add_sync(0xffffffffu, part) * (1.0f / 536870912.0f);
    ga = gn * ((al * m) * be);
  } else {
    ga = row_sum(g0 + g1) * dpq;
    gn = ga * m;
  }
  if (!valid) return false;
  if (!(fabsf(gn) > tol)) return false;                      // also false for NaN
  const float q = fmaf(4.0f * gn, gn, tau2);
  const float h = q * rsqrt_approx(q);
  const float tt = copysignf(2.0f * gn, gn * tau) * rcp_approx(h + atau);
  if (tt == 0.0f) return false;
  const float a = -tt * ratio_qp, b = tt * ratio_pq;
  const uint64_t a2 = pack2(a, a), b2 = pack2(b, b);
#pragma unroll
  for (int t = 0; t < T4; ++t) {
    const float4 u = xp.v[t], w = xq.v[t];
    const uint64_t u01 = pack2(u.x, u.y), u23 = pack2(u.z, u.w), w01 = pack2(w.x, w.y), w23 = pack2(w.z, w.w);
    unpack2(fma2(a2, w01, u01), xp.v[t].x, xp.v[t].y);
    unpack2(fma2(a2, w23, u23), xp.v[t].z, xp.v[t].w);
    unpack2(fma2(b2, u01, w01), xq.v[t].x, xq.v[t].y);
    unpack2(fma2(b2, u23, w23), xq.v[t].z, xq.v[t].w);
  }
  store();
  const float y = fmaf(tt, tt, 1.0f);
  float c = rsqrt_approx(y);
  c = c * fmaf(-0.5f * y * c, c, 1.5f);
  dp *= c; dq *= c;
  const float tg = tt * ga;
  np2 = al - tg; nq2 = be + tg;
  if (np2 < 1e-3f * al) np2 = row_sum(row_norm2_partial<T4>(xp, lane, A4)) * dp * dp;
  if (nq2 < 1e-3f * be) nq2 = row_sum(row_norm2_partial<T4>(xq, lane, A4)) * dq * dq;
  return true;
}

// One block pair (2 B rows, B = 16 / WPR) of one layer, resident in shared memory.  16 warps; a rotation
// is done by WPR warps, each holding one segment of the two rows (WPR = 1 for rows of up to 1024 floats).
// RP = padded short side; ACC: rows are [x | v] (2 RP floats, mode 0), else x only (RP floats, mode 1).
template <int RP, bool ACC, int WPR>
__device__ __forceinline__ void jacobi_block_pair(const SpLayer& L, int slot, int sweep, int local, bool resident,
                                                  float tol, float* smem) {
  constexpr int B = kJB / WPR;
  constexpr int LD = ACC ? 2 * RP : RP;                 // floats per row
  constexpr int SEG = LD / WPR;                         // floats per warp segment
  constexpr int V4 = SEG / 4, T4 = (V4 + 31) / 32;      // float4 per segment, per lane
  constexpr int A4 = ACC ? RP / 4 : V4;                 // float4 of a segment that take part in dot products
  constexpr int NT = 32 * kJB, R4 = LD / 4;
  static_assert(T4 <= 8, "segment too long for one warp");
  static_assert(!ACC || WPR == 1, "route 0 rows are held by one warp");
  float* s_n2 = smem + 2 * B * LD;       // squared norms of the true rows
  float* s_d = s_n2 + 2 * B;             // true row = s_d * stored row
  float* s_part = s_d + 2 * B;           // [B][2][WPR] warp sums of a pair
  const int tid = threadIdx.x, lane = tid % 32, w = tid / 32;
  const int pi = w / WPR, seg = w % WPR; // pair slot, segment
  RowSum<WPR> row_sum{s_part + pi * 2 * WPR, 1 + pi, seg, lane, 0};
  // `resident` (the persistent kernel): the first block stays in shared memory, with its tracked norms, for all
  // steps of a level; it is loaded at the level's first step and stored at its last.
  const StepPlan plan = step_plan(L.nb, local, slot);
  const int bi = plan.bi, bj = plan.bj;
  const bool load_first = !resident || plan.first_in_level, store_first = !resident || plan.last_in_level;
  float* X = L.X;
#ifdef ATOMO_PHASE_TIMING
  long long tk[8]; int nk = 0;
#define ATOMO_TICK() tk[nk++] = clock64()
#else
#define ATOMO_TICK()
#endif
  ATOMO_TICK();
  // ---- load the rows (the first block only when it is not already here) ----
  for (int idx = tid + (load_first ? 0 : B * R4); idx < 2 * B * R4; idx += NT) {
    const int row = idx / R4, q = idx % R4;
    const int grow = (row < B) ? bi * B + row : bj * B + (row - B);
    reinterpret_cast<float4*>(smem + row * LD)[q] = reinterpret_cast<const float4*>(X + (int64_t)grow * LD)[q];
  }
  __syncthreads();
  RowRegs<T4> xp, xq;
  // pair slot pi: squared norms of rows pi and pi + B, computed from every row that was just loaded (a resident
  // row keeps its tracked norm); row pi stays in registers for the cross rounds
  load_row<T4>(xq, smem + (B + pi) * LD + seg * SEG, lane, V4);
  const float nj = row_sum(row_norm2_partial<T4>(xq, lane, A4));
  load_row<T4>(xp, smem + pi * LD + seg * SEG, lane, V4);
  float np2 = load_first ? row_sum(row_norm2_partial<T4>(xp, lane, A4)) : s_n2[pi], dp = 1.0f;
  if (lane == 0 && seg == 0) {
    if (load_first) { s_n2[pi] = np2; s_d[pi] = 1.0f; }
    s_n2[B + pi] = nj; s_d[B + pi] = 1.0f;
  }
  __syncthreads();
  ATOMO_TICK();
  uint32_t nrot = 0;
  // ---- pairs inside each block: once per sweep ----
  if (local == 0) {
    for (int round = 0; round < B - 1; ++round) {
      const int blk = pi / (B / 2), sl = pi % (B / 2);
      int p, q;
      rr_pair(B, round, sl, p, q);
      p += blk * B; q += blk * B;
      float* rowp = smem + p * LD + seg * SEG;
      float* rowq = smem + q * LD + seg * SEG;
      load_row<T4>(xp, rowp, lane, V4);
      load_row<T4>(xq, rowq, lane, V4);
      float a2 = s_n2[p], b2 = s_n2[q], da = s_d[p], db = s_d[q];
      const bool rot = rotate_pair<T4, WPR>(xp, xq, a2, b2, da, db, lane, A4, tol, row_sum, [&] {
        store_row<T4>(xp, rowp, lane, V4);
        store_row<T4>(xq, rowq, lane, V4);
      });
      if (WPR > 1) __syncthreads();       // every warp of the pair has read the old norms and factors
      if (rot) {
        if (lane == 0 && seg == 0) { s_n2[p] = a2; s_n2[q] = b2; s_d[p] = da; s_d[q] = db; }
        if (seg == 0) ++nrot;
      }
      __syncthreads();
    }
    load_row<T4>(xp, smem + pi * LD + seg * SEG, lane, V4);
    np2 = s_n2[pi]; dp = s_d[pi];
  }
  ATOMO_TICK();
  // ---- pairs across the two blocks: slot pi keeps row pi of block bi in registers; the rows of block bj
  //      visit the slots round-robin ----
  for (int round = 0; round < B; ++round) {
    const int j = B + (pi + round) % B;
    float* rowq = smem + j * LD + seg * SEG;
    load_row<T4>(xq, rowq, lane, V4);
    float nq2 = s_n2[j], dq = s_d[j];
    const bool rot = rotate_pair<T4, WPR>(xp, xq, np2, nq2, dp, dq, lane, A4, tol, row_sum,
                                          [&] { store_row<T4>(xq, rowq, lane, V4); });
    if (WPR > 1) __syncthreads();         // every warp of the pair has read the old norm and factor
    if (rot) {
      if (lane == 0 && seg == 0) { s_n2[j] = nq2; s_d[j] = dq; }
      if (seg == 0) ++nrot;
    }
    __syncthreads();
  }
  ATOMO_TICK();
  store_row<T4>(xp, smem + pi * LD + seg * SEG, lane, V4, dp);
  if (lane == 0 && seg == 0) { s_d[pi] = 1.0f; s_n2[pi] = np2; }
  __syncthreads();
  // ---- store, folding the collected cosines back into the rows (the first block only when it leaves) ----
  for (int idx = tid + (store_first ? 0 : B * R4); idx < 2 * B * R4; idx += NT) {
    const int row = idx / R4, q = idx % R4;
    const int grow = (row < B) ? bi * B + row : bj * B + (row - B);
    const float d = s_d[row];
    const float4 a = reinterpret_cast<const float4*>(smem + row * LD)[q];
    reinterpret_cast<float4*>(X + (int64_t)grow * LD)[q] = make_float4(a.x * d, a.y * d, a.z * d, a.w * d);
  }
  if (lane == 0 && nrot) atomicAdd(L.rot_count + sweep, nrot);
  ATOMO_TICK();
#ifdef ATOMO_PHASE_TIMING
  if (tid == 0 && slot == 0 && (sweep == 2 || sweep == 8) && local < 2)
    printf("rp %d acc %d sweep %d local %d: load+norm %lld intra %lld cross %lld store %lld (clk) nrot(w0) %u\n", RP, (int)ACC,
           sweep, local, tk[1] - tk[0], tk[2] - tk[1], tk[3] - tk[2], tk[4] - tk[3], nrot);
#endif
}

constexpr int kJacobiThreads = 32 * kJB;
constexpr int kJacobiThreadsC = kJacobiThreads;

__device__ __forceinline__ void jacobi_dispatch(const SpLayer& L, int slot, int sweep, int local, bool resident, float tol,
                                                float* smem) {
  if (L.acc) {
    switch (L.rp) {
      case 32: jacobi_block_pair<32, true, 1>(L, slot, sweep, local, resident, tol, smem); break;
      case 64: jacobi_block_pair<64, true, 1>(L, slot, sweep, local, resident, tol, smem); break;
      case 128: jacobi_block_pair<128, true, 1>(L, slot, sweep, local, resident, tol, smem); break;
      case 256: jacobi_block_pair<256, true, 1>(L, slot, sweep, local, resident, tol, smem); break;
      case 512: jacobi_block_pair<512, true, 1>(L, slot, sweep, local, resident, tol, smem); break;
      default: break;
    }
  } else {
    switch (L.rp) {
      case 32: jacobi_block_pair<32, false, 1>(L, slot, sweep, local, resident, tol, smem); break;
      case 64: jacobi_block_pair<64, false, 1>(L, slot, sweep, local, resident, tol, smem); break;
      case 128: jacobi_block_pair<128, false, 1>(L, slot, sweep, local, resident, tol, smem); break;
      case 256: jacobi_block_pair<256, false, 1>(L, slot, sweep, local, resident, tol, smem); break;
      case 512: jacobi_block_pair<512, false, 1>(L, slot, sweep, local, resident, tol, smem); break;
      case 1024: jacobi_block_pair<1024, false, 1>(L, slot, sweep, local, resident, tol, smem); break;
      case 2048: jacobi_block_pair<2048, false, 2>(L, slot, sweep, local, resident, tol, smem); break;
      case 4096: jacobi_block_pair<4096, false, 4>(L, slot, sweep, local, resident, tol, smem); break;
      default: break;
    }
  }
}

// One Jacobi step for every layer: mode 1 layers with padded short side <= 4096, mode 0 layers with <= 512.
__global__ void __launch_bounds__(kJacobiThreads) sp_jacobi_step_kernel(const SpLayer* __restrict__ layers,
                                                                        const TileRef* __restrict__ pairs, int t,
                                                                        int max_sweeps, float tol) {
  extern __shared__ __align__(16) float smem[];
  const TileRef ref = pairs[blockIdx.x];
  const SpLayer& L = layers[ref.layer];
  const int steps = L.nb - 1;
  const int sweep = t / steps, local = t % steps;
  if (sweep >= max_sweeps) return;
  if (sweep > 0 && L.rot_count[sweep - 1] == 0) return;   // the previous sweep rotated nothing: converged
  jacobi_dispatch(L, ref.a, sweep, local, false, tol, smem);
}

// The whole eigen-solve in one cooperative launch, for batches whose block pairs are all co-resident (one CTA
// per SM; the cooperative launch is what guarantees that).  The kernel boundary between steps becomes a barrier
// among the CTAs of ONE layer (layers are independent): a counter in global memory that every CTA of the layer
// increments after its stores and then polls until all have arrived.  The poll is bounded: a CTA that gives up
// raises state[0] and leaves, and so will the others of its layer.  A layer stops at the first sweep boundary
// whose finished sweep rotated nothing; its CTAs all read the same, final count there, because every one of them
// has passed the barrier that closes that sweep.  state[1] receives the largest number of steps any layer took.
constexpr uint32_t kStepBarSpinLimit = 1u << 22;

__global__ void __launch_bounds__(kJacobiThreads) sp_jacobi_persistent_kernel(const SpLayer* __restrict__ layers,
                                                                              const TileRef* __restrict__ pairs,
                                                                              int max_sweeps, float tol,
                                                                              uint32_t* __restrict__ state) {
  extern __shared__ __align__(16) float smem[];
  __shared__ int s_fail;
  const TileRef ref = pairs[blockIdx.x];
  const SpLayer& L = layers[ref.layer];
  const int steps = L.nb - 1, n_ctas = L.nb / 2;
  const int t_max = steps * max_sweeps;
  int t = 0;
  for (; t < t_max; ++t) {
    const int sweep = t / steps, local = t % steps;
    if (local == 0 && sweep > 0 && *(volatile uint32_t*)(L.rot_count + sweep - 1) == 0) break;
    jacobi_dispatch(L, ref.a, sweep, local, true, tol, smem);
    __syncthreads();
    if (n_ctas > 1) {
      if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(L.step_bar, 1u);
        const uint32_t target = (uint32_t)(t + 1) * (uint32_t)n_ctas;
        uint32_t spins = 0;
        int fail = 0;
        while (*(volatile uint32_t*)L.step_bar < target)
          if (++spins > kStepBarSpinLimit) { fail = 1; break; }
        __threadfence();
        s_fail = fail;
      }
      __syncthreads();
      if (s_fail) {
        if (threadIdx.x == 0) atomicExch(state, 1u);
        break;
      }
    }
  }
  if (threadIdx.x == 0) atomicMax(state + 1, (uint32_t)t);
}

constexpr int kJacobiSmem = 32 * 1024 * 4 + 1024;   // 32 rows of up to 1024 floats + norms and factors

int sp_jacobi_persistent_capacity(int row_floats_max) {
  int dev = 0, sms = 0, per_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  const int smem = 32 * std::min(row_floats_max, 1024) * 4 + 1024;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sp_jacobi_persistent_kernel, kJacobiThreads, smem) != cudaSuccess) return 0;
  return sms * per_sm;
}

int launch_sp_jacobi_persistent(const SpLayer* d_layers, const TileRef* d_pairs, int n_pairs, int row_floats_max,
                                int max_sweeps, float tol, uint32_t* d_state, cudaStream_t st) {
  const int smem = 32 * std::min(row_floats_max, 1024) * 4 + 1024;
  void* args[] = {(void*)&d_layers, (void*)&d_pairs, (void*)&max_sweeps, (void*)&tol, (void*)&d_state};
  return (int)cudaLaunchCooperativeKernel((const void*)sp_jacobi_persistent_kernel, dim3(n_pairs), dim3(kJacobiThreads), args,
                                          smem, st);
}

void launch_sp_jacobi_step(const SpLayer* d_layers, const TileRef* d_pairs, int n_pairs, int row_floats_max,
                           int t, int max_sweeps, float tol, cudaStream_t st) {
  if (n_pairs <= 0) return;
  const int smem = 32 * std::min(row_floats_max, 1024) * 4 + 1024;
  sp_jacobi_step_kernel<<<n_pairs, kJacobiThreads, smem, st>>>(d_layers, d_pairs, t, max_sweeps, tol);
}

// =================================================================================================
// Cluster form of the persistent eigen-solve, for layers of up to 16 block pairs (padded short side <= 512).
// The CTAs of a layer sit in one thread-block cluster (16 CTAs; smaller layers share a cluster) and the blocks
// never return to global memory between steps: at the end of a step a CTA writes its moving block (and, when a
// level of the schedule ends, its resident block) straight into the shared memory of the CTA that pairs it
// next -- distributed shared memory -- together with the rows' tracked norms, and a cluster barrier takes the
// place of the global-memory barrier.  Four row regions per CTA: resident block x 2 and moving block x 2, so
// that an incoming block never lands in a region that is still being rotated.  Norms are recomputed from
// the rows at the start of every sweep.  A cluster ends when all its layers have converged (or hit the sweep
// cap): every CTA announces the iteration in which it finished in every CTA's `done` table, and after barrier t
// all CTAs take the same decision from the announcements made up to iteration t, so they leave together.  Rotation formulas, pairings and thresholds are those of the kernels above.
// =================================================================================================
constexpr int kClusterCtas = 16;

template <int RP>
struct ClusterRegion {
  static constexpr int kRowFloats = kJB * RP;
  static constexpr int kFloats = kRowFloats + 2 * kJB;            // rows, squared norms, factors
  float* base;
  __device__ __forceinline__ float* row(int i) const { return base + i * RP; }
  __device__ __forceinline__ float* n2() const { return base + kRowFloats; }
  __device__ __forceinline__ float* d() const { return base + kRowFloats + kJB; }
};

template <int RP>
__device__ __forceinline__ void cluster_step(const SpLayer& L, const ClusterCta& me, int t, int& fpar, int& mpar,
                                             int max_sweeps, float tol, float* smem, uint32_t* s_mask,
                                             cg::cluster_group& cluster, bool& done) {
  constexpr int B = kJB, V4 = RP / 4, T4 = (V4 + 31) / 32, NT = kJacobiThreadsC, R4 = RP / 4;
  using Region = ClusterRegion<RP>;
  const int tid = threadIdx.x, lane = tid % 32, pi = tid / 32;
  const int steps = L.nb - 1;
  const int sweep = t / steps, local = t % steps;
  const StepPlan plan = step_plan(L.nb, local, me.slot);
  Region F{smem + fpar * Region::kFloats}, M{smem + (2 + mpar) * Region::kFloats};
  float* X = L.X;
  RowSum<1> row_sum{nullptr, 0, 0, lane, 0};
  if (t == 0) {                                                  // the only load from global memory
    for (int idx = tid; idx < 2 * B * R4; idx += NT) {
      const int row = idx / R4, q = idx % R4;
      const int grow = (row < B) ? plan.bi * B + row : plan.bj * B + (row - B);
      float* dst = row < B ? F.row(row) : M.row(row - B);
      reinterpret_cast<float4*>(dst)[q] = reinterpret_cast<const float4*>(X + (int64_t)grow * RP)[q];
    }
    __syncthreads();
  }
  const bool converged = local == 0 && sweep > 0 && *(volatile uint32_t*)(L.rot_count + sweep - 1) == 0;
  if (converged || sweep >= max_sweeps) {                        // the blocks held now are those of step `local`
    for (int idx = tid; idx < 2 * B * R4; idx += NT) {
      const int row = idx / R4, q = idx % R4;
      const int grow = (row < B) ? plan.bi * B + row : plan.bj * B + (row - B);
      const float* src = row < B ? F.row(row) : M.row(row - B);
      reinterpret_cast<float4*>(X + (int64_t)grow * RP)[q] = reinterpret_cast<const float4*>(src)[q];
    }
    // the rows' squared norms as well: after a sweep that rotated nothing they are the ones computed from the rows
    // at its start, which is what the singular values are taken from
    if (tid < 2 * B) {
      const int grow = (tid < B) ? plan.bi * B + tid : plan.bj * B + (tid - B);
      L.lam[grow] = tid < B ? F.n2()[tid] : M.n2()[tid - B];
    }
    done = true;
    return;
  }
  RowRegs<T4> xp, xq;
  if (local == 0) {                                              // sweep start: norms from the rows (factors are 1)
    load_row<T4>(xq, M.row(pi), lane, V4);
    const float nj = warp_sum(row_norm2_partial<T4>(xq, lane, V4));
    load_row<T4>(xp, F.row(pi), lane, V4);
    const float ni = warp_sum(row_norm2_partial<T4>(xp, lane, V4));
    if (lane == 0) { F.n2()[pi] = ni; M.n2()[pi] = nj; }
  }
  if (lane == 0) { F.d()[pi] = 1.0f; M.d()[pi] = 1.0f; }
  __syncthreads();
  auto rowp_of = [&](int p) { return p < B ? F.row(p) : M.row(p - B); };
  auto n2_of = [&](int p) -> float& { return p < B ? F.n2()[p] : M.n2()[p - B]; };
  auto d_of = [&](int p) -> float& { return p < B ? F.d()[p] : M.d()[p - B]; };
  uint32_t nrot = 0;
  if (local == 0) {                                              // pairs inside each block: once per sweep
    for (int round = 0; round < B - 1; ++round) {
      const int blk = pi / (B / 2), sl = pi % (B / 2);
      int p, q;
      rr_pair(B, round, sl, p, q);
      p += blk * B; q += blk * B;
      float* rowp = rowp_of(p);
      float* rowq = rowp_of(q);
      load_row<T4>(xp, rowp, lane, V4);
      load_row<T4>(xq, rowq, lane, V4);
      float a2 = n2_of(p), b2 = n2_of(q), da = d_of(p), db = d_of(q);
      const bool rot = rotate_pair<T4, 1>(xp, xq, a2, b2, da, db, lane, V4, tol, row_sum, [&] {
        store_row<T4>(xp, rowp, lane, V4);
        store_row<T4>(xq, rowq, lane, V4);
      });
      if (rot) {
        if (lane == 0) { n2_of(p) = a2; n2_of(q) = b2; d_of(p) = da; d_of(q) = db; }
        ++nrot;
      }
      __syncthreads();
    }
  }
  // Late sweeps rotate little: when the finished sweep averaged fewer than 8 rotations per CTA and step, look at
  // all 16 x 16 cosines first (each warp: 2 resident rows against 8 moving rows, no barrier, nothing written)
  // and run only the rounds that hold a pair above tol.  (A rotation changes the other cosines of its two rows
  // only to second order; whatever that lifts above tol is met again in the next sweep, which then takes place
  // because this one rotated.)  Factors are 1 here, so the stored rows are the true rows.
  uint32_t round_mask = 0xffffu;
  if (local != 0 && sweep > 0 && *(volatile uint32_t*)(L.rot_count + sweep - 1) < (uint32_t)(8 * steps * (L.nb / 2))) {
    const int a = pi >> 1, half = pi & 1;
    RowRegs<T4> x0, x1;
    load_row<T4>(x0, F.row(2 * a), lane, V4);
    load_row<T4>(x1, F.row(2 * a + 1), lane, V4);
    const float r0 = rsqrt_approx(F.n2()[2 * a]), r1 = rsqrt_approx(F.n2()[2 * a + 1]);
    const bool ok0 = F.n2()[2 * a] >= kRowFloor, ok1 = F.n2()[2 * a + 1] >= kRowFloor;
    uint32_t need = 0;
#pragma unroll 2
    for (int jj = 0; jj < B / 2; ++jj) {
      const int j = half * (B / 2) + jj;
      load_row<T4>(xq, M.row(j), lane, V4);
      float g0 = 0.f, g1 = 0.f;
#pragma unroll
      for (int u = 0; u < T4; ++u) {
        if (lane + 32 * u < V4) {
          const float4 q4 = xq.v[u], p0 = x0.v[u], p1 = x1.v[u];
          g0 = fmaf(p0.x, q4.x, fmaf(p0.y, q4.y, fmaf(p0.z, q4.z, fmaf(p0.w, q4.w, g0))));
          g1 = fmaf(p1.x, q4.x, fmaf(p1.y, q4.y, fmaf(p1.z, q4.z, fmaf(p1.w, q4.w, g1))));
        }
      }
      const float nq = M.n2()[j];
      const float rq = rsqrt_approx(nq) * 536870912.0f;          // 2^29: the same fixed-point cosine as rotate_pair
      const int c0 = __reduce_add_sync(0xffffffffu, __float2int_rn(g0 * (r0 * rq)));
      const int c1 = __reduce_add_sync(0xffffffffu, __float2int_rn(g1 * (r1 * rq)));
      const float lim = tol * 536870912.0f;
      const bool okq = nq >= kRowFloor;
      // row i of the resident block meets row j of the moving block in round (j - i) mod 16
      if (okq && ok0 && !(fabsf((float)c0) <= lim)) need |= 1u << ((j - 2 * a) & (B - 1));
      if (okq && ok1 && !(fabsf((float)c1) <= lim)) need |= 1u << ((j - 2 * a - 1) & (B - 1));
    }
    if (lane == 0 && need) atomicOr(s_mask, need);
    __syncthreads();
    round_mask = *s_mask;
    __syncthreads();
    if (tid == 0) *s_mask = 0;                                     // for the next step (ordered by the barriers below)
  }
  load_row<T4>(xp, F.row(pi), lane, V4);
  float np2 = F.n2()[pi], dp = F.d()[pi];
  for (int round = 0; round < B; ++round) {                      // pairs across the two blocks
    if (!((round_mask >> round) & 1u)) continue;
    const int j = (pi + round) % B;
    float* rowq = M.row(j);
    load_row<T4>(xq, rowq, lane, V4);
    float nq2 = M.n2()[j], dq = M.d()[j];
    const bool rot = rotate_pair<T4, 1>(xp, xq, np2, nq2, dp, dq, lane, V4, tol, row_sum,
                                        [&] { store_row<T4>(xq, rowq, lane, V4); });
    if (rot) {
      if (lane == 0) { M.n2()[j] = nq2; M.d()[j] = dq; }
      ++nrot;
    }
    __syncthreads();
  }
  store_row<T4>(xp, F.row(pi), lane, V4, dp);
  if (lane == 0) { F.d()[pi] = 1.0f; F.n2()[pi] = np2; }
  if (lane == 0 && nrot) atomicAdd(L.rot_count + sweep, nrot);
  __syncthreads();
  // ---- hand the blocks to the CTAs that pair them at the next step ----
  const int next_local = (local + 1) % steps;
  for (int which = 0; which < 2; ++which) {                      // 0: moving block, 1: resident block (level end only)
    if (which == 1 && !plan.last_in_level) break;
    const int blk = which == 0 ? plan.bj : plan.bi;
    int slot, role;
    find_holder(L.nb, next_local, blk, slot, role);
    const Region src = which == 0 ? M : F;
    const int dst_region = role == 0 ? (fpar ^ 1) : 2 + (mpar ^ 1);
    float* dst_local = smem + dst_region * Region::kFloats;
    float* dst = cluster.map_shared_rank(dst_local, me.base_rank + slot);
    for (int idx = tid; idx < B * R4; idx += NT) {
      const int row = idx / R4, q = idx % R4;
      const float dv = src.d()[row];
      const float4 a = reinterpret_cast<const float4*>(src.row(row))[q];
      reinterpret_cast<float4*>(dst + row * RP)[q] = make_float4(a.x * dv, a.y * dv, a.z * dv, a.w * dv);
    }
    if (tid < B) dst[Region::kRowFloats + tid] = src.n2()[tid];
  }
  mpar ^= 1;
  if (plan.last_in_level) fpar ^= 1;
}

__global__ void __launch_bounds__(kJacobiThreadsC) sp_jacobi_cluster_kernel(const SpLayer* __restrict__ layers,
                                                                            const ClusterCta* __restrict__ ctas,
                                                                            int max_sweeps, float tol) {
  extern __shared__ __align__(16) float smem[];
  __shared__ int s_done[kClusterCtas];
  __shared__ uint32_t s_mask;                            // rounds of the current step that hold a pair to rotate
  cg::cluster_group cluster = cg::this_cluster();
  const ClusterCta me = ctas[blockIdx.x];
  const int my_rank = (int)cluster.block_rank();
  // s_done[r] = the iteration in which CTA r finished (a CTA may already be writing the next iteration's
  // announcement while another still reads the table: comparing with the iteration number makes the
  // decision after barrier t depend only on announcements made before barrier t)
  if (threadIdx.x < kClusterCtas) s_done[threadIdx.x] = 0x7fffffff;
  if (threadIdx.x == 0) s_mask = 0;
  bool done = me.layer < 0, announced = false;
  int fpar = 0, mpar = 0;
  cluster.sync();
  for (int t = 0;; ++t) {
    if (!done) {
      const SpLayer& L = layers[me.layer];
      switch (L.rp) {
        case 32: cluster_step<32>(L, me, t, fpar, mpar, max_sweeps, tol, smem, &s_mask, cluster, done); break;
        case 64: cluster_step<64>(L, me, t, fpar, mpar, max_sweeps, tol, smem, &s_mask, cluster, done); break;
        case 128: cluster_step<128>(L, me, t, fpar, mpar, max_sweeps, tol, smem, &s_mask, cluster, done); break;
        case 256: cluster_step<256>(L, me, t, fpar, mpar, max_sweeps, tol, smem, &s_mask, cluster, done); break;
        case 512: cluster_step<512>(L, me, t, fpar, mpar, max_sweeps, tol, smem, &s_mask, cluster, done); break;
        default: done = true; break;
      }
    }
    if (done && !announced) {
      if (threadIdx.x < kClusterCtas) cluster.map_shared_rank(s_done, threadIdx.x)[my_rank] = t;
      announced = true;
    }
    cluster.sync();
    int pending = 0;
    if (threadIdx.x < kClusterCtas) pending = *(volatile int*)(s_done + threadIdx.x) > t;
    if (!__syncthreads_or(pending)) break;
  }
}

// convergence bookkeeping after t_done steps have been enqueued
__global__ void sp_check_kernel(const SpLayer* __restrict__ layers, int n_layers, int t_done, int max_sweeps,
                                uint32_t* all_done) {
  __shared__ int s_pending;
  if (threadIdx.x == 0) s_pending = 0;
  __syncthreads();
  for (int l = threadIdx.x; l < n_layers; l += blockDim.x) {
    const SpLayer& L = layers[l];
    const int steps = L.nb - 1;
    const int sweeps_done = min(t_done / steps, max_sweeps);
    int conv = -1;
    for (int wv = 0; wv < sweeps_done; ++wv) if (L.rot_count[wv] == 0) { conv = wv; break; }
    if (conv >= 0) L.hdr->sweeps = (uint32_t)(conv + 1);
    else {
      L.hdr->sweeps = (uint32_t)sweeps_done;
      if (sweeps_done < max_sweeps) atomicAdd(&s_pending, 1);
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) *all_done = s_pending == 0 ? 1u : 0u;
}

void launch_sp_check(const SpLayer* d_layers, int n_layers, int t_done, int max_sweeps, uint32_t* d_all_done,
                     cudaStream_t st) {
  sp_check_kernel<<<1, 256, 0, st>>>(d_layers, n_layers, t_done, max_sweeps, d_all_done);
}

// =================================================================================================
// Cholesky factor of the scaled Gram matrix, written transposed: X[c][i] = L[i][c].
// One thread per row, left-looking over panels of 32 columns; a thread keeps its row of the current panel
// in registers.  A pivot below kPivotFloor (trace(A) = 1) is rounding noise of the fp32 Gram matrix: that
// column of L is set to zero (L L^T then differs from A by that noise).
// =================================================================================================
constexpr float kPivotFloor = 1e-9f;
constexpr int kCholPanel = 32;

// Layers of up to 1024 rows: a cluster of 8 CTAs per layer (the panel update would be FMA-bound on one SM);
// each CTA takes max(32, rp / 8) consecutive rows.
// Per panel: every CTA updates its rows; the warp that owns the diagonal block factors it and publishes it in
// global memory; cluster barrier; every CTA solves its rows against it and stores them; cluster barrier (the
// next panel reads rows of L written by other CTAs; those reads bypass L1).
constexpr int kCholClusterCtas = 8, kCholClusterThreads = 128;

__global__ void __launch_bounds__(kCholClusterThreads) sp_cholesky_cluster_kernel(const SpLayer* __restrict__ layers) {
  cg::cluster_group cluster = cg::this_cluster();
  const SpLayer& L = layers[blockIdx.x / kCholClusterCtas];
  if (L.acc || L.rp > 1024) return;                        // the whole cluster leaves: route 0 / sp_cholesky_big_kernel
  __shared__ __align__(16) float s_k[kCholPanel][kCholPanel];
  __shared__ float s_ldd[kCholPanel][kCholPanel + 1];
  __shared__ float s_inv[kCholPanel];
  const int r = L.r, rp = L.rp;
  const int rows_per_cta = max(32, rp / kCholClusterCtas);
  const int tid = threadIdx.x, lane = tid % 32;
  const int i = (int)cluster.block_rank() * rows_per_cta + tid;      // this thread's row
  const bool has_row = tid < rows_per_cta && i < r;
  const float* __restrict__ A = L.A;
  const int64_t lda = L.lda;
  float* X = L.X;
  float* dd = L.chol_dd;                                   // published diagonal block: 32 x 32, then 32 inverses
  for (int j0 = 0; j0 < r; j0 += kCholPanel) {
    const bool active = has_row && i >= j0;
    float p[kCholPanel];
#pragma unroll
    for (int c = 0; c < kCholPanel; ++c) p[c] = (active && j0 + c < r) ? A[(int64_t)(j0 + c) * lda + i] : 0.0f;
    const bool cta_active = (int)cluster.block_rank() * rows_per_cta + rows_per_cta > j0;   // some row of this CTA is >= j0
    if (cta_active) {
      // p[c] -= sum_{k < j0} L[i][k] L[j0+c][k], 32 values of k at a time; the next chunk's operands (this row's
      // L[i][k], and this thread's 8 elements of the 32 x 32 tile of the panel rows) are fetched while the current
      // chunk is multiplied
      constexpr int kTilePer = kCholPanel * kCholPanel / kCholClusterThreads;
      float xc[kCholPanel], tn[kTilePer];
      auto fetch = [&](int k0, float (&xv)[kCholPanel]) {
#pragma unroll
        for (int kk = 0; kk < kCholPanel; ++kk) xv[kk] = active ? X[(int64_t)(k0 + kk) * rp + i] : 0.0f;
#pragma unroll
        for (int u = 0; u < kTilePer; ++u) {
          const int idx = tid + u * kCholClusterThreads;
          tn[u] = __ldcg(X + (int64_t)(k0 + idx / kCholPanel) * rp + j0 + idx % kCholPanel);
        }
      };
      if (j0 > 0) fetch(0, xc);
      for (int k0 = 0; k0 < j0; k0 += kCholPanel) {
        __syncthreads();                                   // the previous chunk's tile has been read by everyone
#pragma unroll
        for (int u = 0; u < kTilePer; ++u) {
          const int idx = tid + u * kCholClusterThreads;
          s_k[idx / kCholPanel][idx % kCholPanel] = tn[u];
        }
        __syncthreads();
        float xn[kCholPanel];
        if (k0 + kCholPanel < j0) fetch(k0 + kCholPanel, xn);
        // packed fp32 pairs: one instruction updates two columns
        uint64_t pk[kCholPanel / 2];
#pragma unroll
        for (int c = 0; c < kCholPanel / 2; ++c) pk[c] = pack2(p[2 * c], p[2 * c + 1]);
#pragma unroll
        for (int kk = 0; kk < kCholPanel; ++kk) {
          const uint64_t xi2 = pack2(-xc[kk], -xc[kk]);
#pragma unroll
          for (int c = 0; c < kCholPanel; c += 4) {
            const ulonglong2 lk = *reinterpret_cast<const ulonglong2*>(&s_k[kk][c]);   // same address in every lane: broadcast
            pk[c / 2] = fma2(xi2, lk.x, pk[c / 2]);
            pk[c / 2 + 1] = fma2(xi2, lk.y, pk[c / 2 + 1]);
          }
        }
#pragma unroll
        for (int c = 0; c < kCholPanel / 2; ++c) unpack2(pk[c], p[2 * c], p[2 * c + 1]);
#pragma unroll
        for (int kk = 0; kk < kCholPanel; ++kk) xc[kk] = xn[kk];
      }
      if (tid < rows_per_cta && i >= j0 && i < j0 + kCholPanel) {        // the warp that owns the diagonal block
#pragma unroll
        for (int c = 0; c < kCholPanel; ++c) {
          const float d = __shfl_sync(0xffffffffu, p[c], c);
          // 1 / sqrt(d) from the approximation and one Newton step (1 ulp), sqrt(d) = d / sqrt(d)
          float inv = rsqrt_approx(fmaxf(d, kPivotFloor));
          inv = inv * fmaf(-0.5f * d * inv, inv, 1.5f);
          inv = d > kPivotFloor ? inv : 0.0f;
          const float lcc = d * inv;
          const float lic = lane > c ? p[c] * inv : (lane == c ? lcc : 0.0f);
          p[c] = lic;
#pragma unroll
          for (int c2 = 0; c2 < kCholPanel; ++c2) {
            if (c2 > c) {
              const float l2 = __shfl_sync(0xffffffffu, lic, c2);
              if (lane > c) p[c2] = fmaf(-lic, l2, p[c2]);
            }
          }
          if (lane == c) dd[kCholPanel * kCholPanel + c] = inv;
        }
#pragma unroll
        for (int c = 0; c < kCholPanel; ++c) dd[lane * kCholPanel + c] = p[c];
      }
    }
    cluster.sync();
    if (cta_active) {
      for (int idx = tid; idx < kCholPanel * kCholPanel; idx += kCholClusterThreads)
        s_ldd[idx / kCholPanel][idx % kCholPanel] = __ldcg(dd + idx);
      if (tid < kCholPanel) s_inv[tid] = __ldcg(dd + kCholPanel * kCholPanel + tid);
      __syncthreads();
      if (active && i >= j0 + kCholPanel) {
#pragma unroll
        for (int c = 0; c < kCholPanel; ++c) {
          float acc = p[c];
#pragma unroll
          for (int k = 0; k < c; ++k) acc = fmaf(-p[k], s_ldd[c][k], acc);
          p[c] = acc * s_inv[c];
        }
      }
      if (active) {
#pragma unroll
        for (int c = 0; c < kCholPanel; ++c)
          if (j0 + c < r) X[(int64_t)(j0 + c) * rp + i] = p[c];
      }
    }
    cluster.sync();
  }
}

// The same factorisation for layers with more than 1024 rows: kCholBigThreads rows per CTA, several CTAs per
// layer in one cooperative launch.  Per panel: every CTA updates its rows; the CTA that owns the diagonal block
// factors it and publishes it; grid barrier; every CTA solves its rows against it and stores them; grid barrier
// (the next panel reads rows of L written by other CTAs).
constexpr int kCholBigThreads = 1024;

__global__ void __launch_bounds__(kCholBigThreads) sp_cholesky_big_kernel(const SpLayer* __restrict__ layers,
                                                                          const TileRef* __restrict__ ctas, int max_panels) {
  cg::grid_group grid = cg::this_grid();
  const TileRef ref = ctas[blockIdx.x];
  const SpLayer& L = layers[ref.layer];
  __shared__ __align__(16) float s_k[kCholPanel][kCholPanel];
  __shared__ float s_ldd[kCholPanel][kCholPanel + 1];
  __shared__ float s_inv[kCholPanel];
  const int r = L.r, rp = L.rp;
  const int tid = threadIdx.x, lane = tid % 32, warp = tid / 32;
  const int i = ref.a * kCholBigThreads + tid;            // this thread's row
  const float* __restrict__ A = L.A;
  const int64_t lda = L.lda;
  float* X = L.X;
  float* dd = L.chol_dd;                                   // published diagonal block: 32 x 32, then 32 inverses
  for (int panel = 0; panel < max_panels; ++panel) {
    const int j0 = panel * kCholPanel;
    const bool live = j0 < r;                              // uniform per CTA
    const bool active = live && i >= j0 && i < r;
    float p[kCholPanel];
#pragma unroll
    for (int c = 0; c < kCholPanel; ++c) p[c] = (active && j0 + c < r) ? A[(int64_t)(j0 + c) * lda + i] : 0.0f;
    if (live) {
      for (int k0 = 0; k0 < j0; k0 += kCholPanel) {
        __syncthreads();
        for (int idx = tid; idx < kCholPanel * kCholPanel; idx += kCholBigThreads) {
          const int kk = idx / kCholPanel, c = idx % kCholPanel;
          s_k[kk][c] = X[(int64_t)(k0 + kk) * rp + j0 + c];
        }
        __syncthreads();
        if (active) {
#pragma unroll 4
          for (int kk = 0; kk < kCholPanel; ++kk) {
            const float xi = -X[(int64_t)(k0 + kk) * rp + i];
#pragma unroll
            for (int c = 0; c < kCholPanel; c += 4) {
              const float4 lk = *reinterpret_cast<const float4*>(&s_k[kk][c]);   // same address in every lane: broadcast
              p[c] = fmaf(xi, lk.x, p[c]); p[c + 1] = fmaf(xi, lk.y, p[c + 1]);
              p[c + 2] = fmaf(xi, lk.z, p[c + 2]); p[c + 3] = fmaf(xi, lk.w, p[c + 3]);
            }
          }
        }
      }
      if (i >= j0 && i < j0 + kCholPanel) {               // the warp that owns the diagonal block
#pragma unroll
        for (int c = 0; c < kCholPanel; ++c) {
          const float d = __shfl_sync(0xffffffffu, p[c], c);
          const float lcc = d > kPivotFloor ? sqrtf(d) : 0.0f;
          const float inv = lcc > 0.0f ? 1.0f / lcc : 0.0f;
          const float lic = lane > c ? p[c] * inv : (lane == c ? lcc : 0.0f);
          p[c] = lic;
#pragma unroll
          for (int c2 = 0; c2 < kCholPanel; ++c2) {
            if (c2 > c) {
              const float l2 = __shfl_sync(0xffffffffu, lic, c2);
              if (lane > c) p[c2] = fmaf(-lic, l2, p[c2]);
            }
          }
          if (lane == c) dd[kCholPanel * kCholPanel + c] = inv;
        }
#pragma unroll
        for (int c = 0; c < kCholPanel; ++c) dd[lane * kCholPanel + c] = p[c];
        __threadfence();
      }
    }
    (void)warp;
    grid.sync();
    if (live) {
      for (int idx = tid; idx < kCholPanel * kCholPanel; idx += kCholBigThreads) s_ldd[idx / kCholPanel][idx % kCholPanel] = dd[idx];
      if (tid < kCholPanel) s_inv[tid] = dd[kCholPanel * kCholPanel + tid];
      __syncthreads();
      if (active && i >= j0 + kCholPanel) {
#pragma unroll
        for (int c = 0; c < kCholPanel; ++c) {
          float acc = p[c];
#pragma unroll
          for (int k = 0; k < c; ++k) acc = fmaf(-p[k], s_ldd[c][k], acc);
          p[c] = acc * s_inv[c];
        }
      }
      if (active) {
#pragma unroll
        for (int c = 0; c < kCholPanel; ++c)
          if (j0 + c < r) X[(int64_t)(j0 + c) * rp + i] = p[c];
      }
      __threadfence();
    }
    grid.sync();
  }
}

int launch_sp_cholesky(const SpLayer* d_layers, int n_layers, int rp_max, cudaStream_t st) {
  (void)rp_max;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_layers * kCholClusterCtas);
  cfg.blockDim = dim3(kCholClusterThreads);
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = kCholClusterCtas; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return (int)cudaLaunchKernelEx(&cfg, sp_cholesky_cluster_kernel, d_layers);
}

int launch_sp_cholesky_big(const SpLayer* d_layers, const TileRef* d_ctas, int n_ctas, int max_panels, cudaStream_t st) {
  if (n_ctas <= 0) return 0;
  void* args[] = {(void*)&d_layers, (void*)&d_ctas, (void*)&max_panels};
  return (int)cudaLaunchCooperativeKernel((const void*)sp_cholesky_big_kernel, dim3(n_ctas), dim3(kCholBigThreads), args, 0, st);
}

int sp_cholesky_big_rows_per_cta() { return kCholBigThreads; }

// ---- cluster form: host side ----
static int cluster_smem_bytes(int rp_max) { return 4 * (kJB * rp_max + 2 * kJB) * (int)sizeof(float); }
int sp_jacobi_cluster_ctas() { return kClusterCtas; }
int sp_jacobi_cluster_max_rp() { return 512; }

// how many clusters of 16 such CTAs the GPU can hold at once (0: this form cannot run here)
int sp_jacobi_cluster_capacity(int rp_max) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kClusterCtas); cfg.blockDim = dim3(kJacobiThreads); cfg.dynamicSmemBytes = cluster_smem_bytes(rp_max);
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = kClusterCtas; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, sp_jacobi_cluster_kernel, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
  return n;
}

int launch_sp_jacobi_cluster(const SpLayer* d_layers, const ClusterCta* d_ctas, int n_clusters, int rp_max, int max_sweeps,
                             float tol, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_clusters * kClusterCtas); cfg.blockDim = dim3(kJacobiThreads);
  cfg.dynamicSmemBytes = cluster_smem_bytes(rp_max); cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = kClusterCtas; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return (int)cudaLaunchKernelEx(&cfg, sp_jacobi_cluster_kernel, d_layers, d_ctas, max_sweeps, tol);
}

int sp_configure_eig() {
  cudaError_t e = cudaFuncSetAttribute(sp_jacobi_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kJacobiSmem);
  if (e != cudaSuccess) return (int)e;
  e = cudaFuncSetAttribute(sp_jacobi_persistent_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kJacobiSmem);
  if (e != cudaSuccess) return (int)e;
  // the cluster form is optional: a GPU that refuses 16-CTA clusters simply reports a capacity of 0
  if (cudaFuncSetAttribute(sp_jacobi_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, cluster_smem_bytes(512)) != cudaSuccess ||
      cudaFuncSetAttribute(sp_jacobi_cluster_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)
    cudaGetLastError();
  return 0;
}

}  // namespace atomo
