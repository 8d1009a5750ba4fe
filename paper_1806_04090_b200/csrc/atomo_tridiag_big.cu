// Tridiagonal route for layers with a short side above 512 (Section 5 of the paper asks for the SVD of every layer
// gradient; the probabilities of Eq. 3 / Algorithm 1 need the singular values of all atoms, Eq. 2 the vectors of the
// kept atoms only).  The scaled Gram matrix A (r x r, r up to 4096) no longer fits the registers of a cluster, so it
// stays in global memory and the reduction is the blocked (panel) form of the Householder tridiagonalisation:
//
//   sp_tridiag_big_kernel : T = Q^T A Q.  A cluster of C CTAs (C = 1, 2, 4, 8 or 16) owns a layer; rows are dealt to
//                           the CTAs in blocks of 32 (block b belongs to CTA b mod C).  Within a panel of 32 columns
//                           the stored matrix A0 is not touched: step c forms column c as it would be after the
//                           panel's earlier reflectors (A0[:, c] - U W[c]^T - W U[c]^T), the unit reflector u_c
//                           (H_c = I - 2 u u^T), the product y = A0 u (the one pass over the trailing block) with the
//                           same correction, and w = 2 y - (2 u^T y) u.  After the panel the trailing block takes the
//                           rank-64 update A0 -= U W^T + W U^T (register-tiled, 4 x 4 outputs per thread).  The
//                           reflectors go to global memory as fp32 unit vectors for the back-transformation.
//                           Storage type T = float: the matrix and the panel vectors are kept in fp32; on clusters the
//                           product goes over the lower triangle in 32 x 32 sub-tiles dealt evenly to all warps of the
//                           cluster, each sub-tile's row and column sums (fp32 over 32 terms) rounded to fixed point
//                           and added as integers; with C = 1 and for T = double (everything in fp64) a warp takes
//                           a row, its lanes along the row.  Column updates, norms and all scalars are fp64.  Every sum has an order that does
//                           not depend on C: a sub-tile's sums are one warp's and integers add in any order, block-wide
//                           sums go over the 32-row blocks in ascending order.
//   sp_eigvec_big_cta_kernel / sp_eigvec_big_kernel (short sides up to 1024 / above)
//                         : vectors of the kept atoms: twisted factorisation of T - lambda I (the routine of the small
//                           route, its work vectors in global memory), back-transformation u = Q z four reflectors at
//                           a time (fp32) by a whole CTA: four warps per kept atom up to a short side of 1024, above it
//                           sixteen warps on up to four atoms at once (the reflectors are then read once per four
//                           atoms).
//
// The eigenvalues of T come from sp_bisect_kernel (atomo_tridiag.cu), as for the small layers.
// Work per layer: the matrix-vector products read sum_c (r - c)^2 / 2 ~ r^3 / 6 matrix entries (one triangle; bytes
// from L2 / HBM), the panel updates cost 2 r^3 / 3 multiply-adds.
#include <cstdio>

#include <cooperative_groups.h>

#include "atomo_kernels.cuh"
#include "atomo_twisted.cuh"

namespace cg = cooperative_groups;

// development builds (-DTB_PROFILE) stamp the phases of the reduction kernels with clock64 and print the sums
#ifdef TB_PROFILE
#define TB_PROF_DECL long long tp[6] = {0, 0, 0, 0, 0, 0}, tl = clock64();
#define TB_MARK(k) { const long long now = clock64(); tp[k] += now - tl; tl = now; }
#else
#define TB_PROF_DECL
#define TB_MARK(k)
#endif

namespace atomo {

namespace {

constexpr int kTbThreads = 1024;
constexpr int kTbWarps = kTbThreads / 32;
constexpr int kTbNB = 32;                    // columns per panel
constexpr int kTbMaxC = 16;                  // CTAs per cluster
constexpr int kTbMaxR = 4096;
constexpr int kTbMaxBlocks = kTbMaxR / 32;   // 32-row blocks of a layer
constexpr int kTbPanRows = 256;              // rows per CTA up to which the panel entries of the CTA's rows live in shared memory

template <typename T> struct Vec4;           // 16-byte (float) / 32-byte (double) groups of four matrix entries
template <> struct Vec4<float> { using type = float4; };
template <> struct Vec4<double> { using type = double4; };

__device__ __forceinline__ float4 ldcg4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ double4 ldcg4(const double* p) {
  const double2 a = __ldcg(reinterpret_cast<const double2*>(p)), b = __ldcg(reinterpret_cast<const double2*>(p) + 1);
  return make_double4(a.x, a.y, b.x, b.y);
}
__device__ __forceinline__ void st4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void st4(double* p, double4 v) {
  reinterpret_cast<double2*>(p)[0] = make_double2(v.x, v.y);
  reinterpret_cast<double2*>(p)[1] = make_double2(v.z, v.w);
}

// the TR consecutive row operands of a thread as one shared-memory load
template <typename T> __device__ __forceinline__ void load_rows(const T* p, T* out);
template <> __device__ __forceinline__ void load_rows<float>(const float* p, float* out) {
  const float4 v = *reinterpret_cast<const float4*>(p);
  out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
template <> __device__ __forceinline__ void load_rows<double>(const double* p, double* out) {
  const double2 v = *reinterpret_cast<const double2*>(p);
  out[0] = v.x; out[1] = v.y;
}

// sum of the per-block partial sums in ascending block order, the same bits in every thread of every CTA
__device__ __forceinline__ double tb_ordered_sum(const double* part, int nblk, int lane) {
  double s = 0.0;
  for (int b = lane; b < nblk; b += 32) s += part[b];
  return warp_sum(s);
}

// this lane's part of sum_{h0 <= h < r} x[h] u[h] (x in global memory, written earlier in this launch; u in shared
// memory), eight loads in flight
template <typename X, typename T>
__device__ __forceinline__ double tb_dot(const X* __restrict__ x, const T* __restrict__ u, int h0, int r, int lane) {
  double acc = 0.0;
  int h = h0 + lane;
  for (; h + 7 * 32 < r; h += 8 * 32) {
    X xb[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) xb[j] = __ldcg(x + h + 32 * j);
#pragma unroll
    for (int j = 0; j < 8; ++j) acc = fma((double)xb[j], (double)u[h + 32 * j], acc);
  }
  for (; h < r; h += 32) acc = fma((double)__ldcg(x + h), (double)u[h], acc);
  return acc;
}

// the same for one of `nsub` warps that share a dot: 32-element blocks of [h0, r) are dealt to the warps in turn
template <typename X, typename T>
__device__ __forceinline__ double tb_dot_part(const X* __restrict__ x, const T* __restrict__ u, int h0, int r, int lane,
                                              int sub, int nsub) {
  double acc = 0.0;
  int h = h0 + 32 * sub + lane;
  const int stride = 32 * nsub;
  for (; h + 3 * stride < r; h += 4 * stride) {
    X xb[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) xb[j] = __ldcg(x + h + stride * j);
#pragma unroll
    for (int j = 0; j < 4; ++j) acc = fma((double)xb[j], (double)u[h + stride * j], acc);
  }
  for (; h < r; h += stride) acc = fma((double)__ldcg(x + h), (double)u[h], acc);
  return acc;
}

// sum over the 8 lanes lx = lane % 8 of v[k]: lane lx ends with the total of k = lx
__device__ __forceinline__ float rs8(float (&v)[8], int lane) {
  const bool b4 = lane & 4, b2 = lane & 2, b1 = lane & 1;
  float a[4];
#pragma unroll
  for (int m = 0; m < 4; ++m) {
    const float send = b4 ? v[m] : v[m + 4], keep = b4 ? v[m + 4] : v[m];
    a[m] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
  }
  float b[2];
#pragma unroll
  for (int m = 0; m < 2; ++m) {
    const float send = b2 ? a[m] : a[m + 2], keep = b2 ? a[m + 2] : a[m];
    b[m] = keep + __shfl_xor_sync(0xffffffffu, send, 2);
  }
  const float send = b1 ? b[0] : b[1], keep = b1 ? b[1] : b[0];
  return keep + __shfl_xor_sync(0xffffffffu, send, 1);
}
// y[row] += v in fixed point: v 2^48 as a 64-bit integer, its upper 40 and lower 24 bits added to two 32-bit words.
// Integer addition commutes, so the sums of y do not depend on the order in which the warps finish their tiles.  (At
// most 64 additions per row and step: the lower word cannot overflow; |v| < 2^7, and the matrix has trace 1.)
__device__ __forceinline__ void t1_add_fix(int32_t* yhi, uint32_t* ylo, int row, float v) {
  const long long q = __float2ll_rn(v * 281474976710656.0f);
  atomicAdd(yhi + row, (int32_t)(q >> 24));
  atomicAdd(ylo + row, (uint32_t)(q & 0xffffffll));
}
// sum over the 4 lanes ly = lane / 8 of v[j]: lane ly ends with the total of j = ly
__device__ __forceinline__ float rs4(float (&v)[4], int lane) {
  const bool b2 = lane & 16, b1 = lane & 8;
  float a[2];
#pragma unroll
  for (int m = 0; m < 2; ++m) {
    const float send = b2 ? v[m] : v[m + 2], keep = b2 ? v[m + 2] : v[m];
    a[m] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
  }
  const float send = b1 ? a[0] : a[1], keep = b1 ? a[1] : a[0];
  return keep + __shfl_xor_sync(0xffffffffu, send, 8);
}

// the same for one array of (upper, lower) word pairs
__device__ __forceinline__ void tb_add_fix(int2* y, int row, float v) {
  const long long q = __float2ll_rn(v * 281474976710656.0f);
  atomicAdd(&y[row].x, (int32_t)(q >> 24));
  atomicAdd(reinterpret_cast<uint32_t*>(&y[row].y), (uint32_t)(q & 0xffffffll));
}
__device__ __forceinline__ long long tb_fix_value(int2 v) { return (long long)v.x * 16777216ll + (long long)(uint32_t)v.y; }

struct alignas(16) TbShared {
  double part_a[kTbMaxBlocks];     // per 32-row block: ||x||^2 partial of the current column
  double part_k[kTbMaxBlocks];     // per 32-row block: u^T p partial
  double dots[2 * kTbNB];          // a_t = w_t^T u, b_t = u_t^T u of the panel's earlier reflectors
  double dot_part[4][8];           // a dot's eight warp partials (four dots in progress per CTA)
  double pc[2 * kTbNB];            // u_t[c], w_t[c]: the panel's entries in row c
  double y[kTbThreads];            // A0 u for this CTA's rows (local row order)
  double x0;                       // first entry of the pivot column
  double p_next;                   // p of the next pivot row (row c + 1), from its owner
};

}  // namespace

template <typename T, int C>
__global__ void __launch_bounds__(kTbThreads, 1) sp_tridiag_big_kernel(const SpLayer* __restrict__ layers,
                                                                       const int* __restrict__ big_layers, int use_pan) {
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ __align__(16) unsigned char tb_smem[];
  TbShared& S = *reinterpret_cast<TbShared*>(tb_smem);
  T* const s_u = reinterpret_cast<T*>(tb_smem + sizeof(TbShared));            // [r4] current reflector, zero up to c
  const int tid = threadIdx.x, lane = tid % 32, w = tid / 32;
  const int q = C == 1 ? 0 : (int)cluster.block_rank();
  const SpLayer& L = layers[big_layers[blockIdx.x / C]];
  const int r = L.r;
  const int64_t lda = L.lda;
  T* const A = reinterpret_cast<T*>(L.tb_A);
  T* const W = reinterpret_cast<T*>(L.tb_W);
  const int64_t ldw = L.tb_ldw;
  float* const V = L.td_V;
  const int64_t ldv = L.td_ldv;
  double* const td_d = L.td_d;
  double* const td_e = L.td_e;
  const int nblk = (r + 31) / 32;
  const int r4 = (r + 3) & ~3;
  T* const s_gemm = s_u + r4;                                                  // operand tiles of the panel update
  // use_pan: this CTA holds at most kTbPanRows rows, and the panel entries of its own rows (u_t[g], w_t[g]) are kept in
  // shared memory beside their copies in global memory: the column update and the correction of y then read them there
  // instead of from L2 (two dependent round trips per step less)
  constexpr int TRg = sizeof(T) == 4 ? 4 : 2;
  T* const pan_u = s_gemm + 2 * kTbNB * 32 * TRg + 2 * kTbNB * 128;            // [kTbNB][kTbPanRows]
  T* const pan_w = pan_u + kTbNB * kTbPanRows;
  // fp32 clusters: the product over the lower triangle adds its sums up in fixed point (tb_add_fix) in ycol, an array
  // over all rows of the layer in every CTA, which the rows' owners read through distributed shared memory after the
  // step's third barrier
  constexpr bool kSym = sizeof(T) == 4 && C > 1;
  int2* const ycol = reinterpret_cast<int2*>(pan_w + kTbNB * kTbPanRows);       // [32 nblk]: whole blocks, a ragged last one included
  // this thread's row: block (tid / 32) of this CTA = global block (tid / 32) * C + q
  const int gb = w * C + q;
  const int g = gb * 32 + lane;
  const bool valid = gb < nblk && g < r;
  const int n_lblk = (nblk - q + C - 1) / C;                                   // 32-row blocks of this CTA (<= 32)

  auto sync_all = [&]() { if (C == 1) __syncthreads(); else cluster.sync(); };
  // a value into the same shared-memory slot of every CTA of the cluster
  auto bcast = [&](double* slot, double v) {
    if (C == 1) { *slot = v; return; }
#pragma unroll
    for (int rk = 0; rk < C; ++rk) *cluster.map_shared_rank(slot, rk) = v;
  };

  for (int i = tid; i < r4; i += kTbThreads) s_u[i] = (T)0;
  if (kSym) {
    for (int i = tid; i < 32 * nblk; i += kTbThreads) ycol[i] = make_int2(0, 0);
  }
  if (C > 1) cluster.sync();                                                   // every CTA runs: remote stores may start

  TB_PROF_DECL
  const int n_ref = r - 2;                                                     // reflectors: columns 0 .. r-3
  double w_carry = 0.0;                                                        // the newest panel column's entry in the next pivot row
  for (int c = 0; c < r; ++c) {
    const int p0 = c / kTbNB * kTbNB;
    const int i = c < n_ref ? c - p0 : 0;                                      // pending reflectors of this panel (the last panel is applied before the last two columns)
    // ---- the panel's entries in row c ----
    // The newest reflector's two entries were stored by the owner of row c after the last barrier of the step before:
    // they are not read from memory but formed here -- u from the copy every CTA has, w from the owner's p and K
    // (w_carry) -- which is what lets a step end without a barrier.  The older ones are a full step old.
    if (tid < 2 * i) {
      const int t = tid >> 1;
      if (t == i - 1) S.pc[tid] = (tid & 1) ? w_carry : (double)(float)s_u[c];
      else S.pc[tid] = (tid & 1) ? (double)__ldcg(W + (int64_t)t * ldw + c) : (double)__ldcg(V + (int64_t)(p0 + t) * ldv + c);
    }
    __syncthreads();
    // ---- column c as the earlier reflectors of the panel left it ----
    double a = 0.0;
    if (valid && g >= c) {
      a = (double)__ldcg(A + (int64_t)c * lda + g);
      if (use_pan) {
        for (int t = 0; t < i; ++t)
          a -= (double)pan_u[t * kTbPanRows + tid] * S.pc[2 * t + 1] + (double)pan_w[t * kTbPanRows + tid] * S.pc[2 * t];
      } else
      for (int t0 = 0; t0 < i; t0 += 8) {                                       // eight reflectors' entries in flight
        float ub[8]; T wb[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int t = min(t0 + j, i - 1);
          ub[j] = __ldcg(V + (int64_t)(p0 + t) * ldv + g); wb[j] = __ldcg(W + (int64_t)t * ldw + g);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (t0 + j < i) a -= (double)ub[j] * S.pc[2 * (t0 + j) + 1] + (double)wb[j] * S.pc[2 * (t0 + j)];
      }
      if (g == c) td_d[c] = a;
    }
    if (c >= n_ref) {                                                          // the last two columns: no reflector
      if (c == r - 2 && valid && g == r - 1) td_e[c] = a;
      continue;                                                                // uniform over the cluster
    }
    TB_MARK(0)
    const bool live = valid && g > c;
    // fp32 clusters: every CTA forms the whole reflector itself from the column's entries, which their owners leave in
    // their own shared memory (the storage of S.y) -- one barrier for the norm and the reflector instead of two
    // (up to 2048 rows: beyond, with every thread of the CTA fetching entries, the second barrier is the cheaper way;
    // config 3's reduction takes 106.5 ms with it and 108.0 ms without)
    double* const a_pub = S.y;
    const bool form_u = kSym && r <= 2048;
    if (form_u) a_pub[tid] = live ? a : 0.0;
    {
      const double sq = warp_sum(live ? a * a : 0.0);
      if (lane == 0 && gb < nblk) bcast(&S.part_a[gb], sq);
      if (valid && g == c + 1) bcast(&S.x0, a);
    }
    sync_all();
    const double nx2 = tb_ordered_sum(S.part_a, nblk, lane);
    const double x0 = S.x0;
    double alpha = 0.0, inv = 0.0;
    if (nx2 > 1.0e-290) {                                                      // below: a zero column, H = I
      const double nx = sqrt(nx2);
      alpha = -copysign(nx, x0);
      inv = rsqrt(2.0 * nx * (nx + fabs(x0)));                                 // 1 / ||x - alpha e_1||
    }
    double u_own = 0.0;
    if (valid) {
      if (live) u_own = (double)(T)((a - (g == c + 1 ? alpha : 0.0)) * inv);   // the stored precision is the one used
      V[(int64_t)c * ldv + g] = (float)u_own;
      if (use_pan) pan_u[(c - p0) * kTbPanRows + tid] = (T)u_own;
      if (g == c + 1) td_e[c] = alpha;
      if (C == 1) s_u[g] = (T)u_own;
      else if (!kSym) {
#pragma unroll
        for (int rk = 0; rk < C; ++rk) cluster.map_shared_rank(s_u, rk)[g] = (T)u_own;
      }
    }
    float* const u_pub = reinterpret_cast<float*>(S.y);                        // fp32 clusters above 2048 rows: the owners' entries of u, fetched after the barrier
    if (kSym && !form_u) u_pub[tid] = (float)u_own;
    if (form_u) {
      const int h0 = 4 * tid;                                                  // this thread's four entries of the reflector
      if (h0 < r4) {
        const int hb = h0 >> 5;                                                // their 32-row block: one owner
        float uo[4] = {0.f, 0.f, 0.f, 0.f};
        if (hb < nblk && h0 + 3 > c) {
          const double* src = cluster.map_shared_rank(a_pub, hb % C) + (hb / C) * 32 + (h0 & 31);
          const double2 a01 = *reinterpret_cast<const double2*>(src), a23 = *reinterpret_cast<const double2*>(src + 2);
          const double av[4] = {a01.x, a01.y, a23.x, a23.y};
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            const int h = h0 + x;
            if (h > c && h < r) uo[x] = (float)((av[x] - (h == c + 1 ? alpha : 0.0)) * inv);   // as its owner forms u_own
          }
        }
        *reinterpret_cast<float4*>(s_u + h0) = make_float4(uo[0], uo[1], uo[2], uo[3]);
      }
      __syncthreads();
    } else {
      sync_all();
      if (kSym) {                                                              // one 16-byte remote load per thread instead of a store to every CTA
        const int h0 = 4 * tid;
        if (h0 < r4) {
          const int hb = h0 >> 5;
          float4 uo = make_float4(0.f, 0.f, 0.f, 0.f);
          if (hb < nblk && h0 + 3 > c) uo = *reinterpret_cast<const float4*>(cluster.map_shared_rank(u_pub, hb % C) + (hb / C) * 32 + (h0 & 31));
          *reinterpret_cast<float4*>(s_u + h0) = uo;
        }
        __syncthreads();
      }
    }
    TB_MARK(1)
    // ---- y = A0 u over this CTA's live rows and the panel dots ----
    if constexpr (kSym) {
      // The lower triangle only, in 32 x 32 sub-tiles (I, J), J <= I: a sub-tile gives its rows' sums to block I of y
      // and, transposed, its columns' sums to block J (half the bytes of a product over full rows).  The layer's live
      // sub-tiles are dealt in equal runs to all warps of the cluster, whoever owns the rows: every CTA has the same
      // work, and a row's owner finds the sums in the CTAs' ycol arrays after the barrier.  In a sub-tile a lane holds
      // rows 8 ly + kk (kk = 0 .. 7) of columns 4 lx .. 4 lx + 3; the sums over the 8 lanes of a row and the 4 lanes
      // of a column are reduce-scatters.  Every sub-tile's sums are rounded to fixed point on their own and added as
      // integers, so y does not depend on which warp or CTA took the sub-tile: the same bits for every cluster size.
      const int sly = lane >> 3, slx = lane & 7;
      const int jb0 = (c + 1) >> 5;                                            // first live block
      const int nbl = nblk - jb0;                                              // live blocks
      const int N = nbl * (nbl + 1) / 2;                                       // live sub-tiles of the layer
      const int per = (N + C * kTbWarps - 1) / (C * kTbWarps);
      int k = (q * kTbWarps + w) * per;
      const int k_end = min(N, k + per);
      if (k < k_end) {
        int ii = (int)((sqrtf(8.0f * (float)k + 1.0f) - 1.0f) * 0.5f);        // row of the triangle that holds sub-tile k
        while ((ii + 1) * (ii + 2) / 2 <= k) ++ii;
        while (ii * (ii + 1) / 2 > k) --ii;
        int I = jb0 + ii, J = jb0 + (k - ii * (ii + 1) / 2);
        for (; k < k_end; ++k) {
          const int row0 = 32 * I, col0 = 32 * J;
          const bool diag = I == J;
          const bool edge = row0 + 32 > r || col0 + 32 > r;                   // the matrix ends inside the sub-tile
          float4 uj;
          if (!edge) uj = *reinterpret_cast<const float4*>(s_u + col0 + 4 * slx);
          else {
            const int cc = col0 + 4 * slx;
            uj = make_float4(cc < r ? s_u[cc] : 0.f, cc + 1 < r ? s_u[cc + 1] : 0.f, cc + 2 < r ? s_u[cc + 2] : 0.f, cc + 3 < r ? s_u[cc + 3] : 0.f);
          }
          const uint64_t uj01 = pack2(uj.x, uj.y), uj23 = pack2(uj.z, uj.w);
          float rp[8];
          uint64_t c01 = pack2(0.f, 0.f), c23 = pack2(0.f, 0.f);
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int rbase = row0 + 8 * sly + 4 * half;                       // first of this lane's four rows
            float4 v[4];
            float ui[4];
            if (!edge) {
              const float* src = A + (int64_t)rbase * lda + col0 + 4 * slx;
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) v[kk] = ldcg4(src + (int64_t)kk * lda);
              const float4 u4 = *reinterpret_cast<const float4*>(s_u + rbase);
              ui[0] = u4.x; ui[1] = u4.y; ui[2] = u4.z; ui[3] = u4.w;
            } else {
              const int cc = col0 + 4 * slx;
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) {
                const int rr = rbase + kk;
                v[kk] = (rr < r && cc < r) ? ldcg4(A + (int64_t)rr * lda + cc) : make_float4(0.f, 0.f, 0.f, 0.f);   // cc < r: the row's padded length holds the group
                if (cc + 1 >= r) v[kk].y = 0.f;
                if (cc + 2 >= r) v[kk].z = 0.f;
                if (cc + 3 >= r) v[kk].w = 0.f;
                ui[kk] = rr < r ? s_u[rr] : 0.f;
              }
            }
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
              float4 x = v[kk];
              const int rr = 8 * sly + 4 * half + kk, cc = 4 * slx;           // position inside the sub-tile
              if (diag) {                                                      // lower triangle only
                if (cc + 0 > rr) x.x = 0.f;
                if (cc + 1 > rr) x.y = 0.f;
                if (cc + 2 > rr) x.z = 0.f;
                if (cc + 3 > rr) x.w = 0.f;
              }
              float s0, s1;
              unpack2(fma2(pack2(x.z, x.w), uj23, fma2(pack2(x.x, x.y), uj01, pack2(0.f, 0.f))), s0, s1);
              rp[4 * half + kk] = s0 + s1;
              if (diag) {                                                      // the diagonal entry counts once (with the rows)
                if (cc + 0 == rr) x.x = 0.f;
                if (cc + 1 == rr) x.y = 0.f;
                if (cc + 2 == rr) x.z = 0.f;
                if (cc + 3 == rr) x.w = 0.f;
              }
              const uint64_t ui2 = pack2(ui[kk], ui[kk]);
              c01 = fma2(pack2(x.x, x.y), ui2, c01);
              c23 = fma2(pack2(x.z, x.w), ui2, c23);
            }
          }
          const float rsum = rs8(rp, lane);                                    // lane 8 ly + lx: row 8 ly + lx
          float cv[4];
          unpack2(c01, cv[0], cv[1]); unpack2(c23, cv[2], cv[3]);
          const float csum = rs4(cv, lane);                                    // lane 8 ly + lx: column 4 lx + ly
          tb_add_fix(ycol, row0 + lane, rsum);
          tb_add_fix(ycol, col0 + 4 * slx + sly, csum);
          if (++J > I) { ++I; J = jb0; }
        }
      }
      TB_MARK(2)
    } else {
      const int c0 = (c + 1) & ~3;
      using V4 = typename Vec4<T>::type;
      constexpr int RB = sizeof(T) == 4 ? 2 : 1;                               // rows per pass of a warp
      for (int lb = 0; lb < n_lblk; lb += RB) {
        int row[RB]; bool on[RB]; bool any = false;
#pragma unroll
        for (int x = 0; x < RB; ++x) {
          row[x] = ((lb + x) * C + q) * 32 + w;
          on[x] = lb + x < n_lblk && row[x] > c && row[x] < r;
          any |= on[x];
        }
        if (!any) continue;
        const int live_row = on[0] ? row[0] : row[RB - 1];                     // a dead row of the pair reads the live one
        const T* ar[RB];
#pragma unroll
        for (int x = 0; x < RB; ++x) ar[x] = A + (int64_t)(on[x] ? row[x] : live_row) * lda;
        T acc[RB][4];
#pragma unroll
        for (int x = 0; x < RB; ++x) { acc[x][0] = 0; acc[x][1] = 0; acc[x][2] = 0; acc[x][3] = 0; }
        int h = c0 + lane * 4;
        for (; h + 3 + 128 < r; h += 256) {                                    // two groups of four per row in flight
          V4 m0[RB], m1[RB];
#pragma unroll
          for (int x = 0; x < RB; ++x) { m0[x] = ldcg4(ar[x] + h); m1[x] = ldcg4(ar[x] + h + 128); }
          const V4 u0 = *reinterpret_cast<const V4*>(s_u + h), u1 = *reinterpret_cast<const V4*>(s_u + h + 128);
#pragma unroll
          for (int x = 0; x < RB; ++x) {
            acc[x][0] = fma(m0[x].x, u0.x, acc[x][0]); acc[x][1] = fma(m0[x].y, u0.y, acc[x][1]);
            acc[x][2] = fma(m0[x].z, u0.z, acc[x][2]); acc[x][3] = fma(m0[x].w, u0.w, acc[x][3]);
            acc[x][0] = fma(m1[x].x, u1.x, acc[x][0]); acc[x][1] = fma(m1[x].y, u1.y, acc[x][1]);
            acc[x][2] = fma(m1[x].z, u1.z, acc[x][2]); acc[x][3] = fma(m1[x].w, u1.w, acc[x][3]);
          }
        }
        for (; h + 3 < r; h += 128) {
          V4 m0[RB];
#pragma unroll
          for (int x = 0; x < RB; ++x) m0[x] = ldcg4(ar[x] + h);
          const V4 u0 = *reinterpret_cast<const V4*>(s_u + h);
#pragma unroll
          for (int x = 0; x < RB; ++x) {
            acc[x][0] = fma(m0[x].x, u0.x, acc[x][0]); acc[x][1] = fma(m0[x].y, u0.y, acc[x][1]);
            acc[x][2] = fma(m0[x].z, u0.z, acc[x][2]); acc[x][3] = fma(m0[x].w, u0.w, acc[x][3]);
          }
        }
        {
          const int ht = (r & ~3) + lane;                                      // the last r mod 4 columns
          if (ht < r) {
#pragma unroll
            for (int x = 0; x < RB; ++x) acc[x][0] = fma(__ldcg(ar[x] + ht), s_u[ht], acc[x][0]);
          }
        }
        double sum[RB];
#pragma unroll
        for (int x = 0; x < RB; ++x) sum[x] = ((double)acc[x][0] + (double)acc[x][1]) + ((double)acc[x][2] + (double)acc[x][3]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
          for (int x = 0; x < RB; ++x) sum[x] += __shfl_xor_sync(0xffffffffu, sum[x], o);
        }
        if (lane == 0) {
#pragma unroll
          for (int x = 0; x < RB; ++x) if (on[x]) S.y[(lb + x) * 32 + w] = sum[x];
        }
      }
      TB_MARK(2)
    }
    {
      // Panel dots.  Dot number id belongs to CTA id mod C; eight warps share a dot (32-element blocks dealt in turn)
      // and their partial sums are added in warp order -- the same order whatever C is.  The owner sends the result to
      // every CTA of the cluster.
      for (int k0 = 0; q + C * k0 < 2 * i; k0 += 4) {
        const int id = q + C * (k0 + (w >> 3));
        if (id < 2 * i) {
          const int t = id >> 1;
          double acc = (id & 1) ? tb_dot_part(V + (int64_t)(p0 + t) * ldv, s_u, c + 1, r, lane, w & 7, 8)
                                : tb_dot_part(W + (int64_t)t * ldw, s_u, c + 1, r, lane, w & 7, 8);
          acc = warp_sum(acc);
          if (lane == 0) S.dot_part[w >> 3][w & 7] = acc;
        }
        __syncthreads();
        if (tid < 4) {
          const int id2 = q + C * (k0 + tid);
          if (id2 < 2 * i) {
            double tot = 0.0;
#pragma unroll
            for (int j = 0; j < 8; ++j) tot += S.dot_part[tid][j];
            bcast(&S.dots[id2], tot);
          }
        }
        __syncthreads();
      }
    }
    sync_all();                                                              // the other CTAs' dots have arrived
    TB_MARK(3)
    // ---- w = p - (u^T p) u with p = 2 (y - U a - W b) ----
    double p = 0.0;
    double y_sym = 0.0;
    if constexpr (kSym) {
      if (live) {                                                              // this row's sums, from every CTA of the cluster (a dead row's are never used)
        long long tot = 0;
#pragma unroll
        for (int rk = 0; rk < C; ++rk) tot += tb_fix_value(cluster.map_shared_rank(ycol, rk)[g]);
        y_sym = (double)tot * 3.552713678800501e-15;                            // 2^-48
      }
    }
    if (live) {
      double y = kSym ? y_sym : S.y[tid];
      if (use_pan) {
        for (int t = 0; t < i; ++t)
          y -= (double)pan_u[t * kTbPanRows + tid] * S.dots[2 * t] + (double)pan_w[t * kTbPanRows + tid] * S.dots[2 * t + 1];
      } else
      for (int t0 = 0; t0 < i; t0 += 8) {
        float ub[8]; T wb[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int t = min(t0 + j, i - 1);
          ub[j] = __ldcg(V + (int64_t)(p0 + t) * ldv + g); wb[j] = __ldcg(W + (int64_t)t * ldw + g);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (t0 + j < i) y -= (double)ub[j] * S.dots[2 * (t0 + j)] + (double)wb[j] * S.dots[2 * (t0 + j) + 1];
      }
      p = 2.0 * y;
    }
    {
      const double kp = warp_sum(u_own * p);
      if (lane == 0 && gb < nblk) bcast(&S.part_k[gb], kp);
      if (valid && g == c + 1) bcast(&S.p_next, p);                            // the next pivot row's p, for everybody's w_carry
    }
    sync_all();
    const double K = tb_ordered_sum(S.part_k, nblk, lane);
    w_carry = (double)(T)fma(-K, (double)s_u[c + 1], S.p_next);               // w[c + 1] exactly as its owner stores it below
    if (kSym) {                                                                // every owner has read its rows: the column sums start the next step at zero
      for (int i = tid; i < 32 * nblk; i += kTbThreads) ycol[i] = make_int2(0, 0);
    }
    if (valid) {
      const T wv = (T)(live ? fma(-K, u_own, p) : 0.0);
      W[(int64_t)(c - p0) * ldw + g] = wv;
      if (use_pan) pan_w[(c - p0) * kTbPanRows + tid] = wv;
    }
    const bool flush = (c - p0 == kTbNB - 1) || (c == n_ref - 1);
    if (!flush) { TB_MARK(4) continue; }                                        // no barrier: see the start of the step
    TB_MARK(4)
    // ---- end of the panel: A0 -= U W^T + W U^T on the rows and columns beyond c (this CTA's rows) ----
    if (C == 1) { __threadfence_block(); __syncthreads(); } else { __threadfence(); cluster.sync(); }
    {
      constexpr int TR = sizeof(T) == 4 ? 4 : 2;                               // rows per thread
      constexpr int MR = 32 * TR;                                              // local rows per tile (whole 32-row blocks)
      const int nr = c - p0 + 1;                                               // reflectors in the panel
      const int g0 = c + 1;
      T* const s_ur = s_gemm;                                                  // [kTbNB][MR]
      T* const s_wr = s_ur + kTbNB * MR;
      T* const s_uc = s_wr + kTbNB * MR;                                       // [kTbNB][128]
      T* const s_wc = s_uc + kTbNB * 128;
      const int wr = w >> 3, wc = w & 7;                                       // warp: 8 TR rows x 16 columns
      const int ly = lane >> 2, lx = lane & 3;
      const int n_lrows = n_lblk * 32;
      // One thread's TR x 4 outputs of the tile of local rows mr0 .. and columns hc0 ..: row operands of reflector t
      // at ur / wrp + t * rstride (indexed by the row inside the tile), column operands at uc / wcp + t * 128.
      // fp32: a warp's piece of a tile is one 32-row block by 16 columns.  A piece strictly above the diagonal is not
      // computed: its mirror image, a piece strictly below the diagonal in another block's rows, writes both (the
      // update is symmetric and so is A0).  Pieces that meet the diagonal are computed and written as they are.
      auto update_piece = [&](const int mr0, const int hc0, const T* ur, const T* wrp, const int rstride, const T* uc, const T* wcp) {
        const int lr0 = wr * (8 * TR) + ly * TR;                               // first local row (in the tile) of this thread
        const int lc0 = wc * 16 + lx * 4;
        bool mirror = false;
        if (sizeof(T) == 4) {
          const int blk_start = (((mr0 >> 5) + wr) * C + q) * 32;              // this warp's 32-row block
          const int pc_start = hc0 + 16 * wc;
          if (pc_start > blk_start + 31) return;                               // above the diagonal: written by its mirror image
          mirror = pc_start + 15 < blk_start;
        }
        T acc[TR][4];
#pragma unroll
        for (int x = 0; x < TR; ++x)
#pragma unroll
          for (int y = 0; y < 4; ++y) acc[x][y] = 0;
        for (int t = 0; t < nr; ++t) {
          T ru[TR], rw[TR];
          load_rows<T>(ur + t * rstride + lr0, ru);
          load_rows<T>(wrp + t * rstride + lr0, rw);
          const typename Vec4<T>::type cu = *reinterpret_cast<const typename Vec4<T>::type*>(uc + t * 128 + lc0);
          const typename Vec4<T>::type cw = *reinterpret_cast<const typename Vec4<T>::type*>(wcp + t * 128 + lc0);
#pragma unroll
          for (int x = 0; x < TR; ++x) {
            acc[x][0] = fma(ru[x], cw.x, acc[x][0]); acc[x][1] = fma(ru[x], cw.y, acc[x][1]);
            acc[x][2] = fma(ru[x], cw.z, acc[x][2]); acc[x][3] = fma(ru[x], cw.w, acc[x][3]);
            acc[x][0] = fma(rw[x], cu.x, acc[x][0]); acc[x][1] = fma(rw[x], cu.y, acc[x][1]);
            acc[x][2] = fma(rw[x], cu.z, acc[x][2]); acc[x][3] = fma(rw[x], cu.w, acc[x][3]);
          }
        }
        const int h = hc0 + lc0;
        const int lrf = mr0 + lr0;
        const int grf = ((lrf >> 5) * C + q) * 32 + (lrf & 31);                // first global row of this thread (its TR rows are consecutive)
#pragma unroll
        for (int x = 0; x < TR; ++x) {
          const int gr = grf + x;
          const bool on = (lrf >> 5) < n_lblk && gr < r && gr >= g0 && h < r;
          if (on) {
            T* dst = A + (int64_t)gr * lda + h;
            if (h + 3 < r) {
              typename Vec4<T>::type o = ldcg4(dst);
              o.x -= acc[x][0]; o.y -= acc[x][1]; o.z -= acc[x][2]; o.w -= acc[x][3];
              st4(dst, o);
              acc[x][0] = o.x; acc[x][1] = o.y; acc[x][2] = o.z; acc[x][3] = o.w;   // the new entries, for the mirror image
            } else {
              for (int y = 0; y < 4 && h + y < r; ++y) { const T o = __ldcg(dst + y) - acc[x][y]; dst[y] = o; acc[x][y] = o; }
            }
          }
        }
        if (mirror && (lrf >> 5) < n_lblk) {
          // A0[h + y][grf .. grf + TR - 1] = the new A0[grf .. ][h + y]: rows h + y >= g0 only (the others are dead)
#pragma unroll
          for (int y = 0; y < 4; ++y) {
            const int hr = h + y;
            if (hr < g0 || hr >= r) continue;
            T* dst = A + (int64_t)hr * lda + grf;
            if (TR == 4 && grf >= g0 && grf + 3 < r) {
              typename Vec4<T>::type o;
              o.x = acc[0][y]; o.y = acc[1][y]; o.z = acc[TR > 2 ? 2 : 0][y]; o.w = acc[TR > 2 ? 3 : 0][y];
              st4(dst, o);
            } else {
#pragma unroll
              for (int x = 0; x < TR; ++x) if (grf + x >= g0 && grf + x < r) dst[x] = acc[x][y];
            }
          }
        }
      };
      // last global row of the tile of local rows mr0 ..
      auto tile_end = [&](int mr0) { return ((min(mr0 / 32 + MR / 32, n_lblk) - 1) * C + q) * 32 + 31; };
      bool done = false;
      if constexpr (sizeof(T) == 4) {
        if (use_pan) {
          // The panel entries of this CTA's rows are in shared memory already (pan_u, pan_w: at most two tiles of rows),
          // so only the column operands are staged: chunks of 128 columns in two buffers, the next chunk on its way
          // (cp.async) while this one is used by both row tiles -- one barrier per chunk and no wait for a load.
          done = true;
          const int row_end = tile_end(((n_lrows - 1) / MR) * MR);              // this CTA's last row
          if (row_end >= g0) {
            float* const s_c = reinterpret_cast<float*>(s_gemm);              // [2][u, w][kTbNB][128]
            const int hc_first = g0 & ~127, hc_last = min(r - 1, row_end) & ~127;
            auto fetch = [&](int hc0, int buf) {
              float* du = s_c + buf * (2 * kTbNB * 128);
              float* dw = du + kTbNB * 128;
              for (int e = tid; e < nr * 128; e += kTbThreads) {
                const int t = e >> 7, h = hc0 + (e & 127);
                const int hs = h < r ? h : 0, nb = h < r ? 4 : 0;              // beyond the matrix: zero fill
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(du + e)),
                             "l"(V + (int64_t)(p0 + t) * ldv + hs), "r"(nb) : "memory");
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(dw + e)),
                             "l"(reinterpret_cast<const float*>(W) + (int64_t)t * ldw + hs), "r"(nb) : "memory");
              }
              asm volatile("cp.async.commit_group;" ::: "memory");
            };
            __syncthreads();                                                   // nobody still reads the buffers' earlier contents
            fetch(hc_first, 0);
            int it = 0;
            for (int hc0 = hc_first; hc0 <= hc_last; hc0 += 128, ++it) {
              asm volatile("cp.async.wait_group 0;" ::: "memory");
              __syncthreads();                                                 // this chunk has landed; the other buffer is free
              if (hc0 + 128 <= hc_last) fetch(hc0 + 128, (it + 1) & 1);
              const float* du = s_c + (it & 1) * (2 * kTbNB * 128);
              const float* dw = du + kTbNB * 128;
              for (int mr0 = 0; mr0 < n_lrows; mr0 += MR) {
                const int te = tile_end(mr0);
                if (te < g0 || hc0 > te) continue;                             // a dead tile, or every piece above the diagonal
                update_piece(mr0, hc0, reinterpret_cast<const T*>(pan_u) + mr0, reinterpret_cast<const T*>(pan_w) + mr0, kTbPanRows,
                             reinterpret_cast<const T*>(du), reinterpret_cast<const T*>(dw));
              }
            }
          }
        }
      }
      if (!done)
      for (int mr0 = 0; mr0 < n_lrows; mr0 += MR) {
        // dead tiles are skipped
        const int tile_row_end = tile_end(mr0);
        if (tile_row_end < g0) continue;
        __syncthreads();
        for (int e = tid; e < nr * MR; e += kTbThreads) {
          const int t = e / MR, lr = mr0 + e % MR;
          const int gr = ((lr >> 5) * C + q) * 32 + (lr & 31);
          const bool in = (lr >> 5) < n_lblk && gr < r;
          s_ur[t * MR + e % MR] = in ? (T)__ldcg(V + (int64_t)(p0 + t) * ldv + gr) : (T)0;
          s_wr[t * MR + e % MR] = in ? __ldcg(W + (int64_t)t * ldw + gr) : (T)0;
        }
        for (int hc0 = g0 & ~127; hc0 < r; hc0 += 128) {
          if (sizeof(T) == 4 && hc0 > tile_row_end) break;                      // every piece of this and the later chunks lies above the diagonal
          __syncthreads();
          for (int e = tid; e < nr * 128; e += kTbThreads) {
            const int t = e >> 7, h = hc0 + (e & 127);
            s_uc[e] = h < r ? (T)__ldcg(V + (int64_t)(p0 + t) * ldv + h) : (T)0;
            s_wc[e] = h < r ? __ldcg(W + (int64_t)t * ldw + h) : (T)0;
          }
          __syncthreads();
          update_piece(mr0, hc0, s_ur, s_wr, MR, s_uc, s_wc);
        }
      }
    }
    if (C == 1) { __threadfence_block(); __syncthreads(); } else { __threadfence(); cluster.sync(); }
    TB_MARK(5)
  }
#ifdef TB_PROFILE
  if (blockIdx.x == 0 && tid == 0)
    printf("tridiag_big C=%d r=%d cycles: column %lld reflector %lld matvec %lld dots %lld w %lld gemm %lld\n", C, r, tp[0], tp[1], tp[2], tp[3], tp[4], tp[5]);
#endif
  if (C > 1) cluster.sync();                                                   // nobody leaves while a peer may still write here
}

// ---- one CTA per layer (short side up to 1024) -------------------------------------------------------------------
// The form a large batch takes (config 5: 96 layers of 1024 rows, one SM each).  Differences from the cluster
// kernel above, all of them about bytes:
//   * only the lower triangle of A0 is read and updated.  The product y = A0 u goes over 64 x 64 tiles of the
//     triangle, one warp per tile: a tile contributes its rows' sums to block I of y and, transposed, its columns'
//     sums to block J, both added to y in fixed point with integer shared-memory atomics (integer addition commutes:
//     the result does not depend on which warp finishes first).  Per 32 x 32 sub-tile a lane holds 8 x 4 entries; the
//     sums over the 8 lanes of a row and the 4 lanes of a column are reduce-scatters (7 + 3 shuffles).  Half the bytes
//     per step of the row-wise product.  A warp has three sub-tiles in work or on their way: two in registers, one in
//     a 4 KB buffer of its own in shared memory filled by cp.async.
//   * the panel (16 columns: u_t and w_t of all rows) lives in shared memory, so the column update, the correction
//     of y and the panel dots never leave the SM, and the rank-32 update at the end of a panel takes its operands
//     from there (4 x 4 outputs per thread on 128 x 128 tiles of the lower triangle).
//   * 512 threads; thread t owns rows t and t + 512 for the whole reduction.
namespace {

constexpr int kT1Threads = 512;              // 128 registers per thread: two sub-tiles of the product in registers per warp
constexpr int kT1Warps = kT1Threads / 32;
constexpr int kT1NB = 16;                    // columns per panel
constexpr int kT1MaxR = 1024;
constexpr int kT1Blk = 64;                   // tile edge of the matrix-vector product

struct alignas(16) T1Shared {
  double part_a[32];
  double part_k[32];
  double dots[2 * kT1NB];
  double x0;
  double pad;
};

// The kernel works on a copy of the lower triangle in tile-major order: 32 x 32 sub-tile (I, J), J <= I, is the
// contiguous 4 KB block number I (I + 1) / 2 + J, row-major inside.  A warp then reads a sub-tile as one contiguous
// piece of memory (with rows of the row-major matrix it would be 32 pieces of 128 bytes, 4 KB apart, which DRAM
// serves at little more than half its streaming rate).  Rows and columns from r on are zero.
__device__ __forceinline__ float* t1_sub(float* At, int I, int J) { return At + ((size_t)(I * (I + 1) / 2 + J) << 10); }

// 16 bytes from global (L2) to shared memory without passing through registers; waited for with cp.async.wait_group
__device__ __forceinline__ void t1_cp16(float* dst_smem, const float* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src) : "memory");
}

}  // namespace

__global__ void __launch_bounds__(kT1Threads, 1) sp_tridiag_big1_kernel(const SpLayer* __restrict__ layers,
                                                                        const int* __restrict__ big_layers) {
  extern __shared__ __align__(16) unsigned char tb_smem[];
  T1Shared& S = *reinterpret_cast<T1Shared*>(tb_smem);
  float* const s_u = reinterpret_cast<float*>(tb_smem + sizeof(T1Shared));     // [1024] current reflector (zero up to c and from r on)
  float* const pan_u = s_u + kT1MaxR;                                          // [16][1024]
  float* const pan_w = pan_u + kT1NB * kT1MaxR;                                // [16][1024]
  int32_t* const yhi = reinterpret_cast<int32_t*>(pan_w + kT1NB * kT1MaxR);    // [1024] y in fixed point, upper word
  uint32_t* const ylo = reinterpret_cast<uint32_t*>(yhi + kT1MaxR);            // [1024] lower word
  float* const stage = reinterpret_cast<float*>(ylo + kT1MaxR) + (threadIdx.x / 32) * 1024;   // this warp's third sub-tile buffer (4 KB)
  const int tid = threadIdx.x, lane = tid % 32, w = tid / 32;
  const SpLayer& L = layers[big_layers[blockIdx.x]];
  const int r = L.r;
  const int64_t lda = L.lda;
  const float* const A = reinterpret_cast<const float*>(L.tb_A);
  float* const At = L.tb_At;
  float* const V = L.td_V;
  const int64_t ldv = L.td_ldv;
  double* const td_d = L.td_d;
  double* const td_e = L.td_e;
  const int nblk = (r + 31) / 32;
  const int nb64 = (r + kT1Blk - 1) / kT1Blk;
  const int g[2] = {tid, tid + kT1Threads};                                    // this thread's two rows (32-row blocks w and w + 16)
  const bool valid[2] = {g[0] < r, g[1] < r};
  const int ly = lane >> 3, lx = lane & 7;                                     // sub-tile layout: rows 8 ly + kk, columns 4 lx .. 4 lx + 3
  const int idx = 4 * lx + ly;                                                 // the column a lane ends up with after the reduce-scatter

  s_u[g[0]] = 0.0f; s_u[g[1]] = 0.0f;
  yhi[g[0]] = 0; yhi[g[1]] = 0; ylo[g[0]] = 0u; ylo[g[1]] = 0u;
  // the lower triangle of A into tile-major order (one warp per sub-tile: 32 rows of 128 bytes in, 4 KB out)
  for (int k = w; k < nblk * (nblk + 1) / 2; k += kT1Warps) {
    int I = (int)((sqrtf(8.0f * (float)k + 1.0f) - 1.0f) * 0.5f);
    while ((I + 1) * (I + 2) / 2 <= k) ++I;
    while (I * (I + 1) / 2 > k) --I;
    const int J = k - I * (I + 1) / 2;
    float* dst = At + ((size_t)k << 10);
    const int col = 32 * J + lane;
#pragma unroll 8
    for (int rr = 0; rr < 32; ++rr) {
      const int row = 32 * I + rr;
      dst[rr * 32 + lane] = (row < r && col < r) ? __ldcg(A + (int64_t)row * lda + col) : 0.0f;
    }
  }
  __threadfence_block();
  __syncthreads();
  const int n_ref = r - 2;
  TB_PROF_DECL
  // element (row, col) of the working copy, col <= row
  auto at = [&](int row, int col) -> float* { return t1_sub(At, row >> 5, col >> 5) + ((row & 31) << 5) + (col & 31); };
  float a_pref[2];
#pragma unroll
  for (int x = 0; x < 2; ++x) a_pref[x] = valid[x] ? __ldcg(at(g[x], 0)) : 0.0f;   // column 0 (lower triangle: every row)
  for (int c = 0; c < r; ++c) {
    const int p0 = c / kT1NB * kT1NB;
    const int i = c < n_ref ? c - p0 : 0;
    // ---- column c as the earlier reflectors of the panel left it ----
    double a[2] = {0.0, 0.0};
#pragma unroll
    for (int x = 0; x < 2; ++x) {
      if (valid[x] && g[x] >= c) {
        a[x] = (double)a_pref[x];
        for (int t = 0; t < i; ++t)
          a[x] -= (double)pan_u[t * kT1MaxR + g[x]] * (double)pan_w[t * kT1MaxR + c] + (double)pan_w[t * kT1MaxR + g[x]] * (double)pan_u[t * kT1MaxR + c];
        if (g[x] == c) td_d[c] = a[x];
      }
    }
    if (c >= n_ref) {
#pragma unroll
      for (int x = 0; x < 2; ++x) {
        if (c == r - 2 && valid[x] && g[x] == r - 1) td_e[c] = a[x];
        if (c + 1 < r) a_pref[x] = (valid[x] && g[x] >= c + 1) ? __ldcg(at(g[x], c + 1)) : 0.0f;
      }
      continue;
    }
    const bool live[2] = {valid[0] && g[0] > c, valid[1] && g[1] > c};
#pragma unroll
    for (int x = 0; x < 2; ++x) {
      const double sq = warp_sum(live[x] ? a[x] * a[x] : 0.0);
      if (lane == 0) S.part_a[w + kT1Warps * x] = sq;
      if (g[x] == c + 1) S.x0 = a[x];
    }
    __syncthreads();
    const double nx2 = tb_ordered_sum(S.part_a, nblk, lane);
    const double x0 = S.x0;
    double alpha = 0.0, inv = 0.0;
    if (nx2 > 1.0e-290) {
      const double nx = sqrt(nx2);
      alpha = -copysign(nx, x0);
      inv = rsqrt(2.0 * nx * (nx + fabs(x0)));
    }
    float u_f[2] = {0.0f, 0.0f};
#pragma unroll
    for (int x = 0; x < 2; ++x) {
      if (valid[x]) {
        if (live[x]) u_f[x] = (float)((a[x] - (g[x] == c + 1 ? alpha : 0.0)) * inv);
        V[(int64_t)c * ldv + g[x]] = u_f[x];
        if (g[x] == c + 1) td_e[c] = alpha;
        s_u[g[x]] = u_f[x];
        pan_u[i * kT1MaxR + g[x]] = u_f[x];
      }
    }
    __syncthreads();
    TB_MARK(1)
    // ---- panel dots (one warp each), then y = A0 u over the tiles of the lower triangle ----
    for (int id = w; id < 2 * i; id += kT1Warps) {
      const int t = id >> 1;
      const float* xv = (id & 1) ? pan_u + t * kT1MaxR : pan_w + t * kT1MaxR;  // odd: b_t = u_t^T u, even: a_t = w_t^T u
      double acc = 0.0;
      for (int h = lane; h < r; h += 32) acc = fma((double)xv[h], (double)s_u[h], acc);
      acc = warp_sum(acc);
      if (lane == 0) S.dots[id] = acc;
    }
    {
      // One warp per 64 x 64 tile (I, J), J <= I, of the live part of the lower triangle, as up to four 32 x 32
      // sub-tiles in the order (row half, column half) = (0,0) (0,1) (1,0) (1,1).  In a sub-tile a lane holds rows
      // 8 ly + kk (kk = 0 .. 7) of columns 4 lx .. 4 lx + 3.  Row sums are accumulated over the sub-tiles of a row half
      // before the eight lanes of a row are added up (reduce-scatter: lane 8 ly + lx ends with row 8 ly + lx), column
      // sums over the sub-tiles of a column half before the four lanes of a column are (lane ends with column
      // 4 lx + ly).  The tile's sums are added to the fixed-point words of y (rows of block I, columns of block J).
      const int j0 = (c + 1) / kT1Blk;                                         // first live block
      const int nbl = nb64 - j0;
      const int n_tiles = nbl * (nbl + 1) / 2;
      struct Sub { int k, q, I, J; };
      auto tile_of = [&](Sub& sbt) {
        int ii = (int)((sqrtf(8.0f * (float)sbt.k + 1.0f) - 1.0f) * 0.5f);
        while ((ii + 1) * (ii + 2) / 2 <= sbt.k) ++ii;
        while (ii * (ii + 1) / 2 > sbt.k) --ii;
        sbt.I = j0 + ii; sbt.J = j0 + (sbt.k - ii * (ii + 1) / 2);
      };
      // first sub-tile at or after (k, q) that exists: inside the matrix and not above the diagonal
      auto settle = [&](Sub& sbt) {
        while (sbt.k < n_tiles) {
          if (sbt.q > 3) { sbt.k += kT1Warps; sbt.q = 0; if (sbt.k < n_tiles) tile_of(sbt); continue; }
          if (2 * sbt.I + (sbt.q >> 1) >= nblk || (sbt.I == sbt.J && (sbt.q & 1) > (sbt.q >> 1))) { ++sbt.q; continue; }
          return;
        }
      };
      auto next_of = [&](const Sub& sbt) { Sub n = sbt; ++n.q; settle(n); return n; };
      auto load = [&](float4 (&t)[8], const Sub& sbt) {
        const float* src = t1_sub(At, 2 * sbt.I + (sbt.q >> 1), 2 * sbt.J + (sbt.q & 1)) + (8 * ly) * 32 + 4 * lx;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) t[kk] = ldcg4(src + kk * 32);
      };
      float rp[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      float racc[2] = {0.f, 0.f};
      uint64_t cp[2][2] = {{pack2(0.f, 0.f), pack2(0.f, 0.f)}, {pack2(0.f, 0.f), pack2(0.f, 0.f)}};   // [column half][pair of columns]
      // the same sub-tile fetched into this warp's buffer in shared memory (each lane copies the sixteen-byte pieces it
      // will read itself)
      auto load_stage = [&](const Sub& sbt) {
        const float* src = t1_sub(At, 2 * sbt.I + (sbt.q >> 1), 2 * sbt.J + (sbt.q & 1)) + (8 * ly) * 32 + 4 * lx;
        float* dst = stage + (8 * ly) * 32 + 4 * lx;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) t1_cp16(dst + kk * 32, src + kk * 32);
        asm volatile("cp.async.commit_group;" ::: "memory");
      };
      auto process = [&](auto get, const Sub& cur, const Sub& nxt) {
        const int sa = cur.q >> 1, sb = cur.q & 1;
        const int row0 = kT1Blk * cur.I + 32 * sa, col0 = kT1Blk * cur.J + 32 * sb;
        const bool diag = row0 == col0;
        const float4 uj = *reinterpret_cast<const float4*>(s_u + col0 + 4 * lx);
        const uint64_t uj01 = pack2(uj.x, uj.y), uj23 = pack2(uj.z, uj.w);
        const float4 ui0 = *reinterpret_cast<const float4*>(s_u + row0 + 8 * ly);
        const float4 ui1 = *reinterpret_cast<const float4*>(s_u + row0 + 8 * ly + 4);
        const float uiv[8] = {ui0.x, ui0.y, ui0.z, ui0.w, ui1.x, ui1.y, ui1.z, ui1.w};
        uint64_t c01 = pack2(0.f, 0.f), c23 = pack2(0.f, 0.f);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          float4 v = get(kk);
          const int rr = 8 * ly + kk, cc = 4 * lx;                             // position inside the sub-tile
          if (diag) {                                                          // lower triangle only
            if (cc + 0 > rr) v.x = 0.f;
            if (cc + 1 > rr) v.y = 0.f;
            if (cc + 2 > rr) v.z = 0.f;
            if (cc + 3 > rr) v.w = 0.f;
          }
          float s0, s1;
          unpack2(fma2(pack2(v.z, v.w), uj23, fma2(pack2(v.x, v.y), uj01, pack2(0.f, 0.f))), s0, s1);
          rp[kk] += s0 + s1;
          if (diag) {                                                          // the diagonal entry counts once (with the rows)
            if (cc + 0 == rr) v.x = 0.f;
            if (cc + 1 == rr) v.y = 0.f;
            if (cc + 2 == rr) v.z = 0.f;
            if (cc + 3 == rr) v.w = 0.f;
          }
          const uint64_t ui2 = pack2(uiv[kk], uiv[kk]);
          c01 = fma2(pack2(v.x, v.y), ui2, c01);
          c23 = fma2(pack2(v.z, v.w), ui2, c23);
        }
        {                                                                      // into the column half's accumulators (added in a fixed order)
          float a0, a1, b0, b1;
          unpack2(c01, a0, a1); unpack2(cp[sb][0], b0, b1); cp[sb][0] = pack2(a0 + b0, a1 + b1);
          unpack2(c23, a0, a1); unpack2(cp[sb][1], b0, b1); cp[sb][1] = pack2(a0 + b0, a1 + b1);
        }
        const bool tile_ends = nxt.k >= n_tiles || nxt.k != cur.k;
        if (tile_ends || (nxt.q >> 1) != sa) {                                 // the row half is complete
          const float rs = rs8(rp, lane);
          if (sa == 0) racc[0] = rs; else racc[1] = rs;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) rp[kk] = 0.f;
        }
        if (tile_ends) {
          float cacc[2];
#pragma unroll
          for (int hb = 0; hb < 2; ++hb) {
            float cv[4];
            unpack2(cp[hb][0], cv[0], cv[1]); unpack2(cp[hb][1], cv[2], cv[3]);
            cacc[hb] = rs4(cv, lane);
            cp[hb][0] = pack2(0.f, 0.f); cp[hb][1] = pack2(0.f, 0.f);
          }
          // lane 8 ly + lx holds row 8 ly + lx of each row half and column 4 lx + ly of each column half
          t1_add_fix(yhi, ylo, kT1Blk * cur.I + lane, racc[0]);
          t1_add_fix(yhi, ylo, kT1Blk * cur.I + 32 + lane, racc[1]);
          t1_add_fix(yhi, ylo, kT1Blk * cur.J + idx, cacc[0]);
          t1_add_fix(yhi, ylo, kT1Blk * cur.J + 32 + idx, cacc[1]);
          racc[0] = 0.f; racc[1] = 0.f;
        }
      };
      // Three sub-tiles per warp on their way or in work: two in registers (ta, tb), one in the warp's buffer in shared
      // memory (filled by cp.async, which holds no registers while it flies).  While one is multiplied the other two
      // are in flight: with a single one in flight the SM's loads stop during the arithmetic, and the latency of DRAM
      // (two to three thousand cycles under load) is more than one sub-tile's arithmetic covers.
      Sub e0{w, 0, 0, 0};
      if (e0.k < n_tiles) tile_of(e0);
      settle(e0);
      if (e0.k < n_tiles) {
        auto ok = [&](const Sub& e) { return e.k < n_tiles; };
        auto after = [&](const Sub& e) { return ok(e) ? next_of(e) : e; };
        float4 ta[8], tb[8];
        Sub e1 = after(e0), e2 = after(e1);
        load(ta, e0);
        if (ok(e1)) load(tb, e1);
        if (ok(e2)) load_stage(e2);
        for (;;) {
          const Sub e3 = after(e2);
          process([&](int kk) { return ta[kk]; }, e0, e1);
          if (!ok(e1)) break;
          if (ok(e3)) load(ta, e3);
          const Sub e4 = after(e3);
          process([&](int kk) { return tb[kk]; }, e1, e2);
          if (!ok(e2)) break;
          if (ok(e4)) load(tb, e4);
          const Sub e5 = after(e4);
          asm volatile("cp.async.wait_group 0;" ::: "memory");
          __syncwarp();
          process([&](int kk) { return *reinterpret_cast<const float4*>(stage + (8 * ly + kk) * 32 + 4 * lx); }, e2, e3);
          if (!ok(e3)) break;
          __syncwarp();                                                        // every lane has read the buffer
          if (ok(e5)) load_stage(e5);
          e0 = e3; e1 = e4; e2 = e5;
        }
      }
    }
    __syncthreads();
    TB_MARK(2)
    // ---- w = p - (u^T p) u with p = 2 (y - U a - W b) ----
    double p[2] = {0.0, 0.0};
    long long yq[2];                                                           // this thread's two rows of y, in fixed point; the words start the next step at zero
#pragma unroll
    for (int x = 0; x < 2; ++x) {
      yq[x] = (long long)yhi[g[x]] * 16777216ll + (long long)ylo[g[x]];
      yhi[g[x]] = 0; ylo[g[x]] = 0u;
    }
#pragma unroll
    for (int x = 0; x < 2; ++x) {
      if (live[x]) {
        double y = (double)yq[x] * 3.552713678800501e-15;                      // 2^-48
        for (int t = 0; t < i; ++t)
          y -= (double)pan_u[t * kT1MaxR + g[x]] * S.dots[2 * t] + (double)pan_w[t * kT1MaxR + g[x]] * S.dots[2 * t + 1];
        p[x] = 2.0 * y;
      }
      const double kp = warp_sum((double)u_f[x] * p[x]);
      if (lane == 0) S.part_k[w + kT1Warps * x] = kp;
      if (c + 1 < r) a_pref[x] = (valid[x] && g[x] >= c + 1) ? __ldcg(at(g[x], c + 1)) : 0.0f;   // next column, in flight over the barrier
    }
    __syncthreads();
    const double K = tb_ordered_sum(S.part_k, nblk, lane);
#pragma unroll
    for (int x = 0; x < 2; ++x)
      if (valid[x]) pan_w[i * kT1MaxR + g[x]] = (float)(live[x] ? p[x] - K * (double)u_f[x] : 0.0);
    const bool flush = (i == kT1NB - 1) || (c == n_ref - 1);
    __syncthreads();
    TB_MARK(4)
    if (!flush) continue;
    // ---- end of the panel: the lower triangle of A0 -= U W^T + W U^T on rows and columns beyond c ----
    {
      const int nr = i + 1, g0 = c + 1;
      const int wr = w >> 3, wc = w & 7;                                       // 2 x 8 warps: 64 rows x 128 columns per pass
      const int qy = lane >> 2, qx = lane & 3;
      const int nb128 = (r + 127) / 128;
      for (int RI = g0 / 64; RI < nb64; ++RI) {
        for (int CJ = g0 / 128; CJ < nb128 && 128 * CJ <= 64 * RI + 63; ++CJ) {
          const int row0 = 64 * RI + 32 * wr + 4 * qy, col0 = 128 * CJ + 16 * wc + 4 * qx;
          if (col0 > row0 + 3 || row0 >= r) continue;                          // this thread's 4 x 4 lies above the diagonal or below the matrix
          float acc[4][4];
#pragma unroll
          for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int y = 0; y < 4; ++y) acc[x][y] = 0.f;
          for (int t = 0; t < nr; ++t) {
            const float4 ru = *reinterpret_cast<const float4*>(pan_u + t * kT1MaxR + row0);
            const float4 rw = *reinterpret_cast<const float4*>(pan_w + t * kT1MaxR + row0);
            const float4 cu = *reinterpret_cast<const float4*>(pan_u + t * kT1MaxR + col0);
            const float4 cw = *reinterpret_cast<const float4*>(pan_w + t * kT1MaxR + col0);
            const float rux[4] = {ru.x, ru.y, ru.z, ru.w}, rwx[4] = {rw.x, rw.y, rw.z, rw.w};
#pragma unroll
            for (int x = 0; x < 4; ++x) {
              acc[x][0] = fmaf(rux[x], cw.x, acc[x][0]); acc[x][1] = fmaf(rux[x], cw.y, acc[x][1]);
              acc[x][2] = fmaf(rux[x], cw.z, acc[x][2]); acc[x][3] = fmaf(rux[x], cw.w, acc[x][3]);
              acc[x][0] = fmaf(rwx[x], cu.x, acc[x][0]); acc[x][1] = fmaf(rwx[x], cu.y, acc[x][1]);
              acc[x][2] = fmaf(rwx[x], cu.z, acc[x][2]); acc[x][3] = fmaf(rwx[x], cu.w, acc[x][3]);
            }
          }
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            const int gr = row0 + x;
            if (gr >= r || gr < g0 || col0 > gr) continue;
            float* dst = at(gr, col0);                                         // four columns of one sub-tile row
            if (col0 >= g0 && col0 + 3 <= gr) {                                // four live entries of the lower triangle
              float4 o = ldcg4(dst);
              o.x -= acc[x][0]; o.y -= acc[x][1]; o.z -= acc[x][2]; o.w -= acc[x][3];
              st4(dst, o);
            } else {
#pragma unroll
              for (int y = 0; y < 4; ++y) if (col0 + y >= g0 && col0 + y <= gr) dst[y] = __ldcg(dst + y) - acc[x][y];
            }
          }
        }
      }
    }
    __threadfence_block();
    __syncthreads();
#pragma unroll
    for (int x = 0; x < 2; ++x)
      if (c + 1 < r) a_pref[x] = (valid[x] && g[x] >= c + 1) ? __ldcg(at(g[x], c + 1)) : 0.0f;   // the update changed it
    TB_MARK(5)
  }
#ifdef TB_PROFILE
  if (blockIdx.x == 0 && tid == 0)
    printf("tridiag_big1 r=%d cycles: column+reflector %lld matvec+dots %lld w %lld gemm %lld\n", r, tp[1], tp[2], tp[4], tp[5]);
#endif
}

// ---- vectors of the kept atoms ------------------------------------------------------------------------------------
// Two phases per CTA.  (A) one warp per kept atom: the eigenvector of T by the twisted factorisation of the small
// route (work vectors in global memory), normalised, filed in the payload's slot of the atom.  (B) the whole CTA
// applies the reflectors to up to four of its atoms at once, u = H_0 H_1 ... H_{r-3} z with H = I - 2 v v^T, from the
// last reflector to the first, four at a time: a thread owns the columns tid, tid + 512, ... of the four reflector rows
// (read once per group, kept in registers between the dot products and the update) and of every z (in shared memory;
// no other thread touches them), so the only exchange per group is the block-wide sum of the products: v_i.z for
// every atom and the six v_i.v_j.  For a group applied in the order 0, 1, 2, 3:  c_0 = 2 v_0.z,
// c_i = 2 (v_i.z - sum_{j<i} c_j v_i.v_j),  z -= sum c_i v_i.  The matrix of reflectors is read once per four atoms
// instead of once per atom, by 512 threads instead of 32.
namespace {
constexpr int kVbThreads = 512;
constexpr int kVbWarps = kVbThreads / 32;
constexpr int kVbSlots = 16;                 // work-vector sets per layer (phase A: 16 atoms at a time over the layer's CTAs)
constexpr int kVbMaxCtas = 4;                // CTAs per layer (the kept atoms are dealt to them)
constexpr int kVbBatch = 4;                  // atoms per pass over the reflectors
constexpr int kVbCols = kTbMaxR / kVbThreads;   // columns per thread and reflector row (8)
constexpr int kVbSums = 4 * kVbBatch + 6;    // products summed per group
constexpr double kVbSameEig = 1.0e-9;        // as on the small route
}  // namespace

namespace {
// The last CTA of a layer to finish orthogonalises kept atoms whose eigenvalues nearly coincide (their vectors are
// determined only as a subspace): modified Gram-Schmidt in payload order, one warp.  Called by every thread of the CTA.
__device__ __forceinline__ void vb_orthogonalise_equal(const SpLayer& L, uint32_t k, int n_ctas) {
  __shared__ uint32_t s_last;
  const int tid = threadIdx.x, lane = tid % 32, w = tid / 32;
  const int r = L.r;
  const double* const gLam = L.lam64; const int* const gPerm = L.perm; const uint32_t* const gIdx = L.idx; float* const gShort = L.shortv;
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = atomicAdd(L.vec_ticket, 1u) == (uint32_t)(n_ctas - 1) ? 1u : 0u;
  __syncthreads();
  if (!s_last || w != 0 || k < 2) return;
  __threadfence();
  for (uint32_t a = 1; a < k; ++a) {
    const double la = gLam[gPerm[gIdx[a]]];
    bool changed = false;
    for (uint32_t b = 0; b < a; ++b) {
      const double lb = gLam[gPerm[gIdx[b]]];
      if (fabs(la - lb) > kVbSameEig) continue;
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
}  // namespace


namespace {
// the columns tid, tid + THREADS, ... of the four reflector rows top, top - 1, top - 2, top - 3 (rows below 0: zeros)
template <int THREADS, int COLS>
__device__ __forceinline__ void vb_load_rows(const float* __restrict__ gV, int64_t ldv, int r, int top, float (&q)[4][COLS]) {
  const int tid = threadIdx.x;
  const float* v0 = gV + (int64_t)top * ldv;
  const float* v1 = gV + (int64_t)max(top - 1, 0) * ldv;
  const float* v2 = gV + (int64_t)max(top - 2, 0) * ldv;
  const float* v3 = gV + (int64_t)max(top - 3, 0) * ldv;
  const bool e1 = top - 1 >= 0, e2 = top - 2 >= 0, e3 = top - 3 >= 0;
  const int h0 = max(top - 3, 0) + 1;                          // reflector kk is zero up to index kk
#pragma unroll
  for (int m = 0; m < COLS; ++m) {
    const int h = tid + m * THREADS;
    const bool in = h >= h0 && h < r;
    q[0][m] = in ? __ldcg(v0 + h) : 0.0f;
    q[1][m] = in && e1 ? __ldcg(v1 + h) : 0.0f;
    q[2][m] = in && e2 ? __ldcg(v2 + h) : 0.0f;
    q[3][m] = in && e3 ? __ldcg(v3 + h) : 0.0f;
  }
}

// z_b <- H_0 ... H_{nref-1} z_b for the nb vectors in s_z, the whole CTA.  PREFETCH: the next group's rows are on their
// way while this group's sums are added up (needs twice the registers for the rows: short sides up to 2048).
template <int THREADS, int BATCH, int COLS, bool PREFETCH>
__device__ __forceinline__ void vb_apply_reflectors(const float* __restrict__ gV, int64_t ldv, int r, int rp, int nref, int nb,
                                                    float* s_z, float (*s_part)[4 * BATCH + 6], float* s_tot) {
  constexpr int kSums = 4 * BATCH + 6, kWarps = THREADS / 32;
  const int tid = threadIdx.x, lane = tid % 32, w = tid / 32;
  float q[4][COLS], qn[4][PREFETCH ? COLS : 1];
  if (PREFETCH && nref > 0) vb_load_rows<THREADS, COLS>(gV, ldv, r, nref - 1, q);
  for (int top = nref - 1; top >= 0; top -= 4) {
    if (!PREFETCH) vb_load_rows<THREADS, COLS>(gV, ldv, r, top, q);
    float acc[kSums];
#pragma unroll
    for (int x = 0; x < kSums; ++x) acc[x] = 0.0f;
#pragma unroll
    for (int m = 0; m < COLS; ++m) {
      const int h = tid + m * THREADS;
      if (h < r) {
        acc[0] = fmaf(q[1][m], q[0][m], acc[0]); acc[1] = fmaf(q[2][m], q[0][m], acc[1]); acc[2] = fmaf(q[2][m], q[1][m], acc[2]);
        acc[3] = fmaf(q[3][m], q[0][m], acc[3]); acc[4] = fmaf(q[3][m], q[1][m], acc[4]); acc[5] = fmaf(q[3][m], q[2][m], acc[5]);
#pragma unroll
        for (int b = 0; b < BATCH; ++b) {
          if (b < nb) {
            const float zh = s_z[(size_t)b * rp + h];
            acc[6 + 4 * b + 0] = fmaf(q[0][m], zh, acc[6 + 4 * b + 0]); acc[6 + 4 * b + 1] = fmaf(q[1][m], zh, acc[6 + 4 * b + 1]);
            acc[6 + 4 * b + 2] = fmaf(q[2][m], zh, acc[6 + 4 * b + 2]); acc[6 + 4 * b + 3] = fmaf(q[3][m], zh, acc[6 + 4 * b + 3]);
          }
        }
      }
    }
    if (PREFETCH && top - 4 >= 0) vb_load_rows<THREADS, COLS>(gV, ldv, r, top - 4, reinterpret_cast<float (&)[4][COLS]>(qn));
    const int n_sums = 6 + 4 * nb;
#pragma unroll
    for (int x = 0; x < kSums; ++x) {
      if (x < n_sums) {
        const float t = warp_sum(acc[x]);
        if (lane == 0) s_part[w][x] = t;
      }
    }
    __syncthreads();
    if (tid < n_sums) {
      float t = 0.0f;
#pragma unroll
      for (int ww = 0; ww < kWarps; ++ww) t += s_part[ww][tid];
      s_tot[tid] = t;
    }
    __syncthreads();
    const float g10 = s_tot[0], g20 = s_tot[1], g21 = s_tot[2], g30 = s_tot[3], g31 = s_tot[4], g32 = s_tot[5];
#pragma unroll
    for (int b = 0; b < BATCH; ++b) {
      if (b < nb) {
        const float c0 = 2.0f * s_tot[6 + 4 * b];
        const float c1 = 2.0f * (s_tot[6 + 4 * b + 1] - c0 * g10);
        const float c2 = 2.0f * (s_tot[6 + 4 * b + 2] - c0 * g20 - c1 * g21);
        const float c3 = 2.0f * (s_tot[6 + 4 * b + 3] - c0 * g30 - c1 * g31 - c2 * g32);
#pragma unroll
        for (int m = 0; m < COLS; ++m) {
          const int h = tid + m * THREADS;
          if (h < r) s_z[(size_t)b * rp + h] -= fmaf(c0, q[0][m], fmaf(c1, q[1][m], fmaf(c2, q[2][m], c3 * q[3][m])));
        }
      }
    }
    // (the next group's partial sums go to s_part only after the barrier that follows them in program order for the
    // slowest reader of s_tot: two barriers separate a write from the reads of the group before)
    if (PREFETCH) {
#pragma unroll
      for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int m = 0; m < COLS; ++m) q[x][m] = qn[x][PREFETCH ? m : 0];
    }
  }
}
}  // namespace

// Short sides up to 1024, any number of layers: a small CTA (four warps) per kept atom at a time, sixteen CTAs per
// layer.  One warp forms the atom's eigenvector of T; the four warps then apply the reflectors together (a thread owns
// eight columns of every reflector row: the 16 loads of a group are in flight at once, the next group's are issued
// before this group's sums are exchanged).  With one warp per atom the same rows took four dependent batches of loads.
namespace {
constexpr int kVcThreads = 128;
constexpr int kVcWarps = kVcThreads / 32;
constexpr int kVcCtas = 16;                  // CTAs per layer = work-vector sets per layer
constexpr int kVcMaxRp = 1024;
}  // namespace

__global__ void __launch_bounds__(kVcThreads) sp_eigvec_big_cta_kernel(const SpLayer* __restrict__ layers,
                                                                       const int* __restrict__ big_layers) {
  const SpLayer& L = layers[big_layers[blockIdx.x]];
  if (L.rp > kVcMaxRp) return;                                 // larger layers: sp_eigvec_big_kernel
  extern __shared__ __align__(16) unsigned char vb_smem[];
  const int r = L.r, rp = L.rp;
  double* s_d = reinterpret_cast<double*>(vb_smem);            // [rp]
  double* s_e = s_d + rp;                                      // [rp]
  float* s_z = reinterpret_cast<float*>(s_e + rp);             // [rp]
  __shared__ float s_part[kVcWarps][10];
  __shared__ float s_tot[10];
  const int tid = threadIdx.x, lane = tid % 32, w = tid / 32;
  const uint32_t k = L.hdr->k;
  const float* const gV = L.td_V; const int64_t ldv = L.td_ldv; const double* const gLam = L.lam64;
  const int* const gPerm = L.perm; const uint32_t* const gIdx = L.idx; float* const gShort = L.shortv;
  const int nref = max(r - 2, 0);
  const int slot = blockIdx.y;                                 // 0 .. 15
  if ((uint32_t)slot < k) {
    for (int i = tid; i < r; i += kVcThreads) { s_d[i] = L.td_d[i]; s_e[i] = i + 1 < r ? L.td_e[i] : 0.0; }
    __syncthreads();
    double* wa = L.tb_vecwork + (size_t)slot * 5 * rp;
    double* wb = wa + rp; double* wc = wb + rp; double* wd = wc + rp; double* zz = wd + rp;
    for (uint32_t a = slot; a < k; a += kVcCtas) {
      if (w == 0) {
        const int ei = gPerm[gIdx[a]];                         // index of the atom's eigenvalue (ascending order)
        double lambda = gLam[ei];
        int skip = 0;                                          // earlier kept atoms with the same eigenvalue: another twist index each
        for (uint32_t b2 = lane; b2 < a; b2 += 32) skip += fabs(gLam[gPerm[gIdx[b2]]] - lambda) <= kVbSameEig ? 1 : 0;
        skip = (int)warp_sum((uint32_t)skip);
        double n2 = 1.0;
        const double corr = twisted_vector(s_d, s_e, r, lambda, wa, wb, wc, wd, zz, lane, skip, &n2);
        double gap = 1.0e300;
        if (ei > 0) gap = fmin(gap, fabs(lambda - gLam[ei - 1]));
        if (ei + 1 < r) gap = fmin(gap, fabs(gLam[ei + 1] - lambda));
        if (finite64(corr) && skip == 0 && !(fabs(corr) <= 1.0e-9 * gap)) {  // one Rayleigh-quotient step, then the vector again
          lambda += corr;
          __syncwarp();
          twisted_vector(s_d, s_e, r, lambda, wa, wb, wc, wd, zz, lane, 0, &n2);
        }
        __syncwarp();
        const double inv = n2 > 0.0 ? rsqrt(n2) : 0.0;
        for (int i = lane; i < r; i += 32) s_z[i] = (float)(zz[i] * inv);
      }
      __syncthreads();
      vb_apply_reflectors<kVcThreads, 1, kVcMaxRp / kVcThreads, true>(gV, ldv, r, rp, nref, 1, s_z, s_part, s_tot);
      float n2f = 0.0f;
      for (int i = tid; i < r; i += kVcThreads) n2f = fmaf(s_z[i], s_z[i], n2f);
      n2f = warp_sum(n2f);
      __syncthreads();
      if (lane == 0) s_part[w][0] = n2f;
      __syncthreads();
      float tot = 0.0f;
#pragma unroll
      for (int ww = 0; ww < kVcWarps; ++ww) tot += s_part[ww][0];
      const float invf = tot > 0.0f ? rsqrtf(tot) : 0.0f;
      for (int i = tid; i < r; i += kVcThreads) gShort[(int64_t)a * r + i] = s_z[i] * invf;
      __syncthreads();
    }
  }
  vb_orthogonalise_equal(L, k, kVcCtas);
}

__global__ void __launch_bounds__(kVbThreads, 1) sp_eigvec_big_kernel(const SpLayer* __restrict__ layers,
                                                                      const int* __restrict__ big_layers) {
  const SpLayer& L = layers[big_layers[blockIdx.x]];
  if (L.rp <= 1024) return;                                    // smaller layers: sp_eigvec_big_cta_kernel
  extern __shared__ __align__(16) unsigned char vb_smem[];
  const int r = L.r, rp = L.rp;
  double* s_d = reinterpret_cast<double*>(vb_smem);            // [rp]
  double* s_e = s_d + rp;                                      // [rp]
  float* s_z = reinterpret_cast<float*>(s_e + rp);             // [kVbBatch][rp]
  __shared__ float s_part[kVbWarps][kVbSums];
  __shared__ float s_tot[kVbSums];
  const int tid = threadIdx.x, lane = tid % 32, w = tid / 32;
  const int n_ctas = gridDim.y, cy = blockIdx.y;
  const uint32_t k = L.hdr->k;
  const float* const gV = L.td_V; const int64_t ldv = L.td_ldv; const double* const gLam = L.lam64;
  const int* const gPerm = L.perm; const uint32_t* const gIdx = L.idx; float* const gShort = L.shortv;
  const int nref = max(r - 2, 0);
  for (int i = tid; i < r; i += kVbThreads) { s_d[i] = L.td_d[i]; s_e[i] = i + 1 < r ? L.td_e[i] : 0.0; }
  __syncthreads();
  // ---- (A) this CTA's atoms are a = cy, cy + n_ctas, ...; warp w < slots-per-CTA takes every (slots-per-CTA)-th of them ----
  const int spc = kVbSlots / n_ctas;                           // work-vector sets of this CTA
  if (w < spc) {
    double* wa = L.tb_vecwork + (size_t)(cy * spc + w) * 5 * rp;
    double* wb = wa + rp; double* wc = wb + rp; double* wd = wc + rp; double* zz = wd + rp;
    for (uint32_t a = cy + (uint32_t)n_ctas * w; a < k; a += (uint32_t)(n_ctas * spc)) {
      const int ei = gPerm[gIdx[a]];                           // index of the atom's eigenvalue (ascending order)
      double lambda = gLam[ei];
      int skip = 0;                                            // earlier kept atoms with the same eigenvalue: another twist index each
      for (uint32_t b2 = lane; b2 < a; b2 += 32) skip += fabs(gLam[gPerm[gIdx[b2]]] - lambda) <= kVbSameEig ? 1 : 0;
      skip = (int)warp_sum((uint32_t)skip);
      double n2 = 1.0;
      const double corr = twisted_vector(s_d, s_e, r, lambda, wa, wb, wc, wd, zz, lane, skip, &n2);
      double gap = 1.0e300;
      if (ei > 0) gap = fmin(gap, fabs(lambda - gLam[ei - 1]));
      if (ei + 1 < r) gap = fmin(gap, fabs(gLam[ei + 1] - lambda));
      if (finite64(corr) && skip == 0 && !(fabs(corr) <= 1.0e-9 * gap)) {    // one Rayleigh-quotient step, then the vector again
        lambda += corr;
        __syncwarp();
        twisted_vector(s_d, s_e, r, lambda, wa, wb, wc, wd, zz, lane, 0, &n2);
      }
      __syncwarp();
      const double inv = n2 > 0.0 ? rsqrt(n2) : 0.0;
      for (int i = lane; i < r; i += 32) gShort[(int64_t)a * r + i] = (float)(zz[i] * inv);
      __syncwarp();
    }
  }
  __syncthreads();
  // ---- (B) back-transformation, kVbBatch of this CTA's atoms per pass over the reflectors ----
  const uint32_t n_mine = k > (uint32_t)cy ? (k - (uint32_t)cy + (uint32_t)n_ctas - 1u) / (uint32_t)n_ctas : 0u;
  for (uint32_t b0 = 0; b0 < n_mine; b0 += kVbBatch) {
    const int nb = (int)min((uint32_t)kVbBatch, n_mine - b0);
    for (int b = 0; b < nb; ++b) {
      const float* src = gShort + (int64_t)(cy + (b0 + b) * n_ctas) * r;
      for (int i = tid; i < r; i += kVbThreads) s_z[(size_t)b * rp + i] = src[i];
    }
    __syncthreads();
    if (rp <= 4 * kVbThreads) vb_apply_reflectors<kVbThreads, kVbBatch, 4, true>(gV, ldv, r, rp, nref, nb, s_z, s_part, s_tot);
    else vb_apply_reflectors<kVbThreads, kVbBatch, 8, true>(gV, ldv, r, rp, nref, nb, s_z, s_part, s_tot);
    // normalise and file
    for (int b = 0; b < nb; ++b) {
      float n2f = 0.0f;
      for (int i = tid; i < r; i += kVbThreads) n2f = fmaf(s_z[(size_t)b * rp + i], s_z[(size_t)b * rp + i], n2f);
      n2f = warp_sum(n2f);
      __syncthreads();
      if (lane == 0) s_part[w][0] = n2f;
      __syncthreads();
      float tot = 0.0f;
#pragma unroll
      for (int ww = 0; ww < kVbWarps; ++ww) tot += s_part[ww][0];
      const float invf = tot > 0.0f ? rsqrtf(tot) : 0.0f;
      float* dst = gShort + (int64_t)(cy + (b0 + b) * n_ctas) * r;
      for (int i = tid; i < r; i += kVbThreads) dst[i] = s_z[(size_t)b * rp + i] * invf;
    }
    __syncthreads();
  }
  vb_orthogonalise_equal(L, k, n_ctas);
}

// ---- host side ---------------------------------------------------------------------------------------------------
namespace {

template <typename T> size_t tb_smem_bytes(int r_max) {
  constexpr int TR = sizeof(T) == 4 ? 4 : 2;
  const size_t r4 = (size_t)((r_max + 3) & ~3);
  return sizeof(TbShared) + (r4 + 2 * (size_t)kTbNB * 32 * TR + 2 * (size_t)kTbNB * 128 + (sizeof(T) == 4 ? 2 * (size_t)kTbNB * kTbPanRows : 0)) * sizeof(T) +
         (sizeof(T) == 4 ? (size_t)((r_max + 31) & ~31) * sizeof(int2) : 0);  // fp32: the column sums of the triangle-only product, whole 32-row blocks
}
size_t t1_smem_bytes() {
  return sizeof(T1Shared) + sizeof(float) * ((size_t)kT1MaxR + 2 * (size_t)kT1NB * kT1MaxR + 2 * (size_t)kT1MaxR + (size_t)kT1Warps * 1024);
}
size_t vb_smem_bytes(int rp_max) { return (size_t)rp_max * (2 * sizeof(double) + kVbBatch * sizeof(float)); }
size_t vc_smem_bytes(int rp_max) { return (size_t)std::min(rp_max, kVcMaxRp) * (2 * sizeof(double) + sizeof(float)); }

template <typename T, int C> int tb_configure_one() {
  auto* fn = sp_tridiag_big_kernel<T, C>;
  if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tb_smem_bytes<T>(kTbMaxR)) != cudaSuccess) return 1;
  if (C > 8 && cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) return 1;
  return 0;
}

template <typename T, int C>
int tb_launch_one(const SpLayer* d_layers, const int* d_big, int n_big, int r_max, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_big * C); cfg.blockDim = dim3(kTbThreads);
  cfg.dynamicSmemBytes = tb_smem_bytes<T>(r_max); cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = C; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  // rows per CTA: the 32-row blocks of the largest layer dealt to C CTAs
  const int rows_per_cta = ((r_max + 31) / 32 + C - 1) / C * 32;
  const int use_pan = (sizeof(T) == 4 && rows_per_cta <= kTbPanRows) ? 1 : 0;   // fp32 only: the fp64 tiles leave no room
  return (int)cudaLaunchKernelEx(&cfg, sp_tridiag_big_kernel<T, C>, d_layers, d_big, use_pan);
}

}  // namespace

namespace {
template <typename T, int C> int tb_max_clusters(int r_max) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(C); cfg.blockDim = dim3(kTbThreads); cfg.dynamicSmemBytes = tb_smem_bytes<T>(r_max);
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = C; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, sp_tridiag_big_kernel<T, C>, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
  return n;
}
}  // namespace

// clusters of `ctas` CTAs of the fp32 cluster kernel that the GPU runs at the same time (they have to sit inside one
// GPC each, so this is less than SMs / ctas); 0 if unknown
int sp_tridiag_big_max_clusters(int ctas, int r_max) {
  switch (ctas) {
    case 2: return tb_max_clusters<float, 2>(r_max);
    case 4: return tb_max_clusters<float, 4>(r_max);
    case 8: return tb_max_clusters<float, 8>(r_max);
    case 16: return tb_max_clusters<float, 16>(r_max);
    default: return 0;
  }
}

int sp_tridiag_big_max_r() { return kTbMaxR; }
int sp_tridiag_big_panel() { return kTbNB; }
int sp_tridiag_big_min_ctas(int r) { int c = 1; while (c < kTbMaxC && (int64_t)c * kTbThreads < r) c <<= 1; return c; }
int sp_eigvec_big_slots() { return kVbSlots; }

// 0 if the route is available on this GPU
int sp_configure_tridiag_big() {
  int bad = 0;
  bad |= tb_configure_one<float, 1>() | tb_configure_one<float, 2>() | tb_configure_one<float, 4>() |
         tb_configure_one<float, 8>() | tb_configure_one<float, 16>();
  bad |= tb_configure_one<double, 1>() | tb_configure_one<double, 2>() | tb_configure_one<double, 4>() |
         tb_configure_one<double, 8>() | tb_configure_one<double, 16>();
  bad |= cudaFuncSetAttribute(sp_tridiag_big1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)t1_smem_bytes()) != cudaSuccess;
  bad |= cudaFuncSetAttribute(sp_eigvec_big_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)vb_smem_bytes(kTbMaxR)) != cudaSuccess;
  if (bad) cudaGetLastError();
  return bad;
}

// d_big: n_big layer indices, all stored as fp32 (fp64 = 0) or all as fp64; ctas = CTAs per layer (1, 2, 4, 8, 16)
int launch_sp_tridiag_big(const SpLayer* d_layers, const int* d_big, int n_big, int r_max, int ctas, int fp64, cudaStream_t st) {
  if (n_big <= 0) return 0;
  if (ctas == 1 && !fp64 && r_max <= kT1MaxR) {               // one CTA per layer: the triangle-only kernel
    sp_tridiag_big1_kernel<<<n_big, kT1Threads, t1_smem_bytes(), st>>>(d_layers, d_big);
    return (int)cudaGetLastError();
  }
#define TB_CASE(CC) case CC: return fp64 ? tb_launch_one<double, CC>(d_layers, d_big, n_big, r_max, st) \
                                         : tb_launch_one<float, CC>(d_layers, d_big, n_big, r_max, st);
  switch (ctas) { TB_CASE(1) TB_CASE(2) TB_CASE(4) TB_CASE(8) TB_CASE(16) default: return (int)cudaErrorInvalidValue; }
#undef TB_CASE
}

void launch_sp_eigvec_big(const SpLayer* d_layers, const int* d_big, int n_big, int rp_max, cudaStream_t st) {
  if (n_big <= 0) return;
  // layers up to a short side of 1024: a four-warp CTA per kept atom (the other kernel's CTAs leave such layers at once,
  // and the other way round)
  sp_eigvec_big_cta_kernel<<<dim3(n_big, kVcCtas), kVcThreads, vc_smem_bytes(rp_max), st>>>(d_layers, d_big);
  if (rp_max <= kVcMaxRp) return;
  // larger layers: CTAs per layer (1, 2 or 4; the kept atoms are dealt to them), as many as keep the launch within one wave
  static int sms = 0;
  if (sms == 0) { int dev = 0; if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) sms = 1; }
  int per = 1;
  while (per < kVbMaxCtas && n_big * per * 2 <= sms) per *= 2;
  sp_eigvec_big_kernel<<<dim3(n_big, per), kVbThreads, vb_smem_bytes(rp_max), st>>>(d_layers, d_big);
}

}  // namespace atomo
