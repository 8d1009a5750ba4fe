// Spectral ATOMO (Section 5 of the paper): atoms are the rank-one terms sigma_i u_i v_i^T of the
// layer gradient seen as a matrix; only the singular values are sparsified.
//
//   sp_gram            A = G G^T (rows <= cols) or G^T G, r x r on the short side, fp32 products
//                      accumulated in short fp32 runs that are flushed into fp64
//   sp_scale           power-of-two normalisation of A by its trace (keeps squared row norms of
//                      small gradients away from the fp32 underflow range)
//   sp_jacobi_step     one step of a one-sided (Hestenes) Jacobi eigen-solver on the rows of
//                      X = [A | I]: row i is (x_i | v_i) with x_i = v_i^T A; orthogonal row
//                      rotations keep that relation and drive the x_i mutually orthogonal, i.e.
//                      x_i -> lambda_i v_i^T.  Blocks of B rows are paired round-robin; a CTA holds
//                      one block pair in shared memory, one warp per rotation.
//   sp_finalize_sample lambda_i = <x_i, v_i>, descending sort, sigma = sqrt(lambda), the
//                      probabilities of Algorithm 1, Philox Bernoulli draws (Eq. 2), ordered
//                      compaction of the kept ranks, short-side vectors of the kept atoms
//   sp_backproject     long-side vector of each kept atom, w_i = G^T u_i (or G v_i)
//   sp_finish_atoms    sigma_i = ||w_i||, coef_i = sigma_i / p_i, w_i normalised
//   sp_decode          G_hat = sum_k coef_k u_k v_k^T, one streaming write pass (8 atoms per pass)
#include <algorithm>

#include "atomo_kernels.cuh"

namespace atomo {

// =================================================================================================
// init: V-part of X = identity (X was zero-filled by the caller)
// =================================================================================================
__global__ void sp_init_kernel(const SpLayer* __restrict__ layers) {
  const SpLayer& L = layers[blockIdx.x];
  if (!L.acc) return;
  const int64_t ldx = L.ldx;
  for (int i = blockIdx.y * blockDim.x + threadIdx.x; i < L.rp; i += gridDim.y * blockDim.x)
    L.X[(int64_t)i * ldx + L.rp + i] = 1.0f;
}

void launch_sp_init(const SpLayer* d_layers, int n_layers, const TileRef*, int, cudaStream_t st) {
  sp_init_kernel<<<dim3(n_layers, 4), 256, 0, st>>>(d_layers);
}

// =================================================================================================
// Gram matrix of the short side.  64 x 64 output tile per CTA, 16 x 16 threads, 4 x 4 per thread.
// Short-side vector i is row i of G (rows <= cols) or column i of G (rows > cols).
// =================================================================================================
constexpr int kGramTile = 64, kGramK = 16;

__global__ void __launch_bounds__(256) sp_gram_kernel(const SpLayer* __restrict__ layers,
                                                      const TileRef* __restrict__ tiles) {
  __shared__ __align__(16) float As[kGramK][kGramTile + 4];
  __shared__ __align__(16) float Bs[kGramK][kGramTile + 4];
  const TileRef ref = tiles[blockIdx.x];
  const SpLayer& L = layers[ref.layer];
  const int i0 = ref.a * kGramTile, j0 = ref.b * kGramTile;
  const bool diag = ref.a == ref.b;
  const float* __restrict__ G = L.G;
  const int64_t ld = L.ld;
  const int r = L.r, len = L.L;
  const int t = threadIdx.x, ty = t / 16, tx = t % 16;
  float acc[4][4];
  double acc64[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) { acc[a][b] = 0.0f; acc64[a][b] = 0.0; }

  int flush = 0;
  for (int c0 = 0; c0 < len; c0 += kGramK) {
    // stage As[kk][i] = x_{i0+i}[c0+kk], Bs likewise for j0
    if (!L.tall) {
      const int row = t / 4, k4 = (t % 4) * 4;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int c = c0 + k4 + j;
        const int ia = i0 + row, ib = j0 + row;
        As[k4 + j][row] = (ia < r && c < len) ? __ldg(G + (int64_t)ia * ld + c) : 0.0f;
        if (!diag) Bs[k4 + j][row] = (ib < r && c < len) ? __ldg(G + (int64_t)ib * ld + c) : 0.0f;
      }
    } else {
      const int kk = t / 16, i4 = (t % 16) * 4;
      const int c = c0 + kk;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int ia = i0 + i4 + j, ib = j0 + i4 + j;
        As[kk][i4 + j] = (ia < r && c < len) ? __ldg(G + (int64_t)c * ld + ia) : 0.0f;
        if (!diag) Bs[kk][i4 + j] = (ib < r && c < len) ? __ldg(G + (int64_t)c * ld + ib) : 0.0f;
      }
    }
    __syncthreads();
    const float(*Bp)[kGramTile + 4] = diag ? As : Bs;
#pragma unroll
    for (int kk = 0; kk < kGramK; ++kk) {
      const float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&Bp[kk][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[p][q] = fmaf(av[p], bv[q], acc[p][q]);
    }
    __syncthreads();
    if (++flush == 2) {   // 32 products per fp32 run, then into fp64
      flush = 0;
#pragma unroll
      for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) { acc64[p][q] += (double)acc[p][q]; acc[p][q] = 0.0f; }
    }
  }
  const int64_t lda = L.lda;
#pragma unroll
  for (int p = 0; p < 4; ++p)
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int i = i0 + ty * 4 + p, j = j0 + tx * 4 + q;
      if (i < r && j < r) {
        const float v = (float)(acc64[p][q] + (double)acc[p][q]);
        L.A[(int64_t)i * lda + j] = v;
        if (!diag) L.A[(int64_t)j * lda + i] = v;
      }
    }
}

void launch_sp_gram(const SpLayer* d_layers, const TileRef* d_tiles, int n_tiles, cudaStream_t st) {
  if (n_tiles > 0) sp_gram_kernel<<<n_tiles, 256, 0, st>>>(d_layers, d_tiles);
}

// =================================================================================================
// scale A by a power of two so that trace(A) is about 1
// =================================================================================================
__global__ void __launch_bounds__(256) sp_trace_kernel(const SpLayer* __restrict__ layers) {
  const SpLayer& L = layers[blockIdx.x];
  const int64_t lda = L.lda;
  __shared__ float s_red[256];
  float tr = 0.0f;
  for (int i = threadIdx.x; i < L.r; i += 256) tr += L.A[(int64_t)i * lda + i];
  s_red[threadIdx.x] = tr;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) { if (threadIdx.x < o) s_red[threadIdx.x] += s_red[threadIdx.x + o]; __syncthreads(); }
  tr = s_red[0];
  float sc = 1.0f;
  if (tr > 0.0f && tr < 3.0e38f) sc = exp2f(-rintf(log2f(tr)));
  if (!(sc > 0.0f) || !(sc < 3.0e38f)) sc = 1.0f;
  if (threadIdx.x == 0) *L.scale = sc;
}

__global__ void __launch_bounds__(256) sp_scale_kernel(const SpLayer* __restrict__ layers) {
  const SpLayer& L = layers[blockIdx.x];
  const int64_t lda = L.lda;
  const float sc = *L.scale;
  if (sc == 1.0f) return;
  for (int i = blockIdx.y; i < L.r; i += gridDim.y)
    for (int j = threadIdx.x; j < L.r; j += 256) L.A[(int64_t)i * lda + j] *= sc;
}

// Start of an encode call: the payload header (passed by value), the layer headers from their template in the table
// cache, the call's flag words and a region of the workspace that starts at zero (n_zero 32-bit words; small: status
// words and tickets) -- a kernel instead of host-to-device copies and memsets, which would queue behind whatever the
// application has on the copy engine.
__global__ void __launch_bounds__(256) begin_kernel(uint8_t* __restrict__ pay, atomo_payload_header gh,
                                                    const atomo_layer_header* __restrict__ tmpl, int n_layers,
                                                    uint32_t* __restrict__ flags, uint32_t* __restrict__ zero, int64_t n_zero) {
  if (blockIdx.x == 0 && threadIdx.x == 0) *reinterpret_cast<atomo_payload_header*>(pay) = gh;
  if (blockIdx.x == 0 && threadIdx.x < 4 && flags != nullptr) flags[threadIdx.x] = 0u;
  for (int64_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n_zero; i += gridDim.x * blockDim.x) zero[i] = 0u;
  static_assert(sizeof(atomo_layer_header) % 16 == 0 && sizeof(atomo_payload_header) % 16 == 0, "headers are copied as 16-byte words");
  uint4* dst = reinterpret_cast<uint4*>(pay + sizeof(atomo_payload_header));
  const uint4* src = reinterpret_cast<const uint4*>(tmpl);
  const int n16 = n_layers * (int)(sizeof(atomo_layer_header) / 16);
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += gridDim.x * blockDim.x) dst[i] = src[i];
}

void launch_sp_begin(uint8_t* pay, const atomo_payload_header& gh, const atomo_layer_header* d_tmpl, int n_layers,
                     uint32_t* d_flags, uint32_t* d_zero, int64_t n_zero, cudaStream_t st) {
  const int64_t n16 = std::max<int64_t>(n_layers * (int64_t)(sizeof(atomo_layer_header) / 16), n_zero);
  begin_kernel<<<(int)std::max<int64_t>(1, std::min<int64_t>(32, (n16 + 255) / 256)), 256, 0, st>>>(pay, gh, d_tmpl, n_layers, d_flags, d_zero, n_zero);
}

// A decomposition supplied by the caller (test entry point): lambda_i = sigma_i^2 in the eigenvalue slots (scale 1),
// short-side vector i (rank-major input) in row i of X, which the caller zero-filled.
__global__ void __launch_bounds__(256) sp_load_svd_kernel(const SpLayer* __restrict__ layers, const float* const* __restrict__ sigma,
                                                          const float* const* __restrict__ vecs) {
  const SpLayer& L = layers[blockIdx.x];
  const float* sg = sigma[blockIdx.x];
  const float* vv = vecs[blockIdx.x];
  const int r = L.r;
  if (blockIdx.y == 0) {
    for (int i = threadIdx.x; i < r; i += 256) { const float x = sg[i]; L.lam[i] = x * x; }
    if (threadIdx.x == 0) *L.scale = 1.0f;
  }
  for (int i = blockIdx.y; i < r; i += gridDim.y)
    for (int j = threadIdx.x; j < r; j += 256) L.X[(int64_t)i * L.ldx + j] = vv[(int64_t)i * r + j];
}

void launch_sp_load_svd(const SpLayer* d_layers, int n_layers, const float* const* d_sigma, const float* const* d_vecs,
                        cudaStream_t st) {
  sp_load_svd_kernel<<<dim3(n_layers, 32), 256, 0, st>>>(d_layers, d_sigma, d_vecs);
}

void launch_sp_scale(const SpLayer* d_layers, int n_layers, cudaStream_t st) {
  sp_trace_kernel<<<n_layers, 256, 0, st>>>(d_layers);
  sp_scale_kernel<<<dim3(n_layers, 32), 256, 0, st>>>(d_layers);
}

// =================================================================================================
// Refinement of the singular values: sigma_i = || G^T u_i || (rows <= cols) or || G v_i || for every
// short-side vector, not only the kept ones.  The Gram route resolves eigenvalues only down to about
// eps * lambda_1, which for a long flat noise tail adds up in the nuclear norm; the norm of the projection
// is second-order accurate in the eigenvector error, so the tail comes out right as long as the
// vectors are orthonormal.  Tile = 64 vectors x 64 positions of the long side; each tile contributes
// one partial sum of squares per vector (summed in a fixed order by sp_finalize_sample).
// =================================================================================================
__global__ void __launch_bounds__(256) sp_rowinv_kernel(const SpLayer* __restrict__ layers) {
  const SpLayer& L = layers[blockIdx.x];
  if (!L.refine) return;
  const int lane = threadIdx.x % 32, w = threadIdx.x / 32;
  const int voff = L.acc ? L.rp : 0;
  for (int i = blockIdx.y * 8 + w; i < L.rp; i += gridDim.y * 8) {
    float n2 = 0.f;
    if (i < L.r) {
      const float* v = L.X + (int64_t)i * L.ldx + voff;
      for (int j = lane; j < L.r; j += 32) n2 = fmaf(v[j], v[j], n2);
    }
    n2 = warp_sum(n2);
    if (lane == 0) L.row_inv[i] = n2 > 0.f ? 1.0f / sqrtf(n2) : 0.f;
  }
}

__global__ void __launch_bounds__(256) sp_refine_kernel(const SpLayer* __restrict__ layers,
                                                        const TileRef* __restrict__ tiles) {
  __shared__ __align__(16) float As[kGramK][kGramTile + 4];   // As[k][a] = u_a[k0 + k]
  __shared__ __align__(16) float Bs[kGramK][kGramTile + 4];   // Bs[k][c] = G(k0 + k, c0 + c) seen from the short side
  __shared__ float s_sq[16][kGramTile];
  const TileRef ref = tiles[blockIdx.x];
  const SpLayer& L = layers[ref.layer];
  const int a0 = ref.a * kGramTile, c0 = ref.b * kGramTile;
  const float* __restrict__ G = L.G;
  const int64_t ld = L.ld, ldx = L.ldx;
  const int r = L.r, len = L.L;
  const int voff = L.acc ? L.rp : 0;
  const int t = threadIdx.x, ty = t / 16, tx = t % 16;
  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.0f;
  for (int k0 = 0; k0 < r; k0 += kGramK) {
    {
      const int row = t / 4, k4 = (t % 4) * 4;               // vector a0 + row, components k0 + k4 ..
      const int a = a0 + row;
      const float inv = a < r ? L.row_inv[a] : 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int k = k0 + k4 + j;
        As[k4 + j][row] = (a < r && k < r) ? L.X[(int64_t)a * ldx + voff + k] * inv : 0.0f;
      }
    }
    if (!L.tall) {                                           // G[k][c]: contiguous in c
      const int kk = t / 16, c4 = (t % 16) * 4;
      const int k = k0 + kk;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int c = c0 + c4 + j;
        Bs[kk][c4 + j] = (k < r && c < len) ? __ldg(G + (int64_t)k * ld + c) : 0.0f;
      }
    } else {                                                 // G[c][k]: contiguous in k
      const int row = t / 4, k4 = (t % 4) * 4;
      const int c = c0 + row;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int k = k0 + k4 + j;
        Bs[k4 + j][row] = (k < r && c < len) ? __ldg(G + (int64_t)c * ld + k) : 0.0f;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kGramK; ++kk) {
      const float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[p][q] = fmaf(av[p], bv[q], acc[p][q]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int p = 0; p < 4; ++p) {
    float sq = 0.f;
#pragma unroll
    for (int q = 0; q < 4; ++q) sq = fmaf(acc[p][q], acc[p][q], sq);
    s_sq[tx][ty * 4 + p] = sq;
  }
  __syncthreads();
  if (t < kGramTile && a0 + t < r) {
    float tot = 0.f;
#pragma unroll
    for (int j = 0; j < 16; ++j) tot += s_sq[j][t];            // fixed order
    L.refine_partials[(int64_t)ref.b * L.rp + a0 + t] = tot;
  }
}

void launch_sp_refine(const SpLayer* d_layers, int n_layers, const TileRef* d_tiles, int n_tiles, cudaStream_t st) {
  if (n_tiles <= 0) return;
  sp_rowinv_kernel<<<dim3(n_layers, 16), 256, 0, st>>>(d_layers);
  sp_refine_kernel<<<n_tiles, 256, 0, st>>>(d_layers, d_tiles);
}

// =================================================================================================
// finalize + probabilities + sampling.  One CTA (512 threads) per layer.
// =================================================================================================
constexpr int kFinThreads = 512;

__global__ void __launch_bounds__(kFinThreads) sp_finalize_sample_kernel(const SpLayer* __restrict__ layers, double s,
                                                                         PhiloxKey key, uint32_t kind_step,
                                                                         int max_sweeps,
                                                                         const uint32_t* __restrict__ timeout_flag) {
  const SpLayer& L = layers[blockIdx.x];
  __shared__ float s_lam[kMaxShort];        // eigenvalues by row, later sigma by rank
  __shared__ float s_sig[kMaxShort];
  __shared__ double s_red[kFinThreads];
  __shared__ uint32_t s_scan[kFinThreads / 32];
  __shared__ double s_T, s_scur;
  __shared__ uint32_t s_nsat, s_bad, s_k;
  const int tid = threadIdx.x, lane = tid % 32, w = tid / 32;
  const int r = L.r, rp = L.rp;
  const int64_t ldx = L.ldx;
  const int voff = L.acc ? rp : 0;          // where the eigenvector sits in a row
  const float inv_scale = 1.0f / *L.scale;
  atomo_layer_header* h = L.hdr;
  if (tid == 0) { s_bad = 0; s_k = 0; }
  __syncthreads();

  // eigenvalue of A per row, one warp per row.  mode 0: lambda_i = <x_i, v_i> (Rayleigh quotient at v_i);
  // mode 1: lambda_i = ||x_i||^2 (row i = sigma_i w_i^T).  With refinement: the sum of the tiles' partial
  // squared norms of the projection (already in the units of G).
  if (L.lam_ready && !L.refine && !L.acc) {
    for (int i = tid; i < r; i += kFinThreads) {
      const float lam = L.lam[i] * inv_scale;
      if (!(fabsf(lam) <= 3.0e38f)) atomicOr(&s_bad, 1u);
      s_lam[i] = fmaxf(lam, 0.0f);
    }
  } else
  for (int i = w; i < r; i += kFinThreads / 32) {
    float lam;
    if (L.refine) {
      double d = 0.0;
      for (int tl = lane; tl < L.refine_tiles; tl += 32) d += (double)L.refine_partials[(int64_t)tl * rp + i];
      lam = (float)warp_sum(d);
    } else {
      // rows are zero-padded to rp floats (a multiple of 32): whole float4, several loads in flight
      const float4* x4 = reinterpret_cast<const float4*>(L.X + (int64_t)i * ldx);
      const float4* v4 = reinterpret_cast<const float4*>(L.X + (int64_t)i * ldx + voff);
      float d0 = 0.f, d1 = 0.f;
#pragma unroll 4
      for (int j = lane; j < rp / 4; j += 32) {
        const float4 a = x4[j], b = v4[j];
        d0 = fmaf(a.x, b.x, fmaf(a.y, b.y, d0));
        d1 = fmaf(a.z, b.z, fmaf(a.w, b.w, d1));
      }
      lam = warp_sum(d0 + d1) * inv_scale;
    }
    if (lane == 0) {
      if (!(fabsf(lam) <= 3.0e38f)) atomicOr(&s_bad, 1u);
      s_lam[i] = fmaxf(lam, 0.0f);
    }
  }
  __syncthreads();
  const bool bad = s_bad != 0;
  // rank by counting (descending, ties: lower row first); sigma = sqrt(lambda)
  for (int i = tid; i < r; i += kFinThreads) {
    const float li = s_lam[i];
    int rank = 0;
    for (int j = 0; j < r; ++j) { const float lj = s_lam[j]; rank += (lj > li) || (lj == li && j < i); }
    s_sig[rank] = bad ? 0.0f : sqrtf(li);
    L.perm[rank] = i;
  }
  __syncthreads();
  // ||sigma||_1 in fp64, fixed tree
  double part = 0.0;
  for (int i = tid; i < r; i += kFinThreads) part += (double)s_sig[i];
  s_red[tid] = part;
  __syncthreads();
  for (int o = kFinThreads / 2; o > 0; o >>= 1) { if (tid < o) s_red[tid] += s_red[tid + o]; __syncthreads(); }
  if (tid == 0) {
    // Algorithm 1 on the sorted sigma: peel atoms while sigma_i * s > sum_{j >= i} sigma_j
    double T = s_red[0], sc = s;
    int i = 0;
    while (i < r && (double)s_sig[i] * sc > T) { T -= (double)s_sig[i]; sc -= 1.0; ++i; }
    if (i == r || !(T > 0.0)) T = 0.0;
    s_T = T; s_scur = sc; s_nsat = (uint32_t)i;
    h->n_sat = (uint32_t)i;
    h->c = (T > 0.0 && sc > 0.0) ? (float)(T / sc) : 0.0f;
    h->l1 = s_red[0];
  }
  __syncthreads();
  const double T = s_T, scur = s_scur;
  const int n_sat = (int)s_nsat;
  const double scale = (T > 0.0 && scur > 0.0) ? scur / T : 0.0;

  // probabilities, Bernoulli draws, ordered compaction of the kept ranks
  uint32_t carry = 0;
  for (int base = 0; base < r; base += kFinThreads) {
    const int i = base + tid;
    float p = 0.0f;
    bool keep = false;
    if (i < r) {
      const float sg = s_sig[i];
      p = (i < n_sat) ? 1.0f : fminf((float)((double)sg * scale), 1.0f);
      if (!(sg > 0.0f)) p = 0.0f;
      const uint4 wd = atom_block_words((uint64_t)(i >> 2), L.layer, kind_step, key);
      const uint32_t word = (i & 3) == 0 ? wd.x : (i & 3) == 1 ? wd.y : (i & 3) == 2 ? wd.z : wd.w;
      keep = !bad && bernoulli_keep(p, word);
      if (L.sigma) L.sigma[i] = sg;
      if (L.prob) L.prob[i] = p;
    }
    const uint32_t ballot = __ballot_sync(0xffffffffu, keep);
    if (lane == 0) {
      s_scan[w] = __popc(ballot);
      if (L.mask_words && base + w * 32 < r) L.mask_words[(base >> 5) + w] = ballot;
    }
    __syncthreads();
    uint32_t off = carry;
    for (int j = 0; j < w; ++j) off += s_scan[j];
    uint32_t total = 0;
    for (int j = 0; j < kFinThreads / 32; ++j) total += s_scan[j];
    if (keep) {
      const uint32_t pos = off + __popc(ballot & ((1u << lane) - 1u));
      if (pos < L.k_cap) { L.idx[pos] = (uint32_t)i; L.p_sel[pos] = p; }
    }
    carry += total;
    __syncthreads();
  }
  if (tid == 0) {
    uint32_t status = ATOMO_OK;
    if (timeout_flag != nullptr && *timeout_flag != 0) status = ATOMO_ERR_TIMEOUT;
    else if (bad) status = ATOMO_ERR_NONFINITE;
    else if (carry > L.k_cap) status = ATOMO_ERR_CAPACITY;
    else if (h->sweeps >= (uint32_t)max_sweeps && L.rot_count[max_sweeps - 1] != 0) status = ATOMO_ERR_NOT_CONVERGED;
    h->status = status;
    // route 0 keeps an orthonormal basis whatever the sweep count, so its unconverged result is still an
    // unbiased estimator; route 1's rows are orthogonal only at convergence, so it keeps nothing
    const uint32_t k = (status == ATOMO_OK || (status == ATOMO_ERR_NOT_CONVERGED && L.acc)) ? carry : 0u;
    h->k = k;
    s_k = k;
  }
  __syncthreads();
  const uint32_t k = s_k;
  if (L.tri) return;                       // tridiagonal route: the vectors of the kept atoms come from sp_eigvec_kernel
  // short-side vectors of the kept atoms, normalised: payload shortv[a][0..r)
  for (uint32_t a = w; a < k; a += kFinThreads / 32) {
    const int row = L.perm[L.idx[a]];
    const float* v = L.X + (int64_t)row * ldx + voff;
    float n2 = 0.f;
    for (int j = lane; j < r; j += 32) n2 = fmaf(v[j], v[j], n2);
    n2 = warp_sum(n2);
    const float inv = n2 > 0.f ? 1.0f / sqrtf(n2) : 0.f;
    for (int j = lane; j < r; j += 32) L.shortv[(int64_t)a * r + j] = v[j] * inv;
  }
  // optional: every short-side vector (normalised), rank-major
  if (L.dbg_short) {
    for (int a = w; a < r; a += kFinThreads / 32) {
      const float* v = L.X + (int64_t)L.perm[a] * ldx + voff;
      float n2 = 0.f;
      for (int j = lane; j < r; j += 32) n2 = fmaf(v[j], v[j], n2);
      n2 = warp_sum(n2);
      const float inv = n2 > 0.f ? 1.0f / sqrtf(n2) : 0.f;
      for (int j = lane; j < r; j += 32) L.dbg_short[(int64_t)a * r + j] = v[j] * inv;
    }
  }
}

void launch_sp_finalize_sample(const SpLayer* d_layers, int n_layers, double s, PhiloxKey key, uint32_t kind_step,
                               int max_sweeps, const uint32_t* timeout_flag, cudaStream_t st) {
  sp_finalize_sample_kernel<<<n_layers, kFinThreads, 0, st>>>(d_layers, s, key, kind_step, max_sweeps, timeout_flag);
}

// =================================================================================================
// back-projection: long-side vector of each kept atom.
//   rows <= cols: w_a[c]   = sum_i G[i][c] u_a[i]   tile = 1024 columns x one chunk of rows (a multiple of 64, set
//                                                     per layer), 4 columns per thread, 8 row loads in flight;
//                                                     chunk partials go to bp_part and are summed in chunk
//                                                     order by sp_finish_atoms
//   rows >  cols: w_a[row] = sum_c G[row][c] v_a[c]   tile = 32 rows, warp per row (one chunk)
// =================================================================================================
constexpr int kBpThreads = 256, kBpAtoms = 8, kBpCols = 1024, kBpRows = 32, kBpChunk = 64;
int sp_bp_cols_per_tile() { return kBpCols; }
int sp_bp_rows_per_tile() { return kBpRows; }
int sp_bp_chunk_rows() { return kBpChunk; }

__global__ void __launch_bounds__(kBpThreads) sp_backproject_kernel(const SpLayer* __restrict__ layers,
                                                                    const TileRef* __restrict__ tiles) {
  __shared__ __align__(16) float s_u[kBpChunk][kBpAtoms];   // wide: the chunk's components of up to 8 short-side vectors
  extern __shared__ __align__(16) float s_v[];              // tall: kBpAtoms x r
  const TileRef ref = tiles[blockIdx.x];
  const SpLayer& L = layers[ref.layer];
  const uint32_t k = L.hdr->k;
  const int r = L.r, len = L.L;
  const int tid = threadIdx.x, lane = tid % 32, w = tid / 32;
  const float* __restrict__ G = L.G;
  const int64_t ld = L.ld;
  const bool vec = (ld % 4 == 0) && ((reinterpret_cast<uintptr_t>(G) & 15u) == 0);
  for (uint32_t a0 = 0; a0 < k; a0 += kBpAtoms) {
    const int na = min((uint32_t)kBpAtoms, k - a0);
    __syncthreads();
    if (!L.tall) {
      // a thread owns 4 consecutive columns: one 16-byte load per row, 8 rows in flight, 32 FMAs per row
      const int row_lo = ref.b * L.bp_chunk_rows, row_hi = min(r, row_lo + L.bp_chunk_rows);
      const int c = ref.a * kBpCols + 4 * tid;
      float acc[kBpAtoms][4];
#pragma unroll
      for (int a = 0; a < kBpAtoms; ++a) { acc[a][0] = 0.f; acc[a][1] = 0.f; acc[a][2] = 0.f; acc[a][3] = 0.f; }
      for (int i0 = row_lo; i0 < row_hi; i0 += kBpChunk) {
        const int ni = min(kBpChunk, row_hi - i0);
        if (i0 > row_lo) __syncthreads();
        for (int idx = tid; idx < kBpAtoms * kBpChunk; idx += kBpThreads) {
          const int i = idx / kBpAtoms, a = idx % kBpAtoms;
          s_u[i][a] = (a < na && i < ni) ? L.shortv[(int64_t)(a0 + a) * r + i0 + i] : 0.0f;
        }
        __syncthreads();
        if (c < len) {
          const float* gp = G + (int64_t)i0 * ld + c;
          const bool full4 = vec && c + 3 < len;
          for (int i = 0; i < ni; i += 8) {
            float4 g[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              g[u] = make_float4(0.f, 0.f, 0.f, 0.f);
              if (i + u < ni) {
                const float* src = gp + (int64_t)(i + u) * ld;
                if (full4) g[u] = __ldg(reinterpret_cast<const float4*>(src));
                else {
                  g[u].x = __ldg(src);
                  if (c + 1 < len) g[u].y = __ldg(src + 1);
                  if (c + 2 < len) g[u].z = __ldg(src + 2);
                  if (c + 3 < len) g[u].w = __ldg(src + 3);
                }
              }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const float4 u0 = *reinterpret_cast<const float4*>(&s_u[i + u][0]);     // rows past ni hold zeros
              const float4 u1 = *reinterpret_cast<const float4*>(&s_u[i + u][4]);
              const float uu[kBpAtoms] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
#pragma unroll
              for (int a = 0; a < kBpAtoms; ++a) {
                acc[a][0] = fmaf(g[u].x, uu[a], acc[a][0]); acc[a][1] = fmaf(g[u].y, uu[a], acc[a][1]);
                acc[a][2] = fmaf(g[u].z, uu[a], acc[a][2]); acc[a][3] = fmaf(g[u].w, uu[a], acc[a][3]);
              }
            }
          }
        }
      }
      if (c < len) {
#pragma unroll
        for (int a = 0; a < kBpAtoms; ++a)
          if (a < na) {
            float* dst = L.bp_part + ((int64_t)ref.b * L.k_cap + a0 + a) * len + c;
            for (int j = 0; j < 4; ++j) if (c + j < len) dst[j] = acc[a][j];
          }
      }
    } else {
      for (int idx = tid; idx < na * r; idx += kBpThreads) s_v[idx] = L.shortv[(int64_t)a0 * r + idx];
      __syncthreads();
      for (int rr = w; rr < kBpRows; rr += kBpThreads / 32) {
        const int row = ref.a * kBpRows + rr;
        if (row >= len) break;
        float acc[kBpAtoms];
#pragma unroll
        for (int a = 0; a < kBpAtoms; ++a) acc[a] = 0.f;
        for (int c = lane; c < r; c += 32) {
          const float g = __ldg(G + (int64_t)row * ld + c);
#pragma unroll
          for (int a = 0; a < kBpAtoms; ++a) if (a < na) acc[a] = fmaf(g, s_v[a * r + c], acc[a]);
        }
#pragma unroll
        for (int a = 0; a < kBpAtoms; ++a) {
          acc[a] = warp_sum(acc[a]);
          if (a < na && lane == 0) L.bp_part[(int64_t)(a0 + a) * len + row] = acc[a];
        }
      }
    }
  }
}

int sp_configure() {
  const int e = sp_configure_eig();
  if (e != 0) return e;
  return (int)cudaFuncSetAttribute(sp_backproject_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   kBpAtoms * kMaxShort * (int)sizeof(float));
}

void launch_sp_backproject(const SpLayer* d_layers, const TileRef* d_tiles, int n_tiles, int r_max_tall, cudaStream_t st) {
  if (n_tiles > 0)
    sp_backproject_kernel<<<n_tiles, kBpThreads, kBpAtoms * r_max_tall * sizeof(float), st>>>(d_layers, d_tiles);
}

// w_a = sum over row chunks (in chunk order), sigma_a = ||w_a||, coef_a = sigma_a / p_a, long vector = w_a / sigma_a.
// One CTA per (layer, kept-atom slot); slots beyond the layer's k leave at once.
constexpr int kFinishThreads = 1024;
__global__ void __launch_bounds__(kFinishThreads) sp_finish_atoms_kernel(const SpLayer* __restrict__ layers, int k_cap_max) {
  const SpLayer& L = layers[blockIdx.x / k_cap_max];
  const uint32_t a = blockIdx.x % k_cap_max;
  if (a >= L.hdr->k) return;
  const int len = L.L, chunks = L.bp_chunks;
  __shared__ double s_red[kFinishThreads / 32];
  __shared__ float s_sg;
  double part = 0.0;
  float* out = L.longv + (int64_t)a * len;
  const float* in = L.bp_part + (int64_t)a * len;
  const int64_t chunk_stride = (int64_t)L.k_cap * len;
  for (int j = threadIdx.x; j < len; j += kFinishThreads) {
    float wv = 0.f;
#pragma unroll 8
    for (int ch = 0; ch < chunks; ++ch) wv += in[ch * chunk_stride + j];
    out[j] = wv;
    part += (double)wv * (double)wv;
  }
  part = warp_sum(part);
  if (threadIdx.x % 32 == 0) s_red[threadIdx.x / 32] = part;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int i = 0; i < kFinishThreads / 32; ++i) t += s_red[i];            // fixed order
    const float sg = (float)sqrt(t);
    L.coef[a] = sg / L.p_sel[a];
    s_sg = sg;
  }
  __syncthreads();
  const float sg = s_sg;
  const float inv = sg > 0.f ? 1.0f / sg : 0.f;
  for (int j = threadIdx.x; j < len; j += kFinishThreads) out[j] *= inv;   // each thread rescales what it wrote itself
}

void launch_sp_finish_atoms(const SpLayer* d_layers, int n_layers, int k_cap_max, cudaStream_t st) {
  sp_finish_atoms_kernel<<<n_layers * k_cap_max, kFinishThreads, 0, st>>>(d_layers, k_cap_max);
}

// =================================================================================================
// decode: out[i][c] = sum_a coef_a rowvec_a[i] colvec_a[c], a streaming write of the output.
// Tile 64 rows x 1024 columns, 256 threads: a thread owns 4 consecutive columns, keeps the column-vector
// entries of up to 8 atoms in registers and walks down the 64 rows, one 16-byte store per row; the row-vector
// entries (times coef) of the tile sit in shared memory and are read as broadcasts.  k is about s, a handful:
// a layer with more than 8 kept atoms takes further passes that add to what the first one wrote.
// =================================================================================================
constexpr int kDecRows = 64, kDecCols = 1024, kDecAtoms = 8, kDecThreads = 256;
int sp_decode_tile_rows() { return kDecRows; }
int sp_decode_tile_cols() { return kDecCols; }

// `single` (one payload) or `list[0 .. n_payloads)`: the kept atoms of all payloads are walked as one sequence,
// payload after payload, 8 per pass; `scale` multiplies every term (1, or 1 / n_payloads for the average).
__global__ void __launch_bounds__(kDecThreads) sp_decode_kernel(const uint8_t* __restrict__ single,
                                                                const uint8_t* const* __restrict__ list, int n_payloads,
                                                                float scale, const SpDecodeLayer* __restrict__ layers,
                                                                const TileRef* __restrict__ tiles) {
  __shared__ __align__(16) float s_rc[kDecRows][kDecAtoms];      // scale * coef_a * rowvec_a[i] of the tile's rows
  const TileRef ref = tiles[blockIdx.x];
  const SpDecodeLayer D = layers[ref.layer];
  const int64_t rows = D.rows, cols = D.cols;
  const bool tall = rows > cols;
  const int64_t r = tall ? cols : rows, len = tall ? rows : cols;
  const int64_t rlen = tall ? len : r, clen = tall ? r : len;     // lengths of the row- and column-indexed vectors
  const int64_t i0 = (int64_t)ref.a * kDecRows, c = (int64_t)ref.b * kDecCols + 4 * threadIdx.x;
  const int n_rows = (int)min((int64_t)kDecRows, rows - i0);
  const bool vec_out = (cols % 4 == 0) && ((reinterpret_cast<uintptr_t>(D.out) & 15u) == 0);
  float* out = D.out + i0 * cols + c;
  int p = 0;                                                     // cursor over (payload, atom)
  uint32_t a_next = 0;
  bool first_pass = true;
  for (;;) {
    // up to 8 atoms for this pass
    const float* rowv[kDecAtoms]; const float* colv[kDecAtoms]; float cf[kDecAtoms];
    int na = 0;
    while (na < kDecAtoms && p < n_payloads) {
      const uint8_t* payload = list ? list[p] : single;
      const atomo_payload_header* gh = reinterpret_cast<const atomo_payload_header*>(payload);
      // a payload normally comes from another rank: its header is checked before anything it points to is read.  The
      // layer headers must exist (layer index below n_layers) and every array must lie inside total_bytes; a header
      // that fails contributes zeros, and the status word is written only where it is known to be a status word
      const bool has_hdr = gh->magic == ATOMO_MAGIC && (uint32_t)ref.layer < gh->n_layers &&
                           sizeof(atomo_payload_header) + (uint64_t)gh->n_layers * sizeof(atomo_layer_header) <= gh->total_bytes;
      const atomo_layer_header* h = reinterpret_cast<const atomo_layer_header*>(payload + sizeof(atomo_payload_header)) +
                                    (has_hdr ? ref.layer : 0);
      bool ok = has_hdr && gh->kind == ATOMO_KIND_SPECTRAL && h->rows == rows && h->cols == cols && h->k <= h->k_cap;
      if (ok) {
        const uint64_t kc = h->k_cap, tb = gh->total_bytes;
        ok = h->off_idx <= tb && kc * 4 <= tb - h->off_idx && h->off_val <= tb && kc * 4 <= tb - h->off_val &&
             h->off_short <= tb && kc * (uint64_t)r * 4 <= tb - h->off_short &&
             h->off_long <= tb && kc * (uint64_t)len * 4 <= tb - h->off_long;
      }
      if (!ok && has_hdr && a_next == 0 && ref.a == 0 && ref.b == 0 && threadIdx.x == 0)
        raise_status(const_cast<atomo_layer_header*>(h), ATOMO_ERR_PAYLOAD);
      const uint32_t k = ok ? h->k : 0u;
      if (a_next >= k) { ++p; a_next = 0; continue; }
      const float* shortv = reinterpret_cast<const float*>(payload + h->off_short);
      const float* longv = reinterpret_cast<const float*>(payload + h->off_long);
      rowv[na] = (tall ? longv : shortv) + (int64_t)a_next * rlen;     // indexed by output row
      colv[na] = (tall ? shortv : longv) + (int64_t)a_next * clen;     // indexed by output column
      cf[na] = __ldg(reinterpret_cast<const float*>(payload + h->off_val) + a_next) * scale;
      ++na; ++a_next;
    }
    if (na == 0 && !first_pass) break;
    __syncthreads();
    for (int idx = threadIdx.x; idx < kDecRows * kDecAtoms; idx += kDecThreads) {
      const int i = idx / kDecAtoms, a = idx % kDecAtoms;
      float v = 0.f;
#pragma unroll
      for (int u = 0; u < kDecAtoms; ++u) if (u == a && u < na && i < n_rows) v = __ldg(rowv[u] + i0 + i) * cf[u];
      s_rc[i][a] = v;
    }
    float4 cv[kDecAtoms];
#pragma unroll
    for (int a = 0; a < kDecAtoms; ++a) {
      cv[a] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (a < na && c < cols) {
        const float* src = colv[a] + c;
        if ((clen % 4 == 0) && ((reinterpret_cast<uintptr_t>(colv[a]) & 15u) == 0) && c + 3 < cols)
          cv[a] = __ldg(reinterpret_cast<const float4*>(src));
        else {
          cv[a].x = __ldg(src);
          if (c + 1 < cols) cv[a].y = __ldg(src + 1);
          if (c + 2 < cols) cv[a].z = __ldg(src + 2);
          if (c + 3 < cols) cv[a].w = __ldg(src + 3);
        }
      }
    }
    __syncthreads();
    if (c < cols) {
      const bool add = !first_pass;
#pragma unroll 4
      for (int i = 0; i < n_rows; ++i) {
        const float4 r0 = *reinterpret_cast<const float4*>(&s_rc[i][0]);
        const float4 r1 = *reinterpret_cast<const float4*>(&s_rc[i][4]);
        const float rc[kDecAtoms] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int a = 0; a < kDecAtoms; ++a) {
          v.x = fmaf(rc[a], cv[a].x, v.x); v.y = fmaf(rc[a], cv[a].y, v.y);
          v.z = fmaf(rc[a], cv[a].z, v.z); v.w = fmaf(rc[a], cv[a].w, v.w);
        }
        float* o = out + (int64_t)i * cols;
        if (vec_out && c + 3 < cols) {
          if (add) { const float4 old = *reinterpret_cast<const float4*>(o); v.x += old.x; v.y += old.y; v.z += old.z; v.w += old.w; }
          *reinterpret_cast<float4*>(o) = v;
        } else {
          const float vv[4] = {v.x, v.y, v.z, v.w};
          for (int j = 0; j < 4; ++j) if (c + j < cols) o[j] = add ? o[j] + vv[j] : vv[j];
        }
      }
    }
    first_pass = false;
    if (na < kDecAtoms) break;                                    // the sequence is exhausted
  }
}

void launch_sp_decode(const uint8_t* payload, const SpDecodeLayer* d_layers, const TileRef* d_tiles, int n_tiles,
                      cudaStream_t st) {
  if (n_tiles > 0) sp_decode_kernel<<<n_tiles, kDecThreads, 0, st>>>(payload, nullptr, 1, 1.0f, d_layers, d_tiles);
}

void launch_sp_decode_average(const uint8_t* const* d_payloads, int n_payloads, const SpDecodeLayer* d_layers,
                              const TileRef* d_tiles, int n_tiles, cudaStream_t st) {
  if (n_tiles > 0)
    sp_decode_kernel<<<n_tiles, kDecThreads, 0, st>>>(nullptr, d_payloads, n_payloads, 1.0f / (float)n_payloads, d_layers, d_tiles);
}

}  // namespace atomo
