// Entry-wise ATOMO on flat gradients: atoms e_i, lambda_i = g_i (Section 3 of the paper; the
// QSGD / TernGrad family of Section 4 are the budgets s = ||g||_1/||g||_2 and ||g||_1/||g||_inf).
//
//   ew_solve (cooperative)     : pass 1: ||g||_1 (fp64 accumulation), ||g||_inf, non-finite scan; then the
//                                water-filling form of Algorithm 1 -- every atom with
//                                |g_i| (s - n_s) > sum_{unsaturated} |g_j| gets p = 1; repeated
//                                until no new atom saturates (zero rounds when g is s-balanced,
//                                Lemma 3); grid barriers instead of host round trips
//   pass 2   ew_sample         : p_i = |g_i| (s-n_s)/T, Philox word, keep bit -> mask words + tile counts
//            ew_scan           : exclusive scan of tile counts, k, capacity check, header
//            ew_pack           : ordered compaction: idx ascending, val = g_i / p_i
//   decode   ew_decode         : zero-fill with vector stores, then the tile's kept values (per-tile
//                                offsets travel in the payload)
#include <algorithm>

#include <cooperative_groups.h>

#include "atomo_kernels.cuh"

namespace cg = cooperative_groups;

namespace atomo {

constexpr int kEwThreads = 256;
constexpr int kEwTile = 4096;                 // elements per tile of the sample / pack / decode passes

__device__ __forceinline__ float4 load4(const float* __restrict__ g, int64_t i, int64_t n, bool aligned) {
  if (aligned && i + 3 < n) return __ldg(reinterpret_cast<const float4*>(g + i));
  float4 v;
  v.x = (i + 0 < n) ? __ldg(g + i + 0) : 0.0f;
  v.y = (i + 1 < n) ? __ldg(g + i + 1) : 0.0f;
  v.z = (i + 2 < n) ? __ldg(g + i + 2) : 0.0f;
  v.w = (i + 3 < n) ? __ldg(g + i + 3) : 0.0f;
  return v;
}

// ---- probabilities: one cooperative kernel (pass 1 + water-filling rounds, no host round trip) ----
// Every CTA owns one contiguous chunk.  After each pass all CTAs meet at a grid barrier and each of them
// reduces the per-chunk partials in the same fixed order, so every CTA holds the same state and takes the
// same decision without a broadcast.  Partials are double-buffered: one barrier per pass.
struct EwAcc { double sum; float amax; uint32_t cnt; uint32_t bad; };

template <bool kRound>
__device__ __forceinline__ EwAcc ew_chunk_pass(const EwVec& v, float theta) {
  const bool aligned = (reinterpret_cast<uintptr_t>(v.g) & 15u) == 0;
  const int64_t beg = (int64_t)blockIdx.x * v.chunk;
  const int64_t end = min(v.n, beg + v.chunk);
  EwAcc acc{0.0, 0.0f, 0u, 0u};
  constexpr int kU = 4;
  for (int64_t base = beg + (int64_t)threadIdx.x * 4; base < end; base += (int64_t)kEwThreads * 4 * kU) {
    float4 x[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) {                       // all loads first: kU requests in flight per thread
      const int64_t i = base + (int64_t)u * kEwThreads * 4;
      x[u] = i < end ? load4(v.g, i, end, aligned) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    float fsum = 0.0f;                                   // short fp32 run (<= 16 terms), then into fp64
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const float a[4] = {fabsf(x[u].x), fabsf(x[u].y), fabsf(x[u].z), fabsf(x[u].w)};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (!kRound) {
          fsum += a[j];
          acc.amax = fmaxf(acc.amax, a[j]);
          acc.bad |= !(a[j] <= 3.402823466e38f);         // NaN or Inf
        } else {
          if (a[j] > theta) ++acc.cnt; else fsum += a[j];
        }
      }
    }
    acc.sum += (double)fsum;
  }
  return acc;
}

// block reduction in a fixed order, result valid in every thread
__device__ __forceinline__ EwAcc ew_block_reduce(EwAcc a, double* s_sum, float* s_max, uint32_t* s_cnt, uint32_t* s_bad) {
  a.sum = warp_sum(a.sum); a.amax = warp_max(a.amax); a.cnt = warp_sum(a.cnt);
  a.bad = __any_sync(0xffffffffu, a.bad) ? 1u : 0u;
  const int w = threadIdx.x / kWarp, l = threadIdx.x % kWarp;
  __syncthreads();
  if (l == 0) { s_sum[w] = a.sum; s_max[w] = a.amax; s_cnt[w] = a.cnt; s_bad[w] = a.bad; }
  __syncthreads();
  EwAcc r{0.0, 0.0f, 0u, 0u};
  for (int i = 0; i < kEwThreads / kWarp; ++i) { r.sum += s_sum[i]; r.amax = fmaxf(r.amax, s_max[i]); r.cnt += s_cnt[i]; r.bad |= s_bad[i]; }
  return r;
}

__global__ void __launch_bounds__(kEwThreads) ew_solve_kernel(EwVec v, double s) {
  cg::grid_group grid = cg::this_grid();
  __shared__ double s_sum[kEwThreads / kWarp];
  __shared__ float s_max[kEwThreads / kWarp];
  __shared__ uint32_t s_cnt[kEwThreads / kWarp], s_bad[kEwThreads / kWarp];
  const int nb = gridDim.x;
  // ---- pass 1: ||g||_1, ||g||_inf, non-finite scan ----
  EwAcc mine = ew_block_reduce(ew_chunk_pass<false>(v, 0.0f), s_sum, s_max, s_cnt, s_bad);
  if (threadIdx.x == 0) v.partials[blockIdx.x] = EwPartial{mine.sum, mine.amax, mine.cnt, mine.bad};
  grid.sync();
  EwAcc tot{0.0, 0.0f, 0u, 0u};
  for (int i = threadIdx.x; i < nb; i += kEwThreads) {
    const EwPartial p = v.partials[i];
    tot.sum += p.sum; tot.amax = fmaxf(tot.amax, p.amax); tot.cnt += p.cnt; tot.bad |= p.nonfinite;
  }
  tot = ew_block_reduce(tot, s_sum, s_max, s_cnt, s_bad);
  const double T0 = tot.sum;
  const float amax = tot.amax;
  const bool nonfinite = tot.bad != 0;
  double T = T0, s_cur = s;
  uint32_t n_sat = 0, rounds = 0;
  // atoms with |g| > theta are unbalanced (Definition 1) for the current (T, s_cur); Lemma 3: none if
  // s <= ||g||_1 / ||g||_inf.  The comparison is made in fp32 everywhere so that every kernel agrees on
  // which atoms are saturated.
  float theta = (float)(T0 / s);
  bool done = nonfinite || !(amax > theta);
  // ---- water-filling rounds ----
  while (!done && rounds < kEwMaxRounds) {
    EwPartial* buf = v.partials + (size_t)((rounds & 1) + 1) * nb;
    mine = ew_block_reduce(ew_chunk_pass<true>(v, theta), s_sum, s_max, s_cnt, s_bad);
    if (threadIdx.x == 0) buf[blockIdx.x] = EwPartial{mine.sum, 0.0f, mine.cnt, 0u};
    grid.sync();
    tot = EwAcc{0.0, 0.0f, 0u, 0u};
    for (int i = threadIdx.x; i < nb; i += kEwThreads) { const EwPartial p = buf[i]; tot.sum += p.sum; tot.cnt += p.cnt; }
    tot = ew_block_reduce(tot, s_sum, s_max, s_cnt, s_bad);
    ++rounds;
    if (tot.cnt == n_sat) { done = true; }             // no new saturated atom: (T, s_cur) stand
    else {
      n_sat = tot.cnt; T = tot.sum; s_cur = s - (double)n_sat;
      const float th = (T > 0.0 && s_cur > 0.0) ? (float)(T / s_cur) : 0.0f;
      theta = fminf(theta, th);
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    EwState* st = v.state;
    const bool live = T > 0.0 && s_cur > 0.0 && !nonfinite;
    st->T0 = T0; st->T = T; st->s_cur = s_cur; st->theta = (double)theta; st->theta_f = theta; st->amax = amax;
    st->n_sat = n_sat; st->rounds = rounds; st->done = 1; st->nonfinite = nonfinite ? 1u : 0u;
    st->scale = live ? (float)(s_cur / T) : 0.0f;         // p_i = |g_i| * scale
    st->c = live ? (float)(T / s_cur) : 0.0f;             // weight of kept unsaturated atoms
  }
}

// ---- sampling -----------------------------------------------------------------------------------
__global__ void __launch_bounds__(kEwThreads) ew_sample_kernel(EwVec v, PhiloxKey key, uint32_t kind_step) {
  const EwState* st = v.state;
  const float scale = st->scale;
  const float theta = st->theta_f;
  const bool dead = st->nonfinite != 0;
  const bool aligned = (reinterpret_cast<uintptr_t>(v.g) & 15u) == 0;
  const int64_t tile_base = (int64_t)blockIdx.x * kEwTile;
  uint32_t kept = 0;
#pragma unroll
  for (int it = 0; it < kEwTile / (kEwThreads * 4); ++it) {
    const int64_t i = tile_base + ((int64_t)it * kEwThreads + threadIdx.x) * 4;
    uint32_t nib = 0;
    float4 pv = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < v.n && !dead) {
      const float4 x = load4(v.g, i, v.n, aligned);
      const uint4 wd = atom_block_words((uint64_t)(i >> 2), v.layer, kind_step, key);
      const float a[4] = {fabsf(x.x), fabsf(x.y), fabsf(x.z), fabsf(x.w)};
      const uint32_t ww[4] = {wd.x, wd.y, wd.z, wd.w};
      float p[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        p[j] = (a[j] > theta) ? 1.0f : fminf(a[j] * scale, 1.0f);
        if (i + j < v.n && bernoulli_keep(p[j], ww[j])) nib |= 1u << j;
      }
      pv = make_float4(p[0], p[1], p[2], p[3]);
    }
    if (v.prob_out != nullptr && i < v.n) {
      if (i + 3 < v.n && (reinterpret_cast<uintptr_t>(v.prob_out) & 15u) == 0)
        *reinterpret_cast<float4*>(v.prob_out + i) = pv;
      else {
        const float pp[4] = {pv.x, pv.y, pv.z, pv.w};
        for (int j = 0; j < 4 && i + j < v.n; ++j) v.prob_out[i + j] = pp[j];
      }
    }
    kept += __popc(nib);
    // 8 consecutive lanes hold the 32 bits of one mask word
    uint32_t word = nib << (4 * (threadIdx.x & 7));
    word |= __shfl_xor_sync(0xffffffffu, word, 1);
    word |= __shfl_xor_sync(0xffffffffu, word, 2);
    word |= __shfl_xor_sync(0xffffffffu, word, 4);
    if ((threadIdx.x & 7) == 0) {
      const int64_t widx = (tile_base >> 5) + it * (kEwThreads / 8) + (threadIdx.x >> 3);
      if (widx < v.n_words) v.mask_words[widx] = word;
    }
  }
  __shared__ uint32_t s_cnt[kEwThreads / kWarp];
  kept = warp_sum(kept);
  if (threadIdx.x % kWarp == 0) s_cnt[threadIdx.x / kWarp] = kept;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t t = 0;
    for (int i = 0; i < kEwThreads / kWarp; ++i) t += s_cnt[i];
    v.tile_counts[blockIdx.x] = t;
  }
}

// exclusive scan of tile_counts (in place), k, capacity check, layer header
__global__ void __launch_bounds__(1024) ew_scan_kernel(EwVec v) {
  __shared__ uint32_t s_warp[32];
  __shared__ uint64_t s_carry;
  if (threadIdx.x == 0) s_carry = 0;
  __syncthreads();
  const int lane = threadIdx.x % kWarp, w = threadIdx.x / kWarp;
  for (int64_t base = 0; base < v.n_tiles; base += 1024) {
    const int64_t i = base + threadIdx.x;
    const uint32_t c = i < v.n_tiles ? v.tile_counts[i] : 0u;
    uint32_t inc = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += t; }
    if (lane == 31) s_warp[w] = inc;
    __syncthreads();
    if (w == 0) {
      uint32_t x = s_warp[lane], y = x;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(0xffffffffu, y, o); if (lane >= o) y += t; }
      s_warp[lane] = y - x;                          // exclusive over warps
    }
    __syncthreads();
    const uint64_t carry = s_carry;
    const uint64_t excl = carry + s_warp[w] + inc - c;
    if (i < v.n_tiles) { v.tile_offsets[i] = excl; v.tile_table[i] = (uint32_t)min(excl, (uint64_t)0xFFFFFFFFull); }
    __syncthreads();
    if (threadIdx.x == 1023) s_carry = excl + c;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const uint64_t k = s_carry;
    const EwState* st = v.state;
    atomo_layer_header* h = v.hdr;
    h->n_sat = st->n_sat; h->c = st->c; h->l1 = st->T0; h->sweeps = st->rounds;
    uint32_t status = ATOMO_OK;
    if (st->nonfinite) status = ATOMO_ERR_NONFINITE;
    else if (k > (uint64_t)v.k_cap) status = ATOMO_ERR_CAPACITY;
    h->status = status;
    h->k = status == ATOMO_OK ? (uint32_t)k : 0u;
    v.tile_table[v.n_tiles] = status == ATOMO_OK ? (uint32_t)k : 0u;
  }
}

// ordered compaction of one tile: indices ascending, value = g_i / p_i
__global__ void __launch_bounds__(kEwThreads) ew_pack_kernel(EwVec v) {
  if (v.hdr->status != ATOMO_OK) return;
  __shared__ uint32_t s_idx[kEwTile];
  __shared__ uint32_t s_woff[kEwTile / 32 + 1];
  __shared__ uint32_t s_wsum[kEwThreads / kWarp];
  const int64_t tile_base = (int64_t)blockIdx.x * kEwTile;
  const int64_t wbase = tile_base >> 5;
  const int t = threadIdx.x, lane = t % kWarp, w = t / kWarp;
  uint32_t word = 0;
  if (t < kEwTile / 32 && wbase + t < v.n_words) word = v.mask_words[wbase + t];
  const uint32_t pc = __popc(word);
  uint32_t inc = pc;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) { const uint32_t x = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += x; }
  if (lane == 31) s_wsum[w] = inc;
  __syncthreads();
  uint32_t woff = inc - pc;
  for (int i = 0; i < w; ++i) woff += s_wsum[i];
  if (t < kEwTile / 32) {
    uint32_t m = word, o = woff;
    while (m) { const int b = __ffs(m) - 1; m &= m - 1; s_idx[o++] = (uint32_t)(t * 32 + b); }
  }
  if (t == kEwTile / 32 - 1) s_woff[0] = woff + pc;     // tile count
  __syncthreads();
  const uint32_t cnt = s_woff[0];
  const uint64_t out0 = v.tile_offsets[blockIdx.x];
  const EwState* st = v.state;
  const float theta = st->theta_f;
  const float c = st->c;
  for (uint32_t j = t; j < cnt; j += kEwThreads) {
    const int64_t i = tile_base + s_idx[j];
    const float g = __ldg(v.g + i);
    // kept atom: saturated (p = 1) keeps g; otherwise g / p = sign(g) * T / (s - n_s)
    const float val = (fabsf(g) > theta) ? g : copysignf(c, g);
    v.idx[out0 + j] = (uint32_t)i;
    v.val[out0 + j] = val;
  }
}

// ---- decode -------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t lower_bound_u32(const uint32_t* __restrict__ a, uint32_t n, uint64_t key) {
  uint32_t lo = 0, hi = n;
  while (lo < hi) { const uint32_t mid = (lo + hi) >> 1; if ((uint64_t)__ldg(a + mid) < key) lo = mid + 1; else hi = mid; }
  return lo;
}

__global__ void __launch_bounds__(kEwThreads) ew_decode_kernel(EwDecode d) {
  const atomo_layer_header* h = d.hdr;
  const bool ok = d.ghdr->magic == ATOMO_MAGIC && d.ghdr->kind == ATOMO_KIND_ENTRYWISE &&
                  h->rows == 1 && h->cols == d.n && h->k <= h->k_cap;
  if (!ok && blockIdx.x == 0 && threadIdx.x == 0) raise_status(const_cast<atomo_layer_header*>(h), ATOMO_ERR_PAYLOAD);
  const uint32_t k = ok ? h->k : 0u;
  const uint32_t* idx = reinterpret_cast<const uint32_t*>(d.payload + h->off_idx);
  const float* val = reinterpret_cast<const float*>(d.payload + h->off_val);
  const uint32_t* table = reinterpret_cast<const uint32_t*>(d.payload + h->off_short);   // kept atoms before each tile
  const int64_t n_tiles = (d.n + kEwTile - 1) / kEwTile;
  const bool vec = (reinterpret_cast<uintptr_t>(d.out) & 15u) == 0;
  // a CTA walks over tiles: zero-fill with vector stores, barrier, then the tile's few kept values
  for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const int64_t tile_base = tile * kEwTile;
    float* out = d.out + tile_base;
    const int64_t left = d.n - tile_base;
    if (left >= kEwTile && vec) {
#pragma unroll
      for (int i = 0; i < kEwTile / 4 / kEwThreads; ++i)
        reinterpret_cast<float4*>(out)[threadIdx.x + i * kEwThreads] = make_float4(0.f, 0.f, 0.f, 0.f);
    } else {
      for (int i = threadIdx.x; i < kEwTile && i < left; i += kEwThreads) out[i] = 0.0f;
    }
    uint32_t lo = 0, hi = 0;
    if (k) { lo = min(__ldg(table + tile), k); hi = min(__ldg(table + tile + 1), k); }
    __syncthreads();                                     // zeros are ordered before the values below
    for (uint32_t j = lo + threadIdx.x; j < hi; j += kEwThreads) {
      const uint32_t i = __ldg(idx + j);
      if ((int64_t)i >= tile_base && (int64_t)i < tile_base + kEwTile && (int64_t)i < d.n) d.out[i] = __ldg(val + j);
    }
  }
}

// ---- host-side launchers --------------------------------------------------------------------------
int ew_solve_max_blocks() {
  int dev = 0, sms = 0, per_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ew_solve_kernel, kEwThreads, 0) != cudaSuccess) return 0;
  return sms * per_sm;
}

int launch_ew_solve(const EwVec& v, double s, cudaStream_t st) {
  EwVec vv = v; double ss = s;
  void* args[] = {&vv, &ss};
  return (int)cudaLaunchCooperativeKernel((const void*)ew_solve_kernel, dim3(v.n_chunks), dim3(kEwThreads), args, 0, st);
}
void launch_ew_sample_pack(const EwVec& v, PhiloxKey key, uint32_t kind_step, cudaStream_t st) {
  ew_sample_kernel<<<(unsigned)v.n_tiles, kEwThreads, 0, st>>>(v, key, kind_step);
  ew_scan_kernel<<<1, 1024, 0, st>>>(v);
  ew_pack_kernel<<<(unsigned)v.n_tiles, kEwThreads, 0, st>>>(v);
}
void launch_ew_decode(const EwDecode& d, cudaStream_t st) {
  const int64_t tiles = (d.n + kEwTile - 1) / kEwTile;
  ew_decode_kernel<<<(unsigned)std::min<int64_t>(tiles, 148 * 16), kEwThreads, 0, st>>>(d);
}
int ew_tile_elems() { return kEwTile; }

}  // namespace atomo
