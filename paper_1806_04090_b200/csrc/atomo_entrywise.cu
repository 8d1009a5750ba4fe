// Entry-wise ATOMO on flat gradients: atoms e_i, lambda_i = g_i (Section 3 of the paper; the
// QSGD / TernGrad family of Section 4 are the budgets s = ||g||_1/||g||_2 and ||g||_1/||g||_inf).
//
//   pass 1   ew_reduce(kAll)   : ||g||_1 (fp64 accumulation), ||g||_inf, non-finite scan
//   rounds   ew_reduce(kRound) : water-filling form of Algorithm 1 -- every atom with
//                                |g_i| (s - n_s) > sum_{unsaturated} |g_j| gets p = 1; repeated
//                                until no new atom saturates (zero rounds when g is s-balanced,
//                                Lemma 3)
//   pass 2   ew_sample         : p_i = |g_i| (s-n_s)/T, Philox word, keep bit -> mask words + tile counts
//            ew_scan           : exclusive scan of tile counts, k, capacity check, header
//            ew_pack           : ordered compaction: idx ascending, val = g_i / p_i
//   decode   ew_decode         : zero-fill + scatter, one coalesced write pass
#include "atomo_kernels.cuh"

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

// ---- reductions --------------------------------------------------------------------------------
// mode kAll  : sum over all atoms of |g|, max |g|, non-finite flag
// mode kRound: with theta from the state: count of atoms with |g| > theta, sum of |g| over the rest
template <int kMode>
__global__ void __launch_bounds__(kEwThreads) ew_reduce_kernel(EwVec v) {
  const bool aligned = (reinterpret_cast<uintptr_t>(v.g) & 15u) == 0;
  const int64_t chunk = v.chunk;                    // multiple of 4
  const int64_t beg = (int64_t)blockIdx.x * chunk;
  const int64_t end = min(v.n, beg + chunk);
  double theta = 0.0;
  if (kMode == kEwRound) {
    if (v.state->done) return;
    theta = v.state->theta;
  }
  double dsum = 0.0;
  float amax = 0.0f;
  uint32_t cnt = 0, bad = 0;
  for (int64_t base = beg + (int64_t)threadIdx.x * 4; base < end; base += (int64_t)kEwThreads * 4 * 4) {
    float fsum = 0.0f;                              // short fp32 run (<= 16 terms), then into fp64
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int64_t i = base + (int64_t)u * kEwThreads * 4;
      if (i >= end) break;
      const float4 x = load4(v.g, i, end, aligned);
      const float a[4] = {fabsf(x.x), fabsf(x.y), fabsf(x.z), fabsf(x.w)};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (kMode == kEwAll) {
          fsum += a[j];
          amax = fmaxf(amax, a[j]);
          bad |= !(a[j] <= 3.402823466e38f);        // NaN or Inf
        } else {
          if ((double)a[j] > theta) ++cnt; else fsum += a[j];
        }
      }
    }
    dsum += (double)fsum;
  }
  __shared__ double s_sum[kEwThreads / kWarp];
  __shared__ float s_max[kEwThreads / kWarp];
  __shared__ uint32_t s_cnt[kEwThreads / kWarp], s_bad[kEwThreads / kWarp];
  dsum = warp_sum(dsum); amax = warp_max(amax); cnt = warp_sum(cnt);
  bad = __any_sync(0xffffffffu, bad);
  const int w = threadIdx.x / kWarp, l = threadIdx.x % kWarp;
  if (l == 0) { s_sum[w] = dsum; s_max[w] = amax; s_cnt[w] = cnt; s_bad[w] = bad; }
  __syncthreads();
  if (threadIdx.x == 0) {
    EwPartial p{0.0, 0.0f, 0u, 0u};
    for (int i = 0; i < kEwThreads / kWarp; ++i) {   // fixed order: deterministic
      p.sum += s_sum[i]; p.amax = fmaxf(p.amax, s_max[i]); p.cnt += s_cnt[i]; p.nonfinite |= s_bad[i];
    }
    v.partials[blockIdx.x] = p;
  }
}

template <int kMode>
__global__ void __launch_bounds__(kEwThreads) ew_finalize_kernel(EwVec v, double s) {
  EwState* st = v.state;
  if (kMode == kEwRound && st->done) return;
  double dsum = 0.0; float amax = 0.0f; uint32_t cnt = 0, bad = 0;
  for (int i = threadIdx.x; i < v.n_chunks; i += kEwThreads) {
    const EwPartial p = v.partials[i];
    dsum += p.sum; amax = fmaxf(amax, p.amax); cnt += p.cnt; bad |= p.nonfinite;
  }
  __shared__ double s_sum[kEwThreads]; __shared__ float s_max[kEwThreads];
  __shared__ uint32_t s_cnt[kEwThreads], s_bad[kEwThreads];
  s_sum[threadIdx.x] = dsum; s_max[threadIdx.x] = amax; s_cnt[threadIdx.x] = cnt; s_bad[threadIdx.x] = bad;
  __syncthreads();
  for (int o = kEwThreads / 2; o > 0; o >>= 1) {     // fixed tree: deterministic
    if (threadIdx.x < o) {
      s_sum[threadIdx.x] += s_sum[threadIdx.x + o];
      s_max[threadIdx.x] = fmaxf(s_max[threadIdx.x], s_max[threadIdx.x + o]);
      s_cnt[threadIdx.x] += s_cnt[threadIdx.x + o];
      s_bad[threadIdx.x] |= s_bad[threadIdx.x + o];
    }
    __syncthreads();
  }
  if (threadIdx.x != 0) return;
  if (kMode == kEwAll) {
    st->T0 = s_sum[0]; st->T = s_sum[0]; st->s_cur = s; st->amax = s_max[0];
    st->n_sat = 0; st->rounds = 0; st->nonfinite = s_bad[0];
    st->theta = s_sum[0] / s;
    // Lemma 3: s-balanced iff s <= ||g||_1 / ||g||_inf  -> no atom saturates
    st->done = (s_bad[0] != 0) || !((double)s_max[0] > st->theta);
  } else {
    const uint32_t n_sat = s_cnt[0];
    const double T = s_sum[0];
    const double s_cur = s - (double)n_sat;
    st->rounds += 1;
    if (n_sat == st->n_sat) { st->done = 1; }         // no new saturated atom: (T, s_cur) unchanged
    else {
      st->n_sat = n_sat; st->T = T; st->s_cur = s_cur;
      const double th = (T > 0.0 && s_cur > 0.0) ? T / s_cur : 0.0;
      st->theta = fmin(st->theta, th);
      if (st->rounds >= kEwMaxRounds) st->done = 1;
    }
  }
  if (st->done) {
    const bool live = st->T > 0.0 && st->s_cur > 0.0 && !st->nonfinite;
    st->scale = live ? (float)(st->s_cur / st->T) : 0.0f;   // p_i = |g_i| * scale
    st->c = live ? (float)(st->T / st->s_cur) : 0.0f;       // weight of kept unsaturated atoms
    st->theta_f = (float)st->theta;
  }
}

// ---- sampling -----------------------------------------------------------------------------------
__global__ void __launch_bounds__(kEwThreads) ew_sample_kernel(EwVec v, PhiloxKey key, uint32_t kind_step) {
  const EwState* st = v.state;
  const float scale = st->scale;
  const double theta = st->theta;
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
        p[j] = ((double)a[j] > theta) ? 1.0f : fminf(a[j] * scale, 1.0f);
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
    if (i < v.n_tiles) v.tile_offsets[i] = excl;
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
  const double theta = st->theta;
  const float c = st->c;
  for (uint32_t j = t; j < cnt; j += kEwThreads) {
    const int64_t i = tile_base + s_idx[j];
    const float g = __ldg(v.g + i);
    // kept atom: saturated (p = 1) keeps g; otherwise g / p = sign(g) * T / (s - n_s)
    const float val = ((double)fabsf(g) > theta) ? g : copysignf(c, g);
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
  __shared__ __align__(16) float s_out[kEwTile];
  __shared__ uint32_t s_range[2];
  const atomo_layer_header* h = d.hdr;
  const bool ok = d.ghdr->magic == ATOMO_MAGIC && d.ghdr->kind == ATOMO_KIND_ENTRYWISE &&
                  h->rows == 1 && h->cols == d.n && h->k <= h->k_cap;
  const int64_t tile_base = (int64_t)blockIdx.x * kEwTile;
  for (int i = threadIdx.x; i < kEwTile; i += kEwThreads) s_out[i] = 0.0f;
  const uint32_t k = ok ? h->k : 0u;
  if (!ok && blockIdx.x == 0 && threadIdx.x == 0) raise_status(const_cast<atomo_layer_header*>(h), ATOMO_ERR_PAYLOAD);
  const uint32_t* idx = reinterpret_cast<const uint32_t*>(d.payload + h->off_idx);
  const float* val = reinterpret_cast<const float*>(d.payload + h->off_val);
  if (threadIdx.x < 2 && k) s_range[threadIdx.x] = lower_bound_u32(idx, k, (uint64_t)tile_base + (threadIdx.x ? kEwTile : 0));
  __syncthreads();
  if (k) {
    const uint32_t lo = s_range[0], hi = s_range[1];
    for (uint32_t j = lo + threadIdx.x; j < hi; j += kEwThreads) {
      const uint32_t i = __ldg(idx + j);
      s_out[i - (uint32_t)tile_base] = __ldg(val + j);   // idx < 2^32 and inside this tile
    }
  }
  __syncthreads();
  float* out = d.out + tile_base;
  const int64_t left = d.n - tile_base;
  if (left >= kEwTile && (reinterpret_cast<uintptr_t>(out) & 15u) == 0) {
    for (int i = threadIdx.x; i < kEwTile / 4; i += kEwThreads)
      reinterpret_cast<float4*>(out)[i] = reinterpret_cast<const float4*>(s_out)[i];
  } else {
    for (int i = threadIdx.x; i < kEwTile && i < left; i += kEwThreads) out[i] = s_out[i];
  }
}

// ---- host-side launchers --------------------------------------------------------------------------
void launch_ew_reduce_all(const EwVec& v, double s, cudaStream_t st) {
  ew_reduce_kernel<kEwAll><<<v.n_chunks, kEwThreads, 0, st>>>(v);
  ew_finalize_kernel<kEwAll><<<1, kEwThreads, 0, st>>>(v, s);
}
void launch_ew_round(const EwVec& v, double s, cudaStream_t st) {
  ew_reduce_kernel<kEwRound><<<v.n_chunks, kEwThreads, 0, st>>>(v);
  ew_finalize_kernel<kEwRound><<<1, kEwThreads, 0, st>>>(v, s);
}
void launch_ew_sample_pack(const EwVec& v, PhiloxKey key, uint32_t kind_step, cudaStream_t st) {
  ew_sample_kernel<<<(unsigned)v.n_tiles, kEwThreads, 0, st>>>(v, key, kind_step);
  ew_scan_kernel<<<1, 1024, 0, st>>>(v);
  ew_pack_kernel<<<(unsigned)v.n_tiles, kEwThreads, 0, st>>>(v);
}
void launch_ew_decode(const EwDecode& d, cudaStream_t st) {
  const int64_t tiles = (d.n + kEwTile - 1) / kEwTile;
  ew_decode_kernel<<<(unsigned)tiles, kEwThreads, 0, st>>>(d);
}
int ew_tile_elems() { return kEwTile; }

}  // namespace atomo
