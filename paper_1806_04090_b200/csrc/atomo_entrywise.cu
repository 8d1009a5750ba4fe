// Entry-wise ATOMO on flat gradients: atoms e_i, lambda_i = g_i (Section 3 of the paper; the
// QSGD / TernGrad family of Section 4 are the budgets s = ||g||_1/||g||_2 and ||g||_1/||g||_inf).
//
//   ew_solve (cooperative)     : pass 1: ||g||_1 (fp64 accumulation), ||g||_inf, non-finite scan; then the
//                                water-filling form of Algorithm 1 -- every atom with
//                                |g_i| (s - n_s) > sum_{unsaturated} |g_j| gets p = 1; repeated
//                                until no new atom saturates (zero rounds when g is s-balanced,
//                                Lemma 3); grid barriers instead of host round trips
//   pass 2   ew_sample_pack    : per chunk of tiles: p_i = |g_i| (s-n_s)/T, Philox word, keep bit -> mask words
//                                and counts; the counts of the earlier chunks are added (one bounded wait, no
//                                chain); ordered compaction from the mask words: idx ascending, val = g_i / p_i;
//                                the last chunk writes k, the capacity check and the header.  Compact format
//                                (the ternary form of Section 4): a kept atom with p < 1 weighs sign(g_i) c, so
//                                it travels as a 16-bit entry (index inside its tile, sign bit); the atoms with
//                                p = 1 keep (idx, val) in a list of their own
//   decode   ew_decode         : zero-fill with vector stores, then the tile's kept values (per-tile
//                                offsets travel in the payload), either format
#include <algorithm>

#include <cooperative_groups.h>

#include "atomo_kernels.cuh"

namespace cg = cooperative_groups;

// development builds (-DEW_PROFILE) print the phase times of a few CTAs of the one-kernel form
#ifdef EW_PROFILE
#include <cstdio>
__device__ __forceinline__ unsigned long long ew_now() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#define EW_STAMP(k) if (threadIdx.x == 0) ew_t[k] = ew_now();
#else
#define EW_STAMP(k)
#endif

namespace atomo {

constexpr int kEwThreads = 256;
constexpr int kEwTile = 4096;                 // elements per tile of the sample / pack / decode passes
#ifndef EW_MIN_BLOCKS
#define EW_MIN_BLOCKS 5
#endif
constexpr int kEwMinBlocks = EW_MIN_BLOCKS;   // resident CTAs per SM the sample / pack kernel is compiled for
#ifndef EW_ENCODE_BLOCKS
#define EW_ENCODE_BLOCKS 4
#endif
constexpr int kEwEncodeBlocks = EW_ENCODE_BLOCKS;   // ... and the one-kernel form (64 registers: two tiles' loads per thread)

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
__device__ __forceinline__ EwAcc ew_chunk_pass(const EwVec& v, float theta, const int64_t beg, const int64_t end) {
  const bool aligned = (reinterpret_cast<uintptr_t>(v.g) & 15u) == 0;
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

// ---- the first pass of the one-kernel form, with a list of candidates --------------------------------------------
// The keep decision of an atom needs ||g||_1, which only the end of the first pass knows; but the Philox word of an
// atom depends on its index alone.  So the first pass already draws the words and keeps a list of the few atoms that
// can still be kept: an atom is kept (Eq. 2 with p < 1) iff word < floor(|g| scale 2^32), and the pass tests
// word <= |g| M with M = 1.25 scale_est 2^32, where scale_est comes from the sum over the chunk's first tile, scaled to
// the vector's length.  A thread keeps its candidates (index, value) in slots of its own, so the list needs neither
// atomics nor votes.  After the grid barrier the true scale is known.  If M >= scale 2^32 (1 + 2^-22) (the slack
// covers the roundings of both products), the vector is s-balanced (no atom with p = 1) and no thread ran out of
// slots, the list holds every kept atom of the chunk and the exact decision is taken on its entries alone (their
// words are drawn again): the chunk is read once.  Otherwise the CTA reads its chunk a second time as the two-kernel form does.  Either way
// the decision is the same integer comparison on the same operands, so the payload does not depend on which way a
// chunk went.  The sums are formed exactly as in ew_chunk_pass (same terms per thread, same order).
constexpr int kEwCandPerThread = 16;             // list entries per thread; 1.25 s (atoms per thread) / n are expected
constexpr int kEwCandSlots = (kEwCandPerThread + 1) * kEwThreads;   // one more row takes what does not fit (never read)
struct EwCands {
  uint32_t* idx;      // [kEwCandPerThread + 1][kEwThreads] atom index inside the chunk, then (same layout) its gradient entry
  uint32_t* stop;     // set by the first thread that runs out of slots: the CTA stops listing
  float m32;          // the multiplier M the list was made with (0: no list)
  uint32_t addr;      // shared-memory address of this thread's next slot: rows of kEwThreads 4-byte entries
  uint32_t addr0;     // ... of its first slot
};
__device__ __forceinline__ uint32_t ew_cand_count(const EwCands& C) { return (C.addr - C.addr0) / (4u * kEwThreads); }

// One tile of the pass: 16 atoms per thread (float4 number tid + 256 u of the tile, u = 0 .. 3).  local0: index of
// x[0].x inside the chunk; blk0: its Philox block (atom index / 4); left: elements of the chunk from x[0].x on
// (FULL: the whole tile lies inside the chunk).  amax ignores NaN (and the sum keeps it), so "some entry is NaN" is
// "the sum is NaN" and "some entry is infinite" is "amax is infinite": no test per entry.
template <bool FULL>
__device__ __forceinline__ void ew_cand_tile(const float4 (&x)[4], const uint32_t local0, const uint32_t blk0, const int64_t left,
                                             const uint32_t layer, const PhiloxKey key, const uint32_t kind_step,
                                             const bool listing, float& fsum, float& amax, EwCands& C) {
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const float a[4] = {fabsf(x[u].x), fabsf(x[u].y), fabsf(x[u].z), fabsf(x[u].w)};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      fsum += a[j];
      amax = fmaxf(amax, a[j]);
    }
  }
  if (!listing) return;
  const float m32 = C.m32;
  const uint32_t spill = C.addr0 + (uint32_t)(kEwCandPerThread * kEwThreads * 4);   // this thread's slot in the extra row
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    if (!FULL && (int64_t)u * kEwThreads * 4 >= left) continue;
    const uint4 wd = philox4x32_10(make_uint4(blk0 + (uint32_t)(u * kEwThreads), 0u, layer, kind_step), key);
    const float gg[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
    const uint32_t ww[4] = {wd.x, wd.y, wd.z, wd.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      // candidate: two predicated stores (index, value) to the thread's next slot and the slot moves on; no branch
      const uint32_t o = min(C.addr, spill);
      const uint32_t li = local0 + (uint32_t)(u * kEwThreads * 4 + j);
      asm volatile(
          "{\n\t.reg .pred p;\n\t.reg .f32 t, wf;\n\t"
          "cvt.rz.f32.u32 wf, %3;\n\t"
          "abs.f32 t, %2;\n\t"
          "mul.f32 t, t, %4;\n\t"
          "setp.ge.f32 p, t, wf;\n\t"
          "@p st.shared.u32 [%1], %5;\n\t"
          "@p st.shared.f32 [%1 + %6], %2;\n\t"
          "@p add.u32 %0, %0, %7;\n\t}"
          : "+r"(C.addr)
          : "r"(o), "f"(gg[j]), "r"(ww[j]), "f"(m32), "r"(li), "n"(kEwCandSlots * 4), "n"(kEwThreads * 4)
          : "memory");
    }
  }
  if (C.addr > spill) *(volatile uint32_t*)C.stop = 1u;    // more candidates than slots: this chunk will be read twice
}

__device__ __forceinline__ EwAcc ew_chunk_pass_cand(const EwVec& v, const PhiloxKey key, const uint32_t kind_step, const double s,
                                                    const int64_t beg, const int64_t end, const int n_my, EwCands& C,
                                                    float* s_red) {
  const bool aligned = (reinterpret_cast<uintptr_t>(v.g) & 15u) == 0;
  const int tid = threadIdx.x, lane = tid % kWarp, w = tid / kWarp;
  constexpr int kU = 4;
  double sum = 0.0;
  float amax = 0.0f;
  C.m32 = 0.0f; C.addr = C.addr0;
  // tiles that lie inside the chunk and can be read with 16-byte loads; the next tile's loads are issued before this
  // tile's words are drawn, so a warp always has requests in flight
  const int n_full = aligned ? (int)((end - beg) / kEwTile) : 0;
  auto load_tile = [&](int tl, float4 (&x)[kU]) {
    const int64_t base = beg + (int64_t)tl * kEwTile + (int64_t)tid * 4;
    if (tl < n_full) {
#pragma unroll
      for (int u = 0; u < kU; ++u) x[u] = __ldg(reinterpret_cast<const float4*>(v.g + base) + u * kEwThreads);
    } else {
#pragma unroll
      for (int u = 0; u < kU; ++u) {
        const int64_t i = base + (int64_t)u * kEwThreads * 4;
        x[u] = i < end ? load4(v.g, i, end, aligned) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
  };
  // one tile: its sums, and its candidates while the CTA is still listing
  auto do_tile = [&](int tl, const float4 (&x)[kU]) {
    const uint32_t local0 = (uint32_t)(tl * kEwTile + tid * 4);
    const uint32_t blk0 = (uint32_t)(beg >> 2) + (uint32_t)(tl * (kEwTile / 4) + tid);
    float fsum = 0.0f;                                     // short fp32 run (16 terms), then into fp64: as in ew_chunk_pass
    if (tl == 0) {                                         // the estimate: this tile's sum, scaled to the vector
      ew_cand_tile<false>(x, local0, blk0, 0, v.layer, key, kind_step, false, fsum, amax, C);
      const float ws = warp_sum(fsum);
      if (lane == 0) s_red[w] = ws;
      __syncthreads();
      float ts = 0.0f;
      for (int i2 = 0; i2 < kEwThreads / kWarp; ++i2) ts += s_red[i2];
      const double in_tile = (double)min((int64_t)kEwTile, end - beg);
      // M = 1.25 (s / l1_est) 2^32 with l1_est = ts n / in_tile.  A zero or non-finite ts gives inf or NaN: the threads'
      // lists overflow or stay empty and the check after the barrier sends the chunk the other way.  No list either
      // where a thread would expect more than a quarter of its slots to fill (budgets above about 1.5 % of the length:
      // the list would cost more than the second read)
      float m32 = (float)(1.25 * s * in_tile * 4294967296.0 / ((double)ts * (double)v.n));
      const double expect = 1.25 * s * (double)(end - beg) / ((double)v.n * kEwThreads);
      if (!(m32 > 0.0f) || expect > 0.25 * kEwCandPerThread) m32 = 0.0f;
      C.m32 = m32;
      float f2 = 0.0f, u2 = 0.0f;                          // the tile again, for its candidates (sums discarded)
      if (m32 != 0.0f) ew_cand_tile<false>(x, local0, blk0, end - beg - (int64_t)local0, v.layer, key, kind_step, true, f2, u2, C);
    } else {
      const bool listing = C.m32 != 0.0f && *(volatile uint32_t*)C.stop == 0u;
      if (tl < n_full) ew_cand_tile<true>(x, local0, blk0, 0, v.layer, key, kind_step, listing, fsum, amax, C);
      else ew_cand_tile<false>(x, local0, blk0, end - beg - (int64_t)local0, v.layer, key, kind_step, listing, fsum, amax, C);
    }
    sum += (double)fsum;
  };
  float4 x[kU], xn[kU];
  load_tile(0, x);
  for (int tl = 0; tl < n_my; ++tl) {
    if (tl + 1 < n_my) load_tile(tl + 1, xn);
    do_tile(tl, x);
#pragma unroll
    for (int u = 0; u < kU; ++u) x[u] = xn[u];
  }
  EwAcc acc;
  acc.sum = sum; acc.cnt = 0u; acc.amax = amax;
  acc.bad = (!(sum == sum) || !(amax <= 3.402823466e38f)) ? 1u : 0u;   // an entry is NaN or infinite
  return acc;
}

// what the probability solve leaves for the sampling pass (every CTA computes the same values)
struct EwSolved { double T0; float scale, theta, c; uint32_t n_sat, rounds; bool nonfinite; };

// The solve over this CTA's elements [beg, end) (a multiple of 4 from the start of the vector); all CTAs of the grid
// call it together (cooperative launch).  `first`: the sums of the first pass, if the caller has made it already.
__device__ __forceinline__ EwSolved ew_solve_body(const EwVec& v, const double s, const int64_t beg, const int64_t end,
                                                  const EwAcc* first = nullptr) {
  cg::grid_group grid = cg::this_grid();
  __shared__ double s_sum[kEwThreads / kWarp];
  __shared__ float s_max[kEwThreads / kWarp];
  __shared__ uint32_t s_cnt[kEwThreads / kWarp], s_bad[kEwThreads / kWarp];
  const int nb = gridDim.x;
  // ---- pass 1: ||g||_1, ||g||_inf, non-finite scan ----
  EwAcc mine = ew_block_reduce(first != nullptr ? *first : ew_chunk_pass<false>(v, 0.0f, beg, end), s_sum, s_max, s_cnt, s_bad);
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
    mine = ew_block_reduce(ew_chunk_pass<true>(v, theta, beg, end), s_sum, s_max, s_cnt, s_bad);
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
  const bool live = T > 0.0 && s_cur > 0.0 && !nonfinite;
  EwSolved r;
  r.T0 = T0; r.theta = theta; r.n_sat = n_sat; r.rounds = rounds; r.nonfinite = nonfinite;
  r.scale = live ? (float)(s_cur / T) : 0.0f;            // p_i = |g_i| * scale
  r.c = live ? (float)(T / s_cur) : 0.0f;                // weight of kept unsaturated atoms
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    EwState* st = v.state;
    st->T0 = T0; st->T = T; st->s_cur = s_cur; st->theta = (double)theta; st->theta_f = theta; st->amax = amax;
    st->n_sat = n_sat; st->rounds = rounds; st->done = 1; st->nonfinite = nonfinite ? 1u : 0u;
    st->scale = r.scale; st->c = r.c;
  }
  return r;
}

__global__ void __launch_bounds__(kEwThreads) ew_solve_kernel(EwVec v, double s) {
  const int64_t beg = (int64_t)blockIdx.x * v.chunk;
  ew_solve_body(v, s, beg, min(v.n, beg + v.chunk));
}

// ---- sampling + ordered compaction, one kernel -----------------------------------------------------
// A CTA takes the next chunk of consecutive tiles (the tiles are spread evenly over the chunks) (a ticket, so that every chunk it will wait for
// is already running).  Phase 1: the keep bit of every atom of the chunk (Eq. 2: p_i = 1 on the saturated set,
// |g_i| (s - n_s) / T elsewhere; Philox word against floor(p 2^32)); mask words go to shared memory (and to the
// mask output), kept atoms are counted per tile.  The chunk's count is published; the CTA then waits (bounded)
// until every earlier chunk has published and adds their counts -- all chunks of a wave finish phase 1 together,
// so nobody waits on a chain.  Phase 2: ordered compaction of the chunk from the mask words in shared memory;
// only the kept atoms' values are read again (they are still in L2).  The last chunk writes k, the capacity
// check and the layer header.  A wait that runs out raises ATOMO_ERR_TIMEOUT in the layer header.
constexpr uint64_t kFlagReady = 1ull << 63;
constexpr uint32_t kChunkSpinLimit = 1u << 20;
constexpr int kEwMaxTilesPerCta = 64;
constexpr int kEwWordsPerTile = kEwTile / 32;

// Phase 1 of the sample / pack kernel over the chunk's tiles: keep bits into the mask words, kept atoms counted per
// tile.  A thread takes 16 consecutive atoms of a tile (four Philox blocks), so two neighbouring lanes hold a mask
// word between them.  SAT also records which kept atoms are saturated (a second mask and count; the compact format
// of a vector that is not s-balanced needs them); UNBAL: the vector is not s-balanced, so some atoms have p = 1 (an
// s-balanced vector, Lemma 3, skips that test); FULL: the tile lies inside the vector and is 16-byte aligned;
// PROB: the probabilities are wanted too (debug output).  The tiles are taken from the chunk's last to its first:
// the reduction kernel read them in ascending order just before, so the end of the chunk is what the L2 still holds.
template <bool SAT, bool UNBAL, bool FULL, bool PROB>
__device__ __forceinline__ void ew_tile_bits(const EwVec& v, const PhiloxKey key, const uint32_t kind_step, const uint32_t tile,
                                             const float scale, const float scale32, const float theta, const bool dead,
                                             const bool aligned, uint32_t& nb_out, uint32_t& sb_out) {
  const int tid = threadIdx.x;
  const int64_t i0 = (int64_t)tile * kEwTile + 16 * tid;
  float4 x[4];
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    const int64_t i = i0 + 4 * it;
    x[it] = FULL ? __ldg(reinterpret_cast<const float4*>(v.g + i))
                 : (i < v.n ? load4(v.g, i, v.n, aligned) : make_float4(0.f, 0.f, 0.f, 0.f));
  }
  uint32_t nb = 0, sb = 0;
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    // block of 4 atoms = atom >> 2 < 2^30 (n < 2^32): the high counter word is zero
    const uint4 wd = philox4x32_10(make_uint4(tile * (uint32_t)(kEwTile / 4) + (uint32_t)(4 * tid + it), 0u, v.layer, kind_step), key);
    const float a[4] = {fabsf(x[it].x), fabsf(x[it].y), fabsf(x[it].z), fabsf(x[it].w)};
    const uint32_t ww[4] = {wd.x, wd.y, wd.z, wd.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      // p = 1 if saturated, else min(a scale, 1); keep iff p >= 1 or word < floor(p 2^32).  a scale32 is the
      // same product times 2^32 (exact), and the truncating conversion gives the floor.
      const float t = a[j] * scale32;
      const bool sat = UNBAL && a[j] > theta;
      bool keep = sat || t >= 4294967296.0f || ww[j] < __float2uint_rz(t);
      if (!FULL) keep = keep && i0 + 4 * it + j < v.n;
      if (keep) { nb |= 1u << (4 * it + j); if (SAT && sat) sb |= 1u << (4 * it + j); }
    }
    if (PROB) {
      const int64_t i = i0 + 4 * it;
      if (i < v.n) {
        float pp[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) pp[j] = dead ? 0.0f : ((a[j] > theta) ? 1.0f : fminf(a[j] * scale, 1.0f));
        if (i + 3 < v.n && (reinterpret_cast<uintptr_t>(v.prob_out) & 15u) == 0)
          *reinterpret_cast<float4*>(v.prob_out + i) = make_float4(pp[0], pp[1], pp[2], pp[3]);
        else
          for (int j = 0; j < 4 && i + j < v.n; ++j) v.prob_out[i + j] = pp[j];
      }
    }
  }
  if (dead) { nb = 0; sb = 0; }
  nb_out = nb; sb_out = sb;
}

template <bool SAT, bool UNBAL>
__device__ __forceinline__ void ew_keep_bits(const EwVec& v, const PhiloxKey key, const uint32_t kind_step,
                                             const int64_t tile0, const int n_my, const float scale, const float theta,
                                             const bool dead, const bool aligned, uint32_t* s_mask, uint32_t* s_sat,
                                             uint32_t* s_tcnt, uint32_t* s_tsat) {
  const int tid = threadIdx.x, lane = tid % kWarp;
  const float scale32 = scale * 4294967296.0f;    // exact: a power-of-two factor
  for (int tl = n_my - 1; tl >= 0; --tl) {
    const uint32_t tile = (uint32_t)(tile0 + tl);
    const int64_t tile_base = (int64_t)tile * kEwTile;
    const bool full = aligned && tile_base + kEwTile <= v.n;
    uint32_t nb, sb;
    if (v.prob_out != nullptr) ew_tile_bits<SAT, UNBAL, false, true>(v, key, kind_step, tile, scale, scale32, theta, dead, aligned, nb, sb);
    else if (full) ew_tile_bits<SAT, UNBAL, true, false>(v, key, kind_step, tile, scale, scale32, theta, dead, aligned, nb, sb);
    else ew_tile_bits<SAT, UNBAL, false, false>(v, key, kind_step, tile, scale, scale32, theta, dead, aligned, nb, sb);
    // two neighbouring lanes hold the 32 bits of one mask word; the even lane stores it
    const uint32_t other = __shfl_xor_sync(0xffffffffu, nb, 1);
    const uint32_t word = nb | (other << 16);
    uint32_t sword = 0;
    if (SAT) sword = sb | (__shfl_xor_sync(0xffffffffu, sb, 1) << 16);
    uint32_t kept = 0, kept_sat = 0;
    if ((lane & 1) == 0) {
      const int wl = tid >> 1;
      s_mask[tl * kEwWordsPerTile + wl] = word;
      if (SAT) s_sat[tl * kEwWordsPerTile + wl] = sword;
      const int64_t widx = (tile_base >> 5) + wl;
      if (widx < v.n_words) v.mask_words[widx] = word;
      kept = __popc(word);
      if (SAT) kept_sat = __popc(sword);
    }
    kept = warp_sum(kept);
    if (lane == 0 && kept) atomicAdd(&s_tcnt[tl], kept);
    if (SAT) {
      kept_sat = warp_sum(kept_sat);
      if (lane == 0 && kept_sat) atomicAdd(&s_tsat[tl], kept_sat);
    }
  }
}

// COMPACT: the payload takes, per kept atom with p < 1, a 16-bit entry (index inside the tile, sign bit) and, per
// atom with p = 1, index and value in a list of its own; both ascending.  The chunk's status word then carries the
// saturated count in bits 32..62 beside the total, and the kernel keeps a second bit mask (saturated and kept).
template <bool COMPACT>
__device__ __forceinline__ void ew_sample_pack_chunk(const EwVec& v, const PhiloxKey key, const uint32_t kind_step,
                                                     const uint32_t chunk, const EwSolved& S, uint32_t* s_mask,
                                                     const EwCands* cands = nullptr
#ifdef EW_PROFILE
                                                     , unsigned long long* ew_t = nullptr
#endif
                                                     ) {
  constexpr int kWarps = kEwThreads / kWarp;
  __shared__ uint32_t s_tcnt[kEwMaxTilesPerCta];  // kept atoms per tile, then their exclusive prefix
  __shared__ uint32_t s_tsat[kEwMaxTilesPerCta];  // the same for the saturated kept atoms (COMPACT)
  __shared__ uint32_t s_chunk, s_chunk_sat;
  __shared__ unsigned long long s_base;           // kept atoms before this chunk (COMPACT: saturated ones in bits 32..62)
  __shared__ int s_fail;
  const float scale = S.scale, theta = S.theta, c = S.c;
  const bool dead = S.nonfinite;
  const bool any_sat = COMPACT && S.n_sat != 0;     // an s-balanced vector (Lemma 3) skips the saturated bookkeeping
  const bool aligned = (reinterpret_cast<uintptr_t>(v.g) & 15u) == 0;
  const int tid = threadIdx.x, lane = tid % kWarp, w = tid / kWarp;
  const int64_t q = v.n_tiles / v.n_ctas, rem = v.n_tiles % v.n_ctas;   // the first `rem` chunks have q + 1 tiles
  if (tid == 0) { s_base = 0ull; s_fail = 0; }
  if (tid < kEwMaxTilesPerCta) { s_tcnt[tid] = 0u; s_tsat[tid] = 0u; }
  __syncthreads();
  const int64_t tile0 = (int64_t)chunk * q + min((int64_t)chunk, rem);
  const int n_my = (int)(q + ((int64_t)chunk < rem ? 1 : 0));
  uint32_t* s_sat = s_mask + (size_t)(q + (rem ? 1 : 0)) * kEwWordsPerTile;   // COMPACT: saturated masks; one-kernel form deciding on its list: the kept atoms' sign bits

  // ---- phase 1 ----
  // the candidate list of the first pass holds every kept atom of the chunk if it was made with a multiplier that
  // covers the true scale, did not overflow and no atom has p = 1
  bool from_list = cands != nullptr && cands->m32 > 0.0f && S.n_sat == 0 && !dead && scale > 0.0f &&
                   cands->m32 >= scale * 4294967296.0f * (1.0f + 2.384185791015625e-07f);
  if (cands != nullptr) from_list = __syncthreads_or(ew_cand_count(*cands) > (uint32_t)kEwCandPerThread ? 1 : 0) == 0 && from_list;
  if (from_list) {
    if (tid == 0) atomicAdd(&v.state->list_chunks, 1u);
    const float scale32 = scale * 4294967296.0f;
    const int n_w = n_my * kEwWordsPerTile;
    for (int wi = tid; wi < n_w; wi += kEwThreads) { s_mask[wi] = 0u; s_sat[wi] = 0u; }
    __syncthreads();
    const uint32_t n_c = ew_cand_count(*cands);
    const uint32_t blk_beg = (uint32_t)(tile0 * (kEwTile / 4));
    for (uint32_t e = 0; e < n_c; ++e) {                   // this thread's own entries; their words are drawn again
      const uint32_t li = cands->idx[e * kEwThreads + tid];
      const uint4 wd = philox4x32_10(make_uint4(blk_beg + (li >> 2), 0u, v.layer, kind_step), key);
      const uint32_t j = li & 3u;
      const uint32_t word = j == 0 ? wd.x : j == 1 ? wd.y : j == 2 ? wd.z : wd.w;
      const uint32_t gbits = cands->idx[kEwCandSlots + e * kEwThreads + tid];
      const float t = fabsf(__uint_as_float(gbits)) * scale32;           // the same product and comparison as ew_tile_bits
      if (t >= 4294967296.0f || word < __float2uint_rz(t)) {
        atomicOr(&s_mask[li >> 5], 1u << (li & 31u));
        if (gbits >> 31) atomicOr(&s_sat[li >> 5], 1u << (li & 31u));    // the value of a kept atom is sign(g) c: its sign is all that phase 2 needs
        atomicAdd(&s_tcnt[li / kEwTile], 1u);
      }
    }
    if (v.n_words > 0) {
      __syncthreads();
      for (int wi = tid; wi < n_w; wi += kEwThreads) {
        const int64_t widx = tile0 * kEwWordsPerTile + wi;
        if (widx < v.n_words) v.mask_words[widx] = s_mask[wi];
      }
    }
  } else
  if (any_sat) ew_keep_bits<true, true>(v, key, kind_step, tile0, n_my, scale, theta, dead, aligned, s_mask, s_sat, s_tcnt, s_tsat);
  else if (S.n_sat != 0) ew_keep_bits<false, true>(v, key, kind_step, tile0, n_my, scale, theta, dead, aligned, s_mask, s_sat, s_tcnt, s_tsat);
  else ew_keep_bits<false, false>(v, key, kind_step, tile0, n_my, scale, theta, dead, aligned, s_mask, s_sat, s_tcnt, s_tsat);
  __syncthreads();
#ifdef EW_PROFILE
  if (ew_t != nullptr) { EW_STAMP(2) }
#endif

  // ---- chunk count out, counts of the earlier chunks in ----
  if (w == 0) {
    uint32_t total = 0, total_sat = 0;
    for (int t = lane; t < n_my; t += kWarp) { total += s_tcnt[t]; total_sat += s_tsat[t]; }
    total = warp_sum(total); total_sat = warp_sum(total_sat);
    if (lane == 0) {
      *(volatile unsigned long long*)(v.tile_status + chunk) =
          kFlagReady | ((unsigned long long)total_sat << 32) | (unsigned long long)total;
      uint32_t run = 0, run_sat = 0;                      // exclusive prefixes over the chunk's tiles
      for (int t = 0; t < n_my; ++t) {
        const uint32_t cnt = s_tcnt[t]; s_tcnt[t] = run; run += cnt;
        const uint32_t cs = s_tsat[t]; s_tsat[t] = run_sat; run_sat += cs;
      }
      s_chunk = total;                                    // reuse: the chunk's counts
      s_chunk_sat = total_sat;
    }
  }
  unsigned long long before = 0;
  int fail = 0;
  for (uint32_t cidx = tid; cidx < chunk; cidx += kEwThreads) {
    unsigned long long sv;
    uint32_t spins = 0;
    for (;;) {
      sv = *(volatile const unsigned long long*)(v.tile_status + cidx);
      if ((sv & kFlagReady) || ++spins > kChunkSpinLimit) break;
      __nanosleep(200);                                   // leave the issue slots to the CTAs that are still sampling
    }
    if (!(sv & kFlagReady)) fail = 1;
    before += sv & ~kFlagReady;                           // totals < 2^32 in all: the two fields never mix
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
  if (lane == 0 && before) atomicAdd(&s_base, before);
  if (fail) s_fail = 1;
  __syncthreads();
#ifdef EW_PROFILE
  if (ew_t != nullptr) { EW_STAMP(3) }
#endif
  const uint64_t base_all = s_base & 0xFFFFFFFFull;       // kept atoms before this chunk
  const uint64_t base_sat = s_base >> 32;                 // of them saturated (0 unless COMPACT)
  const uint64_t base = COMPACT ? base_all - base_sat : base_all;   // position of the chunk's first list entry
  const uint32_t total = s_chunk;
  if (tid == 0) {
    if (s_fail) raise_status(v.hdr, ATOMO_ERR_TIMEOUT);
    for (int t = 0; t < n_my; ++t)
      v.tile_table[tile0 + t] = (uint32_t)min(base + s_tcnt[t] - (COMPACT ? s_tsat[t] : 0u), (uint64_t)0xFFFFFFFFull);
    if (tile0 + n_my == v.n_tiles) {                      // the last chunk knows k: capacity check, layer header
      const uint64_t k = base_all + total;
      const uint64_t k_sat = base_sat + s_chunk_sat;
      const uint64_t k_list = COMPACT ? k - k_sat : k;    // entries of the idx / entry list
      atomo_layer_header* h = v.hdr;
      h->n_sat = S.n_sat; h->c = S.c; h->l1 = S.T0; h->sweeps = S.rounds;
      if (S.nonfinite) raise_status(h, ATOMO_ERR_NONFINITE);
      else if (k_list > (uint64_t)v.k_cap || (COMPACT && k_sat > (uint64_t)v.sat_cap)) raise_status(h, ATOMO_ERR_CAPACITY);
      const bool ok = *(volatile uint32_t*)&h->status == ATOMO_OK;
      h->k = ok ? (uint32_t)k : 0u;
      if (COMPACT) h->n_sat = ok ? (uint32_t)k_sat : 0u;  // the length of the saturated list
      v.tile_table[v.n_tiles] = ok ? (uint32_t)k_list : 0u;
    }
  }
  if (total == 0) return;

  // ---- phase 2: ordered compaction, indices ascending, value = g_i / p_i ----
  // A thread takes a run of consecutive mask words of the chunk; one scan over the threads' counts gives every run
  // its place in the lists.  COMPACT scans two counts at once (list entries in the low half of a 64-bit word,
  // saturated atoms in the high half).
  const int n_w = n_my * kEwWordsPerTile;
  const int wpt = (n_w + kEwThreads - 1) / kEwThreads;                       // words per thread
  const int w_beg = min(tid * wpt, n_w), w_end = min(w_beg + wpt, n_w);
  unsigned long long cnt = 0;
  for (int wi = w_beg; wi < w_end; ++wi) {
    const uint32_t word = s_mask[wi];
    const uint32_t sword = any_sat ? s_sat[wi] : 0u;
    cnt += COMPACT ? ((unsigned long long)__popc(word & ~sword) | ((unsigned long long)__popc(sword) << 32)) : (unsigned long long)__popc(word);
  }
  unsigned long long inc = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) { const unsigned long long t = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += t; }
  __shared__ unsigned long long s_wsum2[kWarps];
  if (lane == 31) s_wsum2[w] = inc;
  __syncthreads();
  unsigned long long off = inc - cnt;
  for (int i = 0; i < w; ++i) off += s_wsum2[i];
  uint64_t pos = base + (off & 0xFFFFFFFFull);
  uint64_t pos_sat = base_sat + (off >> 32);
  for (int wi = w_beg; wi < w_end; ++wi) {
    uint32_t m = s_mask[wi];
    const uint32_t sword = any_sat ? s_sat[wi] : 0u;
    const int tl = wi / kEwWordsPerTile;
    const uint32_t off0 = (uint32_t)(wi % kEwWordsPerTile) * 32u;            // first atom of the word inside its tile
    const int64_t tile_base = (tile0 + tl) * (int64_t)kEwTile;
    while (m) {
      const int bpos = __ffs(m) - 1;
      m &= m - 1;
      const uint32_t o = off0 + (uint32_t)bpos;
      // from the list: no atom has p = 1, so only the sign is needed, and the list left it in the second mask
      const float g = from_list ? (((s_sat[wi] >> bpos) & 1u) ? -1.0f : 1.0f) : __ldg(v.g + tile_base + o);
      if (!COMPACT) {
        if (pos < (uint64_t)v.k_cap) {
          // kept atom: saturated (p = 1) keeps g; otherwise g / p = sign(g) T / (s - n_s)
          v.idx[pos] = (uint32_t)(tile_base + o);
          v.val[pos] = (!from_list && fabsf(g) > theta) ? g : copysignf(c, g);
        }
        ++pos;
      } else if ((sword >> bpos) & 1u) {
        if (pos_sat < (uint64_t)v.sat_cap) { v.sat_idx[pos_sat] = (uint32_t)(tile_base + o); v.sat_val[pos_sat] = g; }
        ++pos_sat;
      } else {
        // value sign(g) c: the entry carries g's sign bit (what copysignf reads in the explicit format)
        if (pos < (uint64_t)v.k_cap) v.ent[pos] = (uint16_t)(o | ((__float_as_uint(g) >> 31) << 15));
        ++pos;
      }
    }
  }
}

// The two-kernel form: the solve has left its result in the state record; a CTA takes the next chunk of consecutive
// tiles by ticket, so that every chunk it will wait for is already running, however many waves the grid takes.
template <bool COMPACT>
__global__ void __launch_bounds__(kEwThreads, kEwMinBlocks) ew_sample_pack_kernel(EwVec v, PhiloxKey key, uint32_t kind_step) {
  extern __shared__ uint32_t s_mask[];            // [tiles_per_cta][128] mask words of the chunk (COMPACT: then the saturated masks)
  __shared__ uint32_t s_ticket;
  const EwState* st = v.state;
  EwSolved S;
  S.T0 = st->T0; S.scale = st->scale; S.theta = st->theta_f; S.c = st->c; S.n_sat = st->n_sat; S.rounds = st->rounds;
  S.nonfinite = st->nonfinite != 0;
  if (threadIdx.x == 0) s_ticket = atomicAdd(v.ticket, 1u);
  __syncthreads();
  ew_sample_pack_chunk<COMPACT>(v, key, kind_step, s_ticket, S, s_mask);
}

// The one-kernel form (cooperative launch, every chunk resident): a CTA solves over its own chunk of tiles and then
// samples and packs the same chunk: from the candidate list of its first pass where that holds every kept atom,
// else from a second read of the chunk, which it finds in the L2 on its own side of the chip.
// LIST: the form with the candidate list (64 registers, four CTAs per SM); without it the kernel is compiled for five.
template <bool COMPACT, bool LIST>
__global__ void __launch_bounds__(kEwThreads, LIST ? kEwEncodeBlocks : kEwMinBlocks)
ew_encode_kernel(EwVec v, double s, PhiloxKey key, uint32_t kind_step, EwBegin begin) {
  extern __shared__ uint32_t s_mask[];
  if (blockIdx.x == 0 && threadIdx.x == 0) v.state->list_chunks = 0u;   // counted after the grid barrier
  if (begin.on) {
    // a call with one vector: the payload header, the layer header and the chunks' status words are set here instead of
    // by a kernel of their own; the grid barrier after the first pass orders them before their first use
    if (blockIdx.x == 0) {
      if (threadIdx.x == 0) *reinterpret_cast<atomo_payload_header*>(begin.pay) = begin.gh;
      if (threadIdx.x < sizeof(atomo_layer_header) / 16)
        reinterpret_cast<uint4*>(v.hdr)[threadIdx.x] = reinterpret_cast<const uint4*>(begin.tmpl + v.layer)[threadIdx.x];
    }
    if (threadIdx.x == 0) v.tile_status[blockIdx.x] = 0ull;
  }
  const int64_t q = v.n_tiles / v.n_ctas, rem = v.n_tiles % v.n_ctas;
  const int64_t chunk = blockIdx.x;
  const int64_t tile0 = chunk * q + min(chunk, rem);
  const int64_t n_my = q + (chunk < rem ? 1 : 0);
#ifdef EW_PROFILE
  unsigned long long ew_t[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#endif
  EW_STAMP(0)
  const int64_t beg = tile0 * kEwTile, end = min(v.n, (tile0 + n_my) * kEwTile);
  if constexpr (LIST) {
    __shared__ uint32_t s_cand[2 * kEwCandSlots], s_cstop;   // indices, then values
    __shared__ float s_red[kEwThreads / kWarp];
    const uint32_t cand0 = (uint32_t)__cvta_generic_to_shared(s_cand) + 4u * threadIdx.x;
    EwCands cands{s_cand, &s_cstop, 0.0f, cand0, cand0};
    const bool with_list = v.prob_out == nullptr;
    EwAcc first;
    if (with_list) {
      if (threadIdx.x == 0) s_cstop = 0u;                    // ordered before its first use by the barrier inside the first tile
      first = ew_chunk_pass_cand(v, key, kind_step, s, beg, end, (int)n_my, cands, s_red);
      EW_STAMP(6)
    }
    const EwSolved S = ew_solve_body(v, s, beg, end, with_list ? &first : nullptr);
    EW_STAMP(1)
#ifdef EW_PROFILE
    ew_sample_pack_chunk<COMPACT>(v, key, kind_step, (uint32_t)chunk, S, s_mask, &cands, ew_t);
    EW_STAMP(5)
    if (threadIdx.x == 0 && (blockIdx.x == 0 || blockIdx.x == gridDim.x / 2 || blockIdx.x == gridDim.x - 1))
      printf("cta %d tiles %d: first pass with list %llu ns (%u candidates in thread 0), solve %llu, keep bits %llu, publish+wait %llu, scan+pack %llu, total %llu\n",
             (int)blockIdx.x, (int)n_my, ew_t[6] ? ew_t[6] - ew_t[0] : 0ull, ew_cand_count(cands), ew_t[1] - ew_t[0], ew_t[2] - ew_t[1], ew_t[3] - ew_t[2],
             ew_t[5] - ew_t[3], ew_t[5] - ew_t[0]);
#else
    ew_sample_pack_chunk<COMPACT>(v, key, kind_step, (uint32_t)chunk, S, s_mask, &cands);
#endif
  } else {
    const EwSolved S = ew_solve_body(v, s, beg, end);
    ew_sample_pack_chunk<COMPACT>(v, key, kind_step, (uint32_t)chunk, S, s_mask);
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
  const bool compact = d.ghdr->ew_format == ATOMO_EW_COMPACT;
  const uint32_t sat_cap = compact ? (uint32_t)min(d.ghdr->ew_sat_cap, (uint64_t)0xFFFFFFFFull) : 0u;
  bool ok = d.ghdr->magic == ATOMO_MAGIC && d.ghdr->kind == ATOMO_KIND_ENTRYWISE && d.ghdr->ew_format <= ATOMO_EW_COMPACT &&
            h->rows == 1 && h->cols == d.n;
  if (compact) ok = ok && h->n_sat <= h->k && h->n_sat <= sat_cap && h->k - h->n_sat <= h->k_cap;
  else ok = ok && h->k <= h->k_cap;
  if (!ok && blockIdx.x == 0 && threadIdx.x == 0) raise_status(const_cast<atomo_layer_header*>(h), ATOMO_ERR_PAYLOAD);
  const uint32_t n_sat = (ok && compact) ? h->n_sat : 0u;
  const uint32_t k = ok ? h->k - n_sat : 0u;               // entries of the idx / entry list
  const float c = h->c;
  const uint32_t* idx = reinterpret_cast<const uint32_t*>(d.payload + h->off_idx);
  const uint16_t* ent = reinterpret_cast<const uint16_t*>(d.payload + h->off_idx);
  const float* val = reinterpret_cast<const float*>(d.payload + h->off_val);
  const uint32_t* table = reinterpret_cast<const uint32_t*>(d.payload + h->off_short);   // list entries before each tile
  const uint32_t* sat_idx = reinterpret_cast<const uint32_t*>(d.payload + h->off_long);
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
    if (!compact) {
      for (uint32_t j = lo + threadIdx.x; j < hi; j += kEwThreads) {
        const uint32_t i = __ldg(idx + j);
        if ((int64_t)i >= tile_base && (int64_t)i < tile_base + kEwTile && (int64_t)i < d.n) d.out[i] = __ldg(val + j);
      }
    } else {
      for (uint32_t j = lo + threadIdx.x; j < hi; j += kEwThreads) {
        const uint32_t e = __ldg(ent + j);
        const int64_t off = e & (uint32_t)(kEwTile - 1);
        if (off < left) out[off] = (e & 0x8000u) ? -c : c;
      }
      if (n_sat) {                                       // the saturated atoms of this tile (ascending list)
        const uint32_t s_lo = lower_bound_u32(sat_idx, n_sat, (uint64_t)tile_base);
        for (uint32_t j = s_lo + threadIdx.x; j < n_sat; j += kEwThreads) {
          const int64_t off = (int64_t)__ldg(sat_idx + j) - tile_base;
          if (off >= kEwTile) break;
          if (off >= 0 && off < left) out[off] = __ldg(val + j);
        }
      }
    }
  }
}

// ---- l_q budget (Section 4: the budget s = ||g||_1 / ||g||_q turns entry-wise ATOMO into QSGD for q = 2 and
//      into TernGrad for q = infinity) --------------------------------------------------------------------
// pass 0: per-CTA sum |g| and max |g|; pass 1 (finite q > 1 only): per-CTA sum (|g| / amax)^q.  fp64 sums.
__global__ void __launch_bounds__(kEwThreads) ew_lq_kernel(const float* __restrict__ g, int64_t n, int pass, double q,
                                                           double inv_amax, double* __restrict__ part_sum,
                                                           float* __restrict__ part_max) {
  __shared__ double s_sum[kEwThreads / kWarp];
  __shared__ float s_max[kEwThreads / kWarp];
  double sum = 0.0;
  float amax = 0.0f;
  for (int64_t i = (int64_t)blockIdx.x * kEwThreads + threadIdx.x; i < n; i += (int64_t)gridDim.x * kEwThreads) {
    const float a = fabsf(__ldg(g + i));
    if (pass == 0) { sum += (double)a; amax = fmaxf(amax, a); if (!(a <= 3.0e38f)) amax = __int_as_float(0x7f800000); }
    else if (a > 0.0f) sum += (q == 2.0) ? ((double)a * inv_amax) * ((double)a * inv_amax) : pow((double)a * inv_amax, q);
  }
  sum = warp_sum(sum); amax = warp_max(amax);
  const int lane = threadIdx.x % kWarp, w = threadIdx.x / kWarp;
  if (lane == 0) { s_sum[w] = sum; s_max[w] = amax; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0; float m = 0.0f;
    for (int i = 0; i < kEwThreads / kWarp; ++i) { t += s_sum[i]; m = fmaxf(m, s_max[i]); }   // fixed order
    part_sum[blockIdx.x] = t;
    if (pass == 0) part_max[blockIdx.x] = m;
  }
}

void launch_ew_lq(const float* g, int64_t n, int pass, double q, double inv_amax, double* part_sum, float* part_max,
                  int n_ctas, cudaStream_t st) {
  ew_lq_kernel<<<n_ctas, kEwThreads, 0, st>>>(g, n, pass, q, inv_amax, part_sum, part_max);
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
namespace {
// co-resident CTAs of a sample / pack style kernel with its largest chunk in shared memory
template <typename K> int64_t ew_wave(K kernel, int dyn_tiles) {
  int dev = 0, sms = 148, per_sm = 4;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kEwThreads, (size_t)dyn_tiles * kEwWordsPerTile * sizeof(uint32_t));
  if (e != cudaSuccess || per_sm < 1) { cudaGetLastError(); per_sm = 4; }
  return (int64_t)sms * per_sm;
}
}  // namespace

int ew_sample_pack_ctas(int64_t n_tiles, bool compact) {
  // one wave of chunks when it fits (at most 64 tiles per chunk, 32 for the compact format): tiles spread evenly, sizes differ by at most one
  const int64_t wave = compact ? ew_wave(ew_sample_pack_kernel<true>, 32) : ew_wave(ew_sample_pack_kernel<false>, 16);
  const int max_tiles = compact ? kEwMaxTilesPerCta / 2 : kEwMaxTilesPerCta;   // compact: two masks per tile in shared memory
  const int64_t min_ctas = (n_tiles + max_tiles - 1) / max_tiles;
  return (int)std::max<int64_t>(1, std::max(min_ctas, std::min(n_tiles, wave)));
}
namespace {
const void* ew_encode_fn(bool compact, bool list) {
  if (list) return compact ? (const void*)ew_encode_kernel<true, true> : (const void*)ew_encode_kernel<false, true>;
  return compact ? (const void*)ew_encode_kernel<true, false> : (const void*)ew_encode_kernel<false, false>;
}
}  // namespace
// CTAs of the one-kernel form, or 0 if the vector does not fit one wave of resident chunks.  `list`: the form that
// keeps a candidate list during its first pass.
int ew_encode_ctas(int64_t n_tiles, bool compact, bool list) {
  static int64_t waves[2][2] = {{0, 0}, {0, 0}};
  // chunks of at most 12 tiles with the list: with the two masks (12 KB) and the list a CTA stays below 48 KB, so that
  // four CTAs per SM fit the 196 KB carve-out a cooperative launch is checked against; 16 without (8 or 16 KB of masks)
  const int64_t fit_tiles = list ? 12 : 16;
  if (waves[compact][list] == 0) {
    int dev = 0, sms = 148, per_sm = 4;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const size_t dyn = (size_t)fit_tiles * kEwWordsPerTile * sizeof(uint32_t) * ((compact || list) ? 2 : 1);
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ew_encode_fn(compact, list), kEwThreads, dyn) != cudaSuccess || per_sm < 1) {
      cudaGetLastError(); per_sm = 4;
    }
    waves[compact][list] = (int64_t)sms * per_sm;
  }
  const int max_tiles = compact ? kEwMaxTilesPerCta / 2 : kEwMaxTilesPerCta;
  const int64_t ctas = std::min(n_tiles, waves[compact][list]);
  if (ctas < 1 || (n_tiles + ctas - 1) / ctas > std::min<int64_t>(max_tiles, fit_tiles)) return 0;
  return (int)ctas;
}
// Whether the list pays for a vector of n elements in `ctas` chunks at budget s: a thread expects 1.25 s (its atoms) / n
// candidates and has kEwCandPerThread slots; beyond a quarter of them (budgets above about 1.5 % of the length) the
// appends cost more than the second read saves and overflows become likely.
bool ew_list_pays(int64_t n, int64_t n_tiles, int ctas, double s) {
  if (ctas < 1) return false;
  const double chunk = (double)((n_tiles + ctas - 1) / ctas) * kEwTile;
  return 1.25 * s * chunk / ((double)n * kEwThreads) <= 0.25 * kEwCandPerThread;
}
void launch_ew_sample_pack(const EwVec& v, PhiloxKey key, uint32_t kind_step, cudaStream_t st) {
  const int64_t most = (v.n_tiles + v.n_ctas - 1) / v.n_ctas;
  const size_t smem = (size_t)most * kEwWordsPerTile * sizeof(uint32_t);
  if (v.compact) {
    // two masks per tile; chunks of at most 32 tiles keep them inside the default 48 KB of dynamic shared memory
    ew_sample_pack_kernel<true><<<(unsigned)v.n_ctas, kEwThreads, 2 * smem, st>>>(v, key, kind_step);
  } else {
    ew_sample_pack_kernel<false><<<(unsigned)v.n_ctas, kEwThreads, smem, st>>>(v, key, kind_step);
  }
}
int launch_ew_encode(const EwVec& v, double s, PhiloxKey key, uint32_t kind_step, const EwBegin& begin, cudaStream_t st) {
  const int64_t most = (v.n_tiles + v.n_ctas - 1) / v.n_ctas;
  // mask words; a second mask for the saturated atoms (compact format) or the sign bits (list)
  const size_t smem = (size_t)most * kEwWordsPerTile * sizeof(uint32_t) * ((v.compact || v.candidates) ? 2 : 1);
  EwVec vv = v; double ss = s; PhiloxKey kk = key; uint32_t ks = kind_step; EwBegin bb = begin;
  void* args[] = {&vv, &ss, &kk, &ks, &bb};
  return (int)cudaLaunchCooperativeKernel(ew_encode_fn(v.compact != 0, v.candidates != 0), dim3((unsigned)v.n_ctas), dim3(kEwThreads), args, smem, st);
}
void launch_ew_decode(const EwDecode& d, cudaStream_t st) {
  const int64_t tiles = (d.n + kEwTile - 1) / kEwTile;
  ew_decode_kernel<<<(unsigned)std::min<int64_t>(tiles, 1 << 20), kEwThreads, 0, st>>>(d);   // a tile per CTA: the CTAs of a wave hide one another's barriers
}
int ew_tile_elems() { return kEwTile; }

}  // namespace atomo
