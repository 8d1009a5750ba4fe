// Combine step of data-parallel training (Section 2 of the paper: every worker sends its sparsified gradient
// g_hat_p, the receiver forms their average): out = (1/P) sum_p decode(payload_p), in one pass over the output.
//   spectral   : the decode kernel of atomo_spectral.cu walks the kept atoms of all P payloads as one sequence
//                (payload after payload, atom after atom: a fixed order), each term scaled by 1/P
//   entry-wise : per tile of 4096 elements, a zeroed tile in shared memory receives payload 0's kept values, then
//                payload 1's, ... (indices are unique inside a payload, so no two threads meet between barriers),
//                then the tile is scaled and written once; explicit and compact payloads may be mixed
#include <algorithm>

#include "atomo_kernels.cuh"

namespace atomo {

namespace {
constexpr int kAvgThreads = 256;
constexpr int kAvgEwTile = ATOMO_EW_TILE;

__device__ __forceinline__ const atomo_layer_header* layer_header(const uint8_t* payload, int layer) {
  return reinterpret_cast<const atomo_layer_header*>(payload + sizeof(atomo_payload_header)) + layer;
}
}  // namespace

__global__ void __launch_bounds__(kAvgThreads) ew_decode_average_kernel(const uint8_t* const* __restrict__ payloads,
                                                                        int n_payloads, float inv_p, int layer,
                                                                        float* __restrict__ out, int64_t n) {
  __shared__ __align__(16) float s_tile[kAvgEwTile];
  const int64_t n_tiles = (n + kAvgEwTile - 1) / kAvgEwTile;
  const bool vec = (reinterpret_cast<uintptr_t>(out) & 15u) == 0;
  for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const int64_t tile_base = tile * kAvgEwTile;
    const int64_t left = n - tile_base;
    __syncthreads();                                     // the previous tile has been written out
    for (int i = threadIdx.x; i < kAvgEwTile / 4; i += kAvgThreads)
      reinterpret_cast<float4*>(s_tile)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int p = 0; p < n_payloads; ++p) {
      const uint8_t* payload = payloads[p];
      const atomo_payload_header* gh = reinterpret_cast<const atomo_payload_header*>(payload);
      const atomo_layer_header* h = layer_header(payload, layer);
      const bool compact = gh->ew_format == ATOMO_EW_COMPACT;
      const uint32_t sat_cap = compact ? (uint32_t)min(gh->ew_sat_cap, (uint64_t)0xFFFFFFFFull) : 0u;
      bool ok = gh->magic == ATOMO_MAGIC && gh->kind == ATOMO_KIND_ENTRYWISE && gh->ew_format <= ATOMO_EW_COMPACT &&
                h->rows == 1 && h->cols == n;
      if (compact) ok = ok && h->n_sat <= h->k && h->n_sat <= sat_cap && h->k - h->n_sat <= h->k_cap;
      else ok = ok && h->k <= h->k_cap;
      if (!ok && tile == 0 && threadIdx.x == 0) raise_status(const_cast<atomo_layer_header*>(h), ATOMO_ERR_PAYLOAD);
      const uint32_t n_sat = (ok && compact) ? h->n_sat : 0u;
      const uint32_t k = ok ? h->k - n_sat : 0u;          // entries of the idx / entry list
      const float c = h->c;
      const uint32_t* idx = reinterpret_cast<const uint32_t*>(payload + h->off_idx);
      const uint16_t* ent = reinterpret_cast<const uint16_t*>(payload + h->off_idx);
      const float* val = reinterpret_cast<const float*>(payload + h->off_val);
      const uint32_t* table = reinterpret_cast<const uint32_t*>(payload + h->off_short);   // list entries before each tile
      const uint32_t* sat_idx = reinterpret_cast<const uint32_t*>(payload + h->off_long);
      uint32_t lo = 0, hi = 0;
      if (k) { lo = min(__ldg(table + tile), k); hi = min(__ldg(table + tile + 1), k); }
      __syncthreads();                                   // zeros / the previous payload's values are in place
      if (!compact) {
        for (uint32_t j = lo + threadIdx.x; j < hi; j += kAvgThreads) {
          const int64_t i = (int64_t)__ldg(idx + j) - tile_base;
          if (i >= 0 && i < kAvgEwTile) s_tile[i] += __ldg(val + j);
        }
      } else {
        // an atom is in the entry list or in the saturated list, never both: still one writer per element
        for (uint32_t j = lo + threadIdx.x; j < hi; j += kAvgThreads) {
          const uint32_t e = __ldg(ent + j);
          s_tile[e & (uint32_t)(kAvgEwTile - 1)] += (e & 0x8000u) ? -c : c;
        }
        if (n_sat) {
          uint32_t s_lo = 0, s_hi = n_sat;               // first saturated atom at or after the tile's start
          while (s_lo < s_hi) { const uint32_t mid = (s_lo + s_hi) >> 1; if ((int64_t)__ldg(sat_idx + mid) < tile_base) s_lo = mid + 1; else s_hi = mid; }
          for (uint32_t j = s_lo + threadIdx.x; j < n_sat; j += kAvgThreads) {
            const int64_t i = (int64_t)__ldg(sat_idx + j) - tile_base;
            if (i >= kAvgEwTile) break;
            if (i >= 0) s_tile[i] += __ldg(val + j);
          }
        }
      }
    }
    __syncthreads();
    float* o = out + tile_base;
    if (left >= kAvgEwTile && vec) {
      for (int i = threadIdx.x; i < kAvgEwTile / 4; i += kAvgThreads) {
        const float4 t = reinterpret_cast<const float4*>(s_tile)[i];
        reinterpret_cast<float4*>(o)[i] = make_float4(t.x * inv_p, t.y * inv_p, t.z * inv_p, t.w * inv_p);
      }
    } else {
      for (int i = threadIdx.x; i < kAvgEwTile && i < left; i += kAvgThreads) o[i] = s_tile[i] * inv_p;
    }
  }
}

void launch_ew_decode_average(const uint8_t* const* d_payloads, int n_payloads, int layer, float* out, int64_t n,
                              cudaStream_t st) {
  const int64_t tiles = (n + kAvgEwTile - 1) / kAvgEwTile;
  ew_decode_average_kernel<<<(unsigned)std::min<int64_t>(tiles, 148 * 8), kAvgThreads, 0, st>>>(
      d_payloads, n_payloads, 1.0f / (float)n_payloads, layer, out, n);
}

}  // namespace atomo
