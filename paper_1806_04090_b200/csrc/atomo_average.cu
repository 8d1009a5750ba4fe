// Combine step of data-parallel training (Section 2 of the paper: every worker sends its sparsified gradient
// g_hat_p, the receiver forms their average): out = (1/P) sum_p decode(payload_p), in one pass over the output.
//   spectral   : per 32 x 256 output tile, the rank-one terms of all P payloads are accumulated in registers,
//                payload after payload, atom after atom (a fixed order), then scaled by 1/P and written once
//   entry-wise : per tile of 4096 elements, a zeroed tile in shared memory receives payload 0's kept values, then
//                payload 1's, ... (indices are unique inside a payload, so no two threads meet between barriers),
//                then the tile is scaled and written once
#include <algorithm>

#include "atomo_kernels.cuh"

namespace atomo {

namespace {
constexpr int kAvgRows = 32, kAvgCols = 256, kAvgAtoms = 16;
constexpr int kAvgThreads = 256;
constexpr int kAvgEwTile = ATOMO_EW_TILE;

__device__ __forceinline__ const atomo_layer_header* layer_header(const uint8_t* payload, int layer) {
  return reinterpret_cast<const atomo_layer_header*>(payload + sizeof(atomo_payload_header)) + layer;
}
}  // namespace

__global__ void __launch_bounds__(kAvgThreads) sp_decode_average_kernel(const uint8_t* const* __restrict__ payloads,
                                                                        int n_payloads, float inv_p,
                                                                        const SpDecodeLayer* __restrict__ layers,
                                                                        const TileRef* __restrict__ tiles) {
  __shared__ __align__(16) float s_col[kAvgAtoms][kAvgCols];
  __shared__ float s_row[kAvgAtoms][kAvgRows];
  const TileRef ref = tiles[blockIdx.x];
  const SpDecodeLayer D = layers[ref.layer];
  const int64_t rows = D.rows, cols = D.cols;
  const bool tall = rows > cols;
  const int64_t r = tall ? cols : rows, len = tall ? rows : cols;
  const int64_t rlen = tall ? len : r, clen = tall ? r : len;
  const int64_t i0 = (int64_t)ref.a * kAvgRows, c0 = (int64_t)ref.b * kAvgCols;
  const int tid = threadIdx.x;
  const int cg = tid % 64, rg = tid / 64;            // 64 column groups of 4, 4 row groups of 8
  float acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  for (int p = 0; p < n_payloads; ++p) {
    const uint8_t* payload = payloads[p];
    const atomo_payload_header* gh = reinterpret_cast<const atomo_payload_header*>(payload);
    const atomo_layer_header* h = layer_header(payload, ref.layer);
    const bool ok = gh->magic == ATOMO_MAGIC && gh->kind == ATOMO_KIND_SPECTRAL && h->rows == rows && h->cols == cols &&
                    h->k <= h->k_cap;
    if (!ok && ref.a == 0 && ref.b == 0 && tid == 0) raise_status(const_cast<atomo_layer_header*>(h), ATOMO_ERR_PAYLOAD);
    const uint32_t k = ok ? h->k : 0u;
    const float* coef = reinterpret_cast<const float*>(payload + h->off_val);
    const float* shortv = reinterpret_cast<const float*>(payload + h->off_short);
    const float* longv = reinterpret_cast<const float*>(payload + h->off_long);
    const float* rowvec = tall ? longv : shortv;   // indexed by output row
    const float* colvec = tall ? shortv : longv;   // indexed by output column
    for (uint32_t a0 = 0; a0 < k; a0 += kAvgAtoms) {
      const int na = min((uint32_t)kAvgAtoms, k - a0);
      __syncthreads();
      for (int idx = tid; idx < na * kAvgCols; idx += kAvgThreads) {
        const int a = idx / kAvgCols, c = idx % kAvgCols;
        s_col[a][c] = (c0 + c < clen) ? __ldg(colvec + (int64_t)(a0 + a) * clen + c0 + c) : 0.f;
      }
      for (int idx = tid; idx < na * kAvgRows; idx += kAvgThreads) {
        const int a = idx / kAvgRows, i = idx % kAvgRows;
        s_row[a][i] = (i0 + i < rlen) ? __ldg(rowvec + (int64_t)(a0 + a) * rlen + i0 + i) * __ldg(coef + a0 + a) : 0.f;
      }
      __syncthreads();
      for (int a = 0; a < na; ++a) {
        const float4 cv = *reinterpret_cast<const float4*>(&s_col[a][cg * 4]);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float rv = s_row[a][rg * 8 + i];
          acc[i][0] = fmaf(rv, cv.x, acc[i][0]); acc[i][1] = fmaf(rv, cv.y, acc[i][1]);
          acc[i][2] = fmaf(rv, cv.z, acc[i][2]); acc[i][3] = fmaf(rv, cv.w, acc[i][3]);
        }
      }
    }
  }
  const bool vec_ok = (cols % 4 == 0) && ((reinterpret_cast<uintptr_t>(D.out) & 15u) == 0);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int64_t row = i0 + rg * 8 + i;
    if (row >= rows) continue;
    const int64_t c = c0 + cg * 4;
    float* o = D.out + row * cols + c;
    if (vec_ok && c + 3 < cols)
      *reinterpret_cast<float4*>(o) = make_float4(acc[i][0] * inv_p, acc[i][1] * inv_p, acc[i][2] * inv_p, acc[i][3] * inv_p);
    else for (int j = 0; j < 4; ++j) if (c + j < cols) o[j] = acc[i][j] * inv_p;
  }
}

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
      const bool ok = gh->magic == ATOMO_MAGIC && gh->kind == ATOMO_KIND_ENTRYWISE && h->rows == 1 && h->cols == n &&
                      h->k <= h->k_cap;
      if (!ok && tile == 0 && threadIdx.x == 0) raise_status(const_cast<atomo_layer_header*>(h), ATOMO_ERR_PAYLOAD);
      const uint32_t k = ok ? h->k : 0u;
      const uint32_t* idx = reinterpret_cast<const uint32_t*>(payload + h->off_idx);
      const float* val = reinterpret_cast<const float*>(payload + h->off_val);
      const uint32_t* table = reinterpret_cast<const uint32_t*>(payload + h->off_short);   // kept atoms before each tile
      uint32_t lo = 0, hi = 0;
      if (k) { lo = min(__ldg(table + tile), k); hi = min(__ldg(table + tile + 1), k); }
      __syncthreads();                                   // zeros / the previous payload's values are in place
      for (uint32_t j = lo + threadIdx.x; j < hi; j += kAvgThreads) {
        const int64_t i = (int64_t)__ldg(idx + j) - tile_base;
        if (i >= 0 && i < kAvgEwTile) s_tile[i] += __ldg(val + j);
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

void launch_sp_decode_average(const uint8_t* const* d_payloads, int n_payloads, const SpDecodeLayer* d_layers,
                              const TileRef* d_tiles, int n_tiles, cudaStream_t st) {
  if (n_tiles > 0)
    sp_decode_average_kernel<<<n_tiles, kAvgThreads, 0, st>>>(d_payloads, n_payloads, 1.0f / (float)n_payloads, d_layers, d_tiles);
}

void launch_ew_decode_average(const uint8_t* const* d_payloads, int n_payloads, int layer, float* out, int64_t n,
                              cudaStream_t st) {
  const int64_t tiles = (n + kAvgEwTile - 1) / kAvgEwTile;
  ew_decode_average_kernel<<<(unsigned)std::min<int64_t>(tiles, 148 * 8), kAvgThreads, 0, st>>>(
      d_payloads, n_payloads, 1.0f / (float)n_payloads, layer, out, n);
}

}  // namespace atomo
