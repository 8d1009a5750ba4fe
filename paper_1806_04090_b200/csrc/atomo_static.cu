// atomo_decode_spectral_static: the spectral decode for callers that must not allocate.
//
// atomo_decode() keeps its per-call tables (one descriptor per layer, one entry per output tile)
// in the context's workspace, which is obtained with cudaMalloc the first time and whenever a
// larger batch arrives.  Some callers cannot afford that: a training process whose framework
// allocator has already reserved the whole device (a raw cudaMalloc then fails or fragments the
// pool), a decode issued from a latency-critical section where cudaMalloc's device-wide
// synchronisation would stall every other stream, or a memory-capped job that is not allowed to
// grow.  For them the tables live in a fixed array that is part of the library image.
#include <mutex>

#include "atomo_kernels.cuh"

using namespace atomo;

namespace {

constexpr int kStaticMaxLayers = ATOMO_STATIC_MAX_LAYERS;
constexpr int kStaticMaxTiles = ATOMO_STATIC_MAX_TILES;
constexpr size_t kLayerBytes = sizeof(SpDecodeLayer) * kStaticMaxLayers;
constexpr size_t kTileBytes = sizeof(TileRef) * kStaticMaxTiles;

// Scratch shared by every call on a device (about 130 KB per GPU that loads the library).
// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[kLayerBytes + kTileBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_ptr[kMaxDevices] = {};     // device address of g_static_scratch, per device

// host-side staging for the tables; cudaMemcpyAsync from pageable memory returns once the source
// has been staged, so one buffer per host thread can be reused by the next call
thread_local SpDecodeLayer t_layers[kStaticMaxLayers];
thread_local TileRef t_tiles[kStaticMaxTiles];

}  // namespace

extern "C" int atomo_decode_spectral_static(int device, const void* payload, const int64_t* rows, const int64_t* cols,
                                            float* const* out, int32_t n_layers, void* stream) {
  if (device < 0 || device >= kMaxDevices || !payload || !rows || !cols || !out || n_layers <= 0)
    return ATOMO_ERR_INVALID_ARG;
  if (n_layers > kStaticMaxLayers) return ATOMO_ERR_CAPACITY;
  const int tr = sp_decode_tile_rows(), tc = sp_decode_tile_cols();
  int64_t n_tiles = 0;
  for (int l = 0; l < n_layers; ++l) {
    if (!out[l] || rows[l] <= 0 || cols[l] <= 0) return ATOMO_ERR_INVALID_ARG;
    n_tiles += ((rows[l] + tr - 1) / tr) * ((cols[l] + tc - 1) / tc);
    if (n_tiles > kStaticMaxTiles) return ATOMO_ERR_CAPACITY;
  }
  if (cudaSetDevice(device) != cudaSuccess) return ATOMO_ERR_CUDA;
  unsigned char* scratch = nullptr;
  {
    // set-up, once per device, with that device current: resolve the array's device address
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_scratch_ptr[device] == nullptr) {
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return ATOMO_ERR_CUDA;
      g_scratch_ptr[device] = static_cast<unsigned char*>(p);
    }
    scratch = g_scratch_ptr[device];
  }
  const uint8_t* pay = static_cast<const uint8_t*>(payload);
  const atomo_layer_header* d_hdr = reinterpret_cast<const atomo_layer_header*>(pay + sizeof(atomo_payload_header));
  int t = 0;
  for (int l = 0; l < n_layers; ++l) {
    t_layers[l] = SpDecodeLayer{d_hdr + l, out[l], rows[l], cols[l]};
    const int na = (int)((rows[l] + tr - 1) / tr), nb = (int)((cols[l] + tc - 1) / tc);
    for (int a = 0; a < na; ++a)
      for (int b = 0; b < nb; ++b) t_tiles[t++] = TileRef{l, a, b, 0};
  }
  cudaStream_t st = (cudaStream_t)stream;
  SpDecodeLayer* d_layers = reinterpret_cast<SpDecodeLayer*>(scratch);
  TileRef* d_tiles = reinterpret_cast<TileRef*>(scratch + kLayerBytes);
  // both tables are fully rewritten for the entries this call uses; nothing has to start at zero
  if (cudaMemcpyAsync(d_layers, t_layers, sizeof(SpDecodeLayer) * n_layers, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return ATOMO_ERR_CUDA;
  if (cudaMemcpyAsync(d_tiles, t_tiles, sizeof(TileRef) * (size_t)t, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return ATOMO_ERR_CUDA;
  launch_sp_decode(pay, d_layers, d_tiles, t, st);
  return cudaGetLastError() == cudaSuccess ? ATOMO_OK : ATOMO_ERR_CUDA;
}
