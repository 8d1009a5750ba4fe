// C ABI of the library (see include/atomo.h): argument checks, payload layout, workspace
// carving and kernel sequencing.  No arithmetic of the method lives here.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include "atomo_kernels.cuh"

using namespace atomo;

// Descriptor tables of a call (layer descriptors, tile lists, tensor maps, header templates) live in a device buffer
// of their own and are uploaded only when they differ from what that buffer already holds: a training loop calls
// with the same pointers and shapes every step, so in steady state a call issues no host-to-device copy at all (a
// copy of a few KB would otherwise queue behind whatever the application has on the copy engine, e.g. the next
// step's inputs).
struct TableCache {
  uint8_t* d = nullptr; size_t cap = 0;        // device buffer
  uint8_t* h = nullptr; size_t hcap = 0;       // pinned staging buffer of the last upload
  std::vector<uint8_t> last;                   // what the device buffer holds
  cudaEvent_t ev = nullptr; bool ev_pending = false;
  cudaStream_t last_stream = nullptr;
};

// A few caches side by side, found by a key over the caller's pointers and shapes: an application that alternates
// between a few sets of buffers (double-buffered gradients, several payloads in flight) still uploads nothing in
// steady state.  The key only picks the way; whether an upload is needed is decided on the table bytes themselves.
struct TableWays {
  static constexpr int kWays = 8;
  TableCache way[kWays];
  uint64_t key[kWays] = {};
  uint64_t used[kWays] = {};                   // 0 = never used, else the tick of the last use
  uint64_t tick = 0;
};

struct atomo_ctx {
  int device = 0;
  TableWays tab_sp, tab_dec, tab_avg;
  TableCache tab_ew;
  int64_t table_uploads = 0, table_reuses = 0;
  uint8_t* ws = nullptr;
  size_t ws_bytes = 0;
  uint32_t* h_flag = nullptr;        // pinned: convergence flag / state mirror
  EwState* h_state = nullptr;        // pinned
  cudaEvent_t ev_sync = nullptr;
  // stage timers: one set of events per API call, a ring of kEvRing sets (a set is read out -- its call is long
  // finished by then -- before it is used again), sums since profiling was switched on
  static constexpr int kEvRing = 32;
  cudaEvent_t ev[kEvRing][ATOMO_N_STAGES][2] = {};
  bool ev_used[kEvRing][ATOMO_N_STAGES] = {};
  int ev_cur = 0;
  int64_t launches[ATOMO_N_STAGES] = {};
  double acc_ms[ATOMO_N_STAGES] = {};
  int64_t acc_launches[ATOMO_N_STAGES] = {};
  int64_t acc_calls = 0;
  bool profiling = false;
  bool configured = false;
  int max_sweeps = 40;
  float tol = 3e-7f;
  int eig_mode = 1;                  // 1: Cholesky factor + Jacobi on its rows; 0: Jacobi on [A | I]
  int refine_min_short = 2048;       // layers with at least this short side get the sigma refinement pass
  bool tc_gram = true;               // Gram matrix on tcgen05 where the layer's layout allows it
  bool tc_ok = false;                // tensor-map entry point found
  int eig_scheme = 3;                // eigen-solve: 0 = Jacobi, one launch per step, 1 = persistent (cooperative), 2 = clusters first, 3 = tridiagonal route first
  int tri_clusters = -1;             // co-resident clusters of the tridiagonal reduction (-1 = not asked yet, 0 = unavailable)
  int tri_big_ok = -1;               // blocked tridiagonal reduction for short sides above 512 (-1 = not asked yet)
  int tri_big_ctas = 0;              // CTAs per layer of that reduction: 0 = chosen per batch, else 1, 2, 4, 8 or 16
  int eig_scheme_used = -1;          // what the last spectral encode actually ran
  int ew_format = ATOMO_EW_EXPLICIT; // payload format of entry-wise encodes
  int ew_launch = 0;                 // 0: one cooperative kernel per vector where it fits one wave; 1: always solve + sample/pack kernels
  std::vector<EwState*> ew_last_state;   // per vector of the last entry-wise encode: its state record (device) ...
  std::vector<int> ew_last_chunks;       // ... and its chunks in the one-kernel form (0: the two-kernel form ran)
  int64_t ew_sat_cap = 0;            // compact format: capacity of the saturated list
  int cluster_capacity[16] = {-1, -1, -1, -1, -1, -1, -1, -1, -1, -1, -1, -1, -1, -1, -1, -1};   // by log2(rp_max), -1 = not asked yet
  std::string err;
};

namespace {

struct Arena {
  uint8_t* base; size_t off = 0;
  explicit Arena(uint8_t* b) : base(b) {}
  template <typename T> T* take(size_t count) {
    off = (off + 255) & ~size_t(255);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
};

int fail_cuda(atomo_ctx* ctx, cudaError_t e, const char* what) {
  ctx->err = std::string(what) + ": " + cudaGetErrorString(e);
  return ATOMO_ERR_CUDA;
}
#define CK(call)                                                            \
  do {                                                                      \
    cudaError_t e__ = (call);                                               \
    if (e__ != cudaSuccess) return fail_cuda(ctx, e__, #call);              \
  } while (0)

// FNV-1a over a block of bytes, chained through h
uint64_t table_key(uint64_t h, const void* data, size_t bytes) {
  const uint8_t* b = static_cast<const uint8_t*>(data);
  for (size_t i = 0; i < bytes; ++i) { h ^= b[i]; h *= 1099511628211ull; }
  return h;
}
constexpr uint64_t kKeySeed = 1469598103934665603ull;

// the way that served this key last, else a way never used, else the one unused for longest
TableCache& table_pick(TableWays& tw, uint64_t key) {
  int pick = -1;
  for (int i = 0; i < TableWays::kWays; ++i) if (tw.used[i] && tw.key[i] == key) { pick = i; break; }
  if (pick < 0) {
    pick = 0;
    for (int i = 1; i < TableWays::kWays; ++i) if (tw.used[i] < tw.used[pick]) pick = i;
  }
  tw.key[pick] = key; tw.used[pick] = ++tw.tick;
  return tw.way[pick];
}
void table_free(TableCache& tc);
void table_free(TableWays& tw) { for (auto& w : tw.way) table_free(w); }

// device buffer of at least `bytes` for a table cache (growing it forgets the cached contents)
int table_reserve(atomo_ctx* ctx, TableCache& tc, size_t bytes) {
  if (bytes <= tc.cap) return ATOMO_OK;
  CK(cudaDeviceSynchronize());
  if (tc.d) CK(cudaFree(tc.d));
  tc.d = nullptr; tc.cap = 0; tc.last.clear();
  const size_t want = bytes + bytes / 4 + 4096;
  CK(cudaMalloc(&tc.d, want));
  tc.cap = want;
  return ATOMO_OK;
}

// makes the device buffer hold host[0 .. bytes): nothing to do if it already does
int table_commit(atomo_ctx* ctx, TableCache& tc, const uint8_t* host, size_t bytes, cudaStream_t st) {
  if (tc.ev == nullptr) CK(cudaEventCreateWithFlags(&tc.ev, cudaEventDisableTiming));
  if (tc.last.size() == bytes && std::memcmp(tc.last.data(), host, bytes) == 0) {
    if (st != tc.last_stream && tc.ev_pending) CK(cudaStreamWaitEvent(st, tc.ev, 0));   // the upload ran on another stream
    ++ctx->table_reuses;
    return ATOMO_OK;
  }
  if (tc.ev_pending) { CK(cudaEventSynchronize(tc.ev)); tc.ev_pending = false; }          // the staging buffer is free again
  if (tc.last_stream != st && tc.last_stream != nullptr) CK(cudaStreamSynchronize(tc.last_stream));   // readers of the old tables
  if (bytes > tc.hcap) {
    if (tc.h) CK(cudaFreeHost(tc.h));
    tc.h = nullptr; tc.hcap = 0;
    CK(cudaMallocHost(&tc.h, bytes + bytes / 4 + 4096));
    tc.hcap = bytes + bytes / 4 + 4096;
  }
  std::memcpy(tc.h, host, bytes);
  CK(cudaMemcpyAsync(tc.d, tc.h, bytes, cudaMemcpyHostToDevice, st));
  CK(cudaEventRecord(tc.ev, st));
  tc.ev_pending = true;
  tc.last.assign(host, host + bytes);
  tc.last_stream = st;
  ++ctx->table_uploads;
  return ATOMO_OK;
}

void table_free(TableCache& tc) {
  if (tc.d) cudaFree(tc.d);
  if (tc.h) cudaFreeHost(tc.h);
  if (tc.ev) cudaEventDestroy(tc.ev);
  tc = TableCache();
}

int ensure_ws(atomo_ctx* ctx, size_t bytes) {
  if (bytes <= ctx->ws_bytes) return ATOMO_OK;
  if (ctx->ws) { CK(cudaDeviceSynchronize()); CK(cudaFree(ctx->ws)); ctx->ws = nullptr; ctx->ws_bytes = 0; }
  const size_t want = bytes + bytes / 8 + (1 << 20);
  CK(cudaMalloc(&ctx->ws, want));
  ctx->ws_bytes = want;
  return ATOMO_OK;
}

void stage_begin(atomo_ctx* ctx, int stage, cudaStream_t st) {
  if (!ctx->profiling) return;
  cudaEventRecord(ctx->ev[ctx->ev_cur][stage][0], st);
  ctx->ev_used[ctx->ev_cur][stage] = true;
}
void stage_end(atomo_ctx* ctx, int stage, cudaStream_t st, int64_t n_launch) {
  ctx->launches[stage] += n_launch;
  ctx->acc_launches[stage] += n_launch;
  if (!ctx->profiling) return;
  cudaEventRecord(ctx->ev[ctx->ev_cur][stage][1], st);
}
// adds the times of one event set to the sums and frees the set (waits for its events: only the newest sets can
// still be running)
void stage_harvest(atomo_ctx* ctx, int slot) {
  for (int i = 0; i < ATOMO_N_STAGES; ++i) {
    if (!ctx->ev_used[slot][i]) continue;
    float ms = 0.0f;
    if (cudaEventSynchronize(ctx->ev[slot][i][1]) == cudaSuccess &&
        cudaEventElapsedTime(&ms, ctx->ev[slot][i][0], ctx->ev[slot][i][1]) == cudaSuccess)
      ctx->acc_ms[i] += (double)ms;
    ctx->ev_used[slot][i] = false;
  }
}
// a new API call: the next event set of the ring
void stage_reset(atomo_ctx* ctx) {
  for (int i = 0; i < ATOMO_N_STAGES; ++i) ctx->launches[i] = 0;
  ++ctx->acc_calls;
  if (!ctx->profiling) return;
  ctx->ev_cur = (ctx->ev_cur + 1) % atomo_ctx::kEvRing;
  stage_harvest(ctx, ctx->ev_cur);
}

int next_pow2_at_least(int x, int lo) { int p = lo; while (p < x) p <<= 1; return p; }

struct SpLayout {                 // payload offsets of one spectral layer
  uint32_t kc; uint64_t off_idx, off_coef, off_short, off_long;
};

uint64_t layout_spectral(const int32_t* rows, const int32_t* cols, int n_layers, int32_t k_cap,
                         std::vector<SpLayout>* out) {
  uint64_t off = sizeof(atomo_payload_header) + (uint64_t)n_layers * sizeof(atomo_layer_header);
  for (int l = 0; l < n_layers; ++l) {
    const int64_t r = std::min(rows[l], cols[l]), L = std::max(rows[l], cols[l]);
    const uint32_t kc = (uint32_t)std::min<int64_t>(k_cap, r);
    SpLayout lo;
    lo.kc = kc;
    off = align_up(off, 16); lo.off_idx = off; off += (uint64_t)kc * 4;
    off = align_up(off, 16); lo.off_coef = off; off += (uint64_t)kc * 4;
    off = align_up(off, 16); lo.off_short = off; off += (uint64_t)kc * r * 4;
    off = align_up(off, 16); lo.off_long = off; off += (uint64_t)kc * L * 4;
    if (out) out->push_back(lo);
  }
  return align_up(off, 16);
}

struct EwLayout { uint32_t kc, sc; uint64_t off_idx, off_val, off_tiles, off_sat; };

// explicit: idx u32[kc], val f32[kc], tile table.  compact: entries u16[kc], saturated values f32[sc], tile table,
// saturated indices u32[sc] (sc = the saturated list's capacity, clamped to n).
uint64_t layout_entrywise(const int64_t* n, int n_vecs, int64_t k_cap, bool compact, int64_t sat_cap,
                          std::vector<EwLayout>* out) {
  uint64_t off = sizeof(atomo_payload_header) + (uint64_t)n_vecs * sizeof(atomo_layer_header);
  for (int l = 0; l < n_vecs; ++l) {
    const uint32_t kc = (uint32_t)std::min<int64_t>(k_cap, n[l]);
    EwLayout lo{};
    lo.kc = kc;
    lo.sc = compact ? (uint32_t)std::min<int64_t>(sat_cap, n[l]) : 0u;
    off = align_up(off, 16); lo.off_idx = off; off += (uint64_t)kc * (compact ? 2 : 4);
    off = align_up(off, 16); lo.off_val = off; off += (uint64_t)(compact ? lo.sc : kc) * 4;
    off = align_up(off, 16); lo.off_tiles = off; off += ((uint64_t)(n[l] + ATOMO_EW_TILE - 1) / ATOMO_EW_TILE + 1) * 4;
    off = align_up(off, 16); lo.off_sat = off; off += (uint64_t)lo.sc * 4;
    if (out) out->push_back(lo);
  }
  return align_up(off, 16);
}

bool bad_budget(double s) { return !(s > 0.0) || !std::isfinite(s); }

}  // namespace

extern "C" {

int atomo_create(atomo_ctx** out, int device) {
  if (!out || device < 0) return ATOMO_ERR_INVALID_ARG;
  atomo_ctx* ctx = new atomo_ctx();
  ctx->device = device;
  *out = ctx;
  CK(cudaSetDevice(device));
  CK(cudaMallocHost(&ctx->h_flag, 256));
  CK(cudaMallocHost(&ctx->h_state, sizeof(EwState)));
  CK(cudaEventCreateWithFlags(&ctx->ev_sync, cudaEventDisableTiming));
  for (int r = 0; r < atomo_ctx::kEvRing; ++r)
    for (int i = 0; i < ATOMO_N_STAGES; ++i) { CK(cudaEventCreate(&ctx->ev[r][i][0])); CK(cudaEventCreate(&ctx->ev[r][i][1])); }
  const int e = sp_configure();
  if (e != 0) return fail_cuda(ctx, (cudaError_t)e, "cudaFuncSetAttribute(max dynamic shared memory)");
  ctx->tc_ok = sp_tc_configure() == 0;
  ctx->configured = true;
  return ATOMO_OK;
}

int atomo_destroy(atomo_ctx* ctx) {
  if (!ctx) return ATOMO_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  cudaDeviceSynchronize();
  if (ctx->ws) cudaFree(ctx->ws);
  table_free(ctx->tab_sp); table_free(ctx->tab_dec); table_free(ctx->tab_avg); table_free(ctx->tab_ew);
  if (ctx->h_flag) cudaFreeHost(ctx->h_flag);
  if (ctx->h_state) cudaFreeHost(ctx->h_state);
  if (ctx->ev_sync) cudaEventDestroy(ctx->ev_sync);
  for (int r = 0; r < atomo_ctx::kEvRing; ++r)
    for (int i = 0; i < ATOMO_N_STAGES; ++i) for (int j = 0; j < 2; ++j) if (ctx->ev[r][i][j]) cudaEventDestroy(ctx->ev[r][i][j]);
  delete ctx;
  return ATOMO_OK;
}

const char* atomo_last_cuda_error(atomo_ctx* ctx) { return ctx ? ctx->err.c_str() : "null context"; }

int64_t atomo_payload_bytes_spectral(const int32_t* rows, const int32_t* cols, int32_t n_layers, int32_t k_cap) {
  if (!rows || !cols || n_layers <= 0 || k_cap <= 0) return -1;
  for (int l = 0; l < n_layers; ++l) if (rows[l] <= 0 || cols[l] <= 0) return -1;
  return (int64_t)layout_spectral(rows, cols, n_layers, k_cap, nullptr);
}

int64_t atomo_payload_bytes_entrywise(const int64_t* n, int32_t n_vecs, int64_t k_cap) {
  if (!n || n_vecs <= 0 || k_cap <= 0) return -1;
  for (int l = 0; l < n_vecs; ++l) if (n[l] <= 0 || n[l] >= (int64_t(1) << 32)) return -1;
  return (int64_t)layout_entrywise(n, n_vecs, k_cap, false, 0, nullptr);
}

int64_t atomo_payload_bytes_entrywise_compact(const int64_t* n, int32_t n_vecs, int64_t k_cap, int64_t sat_cap) {
  if (!n || n_vecs <= 0 || k_cap <= 0 || sat_cap < 0) return -1;
  for (int l = 0; l < n_vecs; ++l) if (n[l] <= 0 || n[l] >= (int64_t(1) << 32)) return -1;
  return (int64_t)layout_entrywise(n, n_vecs, k_cap, true, sat_cap, nullptr);
}

int atomo_set_entrywise_format(atomo_ctx* ctx, int32_t format, int64_t sat_cap) {
  if (!ctx || (format != ATOMO_EW_EXPLICIT && format != ATOMO_EW_COMPACT)) return ATOMO_ERR_INVALID_ARG;
  if (format == ATOMO_EW_COMPACT && sat_cap < 0) return ATOMO_ERR_INVALID_ARG;
  ctx->ew_format = format;
  ctx->ew_sat_cap = format == ATOMO_EW_COMPACT ? sat_cap : 0;
  return ATOMO_OK;
}

int atomo_set_profiling(atomo_ctx* ctx, int enabled) {
  if (!ctx) return ATOMO_ERR_INVALID_ARG;
  CK(cudaSetDevice(ctx->device));
  // switching on starts the sums afresh; event sets still in flight are read out first
  for (int r = 0; r < atomo_ctx::kEvRing; ++r) stage_harvest(ctx, r);
  if (enabled) {
    for (int i = 0; i < ATOMO_N_STAGES; ++i) { ctx->acc_ms[i] = 0.0; ctx->acc_launches[i] = 0; }
    ctx->acc_calls = 0;
  }
  ctx->profiling = enabled != 0;
  return ATOMO_OK;
}

int atomo_get_stage_totals(atomo_ctx* ctx, double* ms, int64_t* launches, int64_t* calls) {
  if (!ctx) return ATOMO_ERR_INVALID_ARG;
  CK(cudaSetDevice(ctx->device));
  // everything recorded so far is added up (this waits for the newest calls' events); the current set stays in use
  // for get_stage_times, so its times are read without freeing it
  for (int r = 0; r < atomo_ctx::kEvRing; ++r) if (r != ctx->ev_cur) stage_harvest(ctx, r);
  for (int i = 0; i < ATOMO_N_STAGES; ++i) {
    double cur = 0.0;
    if (ctx->profiling && ctx->ev_used[ctx->ev_cur][i]) {
      float t = 0.0f;
      CK(cudaEventSynchronize(ctx->ev[ctx->ev_cur][i][1]));
      CK(cudaEventElapsedTime(&t, ctx->ev[ctx->ev_cur][i][0], ctx->ev[ctx->ev_cur][i][1]));
      cur = (double)t;
    }
    if (ms) ms[i] = ctx->acc_ms[i] + cur;
    if (launches) launches[i] = ctx->acc_launches[i];
  }
  if (calls) *calls = ctx->acc_calls;
  return ATOMO_OK;
}

int atomo_get_stage_times(atomo_ctx* ctx, float* ms, int64_t* launches) {
  if (!ctx) return ATOMO_ERR_INVALID_ARG;
  CK(cudaSetDevice(ctx->device));
  for (int i = 0; i < ATOMO_N_STAGES; ++i) {
    if (launches) launches[i] = ctx->launches[i];
    if (!ms) continue;
    ms[i] = 0.0f;
    if (ctx->profiling && ctx->ev_used[ctx->ev_cur][i]) {
      CK(cudaEventSynchronize(ctx->ev[ctx->ev_cur][i][1]));
      CK(cudaEventElapsedTime(&ms[i], ctx->ev[ctx->ev_cur][i][0], ctx->ev[ctx->ev_cur][i][1]));
    }
  }
  return ATOMO_OK;
}

int atomo_set_eig_params(atomo_ctx* ctx, int32_t max_sweeps, float tol) {
  if (!ctx || max_sweeps < 1 || max_sweeps > 1000 || !(tol > 0.0f) || !(tol < 1.0f)) return ATOMO_ERR_INVALID_ARG;
  ctx->max_sweeps = max_sweeps;
  ctx->tol = tol;
  return ATOMO_OK;
}

int atomo_last_eig_scheme(atomo_ctx* ctx) { return ctx ? ctx->eig_scheme_used : -1; }

int atomo_get_table_uploads(atomo_ctx* ctx, int64_t* uploads, int64_t* reuses) {
  if (!ctx) return ATOMO_ERR_INVALID_ARG;
  if (uploads) *uploads = ctx->table_uploads;
  if (reuses) *reuses = ctx->table_reuses;
  return ATOMO_OK;
}

int atomo_set_persistent_eig(atomo_ctx* ctx, int32_t enabled) {
  if (!ctx || enabled < 0 || enabled > 3) return ATOMO_ERR_INVALID_ARG;
  ctx->eig_scheme = enabled;
  return ATOMO_OK;
}

int atomo_set_tridiag_ctas(atomo_ctx* ctx, int32_t ctas_per_layer) {
  if (!ctx) return ATOMO_ERR_INVALID_ARG;
  if (ctas_per_layer != 0 && ctas_per_layer != 1 && ctas_per_layer != 2 && ctas_per_layer != 4 && ctas_per_layer != 8 &&
      ctas_per_layer != 16)
    return ATOMO_ERR_INVALID_ARG;
  ctx->tri_big_ctas = ctas_per_layer;
  return ATOMO_OK;
}

int atomo_set_gram_path(atomo_ctx* ctx, int32_t tensor_cores) {
  if (!ctx) return ATOMO_ERR_INVALID_ARG;
  ctx->tc_gram = tensor_cores != 0;
  return ATOMO_OK;
}

int atomo_set_sigma_refinement(atomo_ctx* ctx, int32_t min_short_side) {
  if (!ctx || min_short_side < 0) return ATOMO_ERR_INVALID_ARG;
  ctx->refine_min_short = min_short_side;
  return ATOMO_OK;
}

int atomo_set_eig_mode(atomo_ctx* ctx, int32_t mode) {
  if (!ctx || (mode != 0 && mode != 1)) return ATOMO_ERR_INVALID_ARG;
  ctx->eig_mode = mode;
  return ATOMO_OK;
}

// ==================================================================================================
static int encode_spectral_impl(atomo_ctx* ctx, const atomo_mat* layers, int32_t n_layers, double s, uint64_t seed,
                                uint64_t step, int32_t k_cap, void* payload, int64_t capacity_bytes,
                                const atomo_debug* dbg, void* stream, const float* const* given_sigma,
                                const float* const* given_short) {
  const bool given = given_sigma != nullptr;                   // the decomposition comes from the caller: S1 is skipped
  if (!ctx || !layers || n_layers <= 0 || k_cap <= 0 || !payload) return ATOMO_ERR_INVALID_ARG;
  if (bad_budget(s)) return ATOMO_ERR_BUDGET;
  if ((reinterpret_cast<uintptr_t>(payload) & 15u) != 0) return ATOMO_ERR_INVALID_ARG;
  std::vector<int32_t> rows(n_layers), cols(n_layers);
  for (int l = 0; l < n_layers; ++l) {
    const atomo_mat& m = layers[l];
    if (!m.data || m.rows <= 0 || m.cols <= 0 || m.ld < m.cols) return ATOMO_ERR_INVALID_ARG;
    if (std::min(m.rows, m.cols) > kSmemRowsMaxRp) return ATOMO_ERR_INVALID_ARG;
    rows[l] = m.rows; cols[l] = m.cols;
  }
  std::vector<SpLayout> lay;
  const uint64_t total = layout_spectral(rows.data(), cols.data(), n_layers, k_cap, &lay);
  if ((int64_t)total > capacity_bytes) return ATOMO_ERR_CAPACITY;
  CK(cudaSetDevice(ctx->device));
  cudaStream_t st = (cudaStream_t)stream;
  stage_reset(ctx);
  const int max_sweeps = ctx->max_sweeps;
  uint8_t* pay = static_cast<uint8_t*>(payload);
  atomo_layer_header* d_hdr = reinterpret_cast<atomo_layer_header*>(pay + sizeof(atomo_payload_header));

  // ---- host descriptors, tiles, workspace carving (two passes: size, then pointers) ----
  std::vector<SpLayer> L(n_layers);
  std::vector<int> tc_layers;
  std::vector<TileRef> gram_tiles, block_pairs, bp_tiles, chol_ctas, refine_tiles, tc_tiles;
  const int map_bytes = sp_tc_map_bytes();
  std::vector<uint8_t> maps_blob((size_t)n_layers * map_bytes, 0);
  int chol_panels = 0;
  int row_floats_max = 0, steps_max = 0, r_max = 0, rp_max = 0, r_max_tall = 0, k_cap_max = 1;
  for (int l = 0; l < n_layers; ++l) {
    SpLayer& d = L[l];
    const atomo_mat& m = layers[l];
    d.G = m.data; d.rows = m.rows; d.cols = m.cols; d.ld = m.ld;
    d.tall = m.rows > m.cols;
    d.r = std::min(m.rows, m.cols); d.L = std::max(m.rows, m.cols);
    d.rp = next_pow2_at_least(d.r, 32);
    d.acc = ctx->eig_mode == 0 ? 1 : 0;
    d.ldx = d.acc ? 2 * d.rp : d.rp;
    if (d.acc && d.ldx > 1024) return ATOMO_ERR_INVALID_ARG;   // route 0 holds rows of 2 rp floats: short side <= 512
    d.B = d.ldx <= 1024 ? 16 : (d.ldx == 2048 ? 8 : 4);          // a rotation is shared by 1, 2 or 4 warps
    d.nb = d.rp / d.B;
    d.layer = (uint32_t)l; d.k_cap = lay[l].kc;
    k_cap_max = std::max(k_cap_max, (int)d.k_cap);
    r_max = std::max(r_max, d.r); rp_max = std::max(rp_max, d.rp);
    const int gt = (d.r + 63) / 64;
    d.tc = 0; d.gram_split = 1;
    // The tensor core's fp32 accumulation truncates, which perturbs sum(sigma) -- and with it the largest p_i -- by a few
    // 1e-6 at a short side of 1024 and more above (measured 6e-6 at 4096): layers with a short side above 1024 take the
    // fp32 FMA kernel, whose sums round to nearest (their Gram matrix is a small part of their cost)
    if (ctx->tc_gram && ctx->tc_ok && !d.acc && d.r <= 1024 && sp_tc_eligible(d.G, d.rows, d.cols, d.ld)) {
      d.tc = 1;
      if (sp_tc_make_map(maps_blob.data() + (size_t)l * map_bytes, d.G, d.rows, d.cols, d.ld) != 0) return ATOMO_ERR_INVALID_ARG;
      tc_layers.push_back(l);
    } else {
      for (int a = 0; a < gt; ++a) for (int b = a; b < gt; ++b) gram_tiles.push_back({l, a, b, 0});
    }
    for (int p = 0; p < d.nb / 2; ++p) block_pairs.push_back({l, p, 0, 0});
    row_floats_max = std::max(row_floats_max, d.ldx); steps_max = std::max(steps_max, d.nb - 1);
    if (!d.acc && d.rp > 1024) {
      const int per = sp_cholesky_big_rows_per_cta();
      for (int c = 0; c < (d.rp + per - 1) / per; ++c) chol_ctas.push_back({l, c, 0, 0});
      chol_panels = std::max(chol_panels, (d.r + 31) / 32);
    }
    d.bp_tiles = d.tall ? (d.L + sp_bp_rows_per_tile() - 1) / sp_bp_rows_per_tile()
                        : (d.L + sp_bp_cols_per_tile() - 1) / sp_bp_cols_per_tile();
    {   // row chunks of the wide back-projection: 64 rows each, fewer and longer when k_cap makes the partials large
      const int64_t per_chunk = (int64_t)d.k_cap * d.L * (int64_t)sizeof(float);
      const int unit = sp_bp_chunk_rows();
      const int want = (d.r + unit - 1) / unit;
      const int fit = (int)std::max<int64_t>(1, ((int64_t)32 << 20) / per_chunk);
      const int chunks = d.tall ? 1 : std::min(want, fit);
      d.bp_chunk_rows = ((d.r + chunks - 1) / chunks + unit - 1) / unit * unit;
      d.bp_chunks = d.tall ? 1 : (d.r + d.bp_chunk_rows - 1) / d.bp_chunk_rows;
    }
    for (int t = 0; t < d.bp_tiles; ++t) for (int c = 0; c < d.bp_chunks; ++c) bp_tiles.push_back({l, t, c, 0});
    if (d.tall) r_max_tall = std::max(r_max_tall, d.r);
    d.refine = d.r >= ctx->refine_min_short ? 1 : 0;
    d.refine_tiles = (d.L + 63) / 64;
    if (d.refine)
      for (int a = 0; a < gt; ++a) for (int b = 0; b < d.refine_tiles; ++b) refine_tiles.push_back({l, a, b, 0});
  }
  // Tridiagonal routes first: eigenvalues of every atom from T = Q^T A Q, vectors for the kept atoms only -- in the
  // registers of a cluster for short sides up to 512, blocked with A in global memory above (no per-atom refinement,
  // no request for the whole short-side basis).  Otherwise the Jacobi routes, the cluster form first.
  bool tri_form = !given && ctx->eig_scheme == 3 && ctx->eig_mode != 0 && !(dbg && dbg->short_vecs);
  bool any_small = false, any_big = false;
  for (int l = 0; l < n_layers && tri_form; ++l) (L[l].rp <= sp_tridiag_max_rp() ? any_small : any_big) = true;
  if (tri_form && any_small) {
    if (ctx->tri_clusters < 0) ctx->tri_clusters = sp_configure_tridiag();
    if (ctx->tri_clusters < 1) tri_form = false;
  }
  if (tri_form && any_big) {
    if (ctx->tri_big_ok < 0) ctx->tri_big_ok = (sp_configure_tridiag_big() == 0 && sp_configure_bisect() == 0) ? 1 : 0;
    if (ctx->tri_big_ok < 1 || r_max > sp_tridiag_big_max_r()) tri_form = false;
  }
  std::vector<int> big_layers;
  for (int l = 0; l < n_layers; ++l) {
    L[l].tri = !tri_form ? 0 : (L[l].rp <= sp_tridiag_max_rp() ? 1 : 2);
    if (L[l].tri) { L[l].refine = 0; }
    if (L[l].tri == 2) big_layers.push_back(l);
  }
  if (tri_form) refine_tiles.clear();
  bool cluster_form = !given && !tri_form && ctx->eig_scheme >= 2 && ctx->eig_mode != 0;
  for (int l = 0; l < n_layers && cluster_form; ++l) cluster_form = L[l].nb / 2 <= sp_jacobi_cluster_ctas() && L[l].rp <= sp_jacobi_cluster_max_rp();
  if (cluster_form) {
    int lg = 0;
    while ((1 << lg) < rp_max) ++lg;
    if (ctx->cluster_capacity[lg] < 0) ctx->cluster_capacity[lg] = sp_jacobi_cluster_capacity(rp_max);
    if (ctx->cluster_capacity[lg] < 1) cluster_form = false;
  }
  for (int l = 0; l < n_layers; ++l) L[l].lam_ready = (cluster_form || tri_form || given) ? 1 : 0;
  if (given) { for (int l = 0; l < n_layers; ++l) L[l].refine = 0; refine_tiles.clear(); }
  // tensor-core Gram tiles: while the batch has fewer CTAs than the GPU has SMs, the K range of the layers with the
  // longest rows is split over 2 or 4 CTAs per tile (at least 16 stages of 32 columns per part)
  {
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    auto tiles_of = [&](int l) { const int tt = (L[l].r + sp_tc_tile() - 1) / sp_tc_tile(); return tt * (tt + 1) / 2; };
    int total = 0;
    for (int l : tc_layers) { L[l].gram_split = 1; total += tiles_of(l); }
    for (;;) {
      int best = -1;
      for (int l : tc_layers) {
        const int stages = (L[l].L + 31) / 32 / L[l].gram_split;
        if (L[l].gram_split < 4 && stages >= 32 && total + tiles_of(l) * L[l].gram_split <= sms &&
            (best < 0 || stages > (L[best].L + 31) / 32 / L[best].gram_split))
          best = l;
      }
      if (best < 0) break;
      total += tiles_of(best) * L[best].gram_split;
      L[best].gram_split *= 2;
    }
    for (int l : tc_layers) {
      const int tt = (L[l].r + sp_tc_tile() - 1) / sp_tc_tile();
      for (int a = 0; a < tt; ++a) for (int b = a; b < tt; ++b)
        for (int c = 0; c < L[l].gram_split; ++c) tc_tiles.push_back({l, a, b, c});
    }
  }
  // cluster tables of the eigen stage: small tridiagonal layers packed into 16-CTA clusters, largest first (a layer
  // takes rp / 32 consecutive ranks of one cluster); or, on the Jacobi cluster route, the block pairs of every layer
  std::vector<ClusterCta> ctas;
  int n_clusters = 0, rp_max_small = 32;
  if (tri_form) {
    const int per = sp_tridiag_cluster_ctas();
    std::vector<int> order;
    for (int l = 0; l < n_layers; ++l) if (L[l].tri == 1) { order.push_back(l); rp_max_small = std::max(rp_max_small, L[l].rp); }
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return L[a].rp > L[b].rp; });
    std::vector<int> used;
    for (int l : order) {
      const int nc = sp_tridiag_ctas_of(L[l].rp);
      size_t c = 0;
      while (c < used.size() && used[c] + nc > per) ++c;
      if (c == used.size()) { used.push_back(0); ctas.resize(ctas.size() + per, ClusterCta{-1, 0, 0, 0}); }
      for (int sl = 0; sl < nc; ++sl) ctas[c * per + used[c] + sl] = ClusterCta{l, sl, used[c], nc};
      used[c] += nc;
    }
    n_clusters = (int)used.size();
  } else if (cluster_form) {
    const int per = sp_jacobi_cluster_ctas();
    std::vector<int> order(n_layers);
    for (int l = 0; l < n_layers; ++l) order[l] = l;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return L[a].nb > L[b].nb; });
    std::vector<int> used;                                 // slots taken in each cluster (first fit, largest first)
    for (int l : order) {
      const int need_slots = L[l].nb / 2;
      size_t c = 0;
      while (c < used.size() && used[c] + need_slots > per) ++c;
      if (c == used.size()) { used.push_back(0); ctas.resize(ctas.size() + per, ClusterCta{-1, 0, 0, 0}); }
      for (int sl = 0; sl < need_slots; ++sl) ctas[c * per + used[c] + sl] = ClusterCta{l, sl, used[c], 0};
      used[c] += need_slots;
    }
    n_clusters = (int)used.size();
  }
  // the tables go to the table cache (device buffer tab_sp, host mirror `tables` with the same offsets), everything
  // the kernels write to the workspace
  SpLayer* d_layers = nullptr; TileRef *d_gram = nullptr, *d_pairs = nullptr, *d_bp = nullptr, *d_chol = nullptr, *d_ref = nullptr, *d_tc = nullptr;
  uint8_t* d_maps = nullptr;
  uint32_t* d_flag = nullptr;
  ClusterCta* d_ctas = nullptr;
  int* d_big = nullptr;
  const float** d_given = nullptr;
  atomo_layer_header* d_hdr_tmpl = nullptr;
  std::vector<uint8_t> tables;
  size_t table_bytes = 0;
  uint64_t tkey = table_key(kKeySeed, layers, (size_t)n_layers * sizeof(atomo_mat));
  tkey = table_key(tkey, &payload, sizeof(payload));
  tkey = table_key(tkey, &k_cap, sizeof(k_cap));
  if (given) { tkey = table_key(tkey, given_sigma, (size_t)n_layers * sizeof(float*)); tkey = table_key(tkey, given_short, (size_t)n_layers * sizeof(float*)); }
  TableCache& tab = table_pick(ctx->tab_sp, tkey);
  for (int pass = 0; pass < 2; ++pass) {
    Arena T(pass ? tab.d : nullptr);
    d_layers = T.take<SpLayer>(n_layers);
    d_gram = T.take<TileRef>(gram_tiles.size());
    d_pairs = T.take<TileRef>(block_pairs.size());
    d_bp = T.take<TileRef>(bp_tiles.size());
    d_chol = T.take<TileRef>(chol_ctas.size());
    d_ref = T.take<TileRef>(refine_tiles.size());
    d_tc = T.take<TileRef>(tc_tiles.size());
    d_maps = T.take<uint8_t>(maps_blob.size());
    d_ctas = T.take<ClusterCta>(ctas.size());
    d_big = T.take<int>(big_layers.size());
    d_given = T.take<const float*>(given ? (size_t)2 * n_layers : 0);
    d_hdr_tmpl = T.take<atomo_layer_header>(n_layers);
    table_bytes = T.off + 256;
    if (pass == 0) { const int rc = table_reserve(ctx, tab, table_bytes); if (rc != ATOMO_OK) return rc; }
  }
  tables.assign(table_bytes, 0);
  auto put = [&](const void* dev_ptr, const void* src, size_t bytes) {
    if (bytes) std::memcpy(tables.data() + (reinterpret_cast<const uint8_t*>(dev_ptr) - tab.d), src, bytes);
  };
  uint8_t* zero_beg = nullptr; size_t zero_bytes = 0;
  size_t need = 0;
  for (int pass = 0; pass < 2; ++pass) {
    Arena A(pass ? ctx->ws : nullptr);
    d_flag = A.take<uint32_t>(4);
    size_t dbg_atoms = 0, dbg_words = 0, dbg_sq = 0;
    for (int l = 0; l < n_layers; ++l) {
      SpLayer& d = L[l];
      d.lam = A.take<float>(d.rp);
      d.perm = A.take<int>(d.r);
      float* sig_ws = A.take<float>(d.r);
      float* prob_ws = A.take<float>(d.r);
      uint32_t* mask_ws = A.take<uint32_t>((d.r + 31) / 32);
      d.sigma = (dbg && dbg->sigma) ? dbg->sigma + dbg_atoms : sig_ws;
      d.prob = (dbg && dbg->prob) ? dbg->prob + dbg_atoms : prob_ws;
      d.mask_words = (dbg && dbg->mask_words) ? dbg->mask_words + dbg_words : mask_ws;
      d.dbg_short = (dbg && dbg->short_vecs) ? dbg->short_vecs + dbg_sq : nullptr;
      dbg_atoms += d.r; dbg_words += (d.r + 31) / 32; dbg_sq += (size_t)d.r * d.r;
      d.p_sel = A.take<float>(d.k_cap);
      d.bp_part = A.take<float>((size_t)d.bp_chunks * d.k_cap * d.L);
      d.scale = A.take<float>(1);
      {
        const int tt = (d.r + sp_tc_tile() - 1) / sp_tc_tile();
        d.gram_part = A.take<float>(d.tc && d.gram_split > 1
                                        ? (size_t)tt * (tt + 1) / 2 * d.gram_split * sp_tc_tile() * sp_tc_tile() : 0);
      }
      d.td_d = A.take<double>(d.tri ? d.rp : 0); d.td_e = A.take<double>(d.tri ? d.rp : 0);
      d.td_tau = A.take<double>(d.tri ? d.rp : 0); d.lam64 = A.take<double>(d.tri ? d.rp : 0);
      d.td_ldv = (d.r + 3) / 4 * 4;
      d.td_V = A.take<float>(d.tri ? (size_t)d.r * d.td_ldv : 0);
      d.tb_fp64 = 0;
      d.tb_ldw = (d.r + 3) / 4 * 4;
      d.tb_W = A.take<float>(d.tri == 2 ? (size_t)sp_tridiag_big_panel() * d.tb_ldw : 0);
      d.tb_vecwork = A.take<double>(d.tri == 2 ? (size_t)sp_eigvec_big_slots() * 5 * d.rp : 0);
      {
        const size_t nb = (size_t)(d.r + 31) / 32;
        d.tb_At = A.take<float>(d.tri == 2 && d.r <= 1024 ? nb * (nb + 1) / 2 * 1024 : 0);
      }
      d.chol_dd = A.take<float>(32 * 32 + 32);
      d.row_inv = A.take<float>(d.rp);
      d.refine_partials = A.take<float>(d.refine ? (size_t)d.refine_tiles * d.rp : 0);
      d.hdr = d_hdr + l;
      d.idx = reinterpret_cast<uint32_t*>(pay + lay[l].off_idx);
      d.coef = reinterpret_cast<float*>(pay + lay[l].off_coef);
      d.shortv = reinterpret_cast<float*>(pay + lay[l].off_short);
      d.longv = reinterpret_cast<float*>(pay + lay[l].off_long);
    }
    // zero-filled region: rotation counters and the X matrices
    uint8_t* zb = reinterpret_cast<uint8_t*>(A.take<uint32_t>(0));
    size_t z0 = A.off;
    for (int l = 0; l < n_layers; ++l) { L[l].rot_count = A.take<uint32_t>(max_sweeps); L[l].step_bar = A.take<uint32_t>(1); L[l].vec_ticket = A.take<uint32_t>(1); }
    for (int l = 0; l < n_layers; ++l) {
      const int tt = (L[l].r + sp_tc_tile() - 1) / sp_tc_tile();
      L[l].gram_ticket = A.take<uint32_t>(L[l].tc && L[l].gram_split > 1 ? (size_t)tt * (tt + 1) / 2 : 0);
    }
    for (int l = 0; l < n_layers; ++l) L[l].X = A.take<float>(L[l].tri ? 0 : (size_t)L[l].rp * L[l].ldx);
    zero_beg = zb; zero_bytes = A.off - z0;
    for (int l = 0; l < n_layers; ++l) {
      SpLayer& d = L[l];
      if (d.acc) { d.A = d.X; d.lda = d.ldx; }
      else if (d.tri == 2) { d.lda = (d.r + 3) / 4 * 4; d.A = A.take<float>((size_t)d.r * d.lda); d.tb_A = d.A; }   // 16-byte rows
      else { d.A = A.take<float>((size_t)d.r * d.r); d.lda = d.r; }
    }
    need = A.off + 256;
    if (pass == 0) { const int rc = ensure_ws(ctx, need); if (rc != ATOMO_OK) return rc; }
  }

  // ---- tables (uploaded only if they changed since the last call), headers, zero-filled regions ----
  atomo_payload_header gh{};
  gh.magic = ATOMO_MAGIC; gh.version = ATOMO_VERSION; gh.kind = ATOMO_KIND_SPECTRAL; gh.n_layers = (uint32_t)n_layers;
  gh.total_bytes = total; gh.seed = seed; gh.step = step; gh.s = s;
  {
    std::vector<atomo_layer_header> tmpl(n_layers);
    for (int l = 0; l < n_layers; ++l) {
      atomo_layer_header h{};
      h.rows = rows[l]; h.cols = cols[l]; h.k_cap = lay[l].kc; h.k = 0; h.status = ATOMO_OK;
      h.off_idx = lay[l].off_idx; h.off_val = lay[l].off_coef; h.off_short = lay[l].off_short; h.off_long = lay[l].off_long;
      tmpl[l] = h;
    }
    put(d_hdr_tmpl, tmpl.data(), tmpl.size() * sizeof(atomo_layer_header));
  }
  put(d_layers, L.data(), L.size() * sizeof(SpLayer));
  put(d_gram, gram_tiles.data(), gram_tiles.size() * sizeof(TileRef));
  put(d_pairs, block_pairs.data(), block_pairs.size() * sizeof(TileRef));
  put(d_bp, bp_tiles.data(), bp_tiles.size() * sizeof(TileRef));
  put(d_chol, chol_ctas.data(), chol_ctas.size() * sizeof(TileRef));
  put(d_ref, refine_tiles.data(), refine_tiles.size() * sizeof(TileRef));
  put(d_tc, tc_tiles.data(), tc_tiles.size() * sizeof(TileRef));
  put(d_maps, maps_blob.data(), maps_blob.size());
  put(d_ctas, ctas.data(), ctas.size() * sizeof(ClusterCta));
  put(d_big, big_layers.data(), big_layers.size() * sizeof(int));
  if (given) {
    std::vector<const float*> ptrs(2 * (size_t)n_layers);
    for (int l = 0; l < n_layers; ++l) { ptrs[l] = given_sigma[l]; ptrs[n_layers + l] = given_short[l]; }
    put(d_given, ptrs.data(), ptrs.size() * sizeof(const float*));
  }
  { const int rc = table_commit(ctx, tab, tables.data(), table_bytes, st); if (rc != ATOMO_OK) return rc; }
  launch_sp_begin(pay, gh, d_hdr_tmpl, n_layers, d_flag, nullptr, 0, st);          // payload header, layer headers, flags
  CK(cudaMemsetAsync(zero_beg, 0, zero_bytes, st));

  // ---- S1: Gram matrix, scaling ----
  stage_begin(ctx, ATOMO_STAGE_GRAM, st);
  if (given) {
    // singular values and short-side vectors as given: squared into the eigenvalue slots, vectors into the rows of X
    launch_sp_load_svd(d_layers, n_layers, d_given, d_given + n_layers, st);
  } else {
  if (ctx->eig_mode == 0) launch_sp_init(d_layers, n_layers, nullptr, 0, st);   // the identity half of [A | I]
  launch_sp_gram(d_layers, d_gram, (int)gram_tiles.size(), st);
  launch_sp_gram_tc(d_layers, d_maps, d_tc, (int)tc_tiles.size(), d_flag + 1, st);
  launch_sp_scale(d_layers, n_layers, st);
  }
  if (!given && ctx->eig_mode != 0 && !tri_form) {
    const int ec = launch_sp_cholesky(d_layers, n_layers, rp_max, st);
    if (ec != 0) return fail_cuda(ctx, (cudaError_t)ec, "cudaLaunchKernelEx(cholesky)");
    const int e = launch_sp_cholesky_big(d_layers, d_chol, (int)chol_ctas.size(), chol_panels, st);
    if (e != 0) return fail_cuda(ctx, (cudaError_t)e, "cudaLaunchCooperativeKernel(cholesky)");
  }
  stage_end(ctx, ATOMO_STAGE_GRAM, st, 5);
  CK(cudaGetLastError());

  // ---- S1: eigen-solver; the host reads a convergence flag once per sweep of the largest layer ----
  stage_begin(ctx, ATOMO_STAGE_EIG, st);
  int t_done = 0;
  int64_t n_eig_launch = 0;
  bool flags_pending = false;
  // Persistent form: the block pairs of a group of whole layers are co-resident (one CTA per SM) and solve their
  // layers in one cooperative launch.  A batch larger than the GPU is cut into such groups, launched one after
  // the other; a single layer with more block pairs than the GPU holds CTAs falls back to one launch per step.
  if (tri_form) {
    if (n_clusters > 0) {
      const int e = launch_sp_tridiag(d_layers, d_ctas, n_clusters, rp_max_small, st);
      if (e != 0) return fail_cuda(ctx, (cudaError_t)e, "cudaLaunchKernelEx(tridiagonal reduction)");
      ++n_eig_launch;
    }
    if (!big_layers.empty()) {
      // larger layers: a cluster of C CTAs each.  C is the smallest that holds the rows; it is doubled while the
      // batch still leaves SMs idle (the result does not depend on C)
      int sms = 148, dev = 0;
      if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
      int cmin = 1, rb = 0;
      for (int l : big_layers) { cmin = std::max(cmin, sp_tridiag_big_min_ctas(L[l].r)); rb = std::max(rb, L[l].r); }
      int cc = cmin;
      if (ctx->tri_big_ctas > 0) cc = std::max(cmin, ctx->tri_big_ctas);
      else {
        // (clusters sit inside one GPC each: the GPU holds fewer of them than SMs / CTAs, so ask)
        auto fits = [&](int c2) {
          const int mc = sp_tridiag_big_max_clusters(c2, rb);
          return mc > 0 ? (int)big_layers.size() <= mc : (int)big_layers.size() * c2 <= sms;
        };
        while (cc < 16 && fits(cc * 2)) cc *= 2;
        // up to a short side of 1024 one CTA per layer runs the triangle-only kernel, which beats a pair of CTAs on full
        // rows (40 layers: 25 ms against 36 ms); clusters pay from four CTAs per layer on
        if (cc == 2 && rb <= 1024) cc = 1;
      }
      const int e = launch_sp_tridiag_big(d_layers, d_big, (int)big_layers.size(), rb, cc, 0, st);
      if (e != 0) return fail_cuda(ctx, (cudaError_t)e, "cudaLaunchKernelEx(blocked tridiagonal reduction)");
      ++n_eig_launch;
    }
    // the eigenvalues (bisection) are timed with the sampling stage.  No host wait on this route: a bounded wait of
    // the Gram kernel that ran out is reported by the sampling kernel in every layer's status word
    // (ATOMO_ERR_TIMEOUT, nothing kept)
  }
  if (cluster_form) {
    const int e = launch_sp_jacobi_cluster(d_layers, d_ctas, n_clusters, rp_max, max_sweeps, ctx->tol, st);
    if (e != 0) return fail_cuda(ctx, (cudaError_t)e, "cudaLaunchKernelEx(jacobi clusters)");
    launch_sp_check(d_layers, n_layers, steps_max * max_sweeps, max_sweeps, d_flag, st);
    n_eig_launch = 2;
    CK(cudaMemsetAsync(d_flag + 2, 0, 2 * sizeof(uint32_t), st));
    CK(cudaMemcpyAsync(ctx->h_flag, d_flag, 4 * sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
    flags_pending = true;                                  // read at the end of the call, after everything is enqueued
  }
  const int capacity = (!given && !cluster_form && !tri_form && ctx->eig_scheme >= 1) ? sp_jacobi_persistent_capacity(row_floats_max) : 0;
  int max_layer_pairs = 0;
  for (int l = 0; l < n_layers; ++l) max_layer_pairs = std::max(max_layer_pairs, L[l].nb / 2);
  const bool persistent = capacity > 0 && max_layer_pairs <= capacity;
  if (!given) ctx->eig_scheme_used = tri_form ? 3 : cluster_form ? 2 : (persistent ? 1 : 0);
  if (cluster_form || tri_form || given) {
    // done above
  } else if (persistent) {
    // d_flag[2] is raised if a step barrier gave up, d_flag[3] receives the steps executed
    CK(cudaMemsetAsync(d_flag + 2, 0, 2 * sizeof(uint32_t), st));
    const int t_max = steps_max * max_sweeps;
    size_t first = 0;                                     // block_pairs is ordered by layer
    while (first < block_pairs.size()) {
      size_t last = first;
      while (last < block_pairs.size()) {
        const int l = block_pairs[last].layer;
        const size_t layer_pairs = (size_t)L[l].nb / 2;
        if (last + layer_pairs - first > (size_t)capacity) break;
        last += layer_pairs;
      }
      const int e = launch_sp_jacobi_persistent(d_layers, d_pairs + first, (int)(last - first), row_floats_max, max_sweeps,
                                                ctx->tol, d_flag + 2, st);
      if (e != 0) return fail_cuda(ctx, (cudaError_t)e, "cudaLaunchCooperativeKernel(jacobi)");
      ++n_eig_launch;
      first = last;
    }
    launch_sp_check(d_layers, n_layers, t_max, max_sweeps, d_flag, st);
    ++n_eig_launch;
    CK(cudaMemcpyAsync(ctx->h_flag, d_flag, 4 * sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
    flags_pending = true;                                  // read at the end of the call, after everything is enqueued
  } else
  for (int it = 0; it < max_sweeps; ++it) {
    for (int j = 0; j < steps_max; ++j, ++t_done, ++n_eig_launch)
      launch_sp_jacobi_step(d_layers, d_pairs, (int)block_pairs.size(), row_floats_max, t_done, max_sweeps, ctx->tol, st);
    launch_sp_check(d_layers, n_layers, t_done, max_sweeps, d_flag, st);
    CK(cudaMemcpyAsync(ctx->h_flag, d_flag, 2 * sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
    CK(cudaStreamSynchronize(st));
    if (ctx->h_flag[1] != 0) { ctx->err = "a bounded wait in the tensor-core Gram kernel ran out"; return ATOMO_ERR_TIMEOUT; }
    if (ctx->h_flag[0]) break;
  }
  stage_end(ctx, ATOMO_STAGE_EIG, st, n_eig_launch);

  // ---- S2-S4: (refined singular values,) probabilities, draws, compaction ----
  stage_begin(ctx, ATOMO_STAGE_SAMPLE, st);
  if (tri_form) {                                                   // all eigenvalues of the tridiagonal matrices
    int64_t n_eig = 0;
    for (int l = 0; l < n_layers; ++l) n_eig += L[l].r;
    launch_sp_bisect(d_layers, n_layers, r_max, n_eig, st);
  }
  launch_sp_refine(d_layers, n_layers, d_ref, (int)refine_tiles.size(), st);
  const PhiloxKey key{(uint32_t)seed, (uint32_t)(seed >> 32)};
  launch_sp_finalize_sample(d_layers, n_layers, s, key, kind_step_word(ATOMO_KIND_SPECTRAL, step), max_sweeps,
                            tri_form ? d_flag + 1 : nullptr, st);
  stage_end(ctx, ATOMO_STAGE_SAMPLE, st, tri_form ? 2 : 1);

  // ---- S4: long-side vectors of the kept atoms ----
  stage_begin(ctx, ATOMO_STAGE_BACKPROJECT, st);
  if (tri_form) {                                                   // short-side vectors of the kept atoms
    if (any_small) launch_sp_eigvec(d_layers, n_layers, rp_max_small, st);
    launch_sp_eigvec_big(d_layers, d_big, (int)big_layers.size(), rp_max, st);
  }
  launch_sp_backproject(d_layers, d_bp, (int)bp_tiles.size(), std::max(r_max_tall, 1), st);
  launch_sp_finish_atoms(d_layers, n_layers, k_cap_max, st);
  stage_end(ctx, ATOMO_STAGE_BACKPROJECT, st, tri_form ? 2 + (any_small ? 1 : 0) + (any_big ? 1 : 0) : 2);
  CK(cudaGetLastError());
  if (flags_pending) {
    // the one host wait of the persistent forms: the kernels' bounded waits report here
    CK(cudaStreamSynchronize(st));
    if (ctx->h_flag[1] != 0) { ctx->err = "a bounded wait in the tensor-core Gram kernel ran out"; return ATOMO_ERR_TIMEOUT; }
    if (ctx->h_flag[2] != 0) { ctx->err = "a step barrier of the persistent eigen-solve ran out of polls"; return ATOMO_ERR_TIMEOUT; }
  }
  return ATOMO_OK;
}

int atomo_encode_spectral(atomo_ctx* ctx, const atomo_mat* layers, int32_t n_layers, double s, uint64_t seed,
                          uint64_t step, int32_t k_cap, void* payload, int64_t capacity_bytes,
                          const atomo_debug* dbg, void* stream) {
  return encode_spectral_impl(ctx, layers, n_layers, s, seed, step, k_cap, payload, capacity_bytes, dbg, stream, nullptr, nullptr);
}

int atomo_encode_spectral_from_svd(atomo_ctx* ctx, const atomo_mat* layers, int32_t n_layers,
                                   const float* const* sigma, const float* const* short_vecs, double s, uint64_t seed,
                                   uint64_t step, int32_t k_cap, void* payload, int64_t capacity_bytes,
                                   const atomo_debug* dbg, void* stream) {
  if (!sigma || !short_vecs || n_layers <= 0) return ATOMO_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l) if (!sigma[l] || !short_vecs[l]) return ATOMO_ERR_INVALID_ARG;
  return encode_spectral_impl(ctx, layers, n_layers, s, seed, step, k_cap, payload, capacity_bytes, dbg, stream, sigma, short_vecs);
}

// ==================================================================================================
int atomo_encode_entrywise(atomo_ctx* ctx, const atomo_vec* vecs, int32_t n_vecs, double s, uint64_t seed,
                           uint64_t step, int64_t k_cap, void* payload, int64_t capacity_bytes,
                           const atomo_debug* dbg, void* stream) {
  if (!ctx || !vecs || n_vecs <= 0 || k_cap <= 0 || !payload) return ATOMO_ERR_INVALID_ARG;
  if (bad_budget(s)) return ATOMO_ERR_BUDGET;
  if ((reinterpret_cast<uintptr_t>(payload) & 15u) != 0) return ATOMO_ERR_INVALID_ARG;
  std::vector<int64_t> ns(n_vecs);
  for (int l = 0; l < n_vecs; ++l) {
    if (!vecs[l].data || vecs[l].n <= 0 || vecs[l].n >= (int64_t(1) << 32)) return ATOMO_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(vecs[l].data) & 3u) != 0) return ATOMO_ERR_INVALID_ARG;
    ns[l] = vecs[l].n;
  }
  std::vector<EwLayout> lay;
  const bool compact = ctx->ew_format == ATOMO_EW_COMPACT;
  const uint64_t total = layout_entrywise(ns.data(), n_vecs, k_cap, compact, ctx->ew_sat_cap, &lay);
  if ((int64_t)total > capacity_bytes) return ATOMO_ERR_CAPACITY;
  CK(cudaSetDevice(ctx->device));
  cudaStream_t st = (cudaStream_t)stream;
  stage_reset(ctx);
  uint8_t* pay = static_cast<uint8_t*>(payload);
  atomo_layer_header* d_hdr = reinterpret_cast<atomo_layer_header*>(pay + sizeof(atomo_payload_header));
  const int tile = ew_tile_elems();

  std::vector<EwVec> V(n_vecs);
  std::vector<char> fused(n_vecs, 0);
  size_t need = 0;
  uint8_t* ew_zero_beg = nullptr; size_t ew_zero_bytes = 0;
  const int max_blocks = ew_solve_max_blocks();
  if (max_blocks <= 0) return fail_cuda(ctx, cudaGetLastError(), "occupancy query for the cooperative solve");
  for (int pass = 0; pass < 2; ++pass) {
    Arena A(pass ? ctx->ws : nullptr);
    size_t dbg_atoms = 0, dbg_words = 0;
    for (int l = 0; l < n_vecs; ++l) {
      EwVec& v = V[l];
      v.g = vecs[l].data; v.n = vecs[l].n; v.layer = (uint32_t)l; v.k_cap = lay[l].kc;
      v.n_tiles = (v.n + tile - 1) / tile;
      int fused_ctas = 0;
      v.candidates = 0;
      if (ctx->ew_launch != 1) {
        // the one-kernel form, with the candidate list where the caller does not ask for the probabilities and the
        // budget is small enough for the list to pay
        const bool want_list = ctx->ew_launch == 0 && !(dbg && dbg->prob);
        const int with_list = want_list ? ew_encode_ctas(v.n_tiles, compact, true) : 0;
        if (with_list > 0 && ew_list_pays(v.n, v.n_tiles, with_list, s)) { fused_ctas = with_list; v.candidates = 1; }
        else fused_ctas = ew_encode_ctas(v.n_tiles, compact, false);
      }
      fused[l] = fused_ctas > 0;
      v.n_ctas = fused[l] ? fused_ctas : ew_sample_pack_ctas(v.n_tiles, compact);
      v.compact = compact ? 1 : 0; v.sat_cap = lay[l].sc;
      v.ent = reinterpret_cast<uint16_t*>(pay + lay[l].off_idx);
      v.sat_idx = reinterpret_cast<uint32_t*>(pay + lay[l].off_sat);
      v.sat_val = reinterpret_cast<float*>(pay + lay[l].off_val);
      const int64_t n_words = (v.n + 31) / 32;
      const bool want_mask = dbg && dbg->mask_words;           // the mask words leave the kernel only when asked for
      v.n_words = want_mask ? n_words : 0;
      const int64_t want_chunks = std::min<int64_t>(max_blocks, (v.n + 4095) / 4096);
      v.chunk = (int64_t)align_up((uint64_t)((v.n + want_chunks - 1) / want_chunks), 4);
      v.n_chunks = (int)((v.n + v.chunk - 1) / v.chunk);
      v.hdr = d_hdr + l;
      v.idx = reinterpret_cast<uint32_t*>(pay + lay[l].off_idx);
      v.val = reinterpret_cast<float*>(pay + lay[l].off_val);
      v.tile_table = reinterpret_cast<uint32_t*>(pay + lay[l].off_tiles);
      v.partials = A.take<EwPartial>((size_t)3 * std::max(v.n_chunks, v.n_ctas));
      v.state = A.take<EwState>(1);
      v.mask_words = want_mask ? dbg->mask_words + dbg_words : nullptr;
      v.prob_out = (dbg && dbg->prob) ? dbg->prob + dbg_atoms : nullptr;
      dbg_atoms += v.n; dbg_words += n_words;
    }
    // zero-filled per call: look-back status words and tile tickets of all vectors, one contiguous region
    uint8_t* zb = reinterpret_cast<uint8_t*>(A.take<uint32_t>(0));
    const size_t z0 = A.off;
    for (int l = 0; l < n_vecs; ++l) { V[l].tile_status = A.take<uint64_t>(V[l].n_ctas); V[l].ticket = A.take<uint32_t>(1); }
    ew_zero_beg = zb; ew_zero_bytes = A.off - z0;
    need = A.off + 256;
    if (pass == 0) { const int rc = ensure_ws(ctx, need); if (rc != ATOMO_OK) return rc; }
  }

  atomo_payload_header gh{};
  gh.magic = ATOMO_MAGIC; gh.version = ATOMO_VERSION; gh.kind = ATOMO_KIND_ENTRYWISE; gh.n_layers = (uint32_t)n_vecs;
  gh.total_bytes = total; gh.seed = seed; gh.step = step; gh.s = s;
  gh.ew_format = (uint64_t)ctx->ew_format; gh.ew_sat_cap = compact ? (uint64_t)ctx->ew_sat_cap : 0;
  {
    // layer header templates through the table cache; the headers themselves are written by a kernel
    std::vector<atomo_layer_header> tmpl(n_vecs);
    for (int l = 0; l < n_vecs; ++l) {
      atomo_layer_header h{};
      h.rows = 1; h.cols = ns[l]; h.k_cap = lay[l].kc; h.status = ATOMO_OK;
      h.off_idx = lay[l].off_idx; h.off_val = lay[l].off_val; h.off_short = lay[l].off_tiles;
      h.off_long = compact ? lay[l].off_sat : 0;
      tmpl[l] = h;
    }
    const size_t tb = tmpl.size() * sizeof(atomo_layer_header);
    { const int rc = table_reserve(ctx, ctx->tab_ew, tb); if (rc != ATOMO_OK) return rc; }
    { const int rc = table_commit(ctx, ctx->tab_ew, reinterpret_cast<const uint8_t*>(tmpl.data()), tb, st); if (rc != ATOMO_OK) return rc; }
  }
  // ... and the look-back status words and tickets of the sample / pack kernels start at zero.  A call with one vector
  // in the one-kernel form does all of this inside that kernel: one launch less.
  auto begin = [&]() {
    launch_sp_begin(pay, gh, reinterpret_cast<const atomo_layer_header*>(ctx->tab_ew.d), n_vecs, nullptr,
                    reinterpret_cast<uint32_t*>(ew_zero_beg), (int64_t)((ew_zero_bytes + 3) / 4), st);
  };
  const bool begin_inside = n_vecs == 1 && fused[0];
  EwBegin eb{};
  eb.pay = pay; eb.tmpl = reinterpret_cast<const atomo_layer_header*>(ctx->tab_ew.d); eb.gh = gh; eb.on = begin_inside ? 1 : 0;
  if (!begin_inside) begin();

  const PhiloxKey key{(uint32_t)seed, (uint32_t)(seed >> 32)};
  const uint32_t ks = kind_step_word(ATOMO_KIND_ENTRYWISE, step);
  // probabilities: one cooperative launch per vector (pass 1 and the water-filling rounds); a vector that fits one
  // wave of resident chunks goes on to sampling and packing inside the same launch (timed with the pack stage)
  int n_two = 0, n_one = 0;
  stage_begin(ctx, ATOMO_STAGE_EW_REDUCE, st);
  for (int l = 0; l < n_vecs; ++l) {
    if (fused[l]) continue;
    const int e = launch_ew_solve(V[l], s, st);
    if (e != 0) return fail_cuda(ctx, (cudaError_t)e, "cudaLaunchCooperativeKernel(ew_solve)");
    ++n_two;
  }
  stage_end(ctx, ATOMO_STAGE_EW_REDUCE, st, n_two);
  stage_begin(ctx, ATOMO_STAGE_EW_PACK, st);
  for (int l = 0; l < n_vecs; ++l) {
    if (!fused[l]) { launch_ew_sample_pack(V[l], key, ks, st); continue; }
    const int e = launch_ew_encode(V[l], s, key, ks, eb, st);
    if (e == (int)cudaErrorCooperativeLaunchTooLarge) {
      // fewer CTAs fit the GPU at once than the occupancy query promised: the two-kernel form takes the same chunks
      cudaGetLastError();
      fused[l] = 0;
      if (begin_inside) begin();
      const int e2 = launch_ew_solve(V[l], s, st);
      if (e2 != 0) return fail_cuda(ctx, (cudaError_t)e2, "cudaLaunchCooperativeKernel(ew_solve)");
      launch_ew_sample_pack(V[l], key, ks, st);
      n_one += 2;
      continue;
    }
    if (e != 0) return fail_cuda(ctx, (cudaError_t)e, "cudaLaunchCooperativeKernel(ew_encode)");
    ++n_one;
  }
  stage_end(ctx, ATOMO_STAGE_EW_PACK, st, (int64_t)(n_two + n_one));
  CK(cudaGetLastError());
  ctx->ew_last_state.resize(n_vecs); ctx->ew_last_chunks.resize(n_vecs);
  for (int l = 0; l < n_vecs; ++l) { ctx->ew_last_state[l] = V[l].state; ctx->ew_last_chunks[l] = fused[l] ? V[l].n_ctas : 0; }
  return ATOMO_OK;
}

int atomo_get_entrywise_list_chunks(atomo_ctx* ctx, int32_t vec, uint32_t* from_list, uint32_t* chunks) {
  if (!ctx || vec < 0 || vec >= (int32_t)ctx->ew_last_state.size()) return ATOMO_ERR_INVALID_ARG;
  CK(cudaSetDevice(ctx->device));
  CK(cudaDeviceSynchronize());
  uint32_t n = 0;
  if (ctx->ew_last_chunks[vec] > 0)
    CK(cudaMemcpy(&n, &ctx->ew_last_state[vec]->list_chunks, sizeof(n), cudaMemcpyDeviceToHost));
  if (from_list) *from_list = n;
  if (chunks) *chunks = (uint32_t)ctx->ew_last_chunks[vec];
  return ATOMO_OK;
}

// ==================================================================================================
int atomo_set_entrywise_launch(atomo_ctx* ctx, int32_t two_kernels) {
  if (!ctx || two_kernels < 0 || two_kernels > 2) return ATOMO_ERR_INVALID_ARG;
  ctx->ew_launch = two_kernels;
  return ATOMO_OK;
}

int atomo_lq_budget(atomo_ctx* ctx, const atomo_vec* vecs, int32_t n_vecs, double q, double* s_out, void* stream) {
  if (!ctx || !vecs || n_vecs <= 0 || !s_out || !(q >= 1.0)) return ATOMO_ERR_INVALID_ARG;
  for (int l = 0; l < n_vecs; ++l) {
    if (!vecs[l].data || vecs[l].n <= 0) return ATOMO_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(vecs[l].data) & 3u) != 0) return ATOMO_ERR_INVALID_ARG;
  }
  CK(cudaSetDevice(ctx->device));
  cudaStream_t st = (cudaStream_t)stream;
  const int n_ctas = 148 * 8;
  double* d_sum = nullptr; float* d_max = nullptr;
  for (int pass = 0; pass < 2; ++pass) {
    Arena A(pass ? ctx->ws : nullptr);
    d_sum = A.take<double>(n_ctas);
    d_max = A.take<float>(n_ctas);
    if (pass == 0) { const int rc = ensure_ws(ctx, A.off + 256); if (rc != ATOMO_OK) return rc; }
  }
  std::vector<double> h_sum(n_ctas);
  std::vector<float> h_max(n_ctas);
  for (int l = 0; l < n_vecs; ++l) {
    launch_ew_lq(vecs[l].data, vecs[l].n, 0, q, 0.0, d_sum, d_max, n_ctas, st);
    CK(cudaMemcpyAsync(h_sum.data(), d_sum, n_ctas * sizeof(double), cudaMemcpyDeviceToHost, st));
    CK(cudaMemcpyAsync(h_max.data(), d_max, n_ctas * sizeof(float), cudaMemcpyDeviceToHost, st));
    CK(cudaStreamSynchronize(st));
    double l1 = 0.0, amax = 0.0;
    for (int i = 0; i < n_ctas; ++i) { l1 += h_sum[i]; amax = std::max(amax, (double)h_max[i]); }
    if (!(amax <= 3.0e38) || !(l1 == l1)) { s_out[l] = std::nan(""); continue; }
    if (amax == 0.0) { s_out[l] = 0.0; continue; }
    double norm_q;
    if (std::isinf(q)) norm_q = amax;
    else if (q == 1.0) norm_q = l1;
    else {
      launch_ew_lq(vecs[l].data, vecs[l].n, 1, q, 1.0 / amax, d_sum, d_max, n_ctas, st);
      CK(cudaMemcpyAsync(h_sum.data(), d_sum, n_ctas * sizeof(double), cudaMemcpyDeviceToHost, st));
      CK(cudaStreamSynchronize(st));
      double t = 0.0;
      for (int i = 0; i < n_ctas; ++i) t += h_sum[i];
      norm_q = amax * std::pow(t, 1.0 / q);
    }
    s_out[l] = l1 / norm_q;
  }
  CK(cudaGetLastError());
  return ATOMO_OK;
}

// ==================================================================================================
int atomo_decode(atomo_ctx* ctx, int32_t kind, const void* payload, const int64_t* rows, const int64_t* cols,
                 float* const* out, int32_t n_layers, void* stream) {
  if (!ctx || !payload || !rows || !cols || !out || n_layers <= 0) return ATOMO_ERR_INVALID_ARG;
  if (kind != ATOMO_KIND_SPECTRAL && kind != ATOMO_KIND_ENTRYWISE) return ATOMO_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l) if (!out[l] || rows[l] <= 0 || cols[l] <= 0) return ATOMO_ERR_INVALID_ARG;
  CK(cudaSetDevice(ctx->device));
  cudaStream_t st = (cudaStream_t)stream;
  stage_reset(ctx);
  const uint8_t* pay = static_cast<const uint8_t*>(payload);
  const atomo_payload_header* d_gh = reinterpret_cast<const atomo_payload_header*>(pay);
  const atomo_layer_header* d_hdr = reinterpret_cast<const atomo_layer_header*>(pay + sizeof(atomo_payload_header));
  stage_begin(ctx, ATOMO_STAGE_DECODE, st);
  if (kind == ATOMO_KIND_ENTRYWISE) {
    for (int l = 0; l < n_layers; ++l) {
      if (rows[l] != 1) return ATOMO_ERR_INVALID_ARG;
      EwDecode d{pay, d_gh, d_hdr + l, out[l], cols[l]};
      launch_ew_decode(d, st);
    }
    stage_end(ctx, ATOMO_STAGE_DECODE, st, n_layers);
  } else {
    std::vector<SpDecodeLayer> D(n_layers);
    std::vector<TileRef> tiles;
    const int tr = sp_decode_tile_rows(), tc = sp_decode_tile_cols();
    for (int l = 0; l < n_layers; ++l) {
      D[l] = SpDecodeLayer{d_hdr + l, out[l], rows[l], cols[l]};
      const int na = (int)((rows[l] + tr - 1) / tr), nbt = (int)((cols[l] + tc - 1) / tc);
      for (int a = 0; a < na; ++a) for (int b = 0; b < nbt; ++b) tiles.push_back({l, a, b, 0});
    }
    SpDecodeLayer* d_layers = nullptr; TileRef* d_tiles = nullptr;
    size_t tb = 0;
    uint64_t key = table_key(kKeySeed, &payload, sizeof(payload));
    key = table_key(key, out, (size_t)n_layers * sizeof(float*));
    TableCache& tab = table_pick(ctx->tab_dec, key);
    for (int pass = 0; pass < 2; ++pass) {
      Arena T(pass ? tab.d : nullptr);
      d_layers = T.take<SpDecodeLayer>(n_layers);
      d_tiles = T.take<TileRef>(tiles.size());
      tb = T.off + 256;
      if (pass == 0) { const int rc = table_reserve(ctx, tab, tb); if (rc != ATOMO_OK) return rc; }
    }
    std::vector<uint8_t> tables(tb, 0);
    std::memcpy(tables.data() + (reinterpret_cast<uint8_t*>(d_layers) - tab.d), D.data(), D.size() * sizeof(SpDecodeLayer));
    std::memcpy(tables.data() + (reinterpret_cast<uint8_t*>(d_tiles) - tab.d), tiles.data(), tiles.size() * sizeof(TileRef));
    { const int rc = table_commit(ctx, tab, tables.data(), tb, st); if (rc != ATOMO_OK) return rc; }
    launch_sp_decode(pay, d_layers, d_tiles, (int)tiles.size(), st);
    stage_end(ctx, ATOMO_STAGE_DECODE, st, 1);
  }
  CK(cudaGetLastError());
  return ATOMO_OK;
}

// ==================================================================================================
int atomo_decode_average(atomo_ctx* ctx, int32_t kind, const void* const* payloads, int32_t n_payloads,
                         const int64_t* rows, const int64_t* cols, float* const* out, int32_t n_layers, void* stream) {
  if (!ctx || !payloads || n_payloads <= 0 || !rows || !cols || !out || n_layers <= 0) return ATOMO_ERR_INVALID_ARG;
  if (kind != ATOMO_KIND_SPECTRAL && kind != ATOMO_KIND_ENTRYWISE) return ATOMO_ERR_INVALID_ARG;
  for (int p = 0; p < n_payloads; ++p) if (!payloads[p]) return ATOMO_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l) {
    if (!out[l] || rows[l] <= 0 || cols[l] <= 0) return ATOMO_ERR_INVALID_ARG;
    if (kind == ATOMO_KIND_ENTRYWISE && rows[l] != 1) return ATOMO_ERR_INVALID_ARG;
  }
  CK(cudaSetDevice(ctx->device));
  cudaStream_t st = (cudaStream_t)stream;
  stage_reset(ctx);
  std::vector<SpDecodeLayer> D;
  std::vector<TileRef> tiles;
  if (kind == ATOMO_KIND_SPECTRAL) {
    D.resize(n_layers);
    const int tr = sp_decode_tile_rows(), tc = sp_decode_tile_cols();
    for (int l = 0; l < n_layers; ++l) {
      D[l] = SpDecodeLayer{nullptr, out[l], rows[l], cols[l]};
      const int na = (int)((rows[l] + tr - 1) / tr), nbt = (int)((cols[l] + tc - 1) / tc);
      for (int a = 0; a < na; ++a) for (int b = 0; b < nbt; ++b) tiles.push_back({l, a, b, 0});
    }
  }
  const uint8_t** d_pay = nullptr; SpDecodeLayer* d_layers = nullptr; TileRef* d_tiles = nullptr;
  size_t tb = 0;
  uint64_t key = table_key(kKeySeed, payloads, (size_t)n_payloads * sizeof(void*));
  key = table_key(key, out, (size_t)n_layers * sizeof(float*));
  TableCache& tab = table_pick(ctx->tab_avg, key);
  for (int pass = 0; pass < 2; ++pass) {
    Arena T(pass ? tab.d : nullptr);
    d_pay = T.take<const uint8_t*>(n_payloads);
    d_layers = T.take<SpDecodeLayer>(D.size());
    d_tiles = T.take<TileRef>(tiles.size());
    tb = T.off + 256;
    if (pass == 0) { const int rc = table_reserve(ctx, tab, tb); if (rc != ATOMO_OK) return rc; }
  }
  {
    std::vector<uint8_t> tables(tb, 0);
    std::memcpy(tables.data() + (reinterpret_cast<uint8_t*>(d_pay) - tab.d), payloads, (size_t)n_payloads * sizeof(void*));
    if (!D.empty()) std::memcpy(tables.data() + (reinterpret_cast<uint8_t*>(d_layers) - tab.d), D.data(), D.size() * sizeof(SpDecodeLayer));
    if (!tiles.empty()) std::memcpy(tables.data() + (reinterpret_cast<uint8_t*>(d_tiles) - tab.d), tiles.data(), tiles.size() * sizeof(TileRef));
    const int rc = table_commit(ctx, tab, tables.data(), tb, st);
    if (rc != ATOMO_OK) return rc;
  }
  stage_begin(ctx, ATOMO_STAGE_DECODE, st);
  if (kind == ATOMO_KIND_SPECTRAL) {
    launch_sp_decode_average(d_pay, n_payloads, d_layers, d_tiles, (int)tiles.size(), st);
    stage_end(ctx, ATOMO_STAGE_DECODE, st, 1);
  } else {
    for (int l = 0; l < n_layers; ++l) launch_ew_decode_average(d_pay, n_payloads, l, out[l], cols[l], st);
    stage_end(ctx, ATOMO_STAGE_DECODE, st, n_layers);
  }
  CK(cudaGetLastError());
  return ATOMO_OK;
}

// ==================================================================================================
int atomo_payload_read_headers(atomo_ctx* ctx, const void* payload, int32_t n_layers, atomo_payload_header* hdr,
                               atomo_layer_header* layers, void* stream) {
  if (!ctx || !payload || n_layers <= 0) return ATOMO_ERR_INVALID_ARG;
  CK(cudaSetDevice(ctx->device));
  cudaStream_t st = (cudaStream_t)stream;
  const uint8_t* pay = static_cast<const uint8_t*>(payload);
  if (hdr) CK(cudaMemcpyAsync(hdr, pay, sizeof(*hdr), cudaMemcpyDeviceToHost, st));
  if (layers)
    CK(cudaMemcpyAsync(layers, pay + sizeof(atomo_payload_header), (size_t)n_layers * sizeof(atomo_layer_header),
                       cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  return ATOMO_OK;
}

int atomo_payload_status(atomo_ctx* ctx, const void* payload, int32_t n_layers, int32_t* worst, int32_t* first_bad_layer,
                         void* stream) {
  if (!ctx || !payload || n_layers <= 0) return ATOMO_ERR_INVALID_ARG;
  std::vector<atomo_layer_header> h(n_layers);
  const int rc = atomo_payload_read_headers(ctx, payload, n_layers, nullptr, h.data(), stream);
  if (rc != ATOMO_OK) return rc;
  int32_t w = ATOMO_OK, first = -1;
  for (int l = 0; l < n_layers; ++l)
    if (h[l].status != ATOMO_OK && first < 0) { w = (int32_t)h[l].status; first = l; }
  if (worst) *worst = w;
  if (first_bad_layer) *first_bad_layer = first;
  return ATOMO_OK;
}

}  // extern "C"
