// Gram matrix of the short side on the 5th-generation tensor cores (tcgen05, sm_100a), for layers with
// rows <= cols (the short-side vectors are rows of G, contiguous along the contraction).
//
//   A = G G^T  in fp32-level accuracy from TF32 instructions: every operand x is split as x = hi + lo with
//   hi = the nearest TF32 number to x and lo = the nearest TF32 number to x - hi (rounding to nearest keeps
//   the split unbiased; x - hi is exact in fp32); each 128 x 128 x 8 step issues three MMAs,
//   hi*hi + hi*lo + lo*hi, into one fp32 accumulator in TMEM (the lo*lo term is below fp32 resolution).
//
//   The tensor core adds into its fp32 accumulator with truncation (measured: about 3e-8 of the running sum per
//   MMA, 5e-5 of a same-sign sum over K = 4608 -- far too coarse for the small eigenvalues).  So an accumulator
//   only ever collects one stage of 32 columns (12 MMAs); it is then drained and added to fp32 registers by the
//   CUDA cores (round to nearest) while the MMAs of the next stage fill the second accumulator.
//
// One CTA per 128 x 128 output tile of the upper triangle (the mirror is written by the epilogue).
//   warp 0      TMA producer: raw fp32 tiles of 128 rows x 32 columns (128-byte rows, 128B swizzle), no multicast
//   warp 1      allocates TMEM and issues the MMAs from one lane; tcgen05.commit frees a stage and hands
//               the accumulator to the drain warps
//   warps 2-5   split the raw tile in place into hi and write lo at the same (swizzled) offsets of a second buffer
//   warps 6-9   drain: TMEM -> registers, running sums in registers, at the end registers -> global
// Every mbarrier wait is bounded; a wait that runs out sets an error word and the CTA leaves through
// the common exit (TMEM is freed).
#include <cuda.h>

#include "atomo_kernels.cuh"

namespace atomo {

constexpr int kTcTile = 128;                       // output tile edge (UMMA M = N = 128)
constexpr int kTcKBlk = 32;                        // fp32 per row per stage = 128 bytes = one swizzle atom
constexpr int kTcStages = 3;
constexpr int kTcTileBytes = kTcTile * kTcKBlk * 4;   // 16 KB
constexpr int kTcStageBytes = 4 * kTcTileBytes;       // a_hi, a_lo, b_hi, b_lo
constexpr int kTcThreads = 320;                    // TMA warp, MMA warp, 4 split warps, 4 drain warps
constexpr int kTcSmemBytes = kTcStages * kTcStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr uint32_t kTcTmemCols = 256;               // two 128-column fp32 accumulators
constexpr int kTcSpin = 1 << 20;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void tc_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void tc_mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// bounded wait for the phase with the given parity; also gives up when another role has set the abort word
__device__ __forceinline__ bool tc_mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_word) {
  for (int it = 0; it < kTcSpin; ++it) {
    uint32_t ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (ok) return true;
    if ((it & 63) == 63 && *abort_word) return false;
  }
  *abort_word = 1u;
  return false;
}
__device__ __forceinline__ void tc_tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
// K-major operand, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t addr) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | (1ull << 16) /*LBO (unused)*/ | (64ull << 32) /*SBO = 1024 B*/ |
         (1ull << 46) /*descriptor version*/ | (2ull << 61) /*SWIZZLE_128B*/;
}
// kind::tf32, fp32 accumulator, A and B K-major, M = 128, N = 128
constexpr uint32_t kTcIdesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(kTcTile >> 3) << 17) | ((uint32_t)(kTcTile >> 4) << 24);

__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}\n"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(kTcIdesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u) : "memory");
}
// nearest TF32 number (10 explicit mantissa bits; ties away from zero): the tensor core then reads it exactly
__device__ __forceinline__ float tf32_round(float x) {
  return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xFFFFE000u);
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__global__ void __launch_bounds__(kTcThreads, 1) sp_gram_tc_kernel(const SpLayer* __restrict__ layers,
                                                                   const CUtensorMap* __restrict__ maps,
                                                                   const TileRef* __restrict__ tiles,
                                                                   uint32_t* __restrict__ err) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;       // 1024-byte aligned tiles
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + kTcStages * kTcStageBytes;
  // barriers: full[s] (TMA landed), conv[s] (hi/lo ready), empty[s] (MMAs of the stage done), acc (all MMAs done)
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto conv_bar = [&](int s) { return bars + 8u * (kTcStages + s); };
  auto empty_bar = [&](int s) { return bars + 8u * (2 * kTcStages + s); };
  auto tfull_bar = [&](int b) { return bars + 8u * (3 * kTcStages + b); };        // accumulator b holds one stage's sum
  auto tempty_bar = [&](int b) { return bars + 8u * (3 * kTcStages + 2 + b); };   // accumulator b has been drained
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(base_ptr + kTcStages * kTcStageBytes + 8 * (3 * kTcStages + 4));
  volatile uint32_t* s_abort = s_tmem + 1;
  volatile uint32_t* s_last = s_tmem + 2;

  const TileRef ref = tiles[blockIdx.x];
  const SpLayer& L = layers[ref.layer];
  const CUtensorMap* map = maps + ref.layer;
  const int ti = ref.a, tj = ref.b;
  const bool diag = ti == tj;
  // a tile's K range may be split over L.gram_split CTAs (ref.c = which part); the parts are added by the last
  // CTA of the tile to finish, in part order
  const int all_kb = (L.L + kTcKBlk - 1) / kTcKBlk;
  const int n_split = L.gram_split;
  const int kb_lo = (int)((int64_t)all_kb * ref.c / n_split), kb_hi = (int)((int64_t)all_kb * (ref.c + 1) / n_split);
  const int num_kb = kb_hi - kb_lo;                         // stage / phase arithmetic below counts from kb_lo
  const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;

  if (tid == 0) {
    for (int s = 0; s < kTcStages; ++s) { tc_mbar_init(full_bar(s), 1); tc_mbar_init(conv_bar(s), 128); tc_mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { tc_mbar_init(tfull_bar(b), 1); tc_mbar_init(tempty_bar(b), 128); }
    *s_abort = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)s_tmem)), "r"(kTcTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_d = *s_tmem;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % kTcStages;
        const uint32_t ph = (uint32_t)(kb / kTcStages) & 1u;
        if (!tc_mbar_wait(empty_bar(s), ph ^ 1u, s_abort)) break;
        const uint32_t stage = base + s * kTcStageBytes;
        tc_mbar_expect_tx(full_bar(s), diag ? kTcTileBytes : 2 * kTcTileBytes);
        tc_tma_load_2d(stage, map, full_bar(s), (kb_lo + kb) * kTcKBlk, ti * kTcTile);
        if (!diag) tc_tma_load_2d(stage + 2 * kTcTileBytes, map, full_bar(s), (kb_lo + kb) * kTcKBlk, tj * kTcTile);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % kTcStages, buf = kb & 1;
        const uint32_t ph = (uint32_t)(kb / kTcStages) & 1u;
        if (!tc_mbar_wait(tempty_bar(buf), ((uint32_t)(kb >> 1) & 1u) ^ 1u, s_abort)) break;   // accumulator drained
        if (!tc_mbar_wait(conv_bar(s), ph, s_abort)) break;                                    // hi / lo ready
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t a_hi = base + s * kTcStageBytes, a_lo = a_hi + kTcTileBytes;
        const uint32_t b_hi = diag ? a_hi : a_hi + 2 * kTcTileBytes, b_lo = diag ? a_lo : a_hi + 3 * kTcTileBytes;
        const uint32_t d = tmem_d + (uint32_t)buf * kTcTile;
#pragma unroll
        for (int k = 0; k < kTcKBlk / 8; ++k) {                       // UMMA K = 8 tf32 = 32 bytes
          const uint32_t off = k * 32;
          tc_mma(d, tc_smem_desc(a_lo + off), tc_smem_desc(b_hi + off), k > 0 ? 1u : 0u);      // small terms first
          tc_mma(d, tc_smem_desc(a_hi + off), tc_smem_desc(b_lo + off), 1u);
          tc_mma(d, tc_smem_desc(a_hi + off), tc_smem_desc(b_hi + off), 1u);
        }
        tc_commit(empty_bar(s));                                       // the stage may be refilled when these are done
        tc_commit(tfull_bar(buf));                                     // ... and the accumulator may be drained
      }
    }
  } else if (warp < 6) {
    // ---------------- hi / lo split (warps 2..5, 128 threads) ----------------
    const int ct = tid - 64;
    for (int kb = 0; kb < num_kb; ++kb) {
      const int s = kb % kTcStages;
      const uint32_t ph = (uint32_t)(kb / kTcStages) & 1u;
      if (!tc_mbar_wait(full_bar(s), ph, s_abort)) break;
      uint8_t* stage = base_ptr + s * kTcStageBytes;
      const int n_op = diag ? 1 : 2;
      for (int op = 0; op < n_op; ++op) {
        float4* hi = reinterpret_cast<float4*>(stage + op * 2 * kTcTileBytes);
        float4* lo = reinterpret_cast<float4*>(stage + op * 2 * kTcTileBytes + kTcTileBytes);
#pragma unroll
        for (int j = 0; j < kTcTileBytes / 16 / 128; ++j) {
          const int idx = ct + 128 * j;
          const float4 x = hi[idx];
          float4 h, l;
          h.x = tf32_round(x.x); l.x = tf32_round(x.x - h.x);
          h.y = tf32_round(x.y); l.y = tf32_round(x.y - h.y);
          h.z = tf32_round(x.z); l.z = tf32_round(x.z - h.z);
          h.w = tf32_round(x.w); l.w = tf32_round(x.w - h.w);
          hi[idx] = h; lo[idx] = l;
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the tensor core
      tc_mbar_arrive(conv_bar(s));
    }
  } else {
    // ---------------- drain (warps 6..9): warp q of the group reads TMEM lanes 32 q .. 32 q + 31 (q = warp % 4) ----------------
    const int q = warp % 4;
    const int row = 32 * q + lane;
    float acc[kTcTile];
#pragma unroll
    for (int j = 0; j < kTcTile; ++j) acc[j] = 0.0f;
    bool ok = true;
    for (int kb = 0; kb < num_kb && ok; ++kb) {
      const int buf = kb & 1;
      if (!tc_mbar_wait(tfull_bar(buf), (uint32_t)(kb >> 1) & 1u, s_abort)) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
      for (int c0 = 0; c0 < kTcTile; c0 += 32) {
        uint32_t v[32];
        const uint32_t taddr = tmem_d + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * kTcTile + c0);
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
            "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
            "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
              "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
              "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
              "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
            : "r"(taddr) : "memory");
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int j = 0; j < 32; ++j) acc[c0 + j] += __uint_as_float(v[j]);
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      tc_mbar_arrive(tempty_bar(buf));
    }
    // Epilogue.  The stage buffers are free now (every load has landed and every MMA has completed): the tile goes
    // through shared memory (row stride 129 floats, conflict-free both ways) so that both triangles of A are written
    // with consecutive lanes on consecutive addresses.
    const int r = L.r;
    const int64_t lda = L.lda;
    float* A = L.A;
    float* s_tile = reinterpret_cast<float*>(base_ptr);
    constexpr int kPad = kTcTile + 1;
    const int dt = tid - 6 * 32;                               // 0 .. 127 among the drain warps (= row)
    bool write_tile = ok;
    if (n_split > 1) {
      // this part's tile to the workspace, column-major (consecutive lanes, consecutive addresses)
      const int tt = (r + kTcTile - 1) / kTcTile;
      const int tile_id = ti * tt - ti * (ti - 1) / 2 + (tj - ti);
      float* part = L.gram_part + ((int64_t)tile_id * n_split + ref.c) * (kTcTile * kTcTile);
#pragma unroll
      for (int j = 0; j < kTcTile; ++j) part[j * kTcTile + row] = acc[j];
      __threadfence();
      asm volatile("bar.sync 2, 128;" ::: "memory");           // the four drain warps
      if (dt == 0) *s_last = atomicAdd(L.gram_ticket + tile_id, 1u) == (uint32_t)(n_split - 1) ? 1u : 0u;
      asm volatile("bar.sync 2, 128;" ::: "memory");
      write_tile = *s_last != 0;                               // the last part to finish adds them all, in part order
      if (write_tile) {
        __threadfence();
        const float* parts = L.gram_part + (int64_t)tile_id * n_split * (kTcTile * kTcTile);
#pragma unroll
        for (int j = 0; j < kTcTile; ++j) acc[j] = 0.f;
        for (int sp = 0; sp < n_split; ++sp) {
          const float* ps = parts + (int64_t)sp * (kTcTile * kTcTile) + row;
#pragma unroll
          for (int j = 0; j < kTcTile; ++j) acc[j] += __ldcg(ps + j * kTcTile);
        }
      }
    }
    if (write_tile) {                                          // uniform over the drain warps
#pragma unroll
      for (int j = 0; j < kTcTile; ++j) s_tile[row * kPad + j] = acc[j];
      asm volatile("bar.sync 2, 128;" ::: "memory");
      const int gcol = tj * kTcTile + dt, grow_m = ti * kTcTile + dt;
      for (int rr = 0; rr < kTcTile; ++rr) {
        const int gi = ti * kTcTile + rr, gj = tj * kTcTile + rr;
        if (gi < r && gcol < r) A[(int64_t)gi * lda + gcol] = s_tile[rr * kPad + dt];
        if (!diag && gj < r && grow_m < r) A[(int64_t)gj * lda + grow_m] = s_tile[dt * kPad + rr];
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(kTcTmemCols) : "memory");
  }
  if (tid == 0 && *s_abort) atomicExch(err, (uint32_t)ATOMO_ERR_TIMEOUT);
}

// ---- host side ------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode_tiled = nullptr;

int sp_tc_configure() {
  if (g_encode_tiled == nullptr) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    const cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return (int)e;
    if (qres != cudaDriverEntryPointSuccess || fn == nullptr) return (int)cudaErrorNotSupported;
    g_encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
  }
  return (int)cudaFuncSetAttribute(sp_gram_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemBytes);
}

// rows <= cols, 16-byte aligned base and row pitch: the layer can take the tensor-core Gram kernel
bool sp_tc_eligible(const float* g, int rows, int cols, int64_t ld) {
  return rows <= cols && (reinterpret_cast<uintptr_t>(g) & 15u) == 0 && (ld % 4) == 0 && g_encode_tiled != nullptr;
}

// tensor map of G (rows x cols, row pitch ld): boxes of 32 columns x 128 rows, 128-byte swizzle, zero fill outside
int sp_tc_make_map(void* out_map /*CUtensorMap, host*/, const float* g, int rows, int cols, int64_t ld) {
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 4};
  const cuuint32_t box[2] = {(cuuint32_t)kTcKBlk, (cuuint32_t)kTcTile};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = g_encode_tiled(reinterpret_cast<CUtensorMap*>(out_map), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                                    const_cast<float*>(g), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : 1;
}

int sp_tc_map_bytes() { return (int)sizeof(CUtensorMap); }
int sp_tc_tile() { return kTcTile; }

void launch_sp_gram_tc(const SpLayer* d_layers, const void* d_maps, const TileRef* d_tiles, int n_tiles, uint32_t* d_err,
                       cudaStream_t st) {
  if (n_tiles > 0)
    sp_gram_tc_kernel<<<n_tiles, kTcThreads, kTcSmemBytes, st>>>(d_layers, reinterpret_cast<const CUtensorMap*>(d_maps),
                                                                 d_tiles, d_err);
}

}  // namespace atomo
