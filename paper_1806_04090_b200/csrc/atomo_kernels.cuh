// Device-side descriptors and kernel launchers shared by the API translation unit.
#pragma once
#include "atomo_common.cuh"

namespace atomo {

// ================================= entry-wise path ===============================================
constexpr int kEwMaxRounds = 64;      // water-filling rounds; Algorithm 1 saturates < ceil(s) atoms,
                                      // a round usually takes many at once

struct EwPartial { double sum; float amax; uint32_t cnt; uint32_t nonfinite; };

struct EwState {
  double T0;        // ||g||_1
  double T;         // sum of |g| over unsaturated atoms
  double s_cur;     // s - n_sat
  double theta;     // atoms with |g| > theta have p = 1
  float scale;      // p_i = |g_i| * scale for the rest
  float c;          // T / s_cur
  float theta_f, amax;
  uint32_t n_sat, rounds, done, nonfinite;
  uint32_t list_chunks; // one-kernel form: chunks whose keep decisions were taken on the candidate list (test introspection)
};

struct EwVec {
  const float* g; int64_t n;
  uint32_t layer; uint32_t k_cap;
  int64_t chunk; int n_chunks;            // reduction split (chunk is a multiple of 4)
  int64_t n_tiles; int64_t n_words;
  atomo_layer_header* hdr; uint32_t* idx; float* val;          // payload
  EwPartial* partials; EwState* state;                         // workspace
  uint32_t* mask_words;
  int n_ctas;                                                  // chunks (CTAs) of the sample / pack kernel
  uint64_t* tile_status;                                       // [chunks] ready flag (bit 63) | kept atoms of the chunk; zeroed per call
  uint32_t* ticket;                                            // next chunk to hand out; zeroed per call
  uint32_t* tile_table;                                        // payload: kept atoms before each tile
  float* prob_out;                                             // debug or nullptr
  // compact payload format (else compact = 0 and the rest unused)
  int compact; uint32_t sat_cap;
  int candidates;                                              // one-kernel form: keep a candidate list during the first pass (else read the chunk twice)
  uint16_t* ent;                                               // [k_cap] tile-local index | sign << 15 of kept atoms with p < 1
  uint32_t* sat_idx; float* sat_val;                           // [sat_cap] atoms with p = 1
};

struct EwDecode {
  const uint8_t* payload; const atomo_payload_header* ghdr; const atomo_layer_header* hdr;
  float* out; int64_t n;
};

int ew_solve_max_blocks();                                     // co-resident CTAs of the cooperative solve
int launch_ew_solve(const EwVec& v, double s, cudaStream_t st); // returns a cudaError_t
void launch_ew_sample_pack(const EwVec& v, PhiloxKey key, uint32_t kind_step, cudaStream_t st);
void launch_ew_decode(const EwDecode& d, cudaStream_t st);
int ew_tile_elems();
void launch_ew_lq(const float* g, int64_t n, int pass, double q, double inv_amax, double* part_sum, float* part_max,
                  int n_ctas, cudaStream_t st);
int ew_sample_pack_ctas(int64_t n_tiles, bool compact);
int ew_encode_ctas(int64_t n_tiles, bool compact, bool list);  // CTAs of the one-kernel form (with or without the candidate list); 0 = the vector needs the two-kernel form
bool ew_list_pays(int64_t n, int64_t n_tiles, int ctas, double s);   // whether the candidate list is worth keeping at this budget
// what the header kernel would do for a call with one vector, done by the one-kernel form itself (on = 0: not asked for)
struct EwBegin { uint8_t* pay; const atomo_layer_header* tmpl; atomo_payload_header gh; int on; };
int launch_ew_encode(const EwVec& v, double s, PhiloxKey key, uint32_t kind_step, const EwBegin& begin, cudaStream_t st);   // cudaError_t

// ================================= spectral path =================================================
constexpr int kMaxShort = 4096;       // largest short side (atoms per layer)
constexpr int kSmemRowsMaxRp = 4096;  // largest padded short side the shared-memory Jacobi kernel holds

struct SpLayer {
  const float* G; int rows, cols; int64_t ld;
  int r, L, tall;              // short side, long side, rows > cols
  int rp, B, nb;               // padded short side, Jacobi block rows, number of blocks (even)
  uint32_t layer, k_cap;
  int acc;                     // eigen-solver route: 1 = rows [x | v] of [A | I] (mode 0), 0 = rows of L^T (mode 1)
  int ldx;                     // floats per row of X: 2 rp (acc) or rp
  float* A; int64_t lda;       // scaled Gram matrix, r x r valid (mode 0: the left half of X)
  float* X;                    // rp x ldx working rows of the Jacobi solver
  atomo_layer_header* hdr;     // payload
  uint32_t* idx; float* coef; float* shortv; float* longv;
  float* lam;                  // rp   squared norm per row of X as the cluster eigen-solve left it (scaled units)
  int lam_ready;               // lam was written by the eigen-solve (cluster form): finalize need not re-read X for it
  int* perm;                   // r    rank -> row
  float* sigma; float* prob;   // r    descending (debug buffers or workspace)
  uint32_t* mask_words;        // ceil(r/32)
  float* p_sel;                // k_cap: p of the kept atoms
  float* bp_part;              // [bp_chunks][k_cap][L] row-chunk partial sums of the long vectors
  int bp_tiles, bp_chunks, bp_chunk_rows;
  uint32_t* rot_count;         // [max_sweeps] rotations applied in each sweep
  uint32_t* step_bar;          // arrivals of the layer's CTAs at the step barrier of the persistent eigen-solve
  float* scale;                // 1 float: power-of-two scaling applied to A
  float* chol_dd;              // 32 x 32 + 32 floats: diagonal block of the current Cholesky panel, published by its owner
  float* dbg_short;            // r x r or nullptr
  int tc;                      // Gram matrix came from the tensor-core kernel (see sp_scale_kernel)
  int gram_split;              // tensor-core Gram: CTAs per output tile (parts of the K range), 1 = no split
  float* gram_part;            // [tiles][gram_split][128 x 128] partial tiles (column-major) when gram_split > 1
  uint32_t* gram_ticket;       // [tiles] parts finished; zeroed per call
  int refine, refine_tiles;    // singular values from the projection norms; tiles along the long side
  float* row_inv;              // rp: 1 / norm of each short-side vector as stored in X
  float* refine_partials;      // [refine_tiles][rp] partial squared norms
  // tridiagonal route (short side <= 512): T = Q^T A Q, eigenvalues by bisection, vectors of the kept atoms only
  int tri;                     // this layer takes the tridiagonal route: 1 = registers of a cluster (rp <= 512), 2 = blocked, A in global memory
  double* td_d; double* td_e;  // rp each: diagonal and off-diagonal of T
  double* td_tau;              // rp: beta_k of the reflectors H_k = I - beta_k v_k v_k^T
  int td_ldv;                  // floats per row of td_V: r rounded up to a multiple of 4 (16-byte rows)
  float* td_V;                 // r x td_ldv: row k = v_k / ||v_k|| (zero up to index k), fp32 for the back-transformation: H_k = I - 2 u u^T
  double* lam64;               // rp: eigenvalues of T, ascending (scaled units); lam holds the same in fp32
  uint32_t* vec_ticket;        // CTAs of the vector kernel that finished this layer; zeroed per call
  // tridiagonal route for short sides above 512 (tri = 2): blocked Householder reduction with A in global memory
  void* tb_A;                  // r x lda matrix the reduction works on: float (= A) or double (tb_fp64)
  void* tb_W;                  // [panel][tb_ldw] the panel's w vectors, same type as tb_A
  int64_t tb_ldw;
  int tb_fp64;                 // matrix and panel vectors in fp64
  double* tb_vecwork;          // [slots][5][rp] work vectors of the twisted factorisation
  float* tb_At;                // short side <= 1024: the lower triangle in tile-major order (32 x 32 sub-tiles of 4 KB), the
                               // working copy of the one-CTA-per-layer kernel
};

struct SpDecodeLayer {
  const atomo_layer_header* hdr; float* out; int64_t rows, cols;
};

struct TileRef { int32_t layer, a, b, c; };

// averaging decode of several payloads (combine step of data-parallel training)
void launch_sp_decode_average(const uint8_t* const* d_payloads, int n_payloads, const SpDecodeLayer* d_layers,
                              const TileRef* d_tiles, int n_tiles, cudaStream_t st);
void launch_ew_decode_average(const uint8_t* const* d_payloads, int n_payloads, int layer, float* out, int64_t n,
                              cudaStream_t st);

// payload header (by value), layer headers from a device template, the call's four flag words (may be null)
void launch_sp_begin(uint8_t* pay, const atomo_payload_header& gh, const atomo_layer_header* d_tmpl, int n_layers,
                     uint32_t* d_flags, uint32_t* d_zero, int64_t n_zero, cudaStream_t st);
void launch_sp_init(const SpLayer* d_layers, int n_layers, const TileRef* d_diag_tiles, int n_diag_tiles, cudaStream_t st);
void launch_sp_gram(const SpLayer* d_layers, const TileRef* d_tiles, int n_tiles, cudaStream_t st);
void launch_sp_scale(const SpLayer* d_layers, int n_layers, cudaStream_t st);   // trace, then scaling
void launch_sp_load_svd(const SpLayer* d_layers, int n_layers, const float* const* d_sigma, const float* const* d_vecs,
                        cudaStream_t st);                                       // a decomposition given by the caller
// one Jacobi step (global step index t) for every layer of the batch
void launch_sp_jacobi_step(const SpLayer* d_layers, const TileRef* d_pairs, int n_pairs, int row_floats_max,
                           int t, int max_sweeps, float tol, cudaStream_t st);
// whole eigen-solve of a group of layers in one cooperative launch (block pairs co-resident); returns a cudaError_t
int sp_jacobi_persistent_capacity(int row_floats_max);
int launch_sp_jacobi_persistent(const SpLayer* d_layers, const TileRef* d_pairs, int n_pairs, int row_floats_max,
                                int max_sweeps, float tol, uint32_t* d_state, cudaStream_t st);
// layers of up to 1024 rows: clusters of 8 CTAs; more rows: cooperative launch.  Both return a cudaError_t
// cluster form of the persistent eigen-solve (layers of up to 16 block pairs); one entry per CTA of a cluster
struct ClusterCta { int32_t layer, slot, base_rank, pad; };       // layer < 0: this CTA only keeps the barriers
int sp_jacobi_cluster_ctas();                                     // CTAs per cluster
int sp_jacobi_cluster_max_rp();                                   // largest padded short side it takes
int sp_jacobi_cluster_capacity(int rp_max);                       // co-resident clusters (0: not available here)
int launch_sp_jacobi_cluster(const SpLayer* d_layers, const ClusterCta* d_ctas, int n_clusters, int rp_max, int max_sweeps,
                             float tol, cudaStream_t st);         // returns a cudaError_t
// tridiagonal route (atomo_tridiag.cu)
int sp_tridiag_max_rp();
int sp_tridiag_cluster_ctas();
int sp_tridiag_ctas_of(int rp);                                   // CTAs a layer of padded short side rp takes
int sp_configure_tridiag();                                       // co-resident clusters (0: route not available)
int launch_sp_tridiag(const SpLayer* d_layers, const ClusterCta* d_ctas, int n_clusters, int rp_max, cudaStream_t st);  // cudaError_t
void launch_sp_bisect(const SpLayer* d_layers, int n_layers, int r_max, int64_t n_eigenvalues, cudaStream_t st);
void launch_sp_eigvec(const SpLayer* d_layers, int n_layers, int rp_max, cudaStream_t st);
// tridiagonal route for short sides above 512 (atomo_tridiag_big.cu)
int sp_tridiag_big_max_r();
int sp_tridiag_big_panel();
int sp_tridiag_big_min_ctas(int r);                               // fewest CTAs per layer that hold r rows
int sp_eigvec_big_slots();                                        // warps per layer of the vector kernel (work vectors)
int sp_configure_tridiag_big();                                   // 0 if available
int sp_tridiag_big_max_clusters(int ctas, int r_max);              // co-resident clusters of that many CTAs (0: unknown)
int sp_configure_bisect();                                        // 0 if the eigenvalue kernel got its shared memory
int launch_sp_tridiag_big(const SpLayer* d_layers, const int* d_big, int n_big, int r_max, int ctas, int fp64, cudaStream_t st);  // cudaError_t
void launch_sp_eigvec_big(const SpLayer* d_layers, const int* d_big, int n_big, int rp_max, cudaStream_t st);
int launch_sp_cholesky(const SpLayer* d_layers, int n_layers, int rp_max, cudaStream_t st);
int launch_sp_cholesky_big(const SpLayer* d_layers, const TileRef* d_ctas, int n_ctas, int max_panels, cudaStream_t st);
int sp_cholesky_big_rows_per_cta();
int sp_configure_eig();
// convergence bookkeeping after t_done steps were enqueued
void launch_sp_check(const SpLayer* d_layers, int n_layers, int t_done, int max_sweeps, uint32_t* d_all_done,
                     cudaStream_t st);
void launch_sp_refine(const SpLayer* d_layers, int n_layers, const TileRef* d_tiles, int n_tiles, cudaStream_t st);
// timeout_flag (device, may be null): non-zero means a bounded wait of an earlier kernel of the call ran out;
// every layer then reports ATOMO_ERR_TIMEOUT and keeps nothing
void launch_sp_finalize_sample(const SpLayer* d_layers, int n_layers, double s, PhiloxKey key,
                               uint32_t kind_step, int max_sweeps, const uint32_t* timeout_flag, cudaStream_t st);
void launch_sp_backproject(const SpLayer* d_layers, const TileRef* d_tiles, int n_tiles, int r_max, cudaStream_t st);
void launch_sp_finish_atoms(const SpLayer* d_layers, int n_layers, int k_cap_max, cudaStream_t st);
void launch_sp_decode(const uint8_t* payload, const SpDecodeLayer* d_layers, const TileRef* d_tiles, int n_tiles,
                      cudaStream_t st);
int sp_configure();          // opt in to large dynamic shared memory; returns cudaError_t
// tensor-core Gram kernel (atomo_tc.cu)
int sp_tc_configure();       // driver entry point for tensor maps + shared memory opt-in; returns cudaError_t
bool sp_tc_eligible(const float* g, int rows, int cols, int64_t ld);
int sp_tc_make_map(void* out_map, const float* g, int rows, int cols, int64_t ld);   // 0 on success
int sp_tc_map_bytes();
int sp_tc_tile();
void launch_sp_gram_tc(const SpLayer* d_layers, const void* d_maps, const TileRef* d_tiles, int n_tiles, uint32_t* d_err,
                       cudaStream_t st);
int sp_bp_rows_per_tile();
int sp_bp_cols_per_tile();
int sp_bp_chunk_rows();
int sp_decode_tile_rows();
int sp_decode_tile_cols();

}  // namespace atomo
