/*
 * atomo.h -- C ABI of the B200 (sm_100a) ATOMO gradient encode / decode library.
 *
 * ATOMO ("atomic sparsification") writes a gradient as g = sum_i lambda_i a_i over unit-norm
 * atoms a_i, keeps atom i with probability p_i and rescales it by 1/p_i, so that the sparse
 * estimator  g_hat = sum_i (lambda_i t_i / p_i) a_i,  t_i ~ Bernoulli(p_i)  (Eq. 2) is unbiased;
 * the p_i minimise its variance under the budget  sum_i p_i = s  (Eq. 3, Algorithm 1).
 * Two decompositions are provided (Section 5): entry-wise (atoms e_i, lambda_i = g_i) and
 * spectral (atoms u_i v_i^T, lambda_i = sigma_i, from the SVD of the layer gradient seen as a
 * matrix).
 *
 * Conventions
 *   - Every pointer marked DEVICE is a CUDA device pointer owned by the caller; arrays of
 *     descriptors (atomo_mat, atomo_vec, pointer lists, shape lists) are HOST memory and are
 *     consumed before the call returns.
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = default stream).
 *     atomo_encode_spectral on the tridiagonal routes (eigen scheme 3, the default) never
 *     waits on the host: a bounded device-side wait that ran out shows as ATOMO_ERR_TIMEOUT in the layers' status
 *     words.  On the Jacobi routes it waits once, after it has enqueued all its work (the kernels' bounded waits
 *     report there), or once per Jacobi sweep in launch scheme 0.  atomo_encode_entrywise and the decode calls
 *     never synchronise.  A call that grows the workspace (first call, or a larger batch) does synchronise the
 *     device (cudaMalloc / cudaFree).  No claim is made about capture in a CUDA graph.
 *   - Matrices are fp32 row-major with leading dimension `ld` (elements, ld >= cols).
 *   - Functions return an atomo_status.  Problems visible on the host (NULL, bad sizes,
 *     s <= 0 or not finite, payload capacity too small) return at once and launch nothing.
 *     Problems only the device can see (more kept atoms than k_cap, NaN/Inf input, sweep cap
 *     hit) set the layer's status word in the payload header, leave that layer with k = 0
 *     (except ATOMO_ERR_NOT_CONVERGED on eigen-solver route 0, whose basis is orthonormal at any
 *     sweep count and is kept) and are read back with
 *     atomo_payload_status().  Nothing is ever silently truncated: dropping kept atoms would
 *     bias the estimator of Eq. (2).
 *   - Randomness is counter based (Philox4x32-10): the output is a pure function of the
 *     inputs, s, seed, step and the position of the layer in the call.  Key = (seed low 32,
 *     seed high 32); counter = (i>>2 low, i>>2 high, layer, (kind<<31)|(step & 0x7fffffff)),
 *     atom i takes word i&3; kind 0 = spectral (i = rank in descending sigma), 1 = entry-wise
 *     (i = flat element index).  Atom i is kept iff p_i >= 1 or word < floor(p_i * 2^32).
 *
 * Payload (DEVICE buffer, caller owned, self-describing; all offsets in bytes from its start,
 * 16-byte aligned):
 *   atomo_payload_header, then n_layers x atomo_layer_header, then per layer
 *     entry-wise: idx  u32[k_cap] ascending flat indices, val f32[k_cap] = g_i / p_i,
 *                 tiles u32[ceil(n / ATOMO_EW_TILE) + 1]: number of kept atoms with index below
 *                 t * ATOMO_EW_TILE (last entry = k), at header field off_short
 *     spectral  : idx  u32[k_cap] ascending ranks, coef f32[k_cap] = sigma_i / p_i,
 *                 short f32[k_cap][r]  unit vectors of the short side (length r = min(rows,cols)),
 *                 long  f32[k_cap][L]  unit vectors of the long side  (length L = max(rows,cols));
 *                 for rows <= cols the short vectors are the u_i and the long ones the v_i,
 *                 otherwise the other way round.
 *   Only the first k entries of each array are meaningful (k is in the layer header).
 */
#ifndef ATOMO_H_
#define ATOMO_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct atomo_ctx atomo_ctx; /* opaque; owns workspace, events and the status mirror */

typedef enum {
  ATOMO_OK = 0,
  ATOMO_ERR_INVALID_ARG = 1,   /* NULL pointer, non-positive size, ld < cols, too many atoms      */
  ATOMO_ERR_BUDGET = 2,        /* s <= 0, NaN or Inf                                               */
  ATOMO_ERR_CAPACITY = 3,      /* host: payload buffer too small; device: kept atoms > k_cap       */
  ATOMO_ERR_NONFINITE = 4,     /* NaN or Inf found in a gradient                                   */
  ATOMO_ERR_NOT_CONVERGED = 5, /* eigen-solver hit its sweep cap (route 1: k = 0; route 0: result kept) */
  ATOMO_ERR_TIMEOUT = 6,       /* a bounded device-side wait (mbarrier, step barrier) ran out      */
  ATOMO_ERR_CUDA = 7,          /* a CUDA runtime call failed; see atomo_last_cuda_error            */
  ATOMO_ERR_PAYLOAD = 8        /* decode: header does not match the shapes given                   */
} atomo_status;

enum { ATOMO_KIND_SPECTRAL = 0, ATOMO_KIND_ENTRYWISE = 1 };
enum { ATOMO_MAGIC = 0x4F4D5441 /* "ATMO" */, ATOMO_VERSION = 2 };
enum { ATOMO_EW_TILE = 4096 };   /* entry-wise payloads carry one offset per tile of this many elements */
/* Entry-wise payload formats.  EXPLICIT: idx u32[k_cap] ascending and val f32[k_cap] = g_i / p_i.
 * COMPACT (the ternary form of Section 4: a kept atom with p_i < 1 has g_i / p_i = sign(g_i) c with one
 * scalar c = sum_unsaturated |g| / (s - n_sat) per vector, so its index and one sign bit say everything):
 *   off_idx   u16[k_cap]  one entry per kept atom with p_i < 1, ascending by index: bits 0..11 = index inside
 *                         its tile of ATOMO_EW_TILE elements, bit 15 = sign of g_i (the tile follows from the
 *                         offset table), value sign * c with c from the layer header
 *   off_short u32[n_tiles + 1]  number of such entries before each tile
 *   off_long  u32[sat_cap] indices of the atoms with p_i = 1 (all kept), ascending
 *   off_val   f32[sat_cap] their values g_i
 * with k = all kept atoms, n_sat = the length of the saturated list, k - n_sat entries in off_idx.
 * Both formats decode to the same dense gradient, bit for bit.                                         */
enum { ATOMO_EW_EXPLICIT = 0, ATOMO_EW_COMPACT = 1 };

typedef struct { const float* data; /* DEVICE */ int32_t rows, cols; int64_t ld; } atomo_mat;
typedef struct { const float* data; /* DEVICE */ int64_t n; } atomo_vec;

/* Payload headers as they sit in DEVICE memory (also what atomo_payload_read_headers copies). */
typedef struct {
  uint32_t magic, version, kind, n_layers;
  uint64_t total_bytes;
  uint64_t seed, step;
  double   s;
  uint64_t ew_format;         /* entry-wise: ATOMO_EW_EXPLICIT or ATOMO_EW_COMPACT; spectral: 0   */
  uint64_t ew_sat_cap;        /* compact entry-wise: capacity of the saturated list; else 0       */
} atomo_payload_header;                       /* 64 bytes */

typedef struct {
  int64_t  rows, cols;        /* entry-wise: rows = 1, cols = n                                  */
  uint32_t k_cap, k;          /* capacity and number of kept atoms                               */
  uint32_t n_sat;             /* atoms with p = 1                                                */
  uint32_t status;            /* atomo_status seen by the device for this layer                  */
  float    c;                 /* common weight |lambda_i|/p_i of the kept atoms with p < 1       */
  uint32_t sweeps;            /* spectral: Jacobi sweeps used                                    */
  uint64_t off_idx, off_val;  /* val = entry-wise values / spectral coefficients                 */
  uint64_t off_short, off_long; /* entry-wise: off_short = the per-tile offset table           */
  double   l1;                /* sum |lambda| over all atoms (||g||_1 or the nuclear norm)       */
} atomo_layer_header;                         /* 80 bytes */

/* Optional per-atom outputs for parity checks (DEVICE; any pointer may be NULL).
 * Layer l's atoms start at element offset sum_{j<l} n_atoms_j in sigma/prob (n_atoms = r for
 * spectral, n for entry-wise) and at word offset sum_{j<l} ceil(n_atoms_j/32) in mask_words
 * (bit i&31 of word i>>5 = t_i).  sigma is spectral only (descending).  short_vecs is spectral
 * only: all r short-side singular vectors, rank-major (r x r per layer, offset sum r_j^2).  */
typedef struct { float* sigma; float* prob; uint32_t* mask_words; float* short_vecs; } atomo_debug;

/* Stage timers (milliseconds of device time, CUDA events on the call's stream) filled while
 * profiling is on.  `launches[i]` counts the kernels of stage i in the last call.  On the
 * tridiagonal route EIG is the Householder reduction alone; the bisection for the eigenvalues
 * is timed with SAMPLE and the vectors of the kept atoms with BACKPROJECT.                    */
enum { ATOMO_STAGE_GRAM = 0, ATOMO_STAGE_EIG, ATOMO_STAGE_SAMPLE, ATOMO_STAGE_BACKPROJECT,
       ATOMO_STAGE_EW_REDUCE, ATOMO_STAGE_EW_PACK, ATOMO_STAGE_DECODE, ATOMO_N_STAGES };

/* --- lifetime ------------------------------------------------------------------------------
 * atomo_create binds the context to CUDA device `device` (made current for each call).
 * Workspace is allocated on first use and grown when a larger batch arrives (cudaMalloc, which
 * synchronises the device); a context serves one call at a time.                               */
int atomo_create(atomo_ctx** out, int device);
int atomo_destroy(atomo_ctx* ctx);
const char* atomo_last_cuda_error(atomo_ctx* ctx);   /* text of the last failing CUDA call       */

/* --- sizes (host only, no CUDA call) --------------------------------------------------------
 * Bytes a payload needs for these shapes when every layer may keep up to k_cap atoms
 * (k_cap is clamped to the layer's atom count).  Returns -1 on bad arguments.
 * Since k = sum of independent Bernoulli(p_i) with sum p_i <= s, a k_cap of about
 * s + 8 sqrt(s) + 8 is never exceeded in practice; k_cap = #atoms can never overflow.          */
int64_t atomo_payload_bytes_spectral(const int32_t* rows, const int32_t* cols, int32_t n_layers,
                                     int32_t k_cap);
int64_t atomo_payload_bytes_entrywise(const int64_t* n, int32_t n_vecs, int64_t k_cap);
/* Compact format: k_cap bounds the kept atoms with p < 1, sat_cap (>= 0, clamped to n) the atoms with p = 1.
 * n_sat < s always (every saturated atom uses one unit of the budget), so sat_cap >= s cannot overflow; at the
 * l_q budgets of Section 4 every vector is s-balanced and sat_cap = 0 is enough.                           */
int64_t atomo_payload_bytes_entrywise_compact(const int64_t* n, int32_t n_vecs, int64_t k_cap, int64_t sat_cap);

/* --- encode ---------------------------------------------------------------------------------
 * Spectral ATOMO (Section 5; Eq. 2, Eq. 3 / Algorithm 1) over a batch of layer gradients.
 * Per layer: thin SVD (Gram matrix of the short side -> eigenvalues of all atoms, hence every sigma ->
 * short-side vectors of the kept atoms; see atomo_set_persistent_eig), probabilities from the descending
 * sigma, Bernoulli draws, and for the kept atoms the long-side vector by back-projection (G^T u_i or G v_i, normalised; its norm
 * is the sigma_i used in coef = sigma_i / p_i).  Each layer needs min(rows, cols) <= 4096.     */
int atomo_encode_spectral(atomo_ctx* ctx, const atomo_mat* layers /*HOST array*/, int32_t n_layers,
                          double s, uint64_t seed, uint64_t step, int32_t k_cap,
                          void* payload /*DEVICE*/, int64_t capacity_bytes,
                          const atomo_debug* dbg /*HOST struct or NULL*/, void* stream);

/* Test entry point: everything downstream of the SVD (Algorithm 1, the draws of Eq. 2, the compaction, the
 * back-projection and the payload) for a decomposition that the caller supplies, so that a test can separate those
 * steps from the conditioning of the SVD.  sigma[l] (DEVICE, r_l floats, descending) and short_vecs[l] (DEVICE,
 * r_l x r_l floats, rank-major: row i = the unit short-side vector of atom i: u_i for rows <= cols, else v_i) replace
 * the Gram matrix and the eigen-solver; both pointer lists are HOST arrays.  Everything else as atomo_encode_spectral
 * (short sides up to 4096; the weights still use the norm of the back-projection G^T u_i, which equals sigma_i for an
 * exact decomposition).                                                                                    */
int atomo_encode_spectral_from_svd(atomo_ctx* ctx, const atomo_mat* layers /*HOST array*/, int32_t n_layers,
                                   const float* const* sigma, const float* const* short_vecs, double s, uint64_t seed,
                                   uint64_t step, int32_t k_cap, void* payload /*DEVICE*/, int64_t capacity_bytes,
                                   const atomo_debug* dbg /*HOST struct or NULL*/, void* stream);

/* Entry-wise ATOMO (Section 3; the QSGD / TernGrad family of Section 4) over a batch of flat
 * gradients, each with n < 2^32 elements and its own budget s (same s for every vector).       */
int atomo_encode_entrywise(atomo_ctx* ctx, const atomo_vec* vecs /*HOST array*/, int32_t n_vecs,
                           double s, uint64_t seed, uint64_t step, int64_t k_cap,
                           void* payload /*DEVICE*/, int64_t capacity_bytes,
                           const atomo_debug* dbg, void* stream);
/* Format of the payloads the context's later atomo_encode_entrywise calls write (default ATOMO_EW_EXPLICIT;
 * sat_cap is read for ATOMO_EW_COMPACT only).  The draws, the kept set and the decoded gradient do not depend
 * on the format.  A vector whose kept unsaturated atoms exceed k_cap or whose saturated atoms exceed sat_cap
 * gets ATOMO_ERR_CAPACITY in its status word and k = 0.  Decoders read the format from the payload.       */
int atomo_set_entrywise_format(atomo_ctx* ctx, int32_t format, int64_t sat_cap);
/* Launch form of the context's later atomo_encode_entrywise calls.  two_kernels = 0 (default): a vector whose tiles
 * fit one wave of resident CTAs (up to about 48 million elements on a B200, 29 million with the list below) is encoded by ONE cooperative kernel -- a CTA
 * computes its part of sum |g| and max |g| (Algorithm 1's inputs), all CTAs meet at a grid barrier, and the same CTA
 * then samples and packs its part.  The Philox word of an atom depends on its index alone, so the first pass already
 * draws the words and lists the atoms that an estimate of sum |g| (with a factor of two to spare) cannot rule out; where
 * the true sum confirms the estimate and no atom has p = 1, the exact keep decision (the same integer comparison) is
 * taken on the list and the vector is read once.  Otherwise a CTA reads its part a second time (from the L2 cache).
 * Longer vectors take the two-kernel form.  two_kernels = 1: always a solve kernel followed by a sample / pack kernel
 * whose chunks are handed out by ticket.  two_kernels = 2: the one-kernel form without the list (every part read
 * twice).  Payloads, masks and decoded gradients are bit-identical in all forms.  Other values:
 * ATOMO_ERR_INVALID_ARG.     */
int atomo_set_entrywise_launch(atomo_ctx* ctx, int32_t two_kernels);
/* Test introspection, for vector `vec` of the context's last atomo_encode_entrywise call: the number of chunks (CTAs)
 * of the one-kernel form (0 if the two-kernel form ran) and how many of them took their keep decisions on the
 * candidate list rather than on a second read.  Synchronises the device.  Either pointer may be NULL.
 * ATOMO_ERR_INVALID_ARG if there was no such vector.                                                     */
int atomo_get_entrywise_list_chunks(atomo_ctx* ctx, int32_t vec, uint32_t* from_list /*HOST*/, uint32_t* chunks /*HOST*/);

/* --- l_q budgets (Section 4) ------------------------------------------------------------------
 * s_out[l] (HOST) = ||g_l||_1 / ||g_l||_q for every vector: the budget at which entry-wise ATOMO is the
 * unbiased l_q quantiser of Section 4 -- QSGD for q = 2, TernGrad for q = INFINITY (every g is s-balanced at
 * this budget, so p_i = |g_i| / ||g||_q).  q >= 1; q = INFINITY is accepted.  fp64 accumulation.  Synchronises
 * the stream (the norms come back to the host).  A zero vector gives s = 0 and a vector with a NaN or Inf gives
 * NaN, which atomo_encode_entrywise then rejects as ATOMO_ERR_BUDGET.                                    */
int atomo_lq_budget(atomo_ctx* ctx, const atomo_vec* vecs /*HOST array*/, int32_t n_vecs, double q,
                    double* s_out /*HOST*/, void* stream);

/* --- decode (Eq. 2 summed back to a dense gradient) ----------------------------------------
 * out[l] (DEVICE, fp32) receives layer l: rows[l] x cols[l] row-major with leading dimension
 * cols[l] (entry-wise: rows[l] = 1).  `kind` and the shapes must match the payload's header;
 * a mismatch sets ATOMO_ERR_PAYLOAD in that layer's status word and writes zeros.
 * Never synchronises; every element of every output is written.                                */
int atomo_decode(atomo_ctx* ctx, int32_t kind, const void* payload /*DEVICE*/,
                 const int64_t* rows, const int64_t* cols, float* const* out /*HOST array of DEVICE ptrs*/,
                 int32_t n_layers, void* stream);

/* --- decode and average (the combine step of data-parallel training, Section 2) ---------------
 * out[l] = (1 / n_payloads) * sum over p of the decoded layer l of payloads[p]: what the receiver of the
 * workers' sparsified gradients computes before the model update.  All payloads must be of `kind` and of the
 * shapes given (they normally come from the same encode call on different workers, with different seeds);
 * a payload that does not match contributes zeros and gets ATOMO_ERR_PAYLOAD in its layer's status word.
 * payloads: HOST array of DEVICE pointers (e.g. the slices of an all-gather buffer).  The sum runs over the
 * payloads in array order and over each payload's atoms in payload order, so the result is reproducible.
 * One pass over the output; never synchronises; every element of every output is written.             */
int atomo_decode_average(atomo_ctx* ctx, int32_t kind, const void* const* payloads /*HOST array of DEVICE ptrs*/,
                         int32_t n_payloads, const int64_t* rows, const int64_t* cols,
                         float* const* out /*HOST array of DEVICE ptrs*/, int32_t n_layers, void* stream);

/* --- decode without allocation ---------------------------------------------------------------
 * (The paper has no counterpart: this entry point exists for deployment, not for the method.)
 * Same result as atomo_decode() for a spectral payload, for callers that must not allocate device
 * memory: a process whose framework allocator already owns the whole GPU, a latency-critical
 * section that cannot take cudaMalloc's device-wide synchronisation, a memory-capped job.  It needs
 * no context and calls no cudaMalloc / cudaFree: the per-call tables (one descriptor per layer, one
 * entry per 64 x 1024 output tile) go into a fixed array inside the library image, about 130 KB that
 * every GPU loading the library holds until the process exits.
 *   - Limits: n_layers <= ATOMO_STATIC_MAX_LAYERS and at most ATOMO_STATIC_MAX_TILES output tiles in
 *     all (sum over layers of ceil(rows/64) * ceil(cols/1024)); beyond that ATOMO_ERR_CAPACITY is
 *     returned and nothing is launched.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress, with
 *     that device made current); make that first call before any stream capture begins.
 *   - All calls on a device share the one array: it still holds the previous call's tables, which
 *     the next call overwrites in stream order.  Two calls whose work overlaps on the GPU (different
 *     streams, no dependency) race on it; serialise them.
 *   - The tables are staged in pageable host memory (up to 128 KB per calling thread): the copy may make
 *     the host wait until earlier work on `stream` has drained, and the staging buffer is reused by the
 *     thread's next call.
 *   - out[l] must hold rows[l] * cols[l] floats: every element is written through the raw pointer.
 * `device` is the CUDA ordinal; payload, rows, cols, out, stream as in atomo_decode().               */
enum { ATOMO_STATIC_MAX_LAYERS = 64, ATOMO_STATIC_MAX_TILES = 8192 };
int atomo_decode_spectral_static(int device, const void* payload /*DEVICE*/, const int64_t* rows,
                                 const int64_t* cols, float* const* out /*HOST array of DEVICE ptrs*/,
                                 int32_t n_layers, void* stream);

/* --- status / introspection -----------------------------------------------------------------
 * Copies the payload header and the n_layers layer headers to HOST memory (synchronises
 * `stream`).  Either output may be NULL.                                                       */
int atomo_payload_read_headers(atomo_ctx* ctx, const void* payload /*DEVICE*/, int32_t n_layers,
                               atomo_payload_header* hdr /*HOST*/, atomo_layer_header* layers /*HOST*/,
                               void* stream);
/* Worst device-side status over the layers of a payload and the first layer that has it.       */
int atomo_payload_status(atomo_ctx* ctx, const void* payload /*DEVICE*/, int32_t n_layers,
                         int32_t* worst /*HOST*/, int32_t* first_bad_layer /*HOST*/, void* stream);

/* Descriptor tables (layer descriptors, tile lists, tensor maps, header templates) are kept in device buffers owned by
 * the context and uploaded only when they differ from the previous call's: a loop that calls with the same pointers
 * and shapes every step issues no host-to-device copy in steady state (the payload header travels as a kernel
 * argument).  Counts since atomo_create: calls that had to upload their tables, and calls that found them in place.
 * Host only; either pointer may be NULL.                                                              */
int atomo_get_table_uploads(atomo_ctx* ctx, int64_t* uploads /*HOST*/, int64_t* reuses /*HOST*/);

/* --- profiling ------------------------------------------------------------------------------ */
int atomo_set_profiling(atomo_ctx* ctx, int enabled);
/* ms[ATOMO_N_STAGES], launches[ATOMO_N_STAGES] for the last encode/decode call (synchronises). */
int atomo_get_stage_times(atomo_ctx* ctx, float* ms /*HOST*/, int64_t* launches /*HOST*/);
/* Sums over all encode / decode calls since profiling was last switched on: ms[ATOMO_N_STAGES] of device time,
 * launches[ATOMO_N_STAGES], and the number of calls (any pointer may be NULL).  The calls themselves record events
 * only and never wait for them; this function waits for the newest ones.  Lets a caller time a run of
 * asynchronous steps without a host wait inside it.                                                        */
int atomo_get_stage_totals(atomo_ctx* ctx, double* ms /*HOST*/, int64_t* launches /*HOST*/, int64_t* calls /*HOST*/);

/* Eigen-solver knobs: max Jacobi sweeps (default 40) and the relative rotation threshold
 * (default 3e-7: rows p, q are rotated while |<x_p,x_q>| > tol ||x_p|| ||x_q||).               */
int atomo_set_eig_params(atomo_ctx* ctx, int32_t max_sweeps, float tol);
/* Eigen-solver route.  1 (default): Cholesky factor of the Gram matrix, then one-sided Jacobi on the
 * rows of its transpose (row i converges to sigma_i times eigenvector i).  0: one-sided Jacobi on the
 * rows of [A | I] with accumulated eigenvectors -- slower, kept as a cross-check of route 1.        */
int atomo_set_eig_mode(atomo_ctx* ctx, int32_t mode);
/* Singular-value refinement: layers whose short side is at least `min_short_side` take sigma_i from the
 * norm of the projection, sigma_i = ||G^T u_i|| (or ||G v_i||), for every atom instead of the square root
 * of the Gram eigenvalue (default 2048; 0 = every layer, a value above 4096 = never).  The Gram route
 * resolves eigenvalues only to about 1e-8 of the largest, which a long flat tail of small singular values
 * turns into a visible error of the nuclear norm and thus of every p_i; the projection norm does not
 * have that floor.  It costs one more pass over G with twice the Gram matrix's arithmetic.              */
int atomo_set_sigma_refinement(atomo_ctx* ctx, int32_t min_short_side);
/* Gram matrix path: 1 (default) = tcgen05 tensor cores with the TF32 hi/lo split for layers with rows <= cols, a short
 * side of at most 1024, a 16-byte aligned base and ld % 4 == 0 (other layers take the fp32 FMA kernel); 0 = fp32 FMA
 * kernel always.  The tensor core accumulates in fp32 with truncation: at a short side of 1024 the probabilities then
 * sit within about 3e-6 of those of an exact decomposition (the few largest p_i; measured), with the FMA kernel within
 * about 5e-7.  A caller that needs every draw to agree with an fp64 computation outside a 1e-6 margin takes 0.    */
int atomo_set_gram_path(atomo_ctx* ctx, int32_t tensor_cores);
/* Eigen-solver scheme (`enabled` = 0, 1, 2 or 3):
 * 3 (default) = the tridiagonal routes: the scaled Gram matrix of every layer is reduced to tridiagonal form by
 *     Householder reflectors, all eigenvalues come from bisection on Sturm counts, and eigenvectors are computed for the
 *     kept atoms only (twisted factorisation, back-transformation with the reflectors): only the singular values of
 *     all atoms enter the probabilities, the vectors of atoms that are not kept are never formed.  Short sides up to
 *     512: the rows sit in the registers of the CTAs of a 16-CTA cluster and are exchanged through distributed shared
 *     memory, fp64 arithmetic, one cluster barrier per step.  Short sides above 512 (up to 4096): the matrix stays in
 *     global memory (fp32) and the reduction is blocked in panels of 32 columns, a cluster of 1 to 16 CTAs per layer
 *     (atomo_set_tridiag_ctas); sums and scalars in fp64.  Both kinds of layer can share one call.  A batch takes
 *     scheme 2 instead when eigen-solver route 0 or the whole short-side basis (atomo_debug.short_vecs) is asked
 *     for, or when the GPU cannot place the clusters;
 * 2 = one-sided Jacobi in thread-block clusters where they apply: when every layer of the batch has at most 16 block
 *     pairs (padded short side <= 512), each layer's CTAs sit in one 16-CTA cluster for the whole solve and hand
 *     their blocks to one another through distributed shared memory, with a cluster barrier per Jacobi step;
 *     other batches, or a GPU that cannot place such clusters, take scheme 1;
 * 1 = cooperative launches in which the block pairs of a group of whole layers are co-resident (one CTA per SM)
 *     and run all their Jacobi steps, blocks exchanged through global memory (L2) with a barrier among the CTAs
 *     of a layer between steps; a batch that fits the GPU is one such launch.  A batch with a layer that alone
 *     needs more CTAs than the GPU holds (short side above 2048) takes scheme 0;
 * 0 = one launch per step and one host wait per sweep.
 * Scheme 3 never waits on the host; schemes 1 and 2 wait once, at the end of the call.  The Jacobi schemes work in
 * fp32 throughout and resolve the probabilities of layers with a short side of 1024 only to a few 1e-5; they are
 * kept as a fallback and as an independent cross-check of scheme 3.                                              */
int atomo_set_persistent_eig(atomo_ctx* ctx, int32_t enabled);
/* CTAs per layer of the blocked tridiagonal reduction that scheme 3 runs for short sides above 512: 0 (default) =
 * chosen per batch (the fewest that hold the layer's rows, doubled while SMs would stay idle; never 2 up to a short side
 * of 1024, where one CTA per layer is faster than a pair), else 1, 2, 4, 8 or 16 (raised to the fewest that hold the rows).  With 2 to 16 CTAs a layer runs the cluster kernel, every sum of which has
 * an order that does not depend on this number: the payload is bit-identical for 2, 4, 8 and 16 (the knob exists for
 * tuning and for checking exactly that).  With 1 CTA per layer (short sides up to 1024; what a batch of 38 layers or
 * more gets) another kernel runs (triangle-only products, panels of 16 columns): same kept atoms, values equal to
 * rounding.                                                                                                    */
int atomo_set_tridiag_ctas(atomo_ctx* ctx, int32_t ctas_per_layer);
/* The scheme (0 to 3 as above) that the last atomo_encode_spectral() of this context actually ran; -1 before
 * the first call.  Host only.                                                                                */
int atomo_last_eig_scheme(atomo_ctx* ctx);

/* --- measured arithmetic peaks (benchmark helper; the paper has no counterpart) ---------------
 * Runs a register-only chain of fused multiply-adds on every SM of `device` for a few milliseconds and writes the
 * rate to *tflops (HOST): fp32 (fp64 = 0) or fp64 (fp64 = 1).  The roofline of the kernels that are bound by plain
 * ALU arithmetic is quoted against these figures.  Allocates and frees a small device buffer; synchronises.     */
int atomo_measure_fma_peak(int device, int fp64, double* tflops /*HOST*/);

#ifdef __cplusplus
}
#endif
#endif /* ATOMO_H_ */
