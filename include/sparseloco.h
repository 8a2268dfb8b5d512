/* sparseloco.h — C ABI of the SparseLoCo outer synchronisation step on NVIDIA B200 (sm_100a).
 *
 * The step is Eq. 2 of the paper (§2.1, "Background: SparseLoCo"), run every H inner steps:
 *
 *   line 1   delta   = theta_global - theta_local                  (pseudo-gradient)
 *   line 2   e'      = beta * e + delta                            (error feedback)
 *   line 3   message = Q(Top-k(e'))   k largest magnitudes of every chunk, then quantised
 *   line 4   e       = e' - message                                (what was sent leaves the buffer)
 *   line 5   update  = (1/R) * sum_r message_r ;  theta_global -= outer_lr * update
 *
 * Conventions shared by every call
 * --------------------------------
 *  - Every data pointer is a DEVICE pointer unless it is marked HOST.  The caller owns every
 *    buffer; the library allocates nothing and keeps no state between calls.
 *  - Calls are asynchronous on `stream` (a cudaStream_t passed as void*, NULL = default stream)
 *    and use the current CUDA device.  Host arrays (layout offsets, pointer tables) are read
 *    before the call returns.  A call only enqueues kernels on `stream` (its tables travel in the
 *    kernels' parameters), so it may be recorded into a CUDA graph by stream capture.
 *  - Return value: SL_OK or a negative SL_ERR_*; nothing throws, aborts or prints.  All argument
 *    checks happen on the host before anything is launched.  Conditions met on the device never
 *    trap: they OR a bit into `*flags`.
 *  - Arithmetic is IEEE binary32, round-to-nearest-even, denormals kept, each operation rounded
 *    once; beta*e + delta and theta - outer_lr*update are single fused roundings.
 *
 * Arena and chunks
 * ----------------
 *  Parameters live in a flat fp32 arena of `n_total` elements holding `n_tensors` tensors back
 *  to back (row-major).  Two chunk geometries (the paper's chunk of 4096 elements is stated as a
 *  64 by 64 block, §3 "Training Configuration", Table 8, which can be read either way):
 *   - consecutive (default): a chunk is a run of `chunk` consecutive elements of ONE tensor; the
 *     last chunk of a tensor may be short.  Position p of a chunk is its p-th element.
 *   - square tiles (sl_layout.cols[t] > 0): tensor t is a matrix of cols[t] columns cut into
 *     s x s tiles, s*s = chunk, numbered row-major over the tile grid.  Position p of a tile is
 *     its row p / s, column p % s; tiles on the matrix's right and bottom edges are smaller and
 *     only the positions inside the matrix exist.
 *  A chunk with fewer than k elements keeps them all (k_eff = min(k, its size)).  Chunks are
 *  numbered through the arena in order: chunk g owns idx[g*k .. g*k+k), codes[g*stride ..
 *  (g+1)*stride), scales[g].
 *
 * Message of one chunk
 * --------------------
 *  idx    uint16[k]  chunk-local positions of the kept elements, ascending; unused slots 0xFFFF.
 *  scales float      s = largest magnitude of e' in the chunk.
 *  codes  bits in {2,4,8}: slot j's code sits at bit j*bits of the chunk's `stride` bytes,
 *         least-significant bits first.  With L = 2^(bits-1): code = sign << (bits-1) | q,
 *         q = number of thresholds s*(j/L), j = 1..L-1, that |e'| reaches; the value it stands
 *         for is sign * s * (2q+1)/(2L).  bits = 32: no quantisation (the paper's own runs, §3),
 *         codes is float[k] per chunk holding e' verbatim.
 *  Ties in magnitude go to the lower position; +0 and -0 tie; values are ordered by the low 31
 *  bits of their pattern, so NaN > Inf > finite and nothing is sanitised (SL_FLAG_NONFINITE).
 */
#ifndef SPARSELOCO_H_
#define SPARSELOCO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  SL_OK = 0,
  SL_ERR_INVALID_ARG = -1, /* null pointer, k < 1, k > chunk, bits not in {2,4,8,32}, R out of range,
                              beta / outer_lr not finite, offsets not ascending or not ending at n_total,
                              tiles asked for with a chunk that is not a square or a tensor that is not
                              a whole number of rows */
  SL_ERR_ALIGNMENT = -2,   /* a float pointer not 4-byte aligned or idx not 2-byte aligned */
  SL_ERR_UNSUPPORTED = -3, /* chunk > SL_MAX_CHUNK, n_tensors > SL_MAX_TENSORS, more than 2^31 chunks */
  SL_ERR_CUDA = -4         /* a CUDA runtime call or a launch failed (the error is not cleared) */
};

enum {
  SL_FLAG_NONFINITE = 1u, /* some chunk's largest magnitude was Inf or NaN */
  SL_FLAG_BAD_INDEX = 2u, /* sl_aggregate*: a message slot named a position past its chunk; skipped */
  SL_FLAG_TIMEOUT = 4u,   /* a bounded wait on an on-chip copy ran out; the outputs are not to be trusted */
  SL_FLAG_BOUNDS = 8u     /* debug build only (libsparseloco_debug.so, -DSL_DEBUG_BOUNDS): a kernel of Eq. 2 formed an
                             index outside the buffer it was about to touch; the access was skipped */
};

#define SL_MAX_CHUNK 8192     /* elements; any chunk size in [1, SL_MAX_CHUNK] is accepted */
#define SL_MAX_TENSORS 1280   /* tensors per call; split larger arenas into several calls */
#define SL_MAX_REPLICAS 64    /* replicas per batched / aggregate call */

/* HOST description of an arena.  offset[0] = 0 < ... (non-decreasing) ... offset[n_tensors] =
 * n_total.  A single tensor is n_tensors = 1, offset = {0, n}.  The tuned kernels need every
 * offset (and every tiled tensor's column count) to be a multiple of 4 elements and every arena
 * pointer 16-byte aligned; otherwise the calls fall back to a slower kernel with identical
 * results. */
typedef struct sl_layout {
  uint64_t n_total;
  uint32_t n_tensors;
  const uint64_t* offset; /* HOST, [n_tensors + 1] */
  const uint64_t* cols;   /* HOST, [n_tensors], or NULL: columns of every tensor that is cut into square
                             tiles, 0 for tensors (and NULL for arenas) with consecutive chunks */
} sl_layout;

/* Number of chunks of the arena: per tensor ceil(n_t / chunk), or ceil(rows / s) * ceil(cols / s)
 * for a tensor cut into tiles.  0 on bad arguments. */
uint64_t sl_num_chunks(const sl_layout* layout, int chunk);

/* Bytes of `codes` ONE chunk owns: ceil(k*bits/8), or 4*k when bits == 32.  0 on bad arguments.
 * A replica's codes buffer is sl_num_chunks() * sl_codes_stride() bytes. */
uint64_t sl_codes_stride(int k, int bits);

/* Bytes of ONE replica's whole `codes` buffer for the arena: sl_num_chunks(layout, chunk) *
 * sl_codes_stride(k, bits) (Eq. 2 line 3: the quantised values of the message).  0 on bad
 * arguments (those of the two calls above, or k > chunk). */
uint64_t sl_codes_bytes(const sl_layout* layout, int chunk, int k, int bits);

/* Eq. 2 lines 1-4 for ONE replica: pseudo-gradient, error feedback, chunk-wise Top-k,
 * quantisation, residual.
 *   theta_local, theta_global  [n_total] read only
 *   err     [n_total] read and overwritten in place with the residual (persists across steps)
 *   idx     [n_c * k], codes [n_c * stride] bytes, scales [n_c]: fully overwritten
 *   flags   optional device word, sticky OR of SL_FLAG_*; never cleared by the library */
int sl_compress(const float* theta_local, const float* theta_global, float* err,
                const sl_layout* layout, float beta, int chunk, int k, int bits,
                uint16_t* idx, uint8_t* codes, float* scales, uint32_t* flags, void* stream);

/* The same for R replicas that share theta_global, in one launch; results are identical to R
 * calls of sl_compress.  The pointer tables are HOST arrays of R DEVICE pointers.  theta_global
 * is fetched from memory once per chunk for all replicas. */
int sl_compress_batch(int R, const float* const* theta_local, const float* theta_global,
                      float* const* err, const sl_layout* layout, float beta, int chunk, int k,
                      int bits, uint16_t* const* idx, uint8_t* const* codes, float* const* scales,
                      uint32_t* flags, void* stream);

/* Eq. 2 line 5, first half: decompress R messages and average them into a dense update.
 * Replicas are added in the order 0..R-1 starting from +0 and the sum is divided by R (always
 * R, however many replicas sent a position).  `update` [n_total] is fully overwritten;
 * positions nobody sent are +0.  A slot whose position is >= its chunk's length (other than the
 * 0xFFFF padding) is skipped and raises SL_FLAG_BAD_INDEX.  Inside one replica's chunk message
 * the positions are distinct (sl_compress writes them so); a message that names a position twice
 * gets an unspecified sum at that position. */
int sl_aggregate(int R, const uint16_t* const* idx, const uint8_t* const* codes,
                 const float* const* scales, const sl_layout* layout, int chunk, int k, int bits,
                 float* update, uint32_t* flags, void* stream);

/* Eq. 2 line 5, second half: plain SGD outer step (no momentum, Table 8),
 * theta_global[i] = fma(-outer_lr, update[i], theta_global[i]) for i < n. */
int sl_outer_apply(float* theta_global, const float* update, uint64_t n, float outer_lr, void* stream);

/* Both halves of line 5 in one pass: the dense update lives in shared memory only and
 * theta_global is read and written once.  Same result as sl_aggregate + sl_outer_apply. */
int sl_aggregate_apply(int R, const uint16_t* const* idx, const uint8_t* const* codes,
                       const float* const* scales, const sl_layout* layout, int chunk, int k,
                       int bits, float* theta_global, float outer_lr, uint32_t* flags, void* stream);

/* The whole of Eq. 2 in one call, for R replicas that live on this device: sl_compress_batch
 * followed by sl_aggregate_apply on the messages it wrote, on the same stream (err, idx, codes,
 * scales and theta_global all updated). */
int sl_outer_step(int R, const float* const* theta_local, float* theta_global, float* const* err,
                  const sl_layout* layout, float beta, int chunk, int k, int bits, float outer_lr,
                  uint16_t* const* idx, uint8_t* const* codes, float* const* scales, uint32_t* flags,
                  void* stream);

/* Eq. 2 with the parameters stored as bfloat16 (the upper 16 bits of a binary32, passed as uint16_t)
 * and everything else as above: error buffers, scales and unquantised values stay float32.  The paper
 * states no storage precision for this step (section 2.1); the reading taken here:
 *   line 1   delta = theta_global - theta_local in float32 on the exactly widened values (one rounding);
 *   lines 2-4 as in the float32 calls, so the error buffer keeps what the coarse parameters cannot;
 *   line 5   theta_global = bf16( fma(-outer_lr, update, widen(theta_global)) ): the float32 step with one
 *            rounding, then one more rounding for storage - to nearest, ties to even; a NaN stays a NaN
 *            (quiet bit set), overflow goes to infinity.  An update below half a bfloat16 unit of a
 *            parameter leaves that parameter unchanged.
 * Messages (idx, codes, scales) are identical in format to the float32 calls', so sl_aggregate works on
 * them unchanged.  The tuned kernels take consecutive chunks of 4096 with every tensor offset a multiple of
 * 8 elements and 16-byte aligned arrays; everything else (tiles included) runs the generic kernels with
 * identical results.  Arguments, flags and errors as in the float32 calls of the same names. */
int sl_compress_batch_bf16(int R, const uint16_t* const* theta_local, const uint16_t* theta_global,
                           float* const* err, const sl_layout* layout, float beta, int chunk, int k, int bits,
                           uint16_t* const* idx, uint8_t* const* codes, float* const* scales, uint32_t* flags,
                           void* stream);
int sl_aggregate_apply_bf16(int R, const uint16_t* const* idx, const uint8_t* const* codes,
                            const float* const* scales, const sl_layout* layout, int chunk, int k, int bits,
                            uint16_t* theta_global, float outer_lr, uint32_t* flags, void* stream);
int sl_outer_apply_bf16(uint16_t* theta_global, const float* update, uint64_t n, float outer_lr, void* stream);
int sl_outer_step_bf16(int R, const uint16_t* const* theta_local, uint16_t* theta_global, float* const* err,
                       const sl_layout* layout, float beta, int chunk, int k, int bits, float outer_lr,
                       uint16_t* const* idx, uint8_t* const* codes, float* const* scales, uint32_t* flags,
                       void* stream);

/* 12-bit wire form of the positions (the message of Eq. 2 line 3 carries "indices and values"; a
 * position of a chunk of at most 4096 elements fits 12 bits, which takes a k = 64, 2-bit message
 * from 148 to 116 bytes per chunk).  Slot j of a chunk occupies bits [12 j, 12 j + 12) of the
 * chunk's sl_idx12_stride(k) = ceil(12 k / 8) bytes, least-significant bits first.  The padding
 * 0xFFFF travels as 0xFFF; on the way back 0xFFF is position 4095 in a chunk that has all 4096
 * positions (such a chunk has no padding) and padding in every other chunk, which is why
 * unpacking needs the layout.  The kernels of this library work on the uint16 form; these two
 * calls convert a replica's positions before and after they cross the network.
 *   sl_pack_idx12:   idx [n_chunks * k] -> packed [n_chunks * stride].  A position above 4095
 *                    (other than the padding) is cut to 12 bits and raises SL_FLAG_BAD_INDEX.
 *   sl_unpack_idx12: packed -> idx, for the arena `layout` describes; chunk <= 4096. */
uint64_t sl_idx12_stride(int k);
int sl_pack_idx12(const uint16_t* idx, uint64_t n_chunks, int k, uint8_t* packed, uint32_t* flags, void* stream);
int sl_unpack_idx12(const uint8_t* packed, const sl_layout* layout, int chunk, int k, uint16_t* idx, void* stream);

/* Token-embedding adaptation applied after every outer synchronisation (paper section 2.4,
 * Eqs. 3-4).  The embedding table is kept as TE = T_S + T_perp; U (section 2.3) spans the
 * compression subspace S, and Pi_S(t) = t U U^T for a row t.  In place:
 *     T_perp[v,:] <- T_perp[v,:] + (T_S[v,:] - Pi_S(T_S[v,:]))
 *     T_S[v,:]    <- Pi_S(T_S[v,:])                                  for v < V.
 * The split made before training (same section: T_S <- TE U U^T, T_perp <- TE - T_S) is the
 * same call on T_S = TE and T_perp = 0.
 * T_S, T_perp: DEVICE, float32, V x d row-major, read and written.  U: DEVICE, float32, d x k
 * row-major (orthonormal columns; not checked), read only.
 * Tuned path (d % 4 == 0, k % 4 == 0, 4 <= k <= 256, all three pointers 16-byte aligned): the two
 * contractions run on the tensor cores in TF32 with float32 accumulation.  The hardware cuts a
 * float32 operand to TF32 (10 mantissa bits) instead of rounding it, which would shorten every
 * product; the kernel therefore rounds the T_S tiles and the intermediate coordinates to the
 * nearest TF32 value itself.  U is read as it is: round it once with sl_round_tf32 (it is a
 * fixed matrix), otherwise the projection comes out about 7e-4 short in magnitude - a difference
 * that stays in T_perp like any other residual.  Any other shape with k <= 4096 (the paper's most aggressive settings reach
 * k = 2) takes a plain float32 kernel (fused multiply-adds in index order), slower and exact to
 * float32 rounding.  In both, the subtraction and the addition are float32, each rounded once,
 * and use the very value that is stored to T_S, so T_S + T_perp is conserved to float32 rounding.
 * V < 2^31 (else SL_ERR_UNSUPPORTED); V = 0 is a no-op.  `flags` (DEVICE, may be NULL) receives
 * SL_FLAG_TIMEOUT if an internal wait of the tuned kernel gave up, in which case the tables'
 * contents are unspecified.  Asynchronous on `stream`. */
int sl_embed_reproject(float* T_S, float* T_perp, const float* U, uint64_t V, uint32_t d, uint32_t k,
                       uint32_t* flags, void* stream);

/* Subspace compression of the activations that cross a pipeline-stage boundary (paper section 2.3).
 * X: n_tok x d activations of a flattened batch (token t sits at position t mod L); ids: the
 * tokens (int32, n_tok); T_perp: V x d, the fixed high-rank part of the embedding table; pos:
 * L x d positional embedding; U: d x k orthonormal basis (round it once with sl_round_tf32).
 *   sl_subspace_project:      Xt[t,:]   = (X[t,:] - T_perp[ids[t],:] - pos[t mod L,:]) U     n_tok x k
 *                             with ids == NULL (activation gradients): Xt = X U
 *   sl_subspace_reconstruct:  Xhat[t,:] = Xt[t,:] U^T + T_perp[ids[t],:] + pos[t mod L,:]    n_tok x d
 *                             with ids == NULL: Xhat = Xt U^T
 * All DEVICE, float32 row-major, inputs read only, the output fully overwritten.  Arithmetic: the
 * differences / sums are float32, one rounding per operation in the order written; the
 * contraction runs on the tensor cores in TF32 (its float32 operand - the difference, resp. Xt -
 * rounded to the nearest TF32 value first) with float32 accumulation, for d % 4 == 0, k % 4 == 0,
 * 4 <= k <= 256 and 16-byte aligned pointers; other shapes up to k = 4096 take plain float32
 * kernels.  A token id outside [0, V) contributes no embedding and no position term and raises
 * SL_FLAG_BAD_INDEX.  n_tok, V < 2^31.  Asynchronous on `stream`. */
int sl_subspace_project(const float* X, const int32_t* ids, const float* T_perp, const float* pos, const float* U,
                        uint64_t n_tok, uint32_t L, uint64_t V, uint32_t d, uint32_t k, float* Xt, uint32_t* flags,
                        void* stream);
int sl_subspace_reconstruct(const float* Xt, const int32_t* ids, const float* T_perp, const float* pos, const float* U,
                            uint64_t n_tok, uint32_t L, uint64_t V, uint32_t d, uint32_t k, float* Xhat, uint32_t* flags,
                            void* stream);

/* x[i] <- the TF32 value nearest to x[i] (ties away from zero), kept as float32, for i < n; in place.
 * For matrices that are fed to the tensor cores many times and never change (U above). */
int sl_round_tf32(float* x, uint64_t n, void* stream);

/* Debugging aid (the paper has no counterpart).  Every wait of a kernel of this library on one of
 * its own on-chip copies is bounded: when the bound runs out the kernel stops issuing copies, lets
 * the copies still in flight land, raises SL_FLAG_TIMEOUT in `*flags` and returns; the call's
 * outputs are then unspecified and the device stays usable.  The default bound is about a second,
 * which a healthy device never reaches.  This call replaces it, for every later call from any
 * thread of the process, by `polls` non-blocking polls per wait (1 = give up unless the data is
 * there already; negative = give up without looking), which lets a test drive that path; 0
 * restores the default. */
void sl_debug_set_wait_limit(int32_t polls);

/* Debugging aid (the paper has no counterpart).  The debug build of the library range-checks every
 * shared- and global-memory index of the Eq. 2 kernels (see SL_FLAG_BOUNDS).  This call launches one
 * tiny kernel that puts an out-of-range index through that check: `*flags` (DEVICE) must come back with
 * SL_FLAG_BOUNDS raised and `*probe` (DEVICE, one word) untouched, which shows that the checks are
 * compiled in and skip the access.  The normal build returns SL_ERR_UNSUPPORTED and launches nothing. */
int sl_debug_bounds_selftest(uint32_t* flags, uint32_t* probe, void* stream);

/* Static description of an SL_* return code. */
const char* sl_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* SPARSELOCO_H_ */
