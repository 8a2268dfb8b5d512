// Host side of the C ABI declared in include/sparseloco.h: argument checks, the by-value
// arena table (built on the caller's stack, about 28 KB for the largest arenas), dispatch.  No
// allocation, no state, no synchronisation.
#include <atomic>
#include <cmath>

#include "sl_common.cuh"

namespace sl {
namespace {
std::atomic<uint32_t> g_wait_polls{0};
}
uint32_t debug_wait_polls() { return g_wait_polls.load(std::memory_order_relaxed); }
#ifdef SL_DEBUG_BOUNDS
__global__ void bounds_selftest_kernel(uint32_t* flags, uint32_t* probe) {
  const uint32_t i = 1 + threadIdx.x;                       // the buffer has one word: index 1 is outside
  if (SL_CHECK(flags, i < 1u)) probe[i] = 0xDEADBEEFu;      // must be skipped
}
#endif
}  // namespace sl

namespace {

using namespace sl;

inline bool bits_ok(int bits) { return bits == 2 || bits == 4 || bits == 8 || bits == 32; }
inline bool aligned(const void* p, uintptr_t a) { return ((uintptr_t)p & (a - 1)) == 0; }

inline uint64_t codes_stride(int k, int bits) {
  return bits == 32 ? (uint64_t)k * 4u : ((uint64_t)k * (uint64_t)bits + 7u) / 8u;
}

// side of the square tile with `chunk` elements, 0 if chunk is not a square
inline uint32_t tile_side(int chunk) {
  uint32_t s = 1;
  while ((uint64_t)s * s < (uint64_t)chunk) ++s;
  return (uint64_t)s * s == (uint64_t)chunk ? s : 0;
}

// chunks of tensor t; false if its description is inconsistent
inline bool tensor_chunks(const sl_layout* L, uint32_t t, int chunk, uint32_t side, uint64_t* out) {
  if (L->offset[t + 1] < L->offset[t]) return false;
  const uint64_t n_t = L->offset[t + 1] - L->offset[t];
  const uint64_t c_t = L->cols ? L->cols[t] : 0;
  if (c_t == 0) { *out = (n_t + (uint64_t)chunk - 1) / (uint64_t)chunk; return true; }
  if (side == 0 || c_t > 0xFFFFFFFFull || n_t % c_t != 0) return false;
  const uint64_t rows = n_t / c_t;
  *out = ((rows + side - 1) / side) * ((c_t + side - 1) / side);
  return true;
}

int check_common(const sl_layout* L, int chunk, int k, int bits) {
  if (!L || !L->offset) return SL_ERR_INVALID_ARG;
  if (chunk < 1 || k < 1 || k > chunk || !bits_ok(bits)) return SL_ERR_INVALID_ARG;
  if (chunk > SL_MAX_CHUNK) return SL_ERR_UNSUPPORTED;
  if (L->n_tensors < 1) return SL_ERR_INVALID_ARG;
  if (L->n_tensors > SL_MAX_TENSORS) return SL_ERR_UNSUPPORTED;
  if (L->offset[0] != 0 || L->offset[L->n_tensors] != L->n_total) return SL_ERR_INVALID_ARG;
  const uint32_t side = tile_side(chunk);
  uint64_t nc = 0;
  for (uint32_t t = 0; t < L->n_tensors; ++t) {
    uint64_t c;
    if (!tensor_chunks(L, t, chunk, side, &c)) return SL_ERR_INVALID_ARG;
    nc += c;
  }
  if (nc > 0x7FFFFFFFull) return SL_ERR_UNSUPPORTED;
  return SL_OK;
}

// *tuned_ok: the layout is one the tuned kernels take (every offset, and every tiled tensor's
// column count, a multiple of 4 elements)
template <int T>
void fill_table(Table<T>& tb, const sl_layout* L, int chunk, bool* tuned_ok) {
  tb.n_tensors = L->n_tensors;
  const uint32_t side = tile_side(chunk);
  uint32_t nc = 0, nt = 0;
  bool m4 = true, tiled = false;
  for (uint32_t t = 0; t < L->n_tensors; ++t) {
    tb.first_chunk[t] = nc;
    tb.first_tail[t] = nt;
    tb.offset[t] = L->offset[t];
    tb.cols[t] = L->cols ? (uint32_t)L->cols[t] : 0u;
    m4 = m4 && (L->offset[t] % 4 == 0) && (tb.cols[t] % 4 == 0);
    uint64_t c = 0;
    tensor_chunks(L, t, chunk, side, &c);
    nc += (uint32_t)c;
    const uint64_t n_t = L->offset[t + 1] - L->offset[t];
    if (tb.cols[t] == 0) {
      nt += (n_t % (uint64_t)chunk) != 0 ? 1u : 0u;
    } else {
      tiled = true;
      const uint64_t rows = n_t / tb.cols[t];
      const uint64_t full = (rows / side) * (tb.cols[t] / side);
      nt += (uint32_t)(c - full);
    }
  }
  tb.first_chunk[L->n_tensors] = nc;
  tb.first_tail[L->n_tensors] = nt;
  tb.offset[L->n_tensors] = L->n_total;
  tb.cols[L->n_tensors] = 0;
  tb.side = tiled ? side : 0;
  m4 = m4 && (L->n_total % 4 == 0);
  tb.n_chunks = nc;
  tb.n_tails = nt;
  *tuned_ok = m4;
}

// step = false: Eq. 2 lines 1-4 only.  step = true: the whole of Eq. 2 (theta_global is updated):
// compress followed by aggregate-apply on the same stream.
template <int T>
int compress_impl(int R, const float* const* theta_local, float* theta_global, float* const* err,
                  const sl_layout* L, float beta, int chunk, int k, int bits, uint16_t* const* idx,
                  uint8_t* const* codes, float* const* scales, uint32_t* flags, cudaStream_t st,
                  bool step, float outer_lr, bool bf16) {
  CompressArgs<T> args;                 // by-value kernel parameters, built on the stack: no allocation
  CompressArgs<T>* a = &args;
  bool m4;
  fill_table(a->tb, L, chunk, &m4);
  bool al16 = m4 && aligned(theta_global, 16);
  for (int r = 0; r < R; ++r) {
    a->p.theta_local[r] = theta_local[r];
    a->p.err[r] = err[r];
    a->p.idx[r] = idx[r];
    a->p.codes[r] = codes[r];
    a->p.scales[r] = scales[r];
    al16 = al16 && aligned(theta_local[r], 16) && aligned(err[r], 16) && aligned(idx[r], 16) &&
           aligned(codes[r], 16) && aligned(scales[r], 4);
  }
  a->theta_global = theta_global;
  a->flags = flags;
  a->beta = beta;
  a->chunk = chunk;
  a->k = k;
  a->bits = bits;
  a->R = R;
  a->stride = (uint32_t)codes_stride(k, bits);
  a->wait_polls = debug_wait_polls();
  a->theta_bf16 = bf16 ? 1 : 0;
  if (!step) return launch_compress<T>(*a, al16, st) == cudaSuccess ? SL_OK : SL_ERR_CUDA;

  AggregateArgs<T> gargs;
  AggregateArgs<T>* g = &gargs;
  g->tb = a->tb;
  for (int r = 0; r < R; ++r) {
    g->m.idx[r] = idx[r];
    g->m.codes[r] = codes[r];
    g->m.scales[r] = scales[r];
  }
  g->out = theta_global;
  g->flags = flags;
  g->outer_lr = outer_lr;
  g->chunk = chunk;
  g->k = k;
  g->bits = bits;
  g->R = R;
  g->stride = a->stride;
  g->wait_polls = a->wait_polls;
  g->theta_bf16 = a->theta_bf16;
  if (launch_compress<T>(*a, al16, st) != cudaSuccess) return SL_ERR_CUDA;
  return launch_aggregate<T>(*g, true, al16, st) == cudaSuccess ? SL_OK : SL_ERR_CUDA;
}

int compress_checked(int R, const float* const* theta_local, float* theta_global,
                     float* const* err, const sl_layout* L, float beta, int chunk, int k, int bits,
                     uint16_t* const* idx, uint8_t* const* codes, float* const* scales,
                     uint32_t* flags, void* stream, bool step = false, float outer_lr = 0.0f, bool bf16 = false) {
  if (R < 1 || R > SL_MAX_REPLICAS) return SL_ERR_INVALID_ARG;
  if (!theta_local || !theta_global || !err || !idx || !codes || !scales) return SL_ERR_INVALID_ARG;
  if (!std::isfinite(beta) || !std::isfinite(outer_lr)) return SL_ERR_INVALID_ARG;
  const int rc = check_common(L, chunk, k, bits);
  if (rc != SL_OK) return rc;
  const uintptr_t th_al = bf16 ? 2 : 4;     // alignment of a parameter array: its element type's
  if (!aligned(theta_global, th_al) || (flags && !aligned(flags, 4))) return SL_ERR_ALIGNMENT;
  for (int r = 0; r < R; ++r) {
    if (!theta_local[r] || !err[r] || !idx[r] || !codes[r] || !scales[r]) return SL_ERR_INVALID_ARG;
    if (!aligned(theta_local[r], th_al) || !aligned(err[r], 4) || !aligned(scales[r], 4) ||
        !aligned(idx[r], 2) || (bits == 32 && !aligned(codes[r], 4)))
      return SL_ERR_ALIGNMENT;
  }
  cudaStream_t st = (cudaStream_t)stream;
  if (L->n_tensors <= 256)
    return compress_impl<256>(R, theta_local, theta_global, err, L, beta, chunk, k, bits, idx, codes,
                              scales, flags, st, step, outer_lr, bf16);
  return compress_impl<SL_MAX_TENSORS>(R, theta_local, theta_global, err, L, beta, chunk, k, bits, idx,
                                       codes, scales, flags, st, step, outer_lr, bf16);
}

template <int T>
int aggregate_impl(int R, const uint16_t* const* idx, const uint8_t* const* codes,
                   const float* const* scales, const sl_layout* L, int chunk, int k, int bits, float* out,
                   float outer_lr, bool apply, uint32_t* flags, cudaStream_t st, bool bf16) {
  AggregateArgs<T> args;
  AggregateArgs<T>* a = &args;
  bool m4;
  fill_table(a->tb, L, chunk, &m4);
  bool al16 = m4 && aligned(out, 16);
  for (int r = 0; r < R; ++r) {
    a->m.idx[r] = idx[r];
    a->m.codes[r] = codes[r];
    a->m.scales[r] = scales[r];
    al16 = al16 && aligned(idx[r], 16) && aligned(codes[r], 16);
  }
  a->out = out;
  a->flags = flags;
  a->outer_lr = outer_lr;
  a->chunk = chunk;
  a->k = k;
  a->bits = bits;
  a->R = R;
  a->stride = (uint32_t)codes_stride(k, bits);
  a->wait_polls = debug_wait_polls();
  a->theta_bf16 = bf16 ? 1 : 0;
  return launch_aggregate<T>(*a, apply, al16, st) == cudaSuccess ? SL_OK : SL_ERR_CUDA;
}

int aggregate_checked(int R, const uint16_t* const* idx, const uint8_t* const* codes,
                      const float* const* scales, const sl_layout* L, int chunk, int k, int bits,
                      float* out, float outer_lr, bool apply, uint32_t* flags, void* stream, bool bf16 = false) {
  if (R < 1 || R > SL_MAX_REPLICAS) return SL_ERR_INVALID_ARG;
  if (!idx || !codes || !scales || !out) return SL_ERR_INVALID_ARG;
  if (!std::isfinite(outer_lr)) return SL_ERR_INVALID_ARG;
  const int rc = check_common(L, chunk, k, bits);
  if (rc != SL_OK) return rc;
  if (!aligned(out, bf16 ? 2 : 4) || (flags && !aligned(flags, 4))) return SL_ERR_ALIGNMENT;
  for (int r = 0; r < R; ++r) {
    if (!idx[r] || !codes[r] || !scales[r]) return SL_ERR_INVALID_ARG;
    if (!aligned(idx[r], 2) || !aligned(scales[r], 4) || (bits == 32 && !aligned(codes[r], 4)))
      return SL_ERR_ALIGNMENT;
  }
  cudaStream_t st = (cudaStream_t)stream;
  if (L->n_tensors <= 256)
    return aggregate_impl<256>(R, idx, codes, scales, L, chunk, k, bits, out, outer_lr, apply, flags, st, bf16);
  return aggregate_impl<SL_MAX_TENSORS>(R, idx, codes, scales, L, chunk, k, bits, out, outer_lr, apply,
                                        flags, st, bf16);
}

template <int T>
int unpack_impl(const uint8_t* packed, const sl_layout* L, int chunk, int k, uint16_t* idx, cudaStream_t st) {
  Table<T> tb;
  bool m4;
  fill_table(tb, L, chunk, &m4);
  return launch_unpack_idx12(tb, packed, chunk, k, idx, st) == cudaSuccess ? SL_OK : SL_ERR_CUDA;
}

}  // namespace

extern "C" {

uint64_t sl_num_chunks(const sl_layout* L, int chunk) {
  if (!L || !L->offset || chunk < 1) return 0;
  const uint32_t side = tile_side(chunk);
  uint64_t nc = 0;
  for (uint32_t t = 0; t < L->n_tensors; ++t) {
    uint64_t c;
    if (!tensor_chunks(L, t, chunk, side, &c)) return 0;
    nc += c;
  }
  return nc;
}

uint64_t sl_codes_stride(int k, int bits) {
  if (k < 1 || !bits_ok(bits)) return 0;
  return codes_stride(k, bits);
}

uint64_t sl_codes_bytes(const sl_layout* L, int chunk, int k, int bits) {
  if (k < 1 || k > chunk || !bits_ok(bits)) return 0;
  return sl_num_chunks(L, chunk) * codes_stride(k, bits);
}

int sl_compress(const float* theta_local, const float* theta_global, float* err, const sl_layout* L,
                float beta, int chunk, int k, int bits, uint16_t* idx, uint8_t* codes, float* scales,
                uint32_t* flags, void* stream) {
  // theta_global is only read when no step is asked for
  return compress_checked(1, &theta_local, const_cast<float*>(theta_global), &err, L, beta, chunk, k, bits,
                          &idx, &codes, &scales, flags, stream);
}

int sl_compress_batch(int R, const float* const* theta_local, const float* theta_global,
                      float* const* err, const sl_layout* L, float beta, int chunk, int k, int bits,
                      uint16_t* const* idx, uint8_t* const* codes, float* const* scales,
                      uint32_t* flags, void* stream) {
  return compress_checked(R, theta_local, const_cast<float*>(theta_global), err, L, beta, chunk, k, bits, idx,
                          codes, scales, flags, stream);
}

int sl_outer_step(int R, const float* const* theta_local, float* theta_global, float* const* err,
                  const sl_layout* L, float beta, int chunk, int k, int bits, float outer_lr,
                  uint16_t* const* idx, uint8_t* const* codes, float* const* scales, uint32_t* flags,
                  void* stream) {
  return compress_checked(R, theta_local, theta_global, err, L, beta, chunk, k, bits, idx, codes, scales,
                          flags, stream, true, outer_lr);
}

int sl_aggregate(int R, const uint16_t* const* idx, const uint8_t* const* codes,
                 const float* const* scales, const sl_layout* L, int chunk, int k, int bits,
                 float* update, uint32_t* flags, void* stream) {
  return aggregate_checked(R, idx, codes, scales, L, chunk, k, bits, update, 0.0f, false, flags, stream);
}

int sl_outer_apply(float* theta_global, const float* update, uint64_t n, float outer_lr, void* stream) {
  if (!theta_global || !update || !std::isfinite(outer_lr)) return SL_ERR_INVALID_ARG;
  if (!aligned(theta_global, 4) || !aligned(update, 4)) return SL_ERR_ALIGNMENT;
  return launch_outer_apply(theta_global, update, n, outer_lr, (cudaStream_t)stream) == cudaSuccess
             ? SL_OK : SL_ERR_CUDA;
}

int sl_aggregate_apply(int R, const uint16_t* const* idx, const uint8_t* const* codes,
                       const float* const* scales, const sl_layout* L, int chunk, int k, int bits,
                       float* theta_global, float outer_lr, uint32_t* flags, void* stream) {
  return aggregate_checked(R, idx, codes, scales, L, chunk, k, bits, theta_global, outer_lr, true, flags,
                           stream);
}

int sl_compress_batch_bf16(int R, const uint16_t* const* theta_local, const uint16_t* theta_global,
                           float* const* err, const sl_layout* L, float beta, int chunk, int k, int bits,
                           uint16_t* const* idx, uint8_t* const* codes, float* const* scales, uint32_t* flags,
                           void* stream) {
  // the kernels take the parameter arrays through the float-typed slots of their argument block and
  // reinterpret them when `theta_bf16` is set; nothing is dereferenced on the host
  return compress_checked(R, reinterpret_cast<const float* const*>(theta_local),
                          reinterpret_cast<float*>(const_cast<uint16_t*>(theta_global)), err, L, beta, chunk, k, bits,
                          idx, codes, scales, flags, stream, false, 0.0f, true);
}

int sl_outer_step_bf16(int R, const uint16_t* const* theta_local, uint16_t* theta_global, float* const* err,
                       const sl_layout* L, float beta, int chunk, int k, int bits, float outer_lr,
                       uint16_t* const* idx, uint8_t* const* codes, float* const* scales, uint32_t* flags,
                       void* stream) {
  return compress_checked(R, reinterpret_cast<const float* const*>(theta_local), reinterpret_cast<float*>(theta_global),
                          err, L, beta, chunk, k, bits, idx, codes, scales, flags, stream, true, outer_lr, true);
}

int sl_aggregate_apply_bf16(int R, const uint16_t* const* idx, const uint8_t* const* codes,
                            const float* const* scales, const sl_layout* L, int chunk, int k, int bits,
                            uint16_t* theta_global, float outer_lr, uint32_t* flags, void* stream) {
  return aggregate_checked(R, idx, codes, scales, L, chunk, k, bits, reinterpret_cast<float*>(theta_global), outer_lr,
                           true, flags, stream, true);
}

int sl_outer_apply_bf16(uint16_t* theta_global, const float* update, uint64_t n, float outer_lr, void* stream) {
  if (!theta_global || !update || !std::isfinite(outer_lr)) return SL_ERR_INVALID_ARG;
  if (!aligned(theta_global, 2) || !aligned(update, 4)) return SL_ERR_ALIGNMENT;
  return launch_outer_apply_bf16(theta_global, update, n, outer_lr, (cudaStream_t)stream) == cudaSuccess
             ? SL_OK : SL_ERR_CUDA;
}

uint64_t sl_idx12_stride(int k) { return k < 1 ? 0 : (12u * (uint64_t)k + 7u) / 8u; }

int sl_pack_idx12(const uint16_t* idx, uint64_t n_chunks, int k, uint8_t* packed, uint32_t* flags, void* stream) {
  if (!idx || !packed || k < 1 || k > 4096) return SL_ERR_INVALID_ARG;
  if (!aligned(idx, 2) || (flags && !aligned(flags, 4))) return SL_ERR_ALIGNMENT;
  if (n_chunks > 0x7FFFFFFFull) return SL_ERR_UNSUPPORTED;
  return launch_pack_idx12(idx, n_chunks, k, packed, flags, (cudaStream_t)stream) == cudaSuccess ? SL_OK : SL_ERR_CUDA;
}

int sl_unpack_idx12(const uint8_t* packed, const sl_layout* L, int chunk, int k, uint16_t* idx, void* stream) {
  if (!packed || !idx) return SL_ERR_INVALID_ARG;
  const int rc = check_common(L, chunk, k, 32);
  if (rc != SL_OK) return rc;
  if (chunk > 4096) return SL_ERR_UNSUPPORTED;
  if (!aligned(idx, 2)) return SL_ERR_ALIGNMENT;
  cudaStream_t st = (cudaStream_t)stream;
  return L->n_tensors <= 256 ? unpack_impl<256>(packed, L, chunk, k, idx, st)
                             : unpack_impl<SL_MAX_TENSORS>(packed, L, chunk, k, idx, st);
}

namespace {
int subspace_check(const float* a, const int32_t* ids, const float* T_perp, const float* pos, const float* U, uint64_t n_tok,
                   uint32_t L, uint64_t V, uint32_t d, uint32_t k, const float* out, const uint32_t* flags) {
  if (!a || !U || !out || d < 1 || k < 1) return SL_ERR_INVALID_ARG;
  if (ids && (!T_perp || !pos || L < 1 || V < 1)) return SL_ERR_INVALID_ARG;
  if (!aligned(a, 4) || !aligned(U, 4) || !aligned(out, 4) || (flags && !aligned(flags, 4))) return SL_ERR_ALIGNMENT;
  if (ids && (!aligned(ids, 4) || !aligned(T_perp, 4) || !aligned(pos, 4))) return SL_ERR_ALIGNMENT;
  if (n_tok > 0x7FFFFFFFull || V > 0x7FFFFFFFull || k > 4096) return SL_ERR_UNSUPPORTED;
  return SL_OK;
}
}  // namespace

int sl_subspace_project(const float* X, const int32_t* ids, const float* T_perp, const float* pos, const float* U,
                        uint64_t n_tok, uint32_t L, uint64_t V, uint32_t d, uint32_t k, float* Xt, uint32_t* flags,
                        void* stream) {
  const int rc = subspace_check(X, ids, T_perp, pos, U, n_tok, L, V, d, k, Xt, flags);
  if (rc != SL_OK || n_tok == 0) return rc;
  return launch_subspace_project(X, ids, T_perp, pos, U, n_tok, L, V, d, k, Xt, flags, (cudaStream_t)stream) == cudaSuccess
             ? SL_OK : SL_ERR_CUDA;
}

int sl_subspace_reconstruct(const float* Xt, const int32_t* ids, const float* T_perp, const float* pos, const float* U,
                            uint64_t n_tok, uint32_t L, uint64_t V, uint32_t d, uint32_t k, float* Xhat, uint32_t* flags,
                            void* stream) {
  const int rc = subspace_check(Xt, ids, T_perp, pos, U, n_tok, L, V, d, k, Xhat, flags);
  if (rc != SL_OK || n_tok == 0) return rc;
  return launch_subspace_reconstruct(Xt, ids, T_perp, pos, U, n_tok, L, V, d, k, Xhat, flags, (cudaStream_t)stream) ==
                 cudaSuccess
             ? SL_OK : SL_ERR_CUDA;
}

int sl_round_tf32(float* x, uint64_t n, void* stream) {
  if (!x && n) return SL_ERR_INVALID_ARG;
  if (!aligned(x, 4)) return SL_ERR_ALIGNMENT;
  return launch_round_tf32(x, n, (cudaStream_t)stream) == cudaSuccess ? SL_OK : SL_ERR_CUDA;
}

int sl_embed_reproject(float* T_S, float* T_perp, const float* U, uint64_t V, uint32_t d, uint32_t k,
                       uint32_t* flags, void* stream) {
  if (!T_S || !T_perp || !U || d < 1 || k < 1) return SL_ERR_INVALID_ARG;
  if (!aligned(T_S, 4) || !aligned(T_perp, 4) || !aligned(U, 4) || (flags && !aligned(flags, 4)))
    return SL_ERR_ALIGNMENT;
  if (V > 0x7FFFFFFFull || k > 4096) return SL_ERR_UNSUPPORTED;
  if (V == 0) return SL_OK;
  return launch_embed_reproject(T_S, T_perp, U, V, d, k, flags, (cudaStream_t)stream) == cudaSuccess
             ? SL_OK : SL_ERR_CUDA;
}

int sl_debug_bounds_selftest(uint32_t* flags, uint32_t* probe, void* stream) {
#ifdef SL_DEBUG_BOUNDS
  if (!flags || !probe) return SL_ERR_INVALID_ARG;
  sl::bounds_selftest_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(flags, probe);
  return cudaPeekAtLastError() == cudaSuccess ? SL_OK : SL_ERR_CUDA;
#else
  (void)flags; (void)probe; (void)stream;
  return SL_ERR_UNSUPPORTED;
#endif
}

void sl_debug_set_wait_limit(int32_t polls) {
  sl::g_wait_polls.store(polls < 0 ? 0xFFFFFFFFu : (uint32_t)polls, std::memory_order_relaxed);
}

const char* sl_strerror(int code) {
  switch (code) {
    case SL_OK: return "ok";
    case SL_ERR_INVALID_ARG: return "invalid argument";
    case SL_ERR_ALIGNMENT: return "misaligned pointer";
    case SL_ERR_UNSUPPORTED: return "size outside what this build supports";
    case SL_ERR_CUDA: return "CUDA runtime or launch failure";
    default: return "unknown status";
  }
}

}  // extern "C"
