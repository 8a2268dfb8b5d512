// Shared device-side pieces of the SparseLoCo outer-step kernels (paper §2.1, Eq. 2).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sparseloco.h"

namespace sl {

// ---------------------------------------------------------------------------
// arena description handed to the kernels BY VALUE (kernel parameter space =
// constant bank), so that the library needs no device-side table and no state.
// first_chunk[t] = number of chunks owned by tensors before t.
// ---------------------------------------------------------------------------
// cols[t] > 0: tensor t is a matrix of cols[t] columns cut into side x side tiles (side*side = chunk).
template <int T>
struct Table {
  uint32_t n_tensors;
  uint32_t n_chunks;
  uint32_t side;      // tile side, 0 when no tensor is tiled
  uint32_t n_tails;   // chunks that are not full (short last chunks, edge tiles)
  uint32_t first_chunk[T + 1];
  uint32_t first_tail[T + 1];   // not-full chunks owned by tensors before t
  uint32_t cols[T + 1];
  uint64_t offset[T + 1];
};

struct ChunkRef {
  uint64_t base;    // element offset of the chunk's first element in the arena
  int len;          // elements in the chunk (1..chunk)
  uint32_t stride;  // 0: consecutive chunk; else the matrix's row length (the chunk is a tile)
  uint32_t w;       // tile: columns of this tile (<= side)
  uint32_t side;    // tile: side of a full tile

  // the d-th element of the chunk (ascending position): its arena offset and its position
  __device__ __forceinline__ uint64_t addr(int d) const {
    if (stride == 0) return base + (uint64_t)d;
    const uint32_t lr = (uint32_t)d / w, lc = (uint32_t)d - lr * w;
    return base + (uint64_t)lr * stride + lc;
  }
  __device__ __forceinline__ uint32_t pos(int d) const {
    if (stride == 0) return (uint32_t)d;
    const uint32_t lr = (uint32_t)d / w, lc = (uint32_t)d - lr * w;
    return lr * side + lc;
  }
  // position -> element number, or -1 if the chunk has no such position
  __device__ __forceinline__ int elem(uint32_t p) const {
    if (stride == 0) return p < (uint32_t)len ? (int)p : -1;
    const uint32_t lr = p / side, lc = p - lr * side;
    return (lc < w && lr * w + lc < (uint32_t)len) ? (int)(lr * w + lc) : -1;
  }
};

// geometry of chunk g, which belongs to tensor lo
template <int T>
__device__ __forceinline__ ChunkRef chunk_of_tensor(const Table<T>& tb, uint32_t lo, uint32_t g, int chunk) {
  ChunkRef c;
  const uint32_t nc = tb.cols[lo];
  const uint32_t in_t = g - tb.first_chunk[lo];
  if (nc == 0) {
    c.base = tb.offset[lo] + (uint64_t)in_t * (uint64_t)chunk;
    const uint64_t left = tb.offset[lo + 1] - c.base;
    c.len = left < (uint64_t)chunk ? (int)left : chunk;
    c.stride = 0; c.w = 0; c.side = 0;
  } else {
    const uint32_t s = tb.side;
    const uint32_t tiles_c = (nc + s - 1) / s;
    const uint32_t tr = in_t / tiles_c, tc = in_t - tr * tiles_c;
    const uint64_t rows = (tb.offset[lo + 1] - tb.offset[lo]) / nc;
    const uint64_t r0 = (uint64_t)tr * s, c0 = (uint64_t)tc * s;
    const uint32_t h = (uint32_t)(rows - r0 < s ? rows - r0 : s);
    c.w = (uint32_t)(nc - c0 < s ? nc - c0 : s);
    c.base = tb.offset[lo] + r0 * nc + c0;
    c.len = (int)(h * c.w);
    c.stride = nc;
    c.side = s;
  }
  return c;
}

// chunk g -> its geometry: binary search over the tensors' first chunks
template <int T>
__device__ __forceinline__ ChunkRef locate(const Table<T>& tb, uint32_t g, int chunk) {
  uint32_t lo = 0, hi = tb.n_tensors;  // first_chunk[lo] <= g < first_chunk[hi]
  while (hi - lo > 1) {
    const uint32_t mid = (lo + hi) >> 1;
    if (tb.first_chunk[mid] <= g) lo = mid; else hi = mid;
  }
  return chunk_of_tensor(tb, lo, g, chunk);
}

// the same, trying the tensor of the caller's previous chunk first (t_lo is updated)
template <int T>
__device__ __forceinline__ ChunkRef locate_cached(const Table<T>& tb, uint32_t g, int chunk, uint32_t& t_lo) {
  if (!(tb.first_chunk[t_lo] <= g && g < tb.first_chunk[t_lo + 1])) {
    uint32_t lo = 0, hi = tb.n_tensors;
    while (hi - lo > 1) {
      const uint32_t mid = (lo + hi) >> 1;
      if (tb.first_chunk[mid] <= g) lo = mid; else hi = mid;
    }
    t_lo = lo;
  }
  return chunk_of_tensor(tb, t_lo, g, chunk);
}

// the e-th chunk of the arena that is not full (e < n_tails) -> its chunk number.  A tensor with
// consecutive chunks has at most one (its last); a tiled matrix has its right edge column of
// tiles (if cols is not a multiple of the side), then its bottom edge row.
template <int T>
__device__ __forceinline__ uint32_t tail_chunk(const Table<T>& tb, uint32_t e, int chunk) {
  uint32_t lo = 0, hi = tb.n_tensors;  // first_tail[lo] <= e < first_tail[hi]
  while (hi - lo > 1) {
    const uint32_t mid = (lo + hi) >> 1;
    if (tb.first_tail[mid] <= e) lo = mid; else hi = mid;
  }
  const uint32_t j = e - tb.first_tail[lo];
  const uint32_t nc = tb.cols[lo];
  if (nc == 0) return tb.first_chunk[lo + 1] - 1;
  const uint32_t s = tb.side;
  const uint64_t rows = (tb.offset[lo + 1] - tb.offset[lo]) / nc;
  const uint32_t fr = (uint32_t)(rows / s), fc = nc / s;
  const uint32_t tr = (uint32_t)((rows + s - 1) / s), tc = (nc + s - 1) / s;
  const uint32_t right = tc > fc ? tr : 0;      // tiles of the right edge column
  uint32_t tile_r, tile_c;
  if (j < right) { tile_r = j; tile_c = fc; } else { tile_r = fr; tile_c = j - right; }
  return tb.first_chunk[lo] + tile_r * tc + tile_c;
}

// per-replica pointer tables, by value as well
struct CompressPtrs {
  const float* theta_local[SL_MAX_REPLICAS];
  float* err[SL_MAX_REPLICAS];
  uint16_t* idx[SL_MAX_REPLICAS];
  uint8_t* codes[SL_MAX_REPLICAS];
  float* scales[SL_MAX_REPLICAS];
};

struct MessagePtrs {
  const uint16_t* idx[SL_MAX_REPLICAS];
  const uint8_t* codes[SL_MAX_REPLICAS];
  const float* scales[SL_MAX_REPLICAS];
};

template <int T>
struct CompressArgs {
  Table<T> tb;
  CompressPtrs p;
  const float* theta_global;
  uint32_t* flags;
  float beta;
  int chunk, k, bits, R;
  uint32_t stride;  // bytes of codes per chunk
  uint32_t wait_polls;  // polls a bounded wait makes before it gives up (0: the default, about a second;
                        // 0xFFFFFFFF: none, every wait gives up at once)
  int theta_bf16;       // 1: theta_local / theta_global point to bfloat16 arrays (error buffers stay float32)
};

template <int T>
struct AggregateArgs {
  Table<T> tb;
  MessagePtrs m;
  float* out;       // dense update (aggregate) or theta_global (aggregate + apply)
  uint32_t* flags;
  float outer_lr;
  int chunk, k, bits, R;
  uint32_t stride;
  uint32_t wait_polls;  // as in CompressArgs
  int theta_bf16;       // 1 (aggregate + apply only): `out` is theta_global stored as bfloat16
};

// ---------------------------------------------------------------------------
// the quantiser Q of Eq. 2 line 3 (paper leaves Q open; this build's reading):
// scale s = chunk maximum, L = 2^(bits-1) levels, thresholds s*(j/L),
// reconstruction at the level's midpoint s*(2q+1)/(2L).  Every product is one
// explicitly rounded multiply so that nothing can be contracted.
// ---------------------------------------------------------------------------
// Parameters stored as bfloat16 (the upper half of a binary32).  Widening is exact; storing rounds to
// nearest, ties to even; a NaN stays a NaN (quiet bit set, sign and upper payload kept).
__device__ __forceinline__ float bf16_widen(uint32_t h) { return __uint_as_float(h << 16); }
__device__ __forceinline__ uint32_t bf16_round(float v) {
  const uint32_t b = __float_as_uint(v);
  if ((b & 0x7FFFFFFFu) > 0x7F800000u) return (b >> 16) | 0x0040u;
  return (b + 0x7FFFu + ((b >> 16) & 1u)) >> 16;      // adds just under half, and the last kept bit: half goes to even
}
// four consecutive bfloat16 values held in a uint2 <-> float4
__device__ __forceinline__ float4 bf16x4_widen(uint2 v) {
  return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u), __uint_as_float(v.y << 16),
                     __uint_as_float(v.y & 0xFFFF0000u));
}
__device__ __forceinline__ uint2 bf16x4_round(float4 v) {
  return make_uint2(bf16_round(v.x) | (bf16_round(v.y) << 16), bf16_round(v.z) | (bf16_round(v.w) << 16));
}

__device__ __forceinline__ uint32_t key_of(float v) { return __float_as_uint(v) & 0x7FFFFFFFu; }

// q = number of thresholds t_j = s*(j/L), j = 1..L-1, with |v| >= t_j.  The t_j are
// non-decreasing in j, so the count is found by bisection on j.
__device__ __forceinline__ uint32_t quant_level(float v, float s, int bits) {
  const float a = fabsf(v);
  if (bits == 2) return (a >= __fmul_rn(s, 0.5f)) ? 1u : 0u;
  const int L = 1 << (bits - 1);
  const float invL = 1.0f / (float)L;  // power of two: j * invL is exact
  int lo = 0, hi = L - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (a >= __fmul_rn(s, (float)mid * invL)) lo = mid; else hi = mid - 1;
  }
  return (uint32_t)lo;
}

__device__ __forceinline__ uint32_t quant_code(float v, float s, int bits) {
  return ((__float_as_uint(v) >> 31) << (bits - 1)) | quant_level(v, s, bits);
}

__device__ __forceinline__ float dequant(uint32_t code, float s, int bits) {
  const int L = 1 << (bits - 1);
  const uint32_t q = code & (uint32_t)(L - 1);
  const uint32_t sign = (code >> (bits - 1)) & 1u;
  const float mag = __fmul_rn(s, (float)(2u * q + 1u) * (0.5f / (float)L));
  return __uint_as_float(__float_as_uint(mag) | (sign << 31));
}

// polls every bounded on-chip wait makes before it gives up, as set by sl_debug_set_wait_limit (0: default)
uint32_t debug_wait_polls();

// number of SMs of the current device (grid sizing); 0 with *e set when the query fails
inline int sm_count(cudaError_t* e) {
  int dev = 0, sms = 0;
  if ((*e = cudaGetDevice(&dev)) != cudaSuccess) return 0;
  if ((*e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return 0;
  return sms;
}

// ---------------------------------------------------------------------------
// Range checks of the debug build (-DSL_DEBUG_BOUNDS; the stand-in for a memory checker).  Every index
// the Eq. 2 kernels form for shared or global memory goes through SL_CHECK(flags, condition): in the
// debug build a false condition raises SL_FLAG_BOUNDS and the expression is false, so that the access
// guarded by it is skipped (never a trap, never an assert); in the normal build the expression is the
// constant true and the condition is not evaluated.
// ---------------------------------------------------------------------------
#ifdef SL_DEBUG_BOUNDS
__device__ __forceinline__ bool bounds_check(uint32_t* flags, bool in_range) {
  if (!in_range && flags) atomicOr(flags, (uint32_t)SL_FLAG_BOUNDS);
  return in_range;
}
#define SL_CHECK(flags, cond) (::sl::bounds_check((flags), (cond)))
#else
#define SL_CHECK(flags, cond) (true)
#endif

__device__ __forceinline__ void named_sync(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }
__device__ __forceinline__ void named_arrive(int id, int n) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(n) : "memory"); }

// ---------------------------------------------------------------------------
// launchers implemented in the kernel files (host side, return cudaError_t)
// ---------------------------------------------------------------------------
template <int T> cudaError_t launch_compress(const CompressArgs<T>& a, bool aligned16, cudaStream_t st);
template <int T> bool compress_is_tuned(const CompressArgs<T>& a, bool aligned16);
template <int T> cudaError_t launch_aggregate(const AggregateArgs<T>& a, bool apply, bool aligned16, cudaStream_t st);
template <int T> cudaError_t launch_aggregate_tails(const AggregateArgs<T>& a, bool apply, cudaStream_t st);
cudaError_t launch_outer_apply(float* theta, const float* update, uint64_t n, float lr, cudaStream_t st);
cudaError_t launch_outer_apply_bf16(uint16_t* theta, const float* update, uint64_t n, float lr, cudaStream_t st);
cudaError_t launch_pack_idx12(const uint16_t* idx, uint64_t n_chunks, int k, uint8_t* packed, uint32_t* flags,
                              cudaStream_t st);
template <int T> cudaError_t launch_unpack_idx12(const Table<T>& tb, const uint8_t* packed, int chunk, int k,
                                                 uint16_t* idx, cudaStream_t st);
cudaError_t launch_subspace_project(const float* X, const int32_t* ids, const float* T_perp, const float* pos,
                                    const float* U, uint64_t n_tok, uint32_t L, uint64_t V, uint32_t d, uint32_t k,
                                    float* Xt, uint32_t* flags, cudaStream_t st);
cudaError_t launch_subspace_reconstruct(const float* Xt, const int32_t* ids, const float* T_perp, const float* pos,
                                        const float* U, uint64_t n_tok, uint32_t L, uint64_t V, uint32_t d, uint32_t k,
                                        float* Xhat, uint32_t* flags, cudaStream_t st);
cudaError_t launch_round_tf32(float* x, uint64_t n, cudaStream_t st);
bool embed_is_tuned(const float* T_S, const float* T_perp, const float* U, uint32_t d, uint32_t k);
cudaError_t launch_embed_reproject(float* T_S, float* T_perp, const float* U, uint64_t V, uint32_t d, uint32_t k,
                                   uint32_t* flags, cudaStream_t st);

}  // namespace sl
