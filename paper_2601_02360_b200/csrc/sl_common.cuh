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
template <int T>
struct Table {
  uint32_t n_tensors;
  uint32_t n_chunks;
  uint32_t first_chunk[T + 1];
  uint64_t offset[T + 1];
};

struct ChunkRef {
  uint64_t base;  // element offset of the chunk in the arena
  int len;        // elements in the chunk (1..chunk)
};

// chunk g -> (base, len): binary search over the tensors' first chunks
template <int T>
__device__ __forceinline__ ChunkRef locate(const Table<T>& tb, uint32_t g, int chunk) {
  uint32_t lo = 0, hi = tb.n_tensors;  // first_chunk[lo] <= g < first_chunk[hi]
  while (hi - lo > 1) {
    const uint32_t mid = (lo + hi) >> 1;
    if (tb.first_chunk[mid] <= g) lo = mid; else hi = mid;
  }
  ChunkRef c;
  c.base = tb.offset[lo] + (uint64_t)(g - tb.first_chunk[lo]) * (uint64_t)chunk;
  const uint64_t left = tb.offset[lo + 1] - c.base;
  c.len = left < (uint64_t)chunk ? (int)left : chunk;
  return c;
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
  float* theta_out;   // fused step only: theta_global again, written with the outer update
  uint32_t* flags;
  float beta;
  float outer_lr;     // fused step only
  int fused;          // 1: the tuned kernel finishes every chunk with the average and the outer update
  int chunk, k, bits, R;
  uint32_t stride;  // bytes of codes per chunk
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
};

// ---------------------------------------------------------------------------
// the quantiser Q of Eq. 2 line 3 (paper leaves Q open; this build's reading):
// scale s = chunk maximum, L = 2^(bits-1) levels, thresholds s*(j/L),
// reconstruction at the level's midpoint s*(2q+1)/(2L).  Every product is one
// explicitly rounded multiply so that nothing can be contracted.
// ---------------------------------------------------------------------------
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

__device__ __forceinline__ void named_sync(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }
__device__ __forceinline__ void named_arrive(int id, int n) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(n) : "memory"); }

// ---------------------------------------------------------------------------
// Eq. 2 line 5 for one full 4096-element chunk, run by 256 threads (tid 0..255) that
// synchronise on named barrier `bar`.  `acc` is a 16 KB shared accumulator, G the thread's
// four float4s of theta_global (APPLY only), P any struct with idx[], codes[], scales[].
//  * the (replica, slot) pairs of the chunk are spread over the threads, up to kAggPairs per
//    thread and round; every pair's position and value are fetched before any is applied, so
//    the R messages cost one memory round trip instead of R (loads are ld.global.cg: the fused
//    step reads messages its own CTA has just written);
//  * the pairs are applied replica by replica (a barrier between replicas keeps the additions
//    in replica order; inside one message positions are distinct: no conflicts, no atomics);
//  * division by R is a multiplication by the exact reciprocal when R is a power of two (bit
//    identical), an IEEE division otherwise.
// Returns true if a slot named a position outside the chunk (skipped).
// ---------------------------------------------------------------------------
constexpr int kAggPairs = 4;

template <bool APPLY, typename P>
__device__ __forceinline__ bool aggregate_chunk_c4096(float* acc, const float4 (&G)[4], const P& m, uint32_t g,
                                                      int k, int bits, int R, uint32_t stride,
                                                      float4* out4, float outer_lr, int tid, int bar) {
#pragma unroll
  for (int j = 0; j < 4; ++j) reinterpret_cast<float4*>(acc)[tid + 256 * j] = make_float4(0.f, 0.f, 0.f, 0.f);
  bool bad = false;
  const int total = R * k;
  const int kshift = (k & (k - 1)) == 0 ? 31 - __clz(k) : -1;
  for (int q0 = 0; q0 < total; q0 += 256 * kAggPairs) {
    uint32_t pos[kAggPairs];
    float val[kAggPairs];
    int rep[kAggPairs];
#pragma unroll
    for (int i = 0; i < kAggPairs; ++i) {
      const int q = q0 + tid + 256 * i;            // pair q = (replica q / k, slot q % k)
      pos[i] = 0xFFFFu;
      val[i] = 0.0f;
      rep[i] = -1;
      if (q < total) {
        const int r = kshift >= 0 ? (q >> kshift) : q / k;
        const int j = q - r * k;
        rep[i] = r;
        const uint32_t p = __ldcg(m.idx[r] + (uint64_t)g * (uint64_t)k + j);
        const uint8_t* codes = m.codes[r] + (uint64_t)g * (uint64_t)stride;
        if (bits == 32) {
          val[i] = __ldcg(reinterpret_cast<const float*>(codes) + j);
        } else {
          const float s = __ldcg(m.scales[r] + g);
          const uint32_t bit = (uint32_t)j * (uint32_t)bits;
          const uint32_t code = ((uint32_t)__ldcg(codes + (bit >> 3)) >> (bit & 7u)) & ((1u << bits) - 1u);
          val[i] = dequant(code, s, bits);
        }
        if (p != 0xFFFFu && p >= 4096u) bad = true; else pos[i] = p;
      }
    }
    const int r_lo = kshift >= 0 ? (q0 >> kshift) : q0 / k;
    const int r_hi = min(R - 1, (q0 + 256 * kAggPairs - 1) / k);
    named_sync(bar, 256);                          // accumulator zeroed / previous round applied
    for (int r = r_lo; r <= r_hi; ++r) {
#pragma unroll
      for (int i = 0; i < kAggPairs; ++i)
        if (rep[i] == r && pos[i] != 0xFFFFu) acc[pos[i]] = __fadd_rn(acc[pos[i]], val[i]);
      named_sync(bar, 256);
    }
  }
  if (total == 0) named_sync(bar, 256);
  const bool pow2 = (R & (R - 1)) == 0;
  const float Rf = (float)R, invR = 1.0f / Rf;
  const float nlr = -outer_lr;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float4 s4 = reinterpret_cast<const float4*>(acc)[tid + 256 * j];
    float4 u;
    if (pow2) {
      u.x = __fmul_rn(s4.x, invR); u.y = __fmul_rn(s4.y, invR); u.z = __fmul_rn(s4.z, invR); u.w = __fmul_rn(s4.w, invR);
    } else {
      u.x = __fdiv_rn(s4.x, Rf); u.y = __fdiv_rn(s4.y, Rf); u.z = __fdiv_rn(s4.z, Rf); u.w = __fdiv_rn(s4.w, Rf);
    }
    if (APPLY) {
      u.x = __fmaf_rn(nlr, u.x, G[j].x); u.y = __fmaf_rn(nlr, u.y, G[j].y);
      u.z = __fmaf_rn(nlr, u.z, G[j].z); u.w = __fmaf_rn(nlr, u.w, G[j].w);
    }
    __stcs(out4 + tid + 256 * j, u);
  }
  return bad;
}

// ---------------------------------------------------------------------------
// launchers implemented in the kernel files (host side, return cudaError_t)
// ---------------------------------------------------------------------------
template <int T> cudaError_t launch_compress(const CompressArgs<T>& a, bool aligned16, cudaStream_t st);
template <int T> bool compress_is_tuned(const CompressArgs<T>& a, bool aligned16);
template <int T> cudaError_t launch_aggregate(const AggregateArgs<T>& a, bool apply, bool aligned16, cudaStream_t st);
template <int T> cudaError_t launch_aggregate_tails(const AggregateArgs<T>& a, bool apply, cudaStream_t st);
cudaError_t launch_outer_apply(float* theta, const float* update, uint64_t n, float lr, cudaStream_t st);

}  // namespace sl
