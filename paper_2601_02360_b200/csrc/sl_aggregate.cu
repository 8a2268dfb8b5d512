// Eq. 2 line 5 (paper §2.1): average of the R sparse messages and the SGD outer step.
#include "sl_common.cuh"

namespace sl {

namespace {

constexpr int kThreads = 256;

// One CTA per chunk.  The chunk's dense update is built in shared memory by R scatter passes
// in replica order (positions inside one message are distinct, so a pass has no conflicts and
// needs no atomics; a barrier separates the passes), then divided by R and either written out
// (APPLY = false) or folded straight into theta_global (APPLY = true).
// TAILS = false: CTA b handles chunk b.  TAILS = true: CTA b handles the short last chunk of
// tensor b (if it has one), which is how the tuned kernel delegates the tensors' ragged ends.
template <int T, bool APPLY, bool TAILS>
__global__ void __launch_bounds__(kThreads)
aggregate_generic_kernel(const __grid_constant__ AggregateArgs<T> a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* acc = reinterpret_cast<float*>(smem_raw);  // [chunk]
  const int tid = threadIdx.x;
  uint32_t g = blockIdx.x;
  if (TAILS) {
    const uint32_t t = g;
    const uint64_t n_t = a.tb.offset[t + 1] - a.tb.offset[t];
    if (n_t % (uint64_t)a.chunk == 0) return;
    g = a.tb.first_chunk[t + 1] - 1;
  }
  const ChunkRef c = locate(a.tb, g, a.chunk);
  const int len = c.len, k = a.k, bits = a.bits;

  for (int i = tid; i < len; i += kThreads) acc[i] = 0.0f;
  __syncthreads();
  bool bad = false;
  for (int r = 0; r < a.R; ++r) {
    const uint16_t* __restrict__ idx = a.m.idx[r] + (uint64_t)g * (uint64_t)k;
    const uint8_t* __restrict__ codes = a.m.codes[r] + (uint64_t)g * (uint64_t)a.stride;
    const float s = a.m.scales[r][g];
    for (int j = tid; j < k; j += kThreads) {
      const uint32_t i = idx[j];
      if (i == 0xFFFFu) continue;                 // padding slot
      if (i >= (uint32_t)len) { bad = true; continue; }
      float v;
      if (bits == 32) {
        v = reinterpret_cast<const float*>(codes)[j];
      } else {
        const uint32_t bit = (uint32_t)j * (uint32_t)bits;
        const uint32_t code = ((uint32_t)codes[bit >> 3] >> (bit & 7u)) & ((1u << bits) - 1u);
        v = dequant(code, s, bits);
      }
      acc[i] = __fadd_rn(acc[i], v);
    }
    __syncthreads();
  }
  const float Rf = (float)a.R;
  float* __restrict__ out = a.out + c.base;
  for (int i = tid; i < len; i += kThreads) {
    const float u = __fdiv_rn(acc[i], Rf);
    out[i] = APPLY ? __fmaf_rn(-a.outer_lr, u, out[i]) : u;
  }
  if (bad && a.flags) atomicOr(a.flags, (uint32_t)SL_FLAG_BAD_INDEX);
}

// Tuned kernel for full 4096-element chunks of a 16-byte aligned arena.  One CTA per chunk:
//  * theta_global's 16 KB are requested first (four 128-bit loads per thread) so that they fly
//    while the messages are handled;
//  * the (replica, slot) pairs of the chunk are spread over all threads, up to kPairs per
//    thread and round, and every pair's position and value are fetched before any is applied,
//    so the R messages cost one memory round trip instead of R;
//  * the pairs are then applied to the shared-memory accumulator replica by replica (a barrier
//    between replicas keeps the additions in replica order; inside one message positions are
//    distinct, so there are no conflicts);
//  * division by R is a multiplication by the exact reciprocal when R is a power of two (bit
//    identical), an IEEE division otherwise.
constexpr int kAC = 4096;
constexpr int kPairs = 4;

template <int T, bool APPLY>
__global__ void __launch_bounds__(kThreads)
aggregate_c4096_kernel(const __grid_constant__ AggregateArgs<T> a) {
  __shared__ __align__(16) float acc[kAC];
  const int tid = threadIdx.x;
  const uint32_t g = blockIdx.x;
  const ChunkRef c = locate(a.tb, g, kAC);
  if (c.len != kAC) return;                       // short chunks go to the generic tail launch
  const int k = a.k, bits = a.bits, R = a.R;

  float4* __restrict__ out4 = reinterpret_cast<float4*>(a.out + c.base);
  float4 G[4];
  if (APPLY) {
#pragma unroll
    for (int j = 0; j < 4; ++j) G[j] = __ldcs(out4 + tid + 256 * j);
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) reinterpret_cast<float4*>(acc)[tid + 256 * j] = make_float4(0.f, 0.f, 0.f, 0.f);

  bool bad = false;
  const int total = R * k;
  for (int q0 = 0; q0 < total; q0 += kThreads * kPairs) {
    // fetch this round's pairs: pair q = (replica q / k, slot q % k); q grows with the replica
    uint32_t pos[kPairs];
    float val[kPairs];
    int rep[kPairs];
#pragma unroll
    for (int i = 0; i < kPairs; ++i) {
      const int q = q0 + tid + kThreads * i;
      pos[i] = 0xFFFFu;
      val[i] = 0.0f;
      rep[i] = -1;
      if (q < total) {
        const int r = q / k, j = q - r * k;
        rep[i] = r;
        const uint32_t p = __ldg(a.m.idx[r] + (uint64_t)g * (uint64_t)k + j);
        const uint8_t* __restrict__ codes = a.m.codes[r] + (uint64_t)g * (uint64_t)a.stride;
        if (bits == 32) {
          val[i] = __ldg(reinterpret_cast<const float*>(codes) + j);
        } else {
          const float s = __ldg(a.m.scales[r] + g);
          const uint32_t bit = (uint32_t)j * (uint32_t)bits;
          const uint32_t code = ((uint32_t)__ldg(codes + (bit >> 3)) >> (bit & 7u)) & ((1u << bits) - 1u);
          val[i] = dequant(code, s, bits);
        }
        if (p != 0xFFFFu && p >= (uint32_t)kAC) bad = true; else pos[i] = p;
      }
    }
    const int r_lo = q0 / k;
    const int r_hi = min(R - 1, (q0 + kThreads * kPairs - 1) / k);
    __syncthreads();                              // accumulator zeroed / previous round applied
    for (int r = r_lo; r <= r_hi; ++r) {
#pragma unroll
      for (int i = 0; i < kPairs; ++i)
        if (rep[i] == r && pos[i] != 0xFFFFu) acc[pos[i]] = __fadd_rn(acc[pos[i]], val[i]);
      __syncthreads();
    }
  }
  if (total == 0) __syncthreads();

  const bool pow2 = (R & (R - 1)) == 0;
  const float Rf = (float)R, invR = 1.0f / Rf;
  const float nlr = -a.outer_lr;
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
  if (bad && a.flags) atomicOr(a.flags, (uint32_t)SL_FLAG_BAD_INDEX);
}

__global__ void __launch_bounds__(256)
outer_apply_kernel(float* __restrict__ theta, const float* __restrict__ update, uint64_t n, float lr,
                   int vec) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  const uint64_t t0 = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const float nlr = -lr;
  if (vec) {
    const uint64_t n4 = n >> 2;
    float4* __restrict__ th4 = reinterpret_cast<float4*>(theta);
    const float4* __restrict__ up4 = reinterpret_cast<const float4*>(update);
    for (uint64_t i = t0; i < n4; i += stride) {
      float4 t = th4[i];
      const float4 u = up4[i];
      t.x = __fmaf_rn(nlr, u.x, t.x);
      t.y = __fmaf_rn(nlr, u.y, t.y);
      t.z = __fmaf_rn(nlr, u.z, t.z);
      t.w = __fmaf_rn(nlr, u.w, t.w);
      th4[i] = t;
    }
    for (uint64_t i = (n4 << 2) + t0; i < n; i += stride) theta[i] = __fmaf_rn(nlr, update[i], theta[i]);
  } else {
    for (uint64_t i = t0; i < n; i += stride) theta[i] = __fmaf_rn(nlr, update[i], theta[i]);
  }
}

}  // namespace

template <int T>
cudaError_t launch_aggregate(const AggregateArgs<T>& a, bool apply, bool aligned16, cudaStream_t st) {
  if (a.tb.n_chunks == 0) return cudaSuccess;
  const size_t smem = (size_t)a.chunk * 4;
  if (aligned16 && a.chunk == kAC) {
    if (apply) aggregate_c4096_kernel<T, true><<<a.tb.n_chunks, kThreads, 0, st>>>(a);
    else aggregate_c4096_kernel<T, false><<<a.tb.n_chunks, kThreads, 0, st>>>(a);
    bool tails = false;
    for (uint32_t t = 0; t < a.tb.n_tensors; ++t)
      tails = tails || ((a.tb.offset[t + 1] - a.tb.offset[t]) % (uint64_t)kAC) != 0;
    if (tails) {
      if (apply) aggregate_generic_kernel<T, true, true><<<a.tb.n_tensors, kThreads, smem, st>>>(a);
      else aggregate_generic_kernel<T, false, true><<<a.tb.n_tensors, kThreads, smem, st>>>(a);
    }
    return cudaPeekAtLastError();
  }
  if (apply) aggregate_generic_kernel<T, true, false><<<a.tb.n_chunks, kThreads, smem, st>>>(a);
  else aggregate_generic_kernel<T, false, false><<<a.tb.n_chunks, kThreads, smem, st>>>(a);
  return cudaPeekAtLastError();
}

template cudaError_t launch_aggregate<256>(const AggregateArgs<256>&, bool, bool, cudaStream_t);
template cudaError_t launch_aggregate<SL_MAX_TENSORS>(const AggregateArgs<SL_MAX_TENSORS>&, bool, bool, cudaStream_t);

cudaError_t launch_outer_apply(float* theta, const float* update, uint64_t n, float lr, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  const int vec = (((uintptr_t)theta | (uintptr_t)update) & 15u) == 0;
  const uint64_t work = vec ? (n + 3) / 4 : n;
  uint64_t blocks = (work + 255) / 256;
  const uint64_t cap = 148ull * 8ull;  // grid-stride over one full wave: 8 CTAs of 256 threads per SM
  if (blocks > cap) blocks = cap;
  outer_apply_kernel<<<(unsigned)blocks, 256, 0, st>>>(theta, update, n, lr, vec);
  return cudaPeekAtLastError();
}

}  // namespace sl
