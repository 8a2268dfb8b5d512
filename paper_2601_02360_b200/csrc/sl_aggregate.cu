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

// Tuned kernel for full 4096-element chunks of a 16-byte aligned arena.  One CTA per chunk;
// theta_global's 16 KB are requested first (four 128-bit loads per thread) so that they fly
// while the messages are handled; the rest is aggregate_chunk_c4096().
constexpr int kAC = 4096;

template <int T, bool APPLY>
__global__ void __launch_bounds__(kThreads)
aggregate_c4096_kernel(const __grid_constant__ AggregateArgs<T> a) {
  __shared__ __align__(16) float acc[kAC];
  const int tid = threadIdx.x;
  const uint32_t g = blockIdx.x;
  const ChunkRef c = locate(a.tb, g, kAC);
  if (c.len != kAC) return;                       // short chunks go to the generic tail launch
  float4* out4 = reinterpret_cast<float4*>(a.out + c.base);
  float4 G[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) G[j] = APPLY ? __ldcs(out4 + tid + 256 * j) : make_float4(0.f, 0.f, 0.f, 0.f);
  const bool bad = aggregate_chunk_c4096<APPLY>(acc, G, a.m, g, a.k, a.bits, a.R, a.stride, out4, a.outer_lr, tid, 0);
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
    const cudaError_t e = launch_aggregate_tails<T>(a, apply, st);
    if (e != cudaSuccess) return e;
    return cudaPeekAtLastError();
  }
  if (apply) aggregate_generic_kernel<T, true, false><<<a.tb.n_chunks, kThreads, smem, st>>>(a);
  else aggregate_generic_kernel<T, false, false><<<a.tb.n_chunks, kThreads, smem, st>>>(a);
  return cudaPeekAtLastError();
}

template <int T>
cudaError_t launch_aggregate_tails(const AggregateArgs<T>& a, bool apply, cudaStream_t st) {
  bool tails = false;
  for (uint32_t t = 0; t < a.tb.n_tensors; ++t)
    tails = tails || ((a.tb.offset[t + 1] - a.tb.offset[t]) % (uint64_t)a.chunk) != 0;
  if (!tails) return cudaSuccess;
  const size_t smem = (size_t)a.chunk * 4;
  if (apply) aggregate_generic_kernel<T, true, true><<<a.tb.n_tensors, kThreads, smem, st>>>(a);
  else aggregate_generic_kernel<T, false, true><<<a.tb.n_tensors, kThreads, smem, st>>>(a);
  return cudaPeekAtLastError();
}

template cudaError_t launch_aggregate_tails<256>(const AggregateArgs<256>&, bool, cudaStream_t);
template cudaError_t launch_aggregate_tails<SL_MAX_TENSORS>(const AggregateArgs<SL_MAX_TENSORS>&, bool, cudaStream_t);
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
