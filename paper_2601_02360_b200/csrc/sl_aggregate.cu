// Eq. 2 line 5 (paper §2.1): average of the R sparse messages and the SGD outer step.
#include <algorithm>

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

// Tuned kernel for full 4096-element chunks of a 16-byte aligned arena.  Persistent grid: CTA b
// walks chunks b, b+G, b+2G, ...  Per chunk:
//  * theta_global's 16 KB are requested first (four 128-bit loads per thread) so that they fly
//    while the messages are handled;
//  * the (replica, slot) pairs of the chunk are spread over the threads, NP per thread: pair
//    q = tid + 256 i is slot q % k of replica q / k.  What does not depend on the chunk (replica,
//    slot, the three pointers, the bit offset of the code) is computed once per thread, outside
//    the chunk loop.  Every pair's position and value are fetched before any is applied, so the R
//    messages cost one memory round trip instead of R;
//  * the pairs are applied to a 16 KB shared accumulator in replica order: one round per replica,
//    a barrier between rounds (inside one message positions are distinct: no conflicts, no
//    atomics; across messages the barrier fixes the order of the additions);
//  * division by R is a multiplication by the exact reciprocal when R is a power of two (bit
//    identical), an IEEE division otherwise; the outer update is one fused multiply-add.
constexpr int kAC = 4096;

template <int T, bool APPLY, int NP>
__global__ void __launch_bounds__(kThreads)
aggregate_c4096_kernel(const __grid_constant__ AggregateArgs<T> a) {
  __shared__ __align__(16) float acc[kAC];
  const int tid = threadIdx.x;
  const int k = a.k, bits = a.bits, R = a.R;
  const int total = R * k;

  // per-thread, chunk-independent description of its pairs
  const uint16_t* p_idx[NP];
  const uint8_t* p_code[NP];
  const float* p_scale[NP];
  int rep[NP];
  uint32_t cshift[NP];
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const int q = tid + kThreads * i;
    rep[i] = -1;
    p_idx[i] = nullptr; p_code[i] = nullptr; p_scale[i] = nullptr; cshift[i] = 0;
    if (q < total) {
      const int r = q / k, j = q - r * k;
      rep[i] = r;
      p_idx[i] = a.m.idx[r] + j;
      const uint32_t bit = (uint32_t)j * (uint32_t)bits;
      p_code[i] = bits == 32 ? a.m.codes[r] + 4 * (size_t)j : a.m.codes[r] + (bit >> 3);
      cshift[i] = bit & 7u;
      p_scale[i] = a.m.scales[r];
    }
  }
  const uint32_t cmask = bits == 32 ? 0xFFFFFFFFu : (1u << bits) - 1u;
  const bool pow2 = (R & (R - 1)) == 0;
  const float Rf = (float)R, invR = 1.0f / Rf;
  const float nlr = -a.outer_lr;
  bool bad = false;
  uint32_t t_lo = 0;                               // tensor of the previous chunk: the next one is usually the same

  for (uint32_t g = blockIdx.x; g < a.tb.n_chunks; g += gridDim.x) {
    // chunk -> (base, full?) with the previous tensor as the first guess
    if (!(a.tb.first_chunk[t_lo] <= g && g < a.tb.first_chunk[t_lo + 1])) {
      uint32_t lo = 0, hi = a.tb.n_tensors;
      while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (a.tb.first_chunk[mid] <= g) lo = mid; else hi = mid;
      }
      t_lo = lo;
    }
    const uint64_t base = a.tb.offset[t_lo] + (uint64_t)(g - a.tb.first_chunk[t_lo]) * (uint64_t)kAC;
    if (a.tb.offset[t_lo + 1] - base < (uint64_t)kAC) continue;   // short chunks go to the generic tail launch

    float4* out4 = reinterpret_cast<float4*>(a.out + base);
    float4 G[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) G[j] = APPLY ? __ldcs(out4 + tid + 256 * j) : make_float4(0.f, 0.f, 0.f, 0.f);
    uint32_t pos[NP];
    float val[NP];
#pragma unroll
    for (int i = 0; i < NP; ++i) {
      pos[i] = 0xFFFFu;
      val[i] = 0.0f;
      if (rep[i] >= 0) {
        const uint32_t p = __ldg(p_idx[i] + (uint64_t)g * (uint64_t)k);
        if (bits == 32) {
          val[i] = __ldg(reinterpret_cast<const float*>(p_code[i] + (uint64_t)g * (uint64_t)a.stride));
        } else {
          const uint32_t code = ((uint32_t)__ldg(p_code[i] + (uint64_t)g * (uint64_t)a.stride) >> cshift[i]) & cmask;
          val[i] = dequant(code, __ldg(p_scale[i] + g), bits);
        }
        if (p != 0xFFFFu && p >= (uint32_t)kAC) bad = true; else pos[i] = p;
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) reinterpret_cast<float4*>(acc)[tid + 256 * j] = make_float4(0.f, 0.f, 0.f, 0.f);
    __syncthreads();                               // accumulator zeroed (and the previous chunk's read of it done)
    for (int r = 0; r < R; ++r) {
#pragma unroll
      for (int i = 0; i < NP; ++i)
        if (rep[i] == r && pos[i] != 0xFFFFu) acc[pos[i]] = __fadd_rn(acc[pos[i]], val[i]);
      __syncthreads();
    }
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
    __syncthreads();                               // everyone has read the accumulator before it is zeroed again
  }
  if (bad && a.flags) atomicOr(a.flags, (uint32_t)SL_FLAG_BAD_INDEX);
}

template <int T, bool APPLY>
cudaError_t launch_aggregate_c4096(const AggregateArgs<T>& a, cudaStream_t st) {
  int dev = 0, sms = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  const int pairs = (a.R * a.k + kThreads - 1) / kThreads;
  // persistent grid: exactly as many CTAs as are resident at once, so that every CTA walks the
  // same number of chunks
  auto launch = [&](auto kernel) -> cudaError_t {
    int per_sm = 0;
    cudaError_t err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, 0);
    if (err != cudaSuccess) return err;
    if (per_sm < 1) per_sm = 1;
    const unsigned grid = (unsigned)std::min<uint64_t>((uint64_t)a.tb.n_chunks, (uint64_t)sms * (uint64_t)per_sm);
    kernel<<<grid, kThreads, 0, st>>>(a);
    return cudaPeekAtLastError();
  };
  if (pairs <= 1) return launch(aggregate_c4096_kernel<T, APPLY, 1>);
  if (pairs <= 2) return launch(aggregate_c4096_kernel<T, APPLY, 2>);
  if (pairs <= 4) return launch(aggregate_c4096_kernel<T, APPLY, 4>);
  return launch(aggregate_c4096_kernel<T, APPLY, 8>);
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
  if (aligned16 && a.chunk == kAC && a.R * a.k <= kThreads * 8) {
    cudaError_t e0 = apply ? launch_aggregate_c4096<T, true>(a, st) : launch_aggregate_c4096<T, false>(a, st);
    if (e0 != cudaSuccess) return e0;
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
