// Eq. 2 lines 1-4 (paper §2.1): pseudo-gradient, error feedback, chunk-wise Top-k,
// quantisation, residual.  One CTA owns one (chunk, replica) pair.
#include "sl_common.cuh"

namespace sl {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

__device__ __forceinline__ uint32_t lanemask_lt() {
  uint32_t m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}

// ---------------------------------------------------------------------------
// Generic exact kernel: any chunk length up to SL_MAX_CHUNK, any k <= chunk,
// any supported code width, no alignment requirement.
//
//  1. e' = fma(beta, e, theta_global - theta_local) into shared memory.
//  2. the k-th largest 31-bit magnitude key by a 4-pass radix select
//     (8+8+8+7 bits, shared-memory histogram, suffix scan by one warp).
//  3. kept set = keys above the k-th key plus the lowest-positioned ties;
//     emitted in ascending position with warp ballots (each warp walks one
//     contiguous region of the chunk, regions are stitched by prefix counts).
//  4. codes packed in shared memory, residual patched in shared memory, then
//     one coalesced write of e and of the message.
// ---------------------------------------------------------------------------
template <int T>
__global__ void __launch_bounds__(kThreads)
compress_generic_kernel(const __grid_constant__ CompressArgs<T> a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* ep = reinterpret_cast<float*>(smem_raw);                          // [chunk]
  uint32_t* hist = reinterpret_cast<uint32_t*>(ep + a.chunk);              // [256]
  uint32_t* cw = hist + 256;                                               // [ceil(stride/4)] packed codes
  __shared__ uint32_t s_wmax[kWarps];
  __shared__ uint32_t s_weq[kWarps], s_wgt[kWarps];
  __shared__ uint32_t s_digit, s_need;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t g = blockIdx.x / (uint32_t)a.R;
  const int r = (int)(blockIdx.x % (uint32_t)a.R);
  const ChunkRef c = locate(a.tb, g, a.chunk);
  const int len = c.len;
  const int k = a.k, bits = a.bits;
  const int k_eff = k < len ? k : len;

  const float* __restrict__ tl = a.p.theta_local[r] + c.base;
  const float* __restrict__ tg = a.theta_global + c.base;
  float* __restrict__ er = a.p.err[r] + c.base;

  // ---- 1. pseudo-gradient and error feedback ------------------------------
  uint32_t tmax = 0;
  for (int i = tid; i < len; i += kThreads) {
    const float d = __fsub_rn(tg[i], tl[i]);
    const float e = __fmaf_rn(a.beta, er[i], d);
    ep[i] = e;
    tmax = max(tmax, key_of(e));
  }
  tmax = __reduce_max_sync(0xFFFFFFFFu, tmax);
  if (lane == 0) s_wmax[warp] = tmax;
  const uint32_t cwords = (a.stride + 3) >> 2;
  if (bits != 32)
    for (uint32_t i = tid; i < cwords; i += kThreads) cw[i] = 0;
  __syncthreads();
  uint32_t smax = 0;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) smax = max(smax, s_wmax[w]);
  const float s = __uint_as_float(smax);

  // ---- 2. radix select of the k_eff-th largest key -------------------------
  uint32_t prefix = 0, need = (uint32_t)k_eff;
#pragma unroll 1
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = pass == 0 ? 23 : pass == 1 ? 15 : pass == 2 ? 7 : 0;
    const int width = pass == 3 ? 7 : 8;
    const int hs = shift + width;                 // bits above this digit are already fixed
    hist[tid] = 0;
    __syncthreads();
    for (int i = tid; i < len; i += kThreads) {
      const uint32_t key = key_of(ep[i]);
      if ((key >> hs) == (prefix >> hs)) atomicAdd(&hist[(key >> shift) & ((1u << width) - 1u)], 1u);
    }
    __syncthreads();
    if (warp == 0) {
      uint32_t h[8], mine = 0;
#pragma unroll
      for (int b = 0; b < 8; ++b) { h[b] = hist[lane * 8 + b]; mine += h[b]; }
      uint32_t suf = mine;                        // inclusive suffix sum over lanes >= lane
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t o = __shfl_down_sync(0xFFFFFFFFu, suf, d);
        if (lane + d < 32) suf += o;
      }
      const uint32_t vote = __ballot_sync(0xFFFFFFFFu, suf >= need);
      const int sel = 31 - __clz(vote);           // highest lane whose suffix still reaches `need`
      if (lane == sel) {
        uint32_t cum = suf - mine, digit = (uint32_t)lane * 8u, left = need;
        bool found = false;
#pragma unroll
        for (int bb = 7; bb >= 0; --bb) {         // walk this lane's bins from the top digit down
          if (!found) {
            if (cum + h[bb] >= need) { found = true; digit = (uint32_t)(lane * 8 + bb); left = need - cum; }
            else cum += h[bb];
          }
        }
        s_digit = digit;
        s_need = left;
      }
    }
    __syncthreads();
    prefix |= s_digit << shift;
    need = s_need;
  }
  const uint32_t kth = prefix;                    // the k_eff-th largest key; `need` ties of it are kept

  // ---- 3. ordered emission --------------------------------------------------
  const int rw = ((len + kThreads - 1) / kThreads) * 32;   // region per warp, multiple of 32
  const int r0 = warp * rw;
  const int r1 = min(len, r0 + rw);
  uint32_t ceq = 0, cgt = 0;
  for (int i0 = r0; i0 < r1; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t key = i < r1 ? key_of(ep[i]) : 0u;
    ceq += __popc(__ballot_sync(0xFFFFFFFFu, i < r1 && key == kth));
    cgt += __popc(__ballot_sync(0xFFFFFFFFu, i < r1 && key > kth));
  }
  if (lane == 0) { s_weq[warp] = ceq; s_wgt[warp] = cgt; }
  __syncthreads();
  uint32_t eq_base = 0, out_base = 0;
  for (int w = 0; w < warp; ++w) {
    const uint32_t weq = s_weq[w];
    const uint32_t room = need > eq_base ? need - eq_base : 0u;
    out_base += s_wgt[w] + min(room, weq);
    eq_base += weq;
  }
  uint16_t* __restrict__ oidx = a.p.idx[r] + (uint64_t)g * (uint64_t)k;
  uint8_t* __restrict__ ocodes = a.p.codes[r] + (uint64_t)g * (uint64_t)a.stride;
  for (int i0 = r0; i0 < r1; i0 += 32) {
    const int i = i0 + lane;
    const bool in = i < r1;
    const float v = in ? ep[i] : 0.0f;
    const uint32_t key = key_of(v);
    const bool eq = in && key == kth;
    const uint32_t eqm = __ballot_sync(0xFFFFFFFFu, eq);
    const bool keep = in && (key > kth || (eq && eq_base + __popc(eqm & lanemask_lt()) < need));
    const uint32_t km = __ballot_sync(0xFFFFFFFFu, keep);
    if (keep) {
      const uint32_t slot = out_base + __popc(km & lanemask_lt());
      oidx[slot] = (uint16_t)i;
      float sent;
      if (bits == 32) {
        reinterpret_cast<float*>(ocodes)[slot] = v;
        sent = v;
      } else {
        const uint32_t code = quant_code(v, s, bits);
        atomicOr(&cw[(slot * (uint32_t)bits) >> 5], code << ((slot * (uint32_t)bits) & 31u));
        sent = dequant(code, s, bits);
      }
      ep[i] = __fsub_rn(v, sent);                 // line 4: the residual
    }
    eq_base += __popc(eqm);
    out_base += __popc(km);
  }
  __syncthreads();

  // ---- 4. write-back ---------------------------------------------------------
  for (int i = tid; i < len; i += kThreads) er[i] = ep[i];
  for (int j = k_eff + tid; j < k; j += kThreads) oidx[j] = 0xFFFFu;
  if (bits != 32) {
    const uint8_t* cb = reinterpret_cast<const uint8_t*>(cw);
    for (uint32_t i = tid; i < a.stride; i += kThreads) ocodes[i] = cb[i];
  } else {
    for (int j = k_eff + tid; j < k; j += kThreads) reinterpret_cast<float*>(ocodes)[j] = 0.0f;
  }
  if (tid == 0) {
    a.p.scales[r][g] = s;
    if (smax >= 0x7F800000u && a.flags) atomicOr(a.flags, (uint32_t)SL_FLAG_NONFINITE);
  }
}

}  // namespace

template <int T>
cudaError_t launch_compress(const CompressArgs<T>& a, bool aligned16, cudaStream_t st) {
  (void)aligned16;
  if (a.tb.n_chunks == 0) return cudaSuccess;
  const size_t smem = (size_t)a.chunk * 4 + 256 * 4 + (a.bits == 32 ? 0 : (size_t)((a.stride + 3) / 4) * 4);
  const uint64_t blocks = (uint64_t)a.tb.n_chunks * (uint64_t)a.R;
  if (blocks > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(compress_generic_kernel<T>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  compress_generic_kernel<T><<<(unsigned)blocks, kThreads, smem, st>>>(a);
  return cudaPeekAtLastError();
}

template cudaError_t launch_compress<256>(const CompressArgs<256>&, bool, cudaStream_t);
template cudaError_t launch_compress<SL_MAX_TENSORS>(const CompressArgs<SL_MAX_TENSORS>&, bool, cudaStream_t);

}  // namespace sl
