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
// TAILS = false: CTA b handles chunk b.  TAILS = true: CTA b handles the b-th chunk that is not
// full (short last chunks, edge tiles), which is how the tuned kernel delegates the ragged ends.
template <int T, bool APPLY, bool TAILS>
__global__ void __launch_bounds__(kThreads)
aggregate_generic_kernel(const __grid_constant__ AggregateArgs<T> a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* acc = reinterpret_cast<float*>(smem_raw);  // [chunk]
  const int tid = threadIdx.x;
  uint32_t g = blockIdx.x;
  if (TAILS) g = tail_chunk(a.tb, g, a.chunk);    // the g-th chunk that is not full
  if (!SL_CHECK(a.flags, g < a.tb.n_chunks)) return;
  const ChunkRef c = locate(a.tb, g, a.chunk);
  const int len = c.len, k = a.k, bits = a.bits;
  const uint64_t n_total = a.tb.offset[a.tb.n_tensors];
  (void)n_total;
  if (!SL_CHECK(a.flags, len >= 1 && len <= a.chunk)) return;

  for (int i = tid; i < len; i += kThreads) acc[i] = 0.0f;   // one accumulator per element of the chunk
  __syncthreads();
  bool bad = false;
  for (int r = 0; r < a.R; ++r) {
    const uint16_t* __restrict__ idx = a.m.idx[r] + (uint64_t)g * (uint64_t)k;
    const uint8_t* __restrict__ codes = a.m.codes[r] + (uint64_t)g * (uint64_t)a.stride;
    const float s = a.m.scales[r][g];
    for (int j = tid; j < k; j += kThreads) {
      const uint32_t p = idx[j];
      if (p == 0xFFFFu) continue;                 // padding slot
      const int i = c.elem(p);                    // position -> element number (they differ in edge tiles)
      if (i < 0) { bad = true; continue; }
      if (!SL_CHECK(a.flags, i < len)) continue;
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
  float* __restrict__ out = a.out;
  for (int i = tid; i < len; i += kThreads) {
    const float u = __fdiv_rn(acc[i], Rf);
    const uint64_t at = c.addr(i);
    if (!SL_CHECK(a.flags, at < n_total)) continue;
    if (APPLY && a.theta_bf16) {
      uint16_t* o16 = reinterpret_cast<uint16_t*>(a.out);
      o16[at] = (uint16_t)bf16_round(__fmaf_rn(-a.outer_lr, u, bf16_widen(o16[at])));
    } else {
      out[at] = APPLY ? __fmaf_rn(-a.outer_lr, u, out[at]) : u;
    }
  }
  if (bad && a.flags) atomicOr(a.flags, (uint32_t)SL_FLAG_BAD_INDEX);
}

// Tuned kernel for full 4096-element chunks of a 16-byte aligned arena.  Persistent grid: CTA b
// walks the full chunks among b, b+G, b+2G, ...  Software pipelined over chunks: while chunk i is
// accumulated and written, the next chunk's theta_global is already on its way into shared memory
// (one 16 KB TMA bulk copy per CTA, double buffered, mbarrier completion) and its message
// entries are on their way into registers.  Per chunk:
//  * the (replica, slot) pairs of the chunk are spread over the threads, NP per thread: pair
//    q = tid + 256 i is slot q % k of replica q / k.  What does not depend on the chunk (replica,
//    slot, the three pointers, the bit offset of the code) is computed once per thread;
//  * the pairs are applied to a 16 KB shared accumulator in replica order: one round per replica
//    (and per group of 256 pairs it has entries in), a barrier between rounds (inside one message
//    positions are distinct: no conflicts, no atomics; across messages the barrier fixes the order
//    of the additions);
//  * division by R is a multiplication by the exact reciprocal when R is a power of two (bit
//    identical), an IEEE division otherwise; the outer update is one fused multiply-add; the
//    result leaves with 128-bit streaming stores.
constexpr int kAC = 4096;
constexpr uint32_t kAggWaitLimit = 1u << 22;

struct AggSmem {
  float acc[kAC];
  float gbuf[2][kAC];                // theta_global of the current / next chunk (APPLY only)
  uint64_t full[2];
  volatile uint32_t abort_it;        // non-zero once the bounded wait has given up
};

__device__ __forceinline__ uint32_t agg_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// the cold end of a give-up, kept out of line so that it does not weigh on the kernel's hot code: waits
// (bounded) for the last two of the `issued` bulk copies of theta_global (the j-th went to buffer j & 1) and
// raises the flag
__device__ __noinline__ void agg_giveup_drain(uint64_t* full, uint32_t issued, uint32_t* flags) {
  for (uint32_t j = issued >= 2 ? issued - 2 : 0; j < issued; ++j) {
    const uint32_t bar = agg_smem_u32(&full[j & 1]), parity = (j >> 1) & 1u;
    for (uint32_t spin = 0; spin < kAggWaitLimit; ++spin) {
      uint32_t done;
      asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                   : "=r"(done) : "r"(bar), "r"(parity) : "memory");
      if (done) break;
    }
  }
  if (flags) atomicOr(flags, (uint32_t)SL_FLAG_TIMEOUT);
}

// first full chunk at or after g (stepping by `step`); t_lo caches the tensor of the last hit;
// stride = elements between the chunk's rows of 64 (64 for a consecutive chunk)
template <int T>
__device__ __forceinline__ bool next_full_chunk(const Table<T>& tb, uint32_t& g, uint32_t step, uint32_t& t_lo,
                                                uint64_t& base, uint32_t& stride) {
  for (; g < tb.n_chunks; g += step) {
    const ChunkRef c = locate_cached(tb, g, kAC, t_lo);
    if (c.len == kAC) { base = c.base; stride = c.stride ? c.stride : 64u; return true; }
  }
  return false;                                    // chunks that are not full go to the generic tail launch
}

// TILED (arenas with matrices cut into 64 x 64 tiles): a chunk is 64 rows of 256 bytes `stride`
// elements apart; theta_global then comes in by 16-byte cp.async copies of all threads instead
// of one bulk copy, and the stores follow the same geometry.
//
// The wait for theta_global is bounded.  If it runs out, a mark is set in shared memory: the threads that
// gave up skip their stores, no further chunk of theta_global is requested (the issuing thread looks at
// the mark first), every later wait returns at once (and its stores are skipped), and the CTA walks the
// rest of its chunks with its barriers in step; at the end the copies still in flight are allowed to
// land (bounded again) and SL_FLAG_TIMEOUT is raised.  The loop carries no exit for this: a branch out
// of it cost 1.6 % of the launch.
//
// GROUPED (k a multiple of NP): a thread owns NP consecutive slots of ONE replica instead of NP
// pairs 256 apart.  Its positions then arrive as one 2*NP-byte load and its codes as a few bytes,
// and the accumulation takes R rounds in which the owners of replica r read their NP accumulator
// cells, add, and write them back (positions inside one message are distinct, so the cells are).
// BF (with APPLY, consecutive chunks): theta_global is a bfloat16 array; a chunk of it is 8 KB, widened as
// it is read and rounded to nearest-even as it is stored.
template <int T, bool APPLY, int NP, bool TILED, bool GROUPED, bool BF = false>
__global__ void __launch_bounds__(kThreads)
aggregate_c4096_kernel(const __grid_constant__ AggregateArgs<T> a) {
  static_assert(!BF || (APPLY && !TILED), "bfloat16 parameters: fused update on consecutive chunks only");
  extern __shared__ __align__(16) unsigned char agg_smem_raw[];
  AggSmem& sm = *reinterpret_cast<AggSmem*>(agg_smem_raw);
  float* acc = sm.acc;
  const int tid = threadIdx.x;
  const int k = a.k, bits = a.bits, R = a.R;
  const int total = R * k;
  constexpr uint32_t kBytes = kAC * 4;
  const uint64_t n_total = a.tb.offset[a.tb.n_tensors];
  (void)n_total;

  // per-thread, chunk-independent description of its pairs
  const uint16_t* p_idx[NP];
  const uint8_t* p_code[NP];
  const float* p_scale[NP];
  int rep[NP];
  uint32_t cshift[NP];
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const int q = GROUPED ? tid * NP + i : tid + kThreads * i;
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
  // GROUPED: all NP pairs of a thread belong to replica rep[0] and start at slot j0 (a multiple of NP);
  // only pair 0's pointers are used, the others are dead and cost no registers
  const int my_r = rep[0];
  const uint32_t cmask = bits == 32 ? 0xFFFFFFFFu : (1u << bits) - 1u;
  const bool pow2 = (R & (R - 1)) == 0;
  const float Rf = (float)R, invR = 1.0f / Rf;
  const float nlr = -a.outer_lr;
  bool bad = false;
  const uint32_t wait_limit = a.wait_polls == 0 ? kAggWaitLimit : a.wait_polls == 0xFFFFFFFFu ? 0u : a.wait_polls;

  if (APPLY && tid == 0) {
    sm.abort_it = 0;
    for (int s = 0; s < 2; ++s)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(agg_smem_u32(&sm.full[s])), "r"(TILED ? kThreads : 1) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  // raw message entries of a chunk: position, code bits (or the float itself), scale
  uint32_t rp[NP], rc[NP];
  float rs[NP];
  uint32_t gi[NP > 1 ? NP / 2 : 1];       // GROUPED: the positions, two per word
  uint64_t gw = 0;                         // GROUPED: the bytes holding the NP codes
  float gs = 0.0f;
  auto fetch = [&](uint32_t g) {
    if (!SL_CHECK(a.flags, g < a.tb.n_chunks)) {     // (debug build) no message is read for such a chunk
#pragma unroll
      for (int i = 0; i < NP; ++i) { rp[i] = 0xFFFFu; rc[i] = 0; rs[i] = 0.0f; }
#pragma unroll
      for (int i = 0; i < (NP > 1 ? NP / 2 : 1); ++i) gi[i] = 0xFFFFFFFFu;
      gw = 0; gs = 0.0f;
      return;
    }
    if constexpr (GROUPED) {
#pragma unroll
      for (int i = 0; i < (NP > 1 ? NP / 2 : 1); ++i) gi[i] = 0xFFFFFFFFu;
      gw = 0; gs = 0.0f;
      if (my_r >= 0) {
        const uint16_t* pi = p_idx[0] + (uint64_t)g * (uint64_t)k;
        if constexpr (NP == 8) {
          const uint4 v = __ldg(reinterpret_cast<const uint4*>(pi));
          gi[0] = v.x; gi[1] = v.y; gi[2] = v.z; gi[3] = v.w;
        } else if constexpr (NP == 4) {
          const uint2 v = __ldg(reinterpret_cast<const uint2*>(pi));
          gi[0] = v.x; gi[1] = v.y;
        } else if constexpr (NP == 2) {
          gi[0] = __ldg(reinterpret_cast<const uint32_t*>(pi));
        } else {
          gi[0] = 0xFFFF0000u | (uint32_t)__ldg(pi);
        }
        const uint8_t* pc = p_code[0] + (uint64_t)g * (uint64_t)a.stride;
        if (bits == 32) {
#pragma unroll
          for (int i = 0; i < NP; ++i) rc[i] = __float_as_uint(__ldg(reinterpret_cast<const float*>(pc) + i));
        } else {
          const uint32_t nb = (cshift[0] + (uint32_t)NP * (uint32_t)bits + 7u) >> 3;   // 1..8 bytes
          for (uint32_t b = 0; b < nb; ++b) gw |= (uint64_t)__ldg(pc + b) << (8u * b);
          gs = __ldg(p_scale[0] + g);
        }
      }
    } else {
#pragma unroll
      for (int i = 0; i < NP; ++i) {
        rp[i] = 0xFFFFu; rc[i] = 0; rs[i] = 0.0f;
        if (rep[i] >= 0) {
          rp[i] = __ldg(p_idx[i] + (uint64_t)g * (uint64_t)k);
          if (bits == 32) {
            rc[i] = __float_as_uint(__ldg(reinterpret_cast<const float*>(p_code[i] + (uint64_t)g * (uint64_t)a.stride)));
          } else {
            rc[i] = (uint32_t)__ldg(p_code[i] + (uint64_t)g * (uint64_t)a.stride);
            rs[i] = __ldg(p_scale[i] + g);
          }
        }
      }
    }
  };
  uint32_t issued = 0;                     // thread 0: bulk copies of theta_global requested so far
  auto load_theta = [&](uint64_t base, uint32_t stride, int buf) {
    const uint32_t bar = agg_smem_u32(&sm.full[buf]);
    if ((TILED || tid == 0) && sm.abort_it != 0) return;     // a wait has given up: nothing more is requested
    if (TILED) {                                   // every thread: four 16-byte copies, then one arrival
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int f = tid + 256 * j;
        const float* src = a.out + base + (size_t)(f >> 4) * stride + (size_t)((f & 15) << 2);
        if (SL_CHECK(a.flags, base + (size_t)(f >> 4) * stride + (size_t)((f & 15) << 2) + 4 <= n_total))
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;"
                     ::"r"(agg_smem_u32(reinterpret_cast<float4*>(sm.gbuf[buf]) + f)), "l"(src) : "memory");
      }
      asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
    } else if (tid == 0 && SL_CHECK(a.flags, base + kAC <= n_total)) {   // one 16 KB bulk copy
      constexpr uint32_t kThBytes = BF ? kBytes / 2 : kBytes;
      const void* src = BF ? (const void*)(reinterpret_cast<const uint16_t*>(a.out) + base) : (const void*)(a.out + base);
      ++issued;
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kThBytes) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(agg_smem_u32(sm.gbuf[buf])), "l"(src), "r"(kThBytes), "r"(bar) : "memory");
    }
  };

  uint32_t g = blockIdx.x, t_lo = 0, stride = 64;
  uint64_t base = 0;
  bool valid = next_full_chunk(a.tb, g, gridDim.x, t_lo, base, stride);
  if (valid) {
    if (APPLY) load_theta(base, stride, 0);
    fetch(g);
  }
  for (uint32_t it = 0; valid; ++it) {
    // this chunk's entries become values; then the next chunk's loads are issued
    uint32_t pos[NP];
    float val[NP];
#pragma unroll
    for (int i = 0; i < NP; ++i) {
      pos[i] = 0xFFFFu;
      val[i] = 0.0f;
      if (rep[i] >= 0) {
        uint32_t p;
        if constexpr (GROUPED) {
          p = (gi[i >> 1] >> (16 * (i & 1))) & 0xFFFFu;
          val[i] = bits == 32 ? __uint_as_float(rc[i])
                              : dequant((uint32_t)(gw >> (cshift[0] + (uint32_t)i * (uint32_t)bits)) & cmask, gs, bits);
        } else {
          p = rp[i];
          val[i] = bits == 32 ? __uint_as_float(rc[i]) : dequant((rc[i] >> cshift[i]) & cmask, rs[i], bits);
        }
        if (p != 0xFFFFu && p >= (uint32_t)kAC) bad = true; else pos[i] = p;
      }
    }
    const uint64_t base_cur = base;
    const uint32_t stride_cur = stride;
    g += gridDim.x;
    valid = next_full_chunk(a.tb, g, gridDim.x, t_lo, base, stride);
    if (valid) {
      if (APPLY) load_theta(base, stride, (it + 1) & 1);   // that buffer was last read before the barrier ending iteration it-1
      fetch(g);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) reinterpret_cast<float4*>(acc)[tid + 256 * j] = make_float4(0.f, 0.f, 0.f, 0.f);
    __syncthreads();
    if constexpr (GROUPED) {
      // one round per replica: its owners read their cells, add, write back
      for (int r = 0; r < R; ++r) {
        if (my_r == r) {
          float cur[NP];
#pragma unroll
          for (int i = 0; i < NP; ++i) cur[i] = pos[i] != 0xFFFFu ? acc[pos[i]] : 0.0f;
#pragma unroll
          for (int i = 0; i < NP; ++i)
            if (pos[i] != 0xFFFFu) acc[pos[i]] = __fadd_rn(cur[i], val[i]);
        }
        __syncthreads();
      }
    } else {
      // pair i of all threads covers pairs 256 i .. 256 i + 255, i.e. the replicas r_lo..r_hi below (non-
      // decreasing with i): one round per (i, replica) in that order applies every replica's entries
      // after all entries of the replicas before it, with one predicated add per thread and round
#pragma unroll
      for (int i = 0; i < NP; ++i) {
        const int q_lo = kThreads * i;
        if (q_lo < total) {
          const int r_lo = q_lo / k, q_hi = min(q_lo + kThreads, total) - 1, r_hi = q_hi / k;
          for (int r = r_lo; r <= r_hi; ++r) {
            if (rep[i] == r && pos[i] != 0xFFFFu) acc[pos[i]] = __fadd_rn(acc[pos[i]], val[i]);
            __syncthreads();
          }
        }
      }
    }
    const float4* g4 = reinterpret_cast<const float4*>(sm.gbuf[it & 1]);
    bool have_theta = true;
    if (APPLY) {                                   // bounded wait for this chunk's theta_global
      const uint32_t bar = agg_smem_u32(&sm.full[it & 1]), parity = (it >> 1) & 1u;
      bool ok = false;
      for (uint32_t spin = 0; spin < wait_limit && !ok; ++spin) {
        uint32_t done;
        if (a.wait_polls)                          // a caller-set limit counts non-blocking polls ...
          asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                       : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        else                                       // ... the default ones that suspend the thread for a while
          asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                       : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        ok = done != 0;
        if (!ok && sm.abort_it) break;
      }
      if (!ok) { sm.abort_it = 1; have_theta = false; }
    }
    float* out_cur = a.out + base_cur;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int f = tid + 256 * j;                 // float4 f of the chunk: row f / 16 of a tile
      const size_t off = TILED ? (size_t)(f >> 4) * stride_cur + (size_t)((f & 15) << 2) : (size_t)f * 4;
      float4* dst = reinterpret_cast<float4*>(out_cur + off);
      if (!SL_CHECK(a.flags, base_cur + off + 4 <= n_total)) continue;
      const float4 s4 = reinterpret_cast<const float4*>(acc)[tid + 256 * j];
      float4 u;
      if (pow2) {
        u.x = __fmul_rn(s4.x, invR); u.y = __fmul_rn(s4.y, invR); u.z = __fmul_rn(s4.z, invR); u.w = __fmul_rn(s4.w, invR);
      } else {
        u.x = __fdiv_rn(s4.x, Rf); u.y = __fdiv_rn(s4.y, Rf); u.z = __fdiv_rn(s4.z, Rf); u.w = __fdiv_rn(s4.w, Rf);
      }
      if (APPLY) {
        float4 G;
        if constexpr (BF) G = bf16x4_widen(reinterpret_cast<const uint2*>(sm.gbuf[it & 1])[tid + 256 * j]);
        else G = g4[tid + 256 * j];
        u.x = __fmaf_rn(nlr, u.x, G.x); u.y = __fmaf_rn(nlr, u.y, G.y);
        u.z = __fmaf_rn(nlr, u.z, G.z); u.w = __fmaf_rn(nlr, u.w, G.w);
      }
      if constexpr (BF) {
        if (have_theta) __stcs(reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(a.out) + base_cur + off), bf16x4_round(u));
      } else {
        if (have_theta) __stcs(dst, u);
      }
    }
    __syncthreads();                               // accumulator and theta buffer read by everyone before they are reused
  }
  if (APPLY) {
    if (sm.abort_it != 0) {                        // gave up somewhere: the copies in flight may land first
      if (TILED) asm volatile("cp.async.wait_all;" ::: "memory");
      if (tid == 0) agg_giveup_drain(sm.full, TILED ? 0u : issued, a.flags);
    }
  }
  if (bad && a.flags) atomicOr(a.flags, (uint32_t)SL_FLAG_BAD_INDEX);
}

// Fused average + update for FEW entries per chunk (R * k <= 256, one per thread), consecutive chunks or
// 64 x 64 tiles, float32 parameters, outer_lr > 0.  An element no replica sent has the mean update +0, and
// theta - outer_lr * (+0) is theta itself, bit for bit: for outer_lr > 0 the product is -0 and x + (-0) = x
// for every x, both zeros included (and a position's sum starts from +0, so it is never -0).  So
// theta_global is neither read nor rewritten as a whole: only the elements some replica sent are loaded,
// updated and stored instead of all 16 KB twice.  Thread q owns slot q % k of replica q / k.  Software pipeline over the group's chunks, three in
// flight (deeper ones were no faster: the launch is bound by DRAM, which moves 64 bytes for every element
// read and as much for every element written back, about 16 KB per chunk at R * k = 128 - half of the dense
// form, not a fifth): raw entries are requested two chunks ahead, one chunk ahead they are decoded and the
// theta_global elements they name are requested, and the oldest chunk - whose elements arrived an
// iteration ago - is processed:
//   every entry clears its accumulator cell; then one round per replica in the order 0..R-1 adds its
//   values (positions inside a message are distinct, so a round has no conflicts; a bit map tells an
//   entry whether an earlier replica already named its position); then the FIRST entry of every position
//   divides the finished sum by R, applies the fused step to the element it loaded, and stores it.
constexpr int kSparseMaxEntries = 256;

struct SparseSmem {
  float acc[kAC];
  uint32_t seen[kAC / 32];
};

// GROUPS: with R * k <= 256 / GROUPS entries per chunk the CTA's threads form GROUPS independent groups, each
// walking its own chunks with its own accumulator, bit map and named barrier (the launch is bound by the
// barriers of a chunk, so smaller groups on more chunks at once are faster).
template <int T, int GROUPS>
__global__ void __launch_bounds__(kThreads)
aggregate_sparse_kernel(const __grid_constant__ AggregateArgs<T> a) {
  extern __shared__ __align__(16) unsigned char sparse_smem_raw[];
  constexpr int GT = kThreads / GROUPS;            // threads of a group (a multiple of 32)
  const int gidx = (int)threadIdx.x / GT;
  SparseSmem& sm = reinterpret_cast<SparseSmem*>(sparse_smem_raw)[gidx];
  const int tid = (int)threadIdx.x - gidx * GT;    // index inside the group = the entry this thread owns
  const uint32_t vcta = blockIdx.x * GROUPS + gidx, vgrid = gridDim.x * GROUPS;    // the group as a CTA of a larger grid
  auto group_sync = [&]() { if (GROUPS == 1) __syncthreads(); else named_sync(1 + gidx, GT); };
  const int k = a.k, bits = a.bits, R = a.R;
  const uint64_t n_total = a.tb.offset[a.tb.n_tensors];
  (void)n_total;
  const int my_r = tid < R * k ? tid / k : -1;
  const int my_j = my_r >= 0 ? tid - my_r * k : 0;
  const uint16_t* p_idx = my_r >= 0 ? a.m.idx[my_r] + my_j : nullptr;
  const uint32_t bit0 = (uint32_t)my_j * (uint32_t)bits;
  const uint8_t* p_code = my_r >= 0 ? (bits == 32 ? a.m.codes[my_r] + 4 * (size_t)my_j : a.m.codes[my_r] + (bit0 >> 3)) : nullptr;
  const float* p_scale = my_r >= 0 ? a.m.scales[my_r] : nullptr;
  const uint32_t cshift = bit0 & 7u, cmask = bits == 32 ? 0xFFFFFFFFu : (1u << bits) - 1u;
  const bool pow2 = (R & (R - 1)) == 0;
  const float Rf = (float)R, invR = 1.0f / Rf, nlr = -a.outer_lr;
  bool bad = false;
  for (int i = tid; i < kAC / 32; i += GT) sm.seen[i] = 0;
  group_sync();

  struct Raw { uint32_t pos, code; float scale; };
  auto fetch = [&](uint32_t g) {
    Raw w{0xFFFFu, 0u, 0.0f};
    if (my_r >= 0 && SL_CHECK(a.flags, g < a.tb.n_chunks)) {
      w.pos = __ldg(p_idx + (uint64_t)g * (uint64_t)k);
      if (bits == 32) {
        w.code = __float_as_uint(__ldg(reinterpret_cast<const float*>(p_code + (uint64_t)g * (uint64_t)a.stride)));
      } else {
        w.code = (uint32_t)__ldg(p_code + (uint64_t)g * (uint64_t)a.stride);
        w.scale = __ldg(p_scale + g);
      }
    }
    return w;
  };
  // decoded entry of a chunk: position (0xFFFF: none), value, and the element of theta_global it names
  // (eoff: the element's offset from the chunk's first element - the position itself in a consecutive
  // chunk, row p / 64 and column p % 64 of a tile whose rows are `stride` elements apart; the one formula
  // serves both, since a consecutive chunk is reported with stride 64)
  struct Dec { uint32_t pos; float val, th; uint64_t eoff; };
  auto decode = [&](const Raw& w, uint64_t base, uint32_t stride) {
    Dec d{0xFFFFu, 0.0f, 0.0f, 0};
    if (my_r < 0 || w.pos == 0xFFFFu) return d;
    if (w.pos >= (uint32_t)kAC) { bad = true; return d; }
    const uint64_t eoff = (uint64_t)(w.pos >> 6) * stride + (w.pos & 63u);
    if (!SL_CHECK(a.flags, base + eoff < n_total)) return d;
    d.pos = w.pos;
    d.eoff = eoff;
    d.val = bits == 32 ? __uint_as_float(w.code) : dequant((w.code >> cshift) & cmask, w.scale, bits);
    d.th = __ldcg(a.out + base + eoff);
    return d;
  };
  // The group's chunks in flight, oldest first: stage 0 is processed in this iteration, stages 1..kDec hold
  // decoded entries whose theta_global elements are on their way, the last kRaw stages raw entries on their way.
  constexpr int kDec = 1, kRaw = 1, kStagesInFlight = 1 + kDec + kRaw;
  uint64_t base_q[kStagesInFlight];
  uint32_t stride_q[kStagesInFlight];
  bool valid_q[kStagesInFlight];
  Dec dec_q[1 + kDec];
  Raw raw_q[kRaw];
  uint32_t g_next = vcta, t_lo = 0;
  bool more = true;
#pragma unroll
  for (int i = 0; i < kStagesInFlight; ++i) {
    base_q[i] = 0;
    stride_q[i] = 64;
    valid_q[i] = more && next_full_chunk(a.tb, g_next, vgrid, t_lo, base_q[i], stride_q[i]);
    more = valid_q[i];
    if (i <= kDec) {
      dec_q[i] = Dec{0xFFFFu, 0.0f, 0.0f, 0};
      if (valid_q[i]) dec_q[i] = decode(fetch(g_next), base_q[i], stride_q[i]);
    } else {
      raw_q[i - 1 - kDec] = Raw{0xFFFFu, 0u, 0.0f};
      if (valid_q[i]) raw_q[i - 1 - kDec] = fetch(g_next);
    }
    if (valid_q[i]) g_next += vgrid;
  }
  while (valid_q[0]) {
    // ---- the oldest chunk ----
    const uint32_t posA = dec_q[0].pos;
    const bool have = posA != 0xFFFFu;
    const uint32_t word = posA >> 5, bit = 1u << (posA & 31u);
    if (have) sm.acc[posA] = 0.0f;
    group_sync();
    bool first = false;
    for (int r = 0; r < R; ++r) {
      if (have && my_r == r) {
        first = (atomicOr(&sm.seen[word], bit) & bit) == 0;
        sm.acc[posA] = __fadd_rn(sm.acc[posA], dec_q[0].val);
      }
      group_sync();
    }
    if (have && first) {
      const float sum = sm.acc[posA];
      const float u = pow2 ? __fmul_rn(sum, invR) : __fdiv_rn(sum, Rf);
      a.out[base_q[0] + dec_q[0].eoff] = __fmaf_rn(nlr, u, dec_q[0].th);
      atomicAnd(&sm.seen[word], ~bit);
    }
    group_sync();                                  // cells and bits are free for the next chunk
    // ---- shift: the oldest raw stage is decoded (its theta_global elements are requested), a new chunk is fetched ----
#pragma unroll
    for (int i = 0; i < kDec; ++i) dec_q[i] = dec_q[i + 1];
#pragma unroll
    for (int i = 0; i + 1 < kStagesInFlight; ++i) { base_q[i] = base_q[i + 1]; stride_q[i] = stride_q[i + 1]; valid_q[i] = valid_q[i + 1]; }
    dec_q[kDec] = Dec{0xFFFFu, 0.0f, 0.0f, 0};
    if (valid_q[kDec]) dec_q[kDec] = decode(raw_q[0], base_q[kDec], stride_q[kDec]);
#pragma unroll
    for (int i = 0; i + 1 < kRaw; ++i) raw_q[i] = raw_q[i + 1];
    valid_q[kStagesInFlight - 1] = more && next_full_chunk(a.tb, g_next, vgrid, t_lo, base_q[kStagesInFlight - 1], stride_q[kStagesInFlight - 1]);
    more = valid_q[kStagesInFlight - 1];
    if (more) { raw_q[kRaw - 1] = fetch(g_next); g_next += vgrid; }
  }
  if (bad && a.flags) atomicOr(a.flags, (uint32_t)SL_FLAG_BAD_INDEX);
}

template <int T, bool APPLY>
cudaError_t launch_aggregate_c4096(const AggregateArgs<T>& a, cudaStream_t st) {
  cudaError_t e;
  const int sms = sm_count(&e);
  if (e != cudaSuccess) return e;
  const int pairs = (a.R * a.k + kThreads - 1) / kThreads;
  const size_t smem = APPLY ? sizeof(AggSmem) : sizeof(float) * kAC;
  // persistent grid: exactly as many CTAs as are resident at once, so that every CTA walks the
  // same number of chunks
  auto launch = [&](auto kernel) -> cudaError_t {
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    int per_sm = 0;
    err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, smem);
    if (err != cudaSuccess) return err;
    if (per_sm < 1) per_sm = 1;
    const unsigned grid = (unsigned)std::min<uint64_t>((uint64_t)a.tb.n_chunks, (uint64_t)sms * (uint64_t)per_sm);
    kernel<<<grid, kThreads, smem, st>>>(a);
    return cudaPeekAtLastError();
  };
  const int np = pairs <= 1 ? 1 : pairs <= 2 ? 2 : pairs <= 4 ? 4 : 8;
  const bool grouped = np > 1 && a.k % np == 0;     // (with one pair per thread the two mappings coincide)
  if constexpr (APPLY) {
    if (!a.theta_bf16 && (a.tb.side == 0 || a.tb.side == 64) && a.outer_lr > 0.0f && a.R * a.k <= kSparseMaxEntries) {
      auto launch_sparse = [&](auto kernel, int groups) -> cudaError_t {
        const size_t sm_bytes = sizeof(SparseSmem) * (size_t)groups;
        cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_bytes);
        if (err != cudaSuccess) return err;
        int per_sm = 0;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, sm_bytes);
        if (err != cudaSuccess) return err;
        if (per_sm < 1) per_sm = 1;
        const uint64_t want = ((uint64_t)a.tb.n_chunks + groups - 1) / groups;
        const unsigned grid = (unsigned)std::min<uint64_t>(want, (uint64_t)sms * (uint64_t)per_sm);
        kernel<<<grid, kThreads, sm_bytes, st>>>(a);
        return cudaPeekAtLastError();
      };
      const int entries = a.R * a.k;
      if (entries <= 64) return launch_sparse(aggregate_sparse_kernel<T, 4>, 4);
      if (entries <= 128) return launch_sparse(aggregate_sparse_kernel<T, 2>, 2);
      return launch_sparse(aggregate_sparse_kernel<T, 1>, 1);
    }
  }
  if (a.tb.side != 0) {
    if (np == 1) return launch(aggregate_c4096_kernel<T, APPLY, 1, true, false>);
    if (np == 2) return grouped ? launch(aggregate_c4096_kernel<T, APPLY, 2, true, true>)
                                : launch(aggregate_c4096_kernel<T, APPLY, 2, true, false>);
    if (np == 4) return grouped ? launch(aggregate_c4096_kernel<T, APPLY, 4, true, true>)
                                : launch(aggregate_c4096_kernel<T, APPLY, 4, true, false>);
    return grouped ? launch(aggregate_c4096_kernel<T, APPLY, 8, true, true>)
                   : launch(aggregate_c4096_kernel<T, APPLY, 8, true, false>);
  }
  if constexpr (APPLY) {
    if (a.theta_bf16) {
      if (np == 1) return launch(aggregate_c4096_kernel<T, true, 1, false, false, true>);
      if (np == 2) return grouped ? launch(aggregate_c4096_kernel<T, true, 2, false, true, true>)
                                  : launch(aggregate_c4096_kernel<T, true, 2, false, false, true>);
      if (np == 4) return grouped ? launch(aggregate_c4096_kernel<T, true, 4, false, true, true>)
                                  : launch(aggregate_c4096_kernel<T, true, 4, false, false, true>);
      return grouped ? launch(aggregate_c4096_kernel<T, true, 8, false, true, true>)
                     : launch(aggregate_c4096_kernel<T, true, 8, false, false, true>);
    }
  }
  if (np == 1) return launch(aggregate_c4096_kernel<T, APPLY, 1, false, false>);
  if (np == 2) return grouped ? launch(aggregate_c4096_kernel<T, APPLY, 2, false, true>)
                              : launch(aggregate_c4096_kernel<T, APPLY, 2, false, false>);
  if (np == 4) return grouped ? launch(aggregate_c4096_kernel<T, APPLY, 4, false, true>)
                              : launch(aggregate_c4096_kernel<T, APPLY, 4, false, false>);
  return grouped ? launch(aggregate_c4096_kernel<T, APPLY, 8, false, true>)
                 : launch(aggregate_c4096_kernel<T, APPLY, 8, false, false>);
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

__global__ void __launch_bounds__(256)
outer_apply_bf16_kernel(uint16_t* __restrict__ theta, const float* __restrict__ update, uint64_t n, float lr) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  const float nlr = -lr;
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
    theta[i] = (uint16_t)bf16_round(__fmaf_rn(nlr, update[i], bf16_widen(theta[i])));
}

}  // namespace

template <int T>
cudaError_t launch_aggregate(const AggregateArgs<T>& a, bool apply, bool aligned16, cudaStream_t st) {
  if (a.tb.n_chunks == 0) return cudaSuccess;
  const size_t smem = (size_t)a.chunk * 4;
  bool tuned = aligned16 && a.chunk == kAC && a.R * a.k <= kThreads * 8;
  if (tuned && apply && a.theta_bf16) {          // bfloat16 parameters: consecutive chunks starting on 16 bytes
    tuned = a.tb.side == 0;
    for (uint32_t t = 0; tuned && t <= a.tb.n_tensors; ++t) tuned = a.tb.offset[t] % 8 == 0;
  }
  if (tuned) {
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
  if (a.tb.n_tails == 0) return cudaSuccess;
  const size_t smem = (size_t)a.chunk * 4;
  if (apply) aggregate_generic_kernel<T, true, true><<<a.tb.n_tails, kThreads, smem, st>>>(a);
  else aggregate_generic_kernel<T, false, true><<<a.tb.n_tails, kThreads, smem, st>>>(a);
  return cudaPeekAtLastError();
}

template cudaError_t launch_aggregate_tails<256>(const AggregateArgs<256>&, bool, cudaStream_t);
template cudaError_t launch_aggregate_tails<SL_MAX_TENSORS>(const AggregateArgs<SL_MAX_TENSORS>&, bool, cudaStream_t);
template cudaError_t launch_aggregate<256>(const AggregateArgs<256>&, bool, bool, cudaStream_t);
template cudaError_t launch_aggregate<SL_MAX_TENSORS>(const AggregateArgs<SL_MAX_TENSORS>&, bool, bool, cudaStream_t);

cudaError_t launch_outer_apply_bf16(uint16_t* theta, const float* update, uint64_t n, float lr, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  cudaError_t e;
  const uint64_t cap = (uint64_t)sm_count(&e) * 8ull;
  if (e != cudaSuccess) return e;
  const uint64_t blocks = (n + 255) / 256;
  outer_apply_bf16_kernel<<<(unsigned)(blocks < cap ? blocks : cap), 256, 0, st>>>(theta, update, n, lr);
  return cudaPeekAtLastError();
}

cudaError_t launch_outer_apply(float* theta, const float* update, uint64_t n, float lr, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  const int vec = (((uintptr_t)theta | (uintptr_t)update) & 15u) == 0;
  const uint64_t work = vec ? (n + 3) / 4 : n;
  uint64_t blocks = (work + 255) / 256;
  cudaError_t e;
  const int sms = sm_count(&e);
  if (e != cudaSuccess) return e;
  const uint64_t cap = (uint64_t)sms * 8ull;  // grid-stride over one full wave: 8 CTAs of 256 threads per SM
  if (blocks > cap) blocks = cap;
  outer_apply_kernel<<<(unsigned)blocks, 256, 0, st>>>(theta, update, n, lr, vec);
  return cudaPeekAtLastError();
}

}  // namespace sl
