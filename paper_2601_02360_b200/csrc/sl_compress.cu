// Eq. 2 lines 1-4 (paper §2.1): pseudo-gradient, error feedback, chunk-wise Top-k,
// quantisation, residual.
//
// Two kernels with identical results:
//   compress_generic_kernel  any chunk length / k / code width / alignment; one CTA per
//                            (chunk, replica); exact 4-pass radix select in shared memory.
//   compress_c4096_kernel    the tuned path for full 4096-element chunks, k <= 128: one CTA per
//                            chunk walks all R replicas with theta_global held in registers, a
//                            cheap lower bound on the k-th magnitude prunes the chunk to a few
//                            hundred candidates, one warp finishes the exact selection.
#include "sl_common.cuh"

namespace sl {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr uint32_t kFull = 0xFFFFFFFFu;

__device__ __forceinline__ uint32_t lanemask_lt() {
  uint32_t m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}

// scratch of the block-wide exact selection (shared by both kernels)
struct SelectScratch {
  uint32_t hist[256];
  uint32_t weq[kWarps], wgt[kWarps];
  uint32_t digit, need;
};

// ---------------------------------------------------------------------------
// Block-wide exact selection + emission on a chunk whose e' sits in shared memory.
//   * k_eff-th largest 31-bit magnitude key by a 4-pass radix select (8+8+8+7 bits);
//   * kept set = keys above it plus the lowest-positioned ties, emitted in ascending
//     position with warp ballots (each warp walks one contiguous region, regions are
//     stitched by prefix counts);
//   * codes OR-ed into `cw` (zeroed by the caller), residual patched into `ep`.
// All threads of the CTA must call it; it ends with a barrier.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void block_select_emit(float* ep, int len, int k_eff, int bits, float s,
                                                  SelectScratch& sc, uint32_t* cw,
                                                  uint16_t* __restrict__ oidx, uint8_t* __restrict__ ocodes) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t prefix = 0, need = (uint32_t)k_eff;
#pragma unroll 1
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = pass == 0 ? 23 : pass == 1 ? 15 : pass == 2 ? 7 : 0;
    const int width = pass == 3 ? 7 : 8;
    const int hs = shift + width;                 // bits above this digit are already fixed
    sc.hist[tid] = 0;
    __syncthreads();
    for (int i = tid; i < len; i += kThreads) {
      const uint32_t key = key_of(ep[i]);
      if ((key >> hs) == (prefix >> hs)) atomicAdd(&sc.hist[(key >> shift) & ((1u << width) - 1u)], 1u);
    }
    __syncthreads();
    if (warp == 0) {
      uint32_t h[8], mine = 0;
#pragma unroll
      for (int b = 0; b < 8; ++b) { h[b] = sc.hist[lane * 8 + b]; mine += h[b]; }
      uint32_t suf = mine;                        // inclusive suffix sum over lanes >= lane
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t o = __shfl_down_sync(kFull, suf, d);
        if (lane + d < 32) suf += o;
      }
      const uint32_t vote = __ballot_sync(kFull, suf >= need);
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
        sc.digit = digit;
        sc.need = left;
      }
    }
    __syncthreads();
    prefix |= sc.digit << shift;
    need = sc.need;
  }
  const uint32_t kth = prefix;                    // the k_eff-th largest key; `need` ties of it are kept

  const int rw = ((len + kThreads - 1) / kThreads) * 32;   // region per warp, multiple of 32
  const int r0 = warp * rw;
  const int r1 = min(len, r0 + rw);
  uint32_t ceq = 0, cgt = 0;
  for (int i0 = r0; i0 < r1; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t key = i < r1 ? key_of(ep[i]) : 0u;
    ceq += __popc(__ballot_sync(kFull, i < r1 && key == kth));
    cgt += __popc(__ballot_sync(kFull, i < r1 && key > kth));
  }
  if (lane == 0) { sc.weq[warp] = ceq; sc.wgt[warp] = cgt; }
  __syncthreads();
  uint32_t eq_base = 0, out_base = 0;
  for (int w = 0; w < warp; ++w) {
    const uint32_t weq = sc.weq[w];
    const uint32_t room = need > eq_base ? need - eq_base : 0u;
    out_base += sc.wgt[w] + min(room, weq);
    eq_base += weq;
  }
  for (int i0 = r0; i0 < r1; i0 += 32) {
    const int i = i0 + lane;
    const bool in = i < r1;
    const float v = in ? ep[i] : 0.0f;
    const uint32_t key = key_of(v);
    const bool eq = in && key == kth;
    const uint32_t eqm = __ballot_sync(kFull, eq);
    const bool keep = in && (key > kth || (eq && eq_base + __popc(eqm & lanemask_lt()) < need));
    const uint32_t km = __ballot_sync(kFull, keep);
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
}

// ---------------------------------------------------------------------------
// Generic kernel.  TAILS = false: CTA b handles chunk b / R of replica b % R.
// TAILS = true: CTA b handles the short last chunk of tensor b / R (if it has one); this is
// how the tuned path delegates the ragged ends of the tensors.
// ---------------------------------------------------------------------------
template <int T, bool TAILS>
__global__ void __launch_bounds__(kThreads)
compress_generic_kernel(const __grid_constant__ CompressArgs<T> a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* ep = reinterpret_cast<float*>(smem_raw);                          // [chunk]
  uint32_t* cw = reinterpret_cast<uint32_t*>(ep + a.chunk);                // [ceil(stride/4)] packed codes
  __shared__ SelectScratch sc;
  __shared__ uint32_t s_wmax[kWarps];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r = (int)(blockIdx.x % (uint32_t)a.R);
  uint32_t g = blockIdx.x / (uint32_t)a.R;
  if (TAILS) {
    const uint32_t t = g;
    const uint64_t n_t = a.tb.offset[t + 1] - a.tb.offset[t];
    if (n_t % (uint64_t)a.chunk == 0) return;     // no short chunk in this tensor
    g = a.tb.first_chunk[t + 1] - 1;
  }
  const ChunkRef c = locate(a.tb, g, a.chunk);
  const int len = c.len;
  const int k = a.k, bits = a.bits;
  const int k_eff = k < len ? k : len;

  const float* __restrict__ tl = a.p.theta_local[r] + c.base;
  const float* __restrict__ tg = a.theta_global + c.base;
  float* __restrict__ er = a.p.err[r] + c.base;

  // pseudo-gradient and error feedback
  uint32_t tmax = 0;
  for (int i = tid; i < len; i += kThreads) {
    const float d = __fsub_rn(tg[i], tl[i]);
    const float e = __fmaf_rn(a.beta, er[i], d);
    ep[i] = e;
    tmax = max(tmax, key_of(e));
  }
  tmax = __reduce_max_sync(kFull, tmax);
  if (lane == 0) s_wmax[warp] = tmax;
  const uint32_t cwords = (a.stride + 3) >> 2;
  if (bits != 32)
    for (uint32_t i = tid; i < cwords; i += kThreads) cw[i] = 0;
  __syncthreads();
  uint32_t smax = 0;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) smax = max(smax, s_wmax[w]);
  const float s = __uint_as_float(smax);

  uint16_t* __restrict__ oidx = a.p.idx[r] + (uint64_t)g * (uint64_t)k;
  uint8_t* __restrict__ ocodes = a.p.codes[r] + (uint64_t)g * (uint64_t)a.stride;
  block_select_emit(ep, len, k_eff, bits, s, sc, cw, oidx, ocodes);

  // write-back
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

// ---------------------------------------------------------------------------
// Tuned kernel: chunk = 4096, k <= 128, (k * bits) % 32 == 0, 16-byte aligned arena.
//
// One CTA per chunk walks all R replicas; theta_global stays in registers.  The CTA is warp
// specialised: 8 producer warps (256 threads) and kSel selector warps; selector q handles the
// replicas r with r % kSel == q, so two selections are in flight while the producers run ahead.
//
//  * theta_local and e of replica r arrive by TMA bulk copies (cp.async.bulk + mbarrier):
//    theta_local in a 2-deep ring (dead after phase A, refilled by producer thread 0), e in a
//    4-deep ring (alive until its bulk store has read it, refilled by the selector that owns it).
//  * Producers, per replica (thread t owns float4s t, t+256, t+512, t+768 of the chunk):
//      A  e' = fma(beta, e, theta_global - theta_local), written in place of e in the stage;
//         per-thread maximum key.  The chunk is cut into kp >= k groups of whole threads
//         (kp a power of two); at least k keys are >= the smallest group maximum T1, so T1 is
//         a lower bound of the k-th largest key.
//      B  the keys >= T1 (a few hundred) are compacted into a candidate list.
//  * Selector, per replica:
//      C  bisects the key range [T1, max] for a threshold that leaves exactly k candidates;
//         if the range collapses first the k-th key is tied, and the lowest positions among
//         its ties are found by a second bisection over positions.
//      D  marks the kept positions in a 4096-bit map, walks it in ascending position (each
//         lane owns 128 positions, slots from a prefix sum of popcounts), writes idx and
//         codes, patches the residual into the stage.
//      E  one TMA bulk store sends the stage's 16 KB of e' to the error buffer; when the
//         store has read the stage, e of replica r+4 is loaded into it.
//  If the candidate list overflows (tie-heavy or constant chunks) the selector runs an exact
//  warp-wide radix select over the whole chunk instead of C.
//
// Hand-offs: named barrier 1 = producers only; 2+q = candidate list q ready (producers
// arrive, selector q waits); 4+q = candidate list q free again (selector q arrives, producers
// wait).  Every mbarrier wait is bounded; running out raises SL_FLAG_TIMEOUT and the kernel
// carries on (no trap, no hang).
// ---------------------------------------------------------------------------
constexpr int kC = 4096;
constexpr int kSel = 2;               // selector warps
constexpr int kTlStages = 2;
constexpr int kEeStages = 4;
constexpr int kCandMax = 1024;
constexpr int kCandReg = 12;          // candidates per lane held in registers (C <= 384)
constexpr int kMaxCodeWords = 32;     // k * bits / 32 <= 128 * 8 / 32
constexpr int kFastThreads = kThreads + 32 * kSel;
constexpr int kPairThreads = kThreads + 32;   // producers + one selector
constexpr uint32_t kWaitLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// bounded wait on a phase; false = gave up
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  const uint32_t addr = smem_u32(bar);
  for (uint32_t it = 0; it < kWaitLimit; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
    if (ok) return true;
  }
  return false;
}
__device__ __forceinline__ void tma_load_1d(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tma_store_1d(void* dst, const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
               ::"l"(dst), "r"(smem_u32(src)), "r"(bytes) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void named_sync(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }
__device__ __forceinline__ void named_arrive(int id, int n) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(n) : "memory"); }

struct alignas(16) FastSmem {
  float tl[kTlStages][kC];            // theta_local of replica r in stage r % 2
  float ee[kEeStages][kC];            // e of replica r in stage r % 4, then e' in place, then the store's source
  uint32_t cand_key[kSel][kCandMax];
  uint16_t cand_pos[kSel][kCandMax];
  uint32_t bitmap[kSel][kC / 32];
  uint32_t hist[kSel][256];
  uint32_t cw[kSel][kMaxCodeWords];
  uint32_t wmin[kEeStages][kWarps], wmax[kEeStages][kWarps];   // ring: producers run up to three replicas ahead
  uint32_t count[kSel];
  uint64_t full_tl[kTlStages];
  uint64_t full_ee[kEeStages];
};

// number of candidate keys >= mid; keys either in registers (NREG > 0) or in shared memory
template <int NREG>
__device__ __forceinline__ uint32_t count_ge(const uint32_t* ck_reg, const uint32_t* ck_smem, uint32_t C,
                                             uint32_t mid, int lane) {
  uint32_t cnt = 0;
  if (NREG > 0) {
#pragma unroll
    for (int i = 0; i < NREG; ++i) cnt += ck_reg[i] >= mid ? 1u : 0u;
  } else {
    for (uint32_t i = lane; i < C; i += 32) cnt += ck_smem[i] >= mid ? 1u : 0u;
  }
  return __reduce_add_sync(kFull, cnt);
}

// Phase C + marking: threshold among C candidates, kept positions OR-ed into the bitmap.
template <int NREG>
__device__ __forceinline__ void select_candidates(const uint32_t* cand_key, const uint16_t* cand_pos, uint32_t C,
                                                  uint32_t k, uint32_t T1, uint32_t smax, uint32_t* bitmap,
                                                  int lane, uint32_t* stats) {
  uint32_t ck[NREG > 0 ? NREG : 1];
  if (NREG > 0) {
#pragma unroll
    for (int i = 0; i < NREG; ++i) {
      const uint32_t at = (uint32_t)lane + 32u * (uint32_t)i;
      ck[i] = at < C ? cand_key[at] : 0u;          // padding 0 is below every probe (probes are > T1 >= 0)
    }
  }
  uint32_t lo = T1, hi = smax + 1u, cnt_hi = 0;
  uint32_t thr_ge = T1;                            // keep key >= thr_ge ...
  uint32_t thr_eq = 0xFFFFFFFFu, pos_le = 0;       // ... and key == thr_eq at position <= pos_le
  if (C != k) {
    bool exact = false;
    while (hi - lo > 1u) {
      const uint32_t mid = lo + ((hi - lo) >> 1);
      const uint32_t cnt = count_ge<NREG>(ck, cand_key, C, mid, lane);
#ifdef SL_STATS
      if (lane == 0) atomicAdd(&stats[1], 1u);
#endif
      if (cnt == k) { thr_ge = mid; exact = true; break; }
      if (cnt > k) lo = mid; else { hi = mid; cnt_hi = cnt; }
    }
    if (!exact) {
      // the k-th key is `lo` and it is tied: keep every key above it and the (k - cnt_hi)
      // lowest positions among the ties
      thr_ge = lo + 1u;
      thr_eq = lo;
      const uint32_t need = k - cnt_hi;
      uint32_t plo = 0, phi = kC - 1;              // smallest P with #(ties at position <= P) >= need
      while (plo < phi) {
        const uint32_t pm = (plo + phi) >> 1;
        uint32_t cnt = 0;
        for (uint32_t i = lane; i < C; i += 32)
          cnt += (cand_key[i] == thr_eq && (uint32_t)cand_pos[i] <= pm) ? 1u : 0u;
        cnt = __reduce_add_sync(kFull, cnt);
        if (cnt >= need) phi = pm; else plo = pm + 1;
      }
      pos_le = plo;
#ifdef SL_STATS
      if (lane == 0) atomicAdd(&stats[2], 1u);
#endif
    }
  }
  if (NREG > 0) {
#pragma unroll
    for (int i = 0; i < NREG; ++i) {
      const uint32_t at = (uint32_t)lane + 32u * (uint32_t)i;
      if (at < C) {
        const uint32_t cp = cand_pos[at];
        if (ck[i] >= thr_ge || (ck[i] == thr_eq && cp <= pos_le)) atomicOr(&bitmap[cp >> 5], 1u << (cp & 31u));
      }
    }
  } else {
    for (uint32_t i = lane; i < C; i += 32) {
      const uint32_t k_i = cand_key[i];
      const uint32_t cp = cand_pos[i];
      if (k_i >= thr_ge || (k_i == thr_eq && cp <= pos_le)) atomicOr(&bitmap[cp >> 5], 1u << (cp & 31u));
    }
  }
}

// Overflow path of the selector: exact radix select over the whole chunk by one warp, kept
// positions written to the bitmap (one ballot = one bitmap word).
__device__ __forceinline__ void warp_select_full(const float* ep, uint32_t k, uint32_t* hist, uint32_t* bitmap,
                                                 int lane) {
  uint32_t prefix = 0, need = k;
#pragma unroll 1
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = pass == 0 ? 23 : pass == 1 ? 15 : pass == 2 ? 7 : 0;
    const int width = pass == 3 ? 7 : 8;
    const int hs = shift + width;
#pragma unroll
    for (int b = 0; b < 8; ++b) hist[lane * 8 + b] = 0;
    __syncwarp();
    for (int i = lane; i < kC; i += 32) {
      const uint32_t key = key_of(ep[i]);
      if ((key >> hs) == (prefix >> hs)) atomicAdd(&hist[(key >> shift) & ((1u << width) - 1u)], 1u);
    }
    __syncwarp();
    uint32_t h[8], mine = 0;
#pragma unroll
    for (int b = 0; b < 8; ++b) { h[b] = hist[lane * 8 + b]; mine += h[b]; }
    uint32_t suf = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t o = __shfl_down_sync(kFull, suf, d);
      if (lane + d < 32) suf += o;
    }
    const uint32_t vote = __ballot_sync(kFull, suf >= need);
    const int sel = 31 - __clz(vote);
    uint32_t cum = suf - mine, digit = (uint32_t)lane * 8u, left = need;
    bool found = false;
#pragma unroll
    for (int bb = 7; bb >= 0; --bb) {
      if (!found) {
        if (cum + h[bb] >= need) { found = true; digit = (uint32_t)(lane * 8 + bb); left = need - cum; }
        else cum += h[bb];
      }
    }
    digit = __shfl_sync(kFull, digit, sel);
    need = __shfl_sync(kFull, left, sel);
    prefix |= digit << shift;
    __syncwarp();
  }
  const uint32_t kth = prefix;
  uint32_t eq_seen = 0;
  for (int w = 0; w < kC / 32; ++w) {
    const uint32_t key = key_of(ep[w * 32 + lane]);
    const bool eq = key == kth;
    const uint32_t eqm = __ballot_sync(kFull, eq);
    const bool keep = key > kth || (eq && eq_seen + __popc(eqm & lanemask_lt()) < need);
    const uint32_t km = __ballot_sync(kFull, keep);
    if (lane == 0) bitmap[w] = km;
    eq_seen += __popc(eqm);
  }
}

template <int T>
__global__ void __launch_bounds__(kFastThreads, 2)
compress_c4096_kernel(const __grid_constant__ CompressArgs<T> a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  FastSmem& sm = *reinterpret_cast<FastSmem*>(smem_raw);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t g = blockIdx.x;
  const ChunkRef c = locate(a.tb, g, kC);
  if (c.len != kC) return;                        // short chunks go to the generic tail launch
  const int k = a.k, bits = a.bits, R = a.R;
  constexpr uint32_t kBytes = kC * 4;

  for (int i = tid; i < kSel * (kC / 32); i += kFastThreads) (&sm.bitmap[0][0])[i] = 0;
  if (tid < kSel * kMaxCodeWords) (&sm.cw[0][0])[tid] = 0;
  if (tid == 0) {
#pragma unroll
    for (int q = 0; q < kSel; ++q) sm.count[q] = 0;
#pragma unroll
    for (int s = 0; s < kTlStages; ++s) mbar_init(&sm.full_tl[s], 1);
#pragma unroll
    for (int s = 0; s < kEeStages; ++s) mbar_init(&sm.full_ee[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  __syncthreads();
  bool timed_out = false;

  if (warp < kWarps) {
    // ======================= producers =======================================
    if (tid == 0) {
      for (int r = 0; r < kTlStages && r < R; ++r) {
        mbar_expect_tx(&sm.full_tl[r], kBytes);
        tma_load_1d(sm.tl[r], a.p.theta_local[r] + c.base, kBytes, &sm.full_tl[r]);
      }
    }
    int kp = 8;                                   // kp = max(8, pow2ceil(k)) groups of 256/kp threads
    while (kp < k) kp <<= 1;
    const int group_lanes = kThreads / kp;        // 32, 16, 8, 4 or 2 lanes
    const float beta = a.beta;
    const float4* __restrict__ tg4 = reinterpret_cast<const float4*>(a.theta_global + c.base);
    float4 G[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) G[j] = __ldcs(tg4 + tid + 256 * j);
    __syncwarp();

#pragma unroll 1
    for (int r = 0; r < R; ++r) {
      const int st = r % kTlStages, se = r % kEeStages, q = r % kSel;
      if (!mbar_wait(&sm.full_tl[st], (uint32_t)((r / kTlStages) & 1))) timed_out = true;
      if (!mbar_wait(&sm.full_ee[se], (uint32_t)((r / kEeStages) & 1))) timed_out = true;
      const float4* tl4 = reinterpret_cast<const float4*>(sm.tl[st]);
      float4* ee4 = reinterpret_cast<float4*>(sm.ee[se]);
      // ---- A ----
      uint32_t key[16];
      uint32_t tmax = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float4 L = tl4[tid + 256 * j];
        const float4 E = ee4[tid + 256 * j];
        float4 v;
        v.x = __fmaf_rn(beta, E.x, __fsub_rn(G[j].x, L.x));
        v.y = __fmaf_rn(beta, E.y, __fsub_rn(G[j].y, L.y));
        v.z = __fmaf_rn(beta, E.z, __fsub_rn(G[j].z, L.z));
        v.w = __fmaf_rn(beta, E.w, __fsub_rn(G[j].w, L.w));
        ee4[tid + 256 * j] = v;
        key[4 * j + 0] = key_of(v.x);
        key[4 * j + 1] = key_of(v.y);
        key[4 * j + 2] = key_of(v.z);
        key[4 * j + 3] = key_of(v.w);
        tmax = max(tmax, max(max(key[4 * j], key[4 * j + 1]), max(key[4 * j + 2], key[4 * j + 3])));
      }
      fence_async_smem();                         // e' must be visible to the later bulk store
      uint32_t gmax = tmax;
      for (int d = 1; d < group_lanes; d <<= 1) gmax = max(gmax, __shfl_xor_sync(kFull, gmax, d));
      const uint32_t wmin = __reduce_min_sync(kFull, gmax);
      const uint32_t wmax = __reduce_max_sync(kFull, tmax);
      if (lane == 0) { sm.wmin[se][warp] = wmin; sm.wmax[se][warp] = wmax; }
      named_sync(1, kThreads);
      if (tid == 0 && r + kTlStages < R) {        // every producer has read theta_local(r): refill its stage
        mbar_expect_tx(&sm.full_tl[st], kBytes);
        tma_load_1d(sm.tl[st], a.p.theta_local[r + kTlStages] + c.base, kBytes, &sm.full_tl[st]);
      }
      uint32_t T1 = 0xFFFFFFFFu;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) T1 = min(T1, sm.wmin[se][w]);
      // ---- B ----
      __syncwarp();
      if (r >= kSel) named_sync(4 + q, kPairThreads);   // selector q is done with its candidate list
      uint32_t mask = 0;
#pragma unroll
      for (int e = 0; e < 16; ++e) mask |= (key[e] >= T1 ? 1u : 0u) << e;
      const uint32_t cnt = __popc(mask);
      uint32_t incl = cnt;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t o = __shfl_up_sync(kFull, incl, d);
        if (lane >= d) incl += o;
      }
      uint32_t base = 0;
      if (lane == 31) base = atomicAdd(&sm.count[q], incl);
      base = __shfl_sync(kFull, base, 31);
      uint32_t at = base + incl - cnt;
      const float* ep = sm.ee[se];
      while (mask) {
        const int b = __ffs(mask) - 1;
        mask &= mask - 1;
        const int pos = ((b >> 2) << 10) + (tid << 2) + (b & 3);
        if (at < (uint32_t)kCandMax) {
          sm.cand_key[q][at] = key_of(ep[pos]);
          sm.cand_pos[q][at] = (uint16_t)pos;
        }
        ++at;
      }
      __syncwarp();                               // bar.* is warp-aligned: reconverge first
      __threadfence_block();
      named_arrive(2 + q, kPairThreads);          // candidate list q is ready
    }
  } else {
    // ======================= selectors =======================================
    const int q = warp - kWarps;
    if (lane == 0) {
      for (int r = q; r < kEeStages && r < R; r += kSel) {
        mbar_expect_tx(&sm.full_ee[r], kBytes);
        tma_load_1d(sm.ee[r], a.p.err[r] + c.base, kBytes, &sm.full_ee[r]);
      }
    }
    __syncwarp();
    const int cwords = (k * bits) >> 5;
    uint32_t* bitmap = sm.bitmap[q];
    uint32_t* cw = sm.cw[q];
#pragma unroll 1
    for (int r = q; r < R; r += kSel) {
      const int se = r % kEeStages;
      float* ep = sm.ee[se];
      named_sync(2 + q, kPairThreads);            // candidate list q is ready
      const uint32_t C = sm.count[q];
      uint32_t T1 = 0xFFFFFFFFu, smax = 0;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) { T1 = min(T1, sm.wmin[se][w]); smax = max(smax, sm.wmax[se][w]); }
      const float sc = __uint_as_float(smax);
      uint16_t* __restrict__ oidx = a.p.idx[r] + (uint64_t)g * (uint64_t)k;
      uint8_t* __restrict__ ocodes = a.p.codes[r] + (uint64_t)g * (uint64_t)a.stride;
#ifdef SL_STATS
      if (lane == 0) { atomicAdd(&a.flags[4], C); atomicAdd(&a.flags[7], 1u); if (C > kCandMax) atomicAdd(&a.flags[8], 1u); }
#endif
      // ---- C ----
      if (C > (uint32_t)kCandMax) warp_select_full(ep, (uint32_t)k, sm.hist[q], bitmap, lane);
      else if (C <= 32u * kCandReg)
        select_candidates<kCandReg>(sm.cand_key[q], sm.cand_pos[q], C, (uint32_t)k, T1, smax, bitmap, lane, a.flags + 4);
      else
        select_candidates<0>(sm.cand_key[q], sm.cand_pos[q], C, (uint32_t)k, T1, smax, bitmap, lane, a.flags + 4);
      __syncwarp();
      if (lane == 0) sm.count[q] = 0;
      __threadfence_block();
      __syncwarp();
      if (r + kSel < R) named_arrive(4 + q, kPairThreads);   // candidate list q may be refilled
      // ---- D ----
      uint4 bm = reinterpret_cast<uint4*>(bitmap)[lane];
      const uint32_t mine = __popc(bm.x) + __popc(bm.y) + __popc(bm.z) + __popc(bm.w);
      uint32_t incl = mine;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t o = __shfl_up_sync(kFull, incl, d);
        if (lane >= d) incl += o;
      }
      uint32_t slot = incl - mine;
      const uint32_t words[4] = {bm.x, bm.y, bm.z, bm.w};
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        uint32_t m = words[w];
        while (m) {
          const int b = __ffs(m) - 1;
          m &= m - 1;
          const int pos = lane * 128 + w * 32 + b;
          const float v = ep[pos];
          oidx[slot] = (uint16_t)pos;
          float sent;
          if (bits == 32) {
            reinterpret_cast<float*>(ocodes)[slot] = v;
            sent = v;
          } else {
            const uint32_t code = quant_code(v, sc, bits);
            atomicOr(&cw[(slot * (uint32_t)bits) >> 5], code << ((slot * (uint32_t)bits) & 31u));
            sent = dequant(code, sc, bits);
          }
          ep[pos] = __fsub_rn(v, sent);           // line 4: the residual
          ++slot;
        }
      }
      reinterpret_cast<uint4*>(bitmap)[lane] = make_uint4(0, 0, 0, 0);
      fence_async_smem();
      __syncwarp();
      // ---- E ----
      if (lane == 0) tma_store_1d(a.p.err[r] + c.base, ep, kBytes);
      if (bits != 32 && lane < cwords) {
        reinterpret_cast<uint32_t*>(ocodes)[lane] = cw[lane];
        cw[lane] = 0;
      }
      if (lane == 0) {
        a.p.scales[r][g] = sc;
        if (smax >= 0x7F800000u && a.flags) atomicOr(a.flags, (uint32_t)SL_FLAG_NONFINITE);
        tma_store_wait_read();                    // the stage has been read: it may be refilled
        if (r + kEeStages < R) {
          mbar_expect_tx(&sm.full_ee[se], kBytes);
          tma_load_1d(sm.ee[se], a.p.err[r + kEeStages] + c.base, kBytes, &sm.full_ee[se]);
        }
      }
      __syncwarp();
    }
  }
  if (timed_out && a.flags) atomicOr(a.flags, (uint32_t)SL_FLAG_TIMEOUT);
}

}  // namespace

template <int T>
cudaError_t launch_compress(const CompressArgs<T>& a, bool aligned16, cudaStream_t st) {
  if (a.tb.n_chunks == 0) return cudaSuccess;
  const size_t gsmem = (size_t)a.chunk * 4 + (a.bits == 32 ? 0 : (size_t)((a.stride + 3) / 4) * 4);
  cudaError_t e;
  if (gsmem > 40 * 1024) {
    e = cudaFuncSetAttribute(compress_generic_kernel<T, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gsmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(compress_generic_kernel<T, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gsmem);
    if (e != cudaSuccess) return e;
  }
  const bool fast = aligned16 && a.chunk == kC && a.k <= 128 && ((a.k * a.bits) % 32) == 0;
  if (fast) {
    e = cudaFuncSetAttribute(compress_c4096_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)sizeof(FastSmem));
    if (e != cudaSuccess) return e;
    compress_c4096_kernel<T><<<a.tb.n_chunks, kFastThreads, sizeof(FastSmem), st>>>(a);
    bool tails = false;
    for (uint32_t t = 0; t < a.tb.n_tensors; ++t)
      tails = tails || ((a.tb.offset[t + 1] - a.tb.offset[t]) % (uint64_t)kC) != 0;
    if (tails)
      compress_generic_kernel<T, true><<<a.tb.n_tensors * (unsigned)a.R, kThreads, gsmem, st>>>(a);
    return cudaPeekAtLastError();
  }
  const uint64_t blocks = (uint64_t)a.tb.n_chunks * (uint64_t)a.R;
  if (blocks > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
  compress_generic_kernel<T, false><<<(unsigned)blocks, kThreads, gsmem, st>>>(a);
  return cudaPeekAtLastError();
}

template cudaError_t launch_compress<256>(const CompressArgs<256>&, bool, cudaStream_t);
template cudaError_t launch_compress<SL_MAX_TENSORS>(const CompressArgs<SL_MAX_TENSORS>&, bool, cudaStream_t);

}  // namespace sl
