// Eq. 2 lines 1-4 (paper §2.1): pseudo-gradient, error feedback, chunk-wise Top-k,
// quantisation, residual.
//
// Two kernels with identical results:
//   compress_generic_kernel  any chunk length / k / code width / alignment, consecutive chunks or
//                            square tiles; one CTA per (chunk, replica); exact 4-pass radix
//                            select in shared memory.
//   compress_c4096_kernel    the tuned path for full 4096-element chunks, k <= 128: persistent
//                            warp-specialised CTAs walk (chunk, replica) items with theta_global
//                            held in registers, a cheap lower bound on the k-th magnitude prunes
//                            the chunk to about a hundred candidates, a selector warp finishes
//                            the exact selection while the producers work on the next items.
#include <algorithm>

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
__device__ __forceinline__ void block_select_emit(float* ep, const ChunkRef& c, int k_eff, int bits, float s,
                                                  SelectScratch& sc, uint32_t* cw,
                                                  uint16_t* __restrict__ oidx, uint8_t* __restrict__ ocodes,
                                                  uint32_t* flags, uint32_t cwords) {
  const int len = c.len;
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
      const uint32_t bin = (key >> shift) & ((1u << width) - 1u);
      if ((key >> hs) == (prefix >> hs) && SL_CHECK(flags, bin < 256u)) atomicAdd(&sc.hist[bin], 1u);
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
    const uint32_t slot = out_base + __popc(km & lanemask_lt());
    if (keep && SL_CHECK(flags, slot < (uint32_t)k_eff && (bits == 32 || ((slot * (uint32_t)bits) >> 5) < cwords))) {
      oidx[slot] = (uint16_t)c.pos(i);            // element number -> position (they differ in edge tiles)
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
// TAILS = true: CTA b handles the (b / R)-th chunk that is not full (short last chunks, edge
// tiles); this is how the tuned path delegates the ragged ends of the tensors.
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
  if (TAILS) g = tail_chunk(a.tb, g, a.chunk);    // the g-th chunk that is not full
  if (!SL_CHECK(a.flags, g < a.tb.n_chunks)) return;
  const ChunkRef c = locate(a.tb, g, a.chunk);
  const int len = c.len;
  const int k = a.k, bits = a.bits;
  const int k_eff = k < len ? k : len;
  const uint64_t n_total = a.tb.offset[a.tb.n_tensors];
  (void)n_total;
  if (!SL_CHECK(a.flags, len >= 1 && len <= a.chunk)) return;

  const float* __restrict__ tl = a.p.theta_local[r];
  const float* __restrict__ tg = a.theta_global;
  float* __restrict__ er = a.p.err[r];

  // pseudo-gradient and error feedback; element i of the chunk (ascending position) sits at c.addr(i)
  uint32_t tmax = 0;
  for (int i = tid; i < len; i += kThreads) {
    const uint64_t at = c.addr(i);
    if (!SL_CHECK(a.flags, at < n_total)) continue;
    const float d = a.theta_bf16 ? __fsub_rn(bf16_widen(reinterpret_cast<const uint16_t*>(tg)[at]),
                                             bf16_widen(reinterpret_cast<const uint16_t*>(tl)[at]))
                                 : __fsub_rn(tg[at], tl[at]);
    const float e = __fmaf_rn(a.beta, er[at], d);
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
  block_select_emit(ep, c, k_eff, bits, s, sc, cw, oidx, ocodes, a.flags, cwords);

  // write-back
  for (int i = tid; i < len; i += kThreads) {
    const uint64_t at = c.addr(i);
    if (SL_CHECK(a.flags, at < n_total)) er[at] = ep[i];
  }
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
// Persistent grid of two CTAs per SM.  CTA b of G owns the full chunks among b, b+G, b+2G, ... and
// walks their (chunk, replica) pairs - "items" - as one continuous stream: item w is replica
// w % R of the CTA's (w / R)-th chunk, so the pipeline below never drains between chunks.
// theta_global of the current chunk stays in registers (one trip through memory per chunk for
// all R replicas); the next chunk's is requested as soon as the last replica has used them.
// The CTA is warp specialised: 8 producer warps (256 threads) and kSel selector warps; selector q
// handles the items w with w % kSel == q, so two selections are in flight while the producers
// run ahead.
//
//  * Bulk data moves by TMA (cp.async.bulk + mbarrier complete_tx, every CTA fetching its own data).  theta_local of
//    item w+2 is loaded by producer thread 0 into a 2-deep ring (a stage is dead after phase A).
//    e lives in a 4-deep ring: loaded four items ahead by the selector that owns the stage,
//    overwritten in place with e' by the producers, patched with the residual by the selector,
//    and sent back to the error buffer as ONE bulk store by that selector.  Under a saturated
//    memory system such a store takes microseconds to drain, so nobody waits for a store it has
//    just issued: the selector checks it only at the start of its next item, where it idles at a
//    barrier anyway, and then refills the stage.
//  * Producers, per item (a thread owns four float4s of the chunk, 256 float4s apart):
//      A  e' = fma(beta, e, theta_global - theta_local), written in place of e in the stage;
//         per-thread maximum key.  Every warp sorts its 32 thread maxima (bitonic network of
//         shuffles) and takes the j-th largest, j = ceil(k/8): at least j keys of the warp's 512
//         are >= it, so at least 8j >= k keys of the chunk are >= T1 = the smallest of the eight
//         values: T1 is a lower bound of the k-th largest key.
//      B  the keys >= T1 (about a hundred for k = 64) are appended to a candidate list and
//         counted in a 256-bin histogram of the key range [T1, max].
//      E  item w-2, finished by its selector in the meantime: warp 0 copies its message from
//         shared memory to idx / codes / scales (three coalesced stores; the selectors issue no
//         ordinary global stores).
//  * Selector, per item:
//      C  a suffix scan of the histogram finds the bin that holds the k-th largest key; a
//         bisection inside that bin (candidates in registers) finds a threshold that leaves
//         exactly k candidates; if the range collapses first the k-th key is tied, and the
//         lowest positions among its ties are found by a second bisection over positions.
//      D  kept positions are marked in a 4096-bit map and compacted (ballots); a prefix sum of
//         the map's popcounts turns a position into its rank = message slot; each lane then
//         handles k/32 kept elements: idx and code into a shared-memory copy of the message,
//         residual patched into the stage.
//  If the candidate list overflows (tie-heavy or constant chunks) the selector runs an exact
//  warp-wide radix select over the whole chunk instead of C.
//
// Hand-offs: named barrier 1 = producers only; 2+q = candidate list q ready (producers arrive,
// selector q waits); 4+q = selector q has finished an item: message final, candidate list free
// (selector q arrives, producers wait).  bar.arrive / bar.sync order the shared-memory accesses
// around them (the producer/consumer idiom of the PTX manual), so no membar is used: it would
// also wait for global stores in flight.  Every mbarrier wait is bounded.  A wait that runs out sets a
// mark in shared memory; from then on nothing more is copied in or out in bulk (the issuing threads look
// at the mark before every copy), every later wait returns at once, the selectors select nothing (the
// stages may still be written by copies in flight) and the roles walk the rest of their items with all
// hand-offs in step, so that nobody is left waiting at a named barrier; at the end the threads that
// issued bulk copies wait (bounded again) until the ones in flight have landed, and the kernel returns
// with SL_FLAG_TIMEOUT raised (no trap, no hang; the outputs of the call are then unspecified).  The hot
// loops carry no exit for this: a branch out of the producers' loop cost 1.7 % of the launch.
// ---------------------------------------------------------------------------
constexpr int kC = 4096;
constexpr int kSel = 2;               // selector warps
constexpr int kTlStages = 2;
constexpr int kEeStages = 4;
static_assert(kEeStages == 2 * kSel && kTlStages == 2, "the give-up path counts copies per stage from these");
constexpr int kCandMax = 512;
constexpr int kCandReg = 6;           // candidates per lane held in registers: C <= 192 (k <= 64) ...
constexpr int kCandRegBig = 11;       // ... or C <= 352 (k = 128); longer lists are walked in shared memory

constexpr int kPtrCache = 16;         // replicas whose pointers are staged in shared memory
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
// bounded wait on a phase; false = gave up, or another thread of the CTA already has (`abort` != 0);
// non-blocking test_wait with a short sleep between polls
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint32_t limit, const volatile uint32_t& abort) {
  const uint32_t addr = smem_u32(bar);
  for (uint32_t it = 0; it < limit; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
    if (ok) return true;
    if (abort) return false;
    __nanosleep(40);
  }
  return false;
}
// after a give-up: lets the last of `uses` bulk copies announced on `bar` land before the CTA's shared
// memory goes away (always with the default bound, whatever limit the waits had)
__device__ __forceinline__ void mbar_drain(uint64_t* bar, uint32_t uses) {
  if (uses == 0) return;
  const uint32_t addr = smem_u32(bar), parity = (uses - 1) & 1u;
  for (uint32_t it = 0; it < kWaitLimit; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
    if (ok) return;
    __nanosleep(40);
  }
}
// the cold end of a give-up, kept out of line so that it does not weigh on the kernels' hot code: waits for
// the copies announced on `n` barriers `step` apart (uses[i] of them on barrier i) and raises the flag
__device__ __noinline__ void giveup_drain(uint64_t* bars, int n, int step, uint32_t issued, int per, uint32_t* flags) {
  for (int i = 0; i < n; ++i) mbar_drain(bars + i * step, (issued + per - 1 - i) / per);
  if (flags) atomicOr(flags, (uint32_t)SL_FLAG_TIMEOUT);
}
__device__ __forceinline__ void tma_load_1d(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// 16-byte asynchronous copy global -> shared (per thread, any address pattern); copies are
// grouped per thread, and a thread can wait until all but its newest N groups have landed
__device__ __forceinline__ void cp_async_16(void* dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }
__device__ __forceinline__ void tma_store_1d(void* dst, const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
               ::"l"(dst), "r"(smem_u32(src)), "r"(bytes) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// wait until all bulk stores of this thread have read their source
__device__ __forceinline__ void tma_store_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

struct alignas(16) FastSmem {
  float tl[kTlStages][kC];            // theta_local of replica r in stage r % 2
  float ee[kEeStages][kC];            // e of replica r in stage r % 4, then e' in place, then the store's source
  uint32_t cand_key[kSel][kCandMax];
  uint16_t cand_pos[kSel][kCandMax];
  uint32_t bitmap[kSel][kC / 32];     // kept positions of the selection in progress
  uint32_t hist[kSel][256];           // candidates per bin of [T1, max]; radix histogram in the overflow path
  uint16_t msg_idx[kEeStages][128];   // the message of the replica in each stage: positions,
  uint32_t msg_codes[kEeStages][128]; // packed codes (or k raw floats when bits == 32),
  float msg_scale[kEeStages];         // scale
  uint16_t kept_pos[kSel][128];
  uint8_t prefix[kSel][kC / 32];      // kept positions before each bitmap word
  uint32_t wmin[kEeStages][kWarps], wmax[kEeStages][kWarps];   // ring: producers run up to three replicas ahead
  uint32_t tmax_x[kThreads];          // TILED: thread maxima, regrouped before the lower bound is taken
  uint32_t count[kSel];
  const float* p_tl[kPtrCache];       // the first kPtrCache replicas' pointers (parameter-space reads
  float* p_err[kPtrCache];            // with a run-time index are slow)
  uint16_t* p_idx[kPtrCache];
  uint8_t* p_codes[kPtrCache];
  float* p_scales[kPtrCache];
  uint64_t full_tl[kTlStages];
  uint64_t full_ee[kEeStages];
  volatile uint32_t abort_item;       // non-zero once a bounded wait has given up: no more bulk copies, later waits return at once
};
static_assert(sizeof(FastSmem) <= 115712, "two CTAs per SM need 2 * (smem + 1 KB) <= 228 KB");

// bins of the candidate histogram: bin = (key - T1) >> sh with (max - T1) >> sh <= 255
__device__ __forceinline__ int hist_shift(uint32_t T1, uint32_t smax) {
  const uint32_t range = smax - T1;
  return range < 256u ? 0 : (32 - __clz(range)) - 8;
}

// number of candidate keys >= mid; keys either in registers (NREG > 0) or in shared memory
template <int NREG>
__device__ __forceinline__ uint32_t count_ge(const uint32_t (&ck)[NREG > 0 ? NREG : 1], const uint32_t* ck_smem,
                                             uint32_t C, uint32_t mid, int lane) {
  uint32_t c0 = 0, c1 = 0, c2 = 0;
  if (NREG > 0) {
#pragma unroll
    for (int i = 0; i < NREG; i += 3) {
      c0 += ck[i] >= mid ? 1u : 0u;
      if (i + 1 < NREG) c1 += ck[i + 1] >= mid ? 1u : 0u;
      if (i + 2 < NREG) c2 += ck[i + 2] >= mid ? 1u : 0u;
    }
  } else {
    for (uint32_t i = lane; i < C; i += 32) c0 += ck_smem[i] >= mid ? 1u : 0u;
  }
  return __reduce_add_sync(kFull, c0 + c1 + c2);
}

// Phase C and the first half of D for a candidate list that did not overflow: threshold, then
// kept positions marked in `bitmap` and compacted into `kept_pos` (any order).
template <int NREG>
__device__ __forceinline__ void select_candidates(const uint32_t* cand_key, const uint16_t* cand_pos, uint32_t C,
                                                  uint32_t k, uint32_t T1, uint32_t smax, uint32_t* hist,
                                                  uint32_t* bitmap, uint16_t* kept_pos, int lane, uint32_t* flags) {
  uint32_t ck[NREG > 0 ? NREG : 1];
  uint32_t cp[NREG > 0 ? NREG : 1];
  if (NREG > 0) {
#pragma unroll
    for (int i = 0; i < NREG; ++i) {
      const uint32_t at = (uint32_t)lane + 32u * (uint32_t)i;
      ck[i] = at < C ? cand_key[at] : 0u;          // padding 0 is below every probe (probes are > T1 >= 0)
      cp[i] = at < C ? (uint32_t)cand_pos[at] : 0u;
    }
  }
  // ---- the bin of the k-th largest key: suffix sums of the histogram, top bin first
  const int sh = hist_shift(T1, smax);
  uint32_t lo, hi, cnt_hi;
  bool exact;
  {
    const uint4 h0 = reinterpret_cast<const uint4*>(hist)[2 * lane];
    const uint4 h1 = reinterpret_cast<const uint4*>(hist)[2 * lane + 1];
    reinterpret_cast<uint4*>(hist)[2 * lane] = make_uint4(0, 0, 0, 0);       // ready for the next replica
    reinterpret_cast<uint4*>(hist)[2 * lane + 1] = make_uint4(0, 0, 0, 0);
    const uint32_t h[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
    uint32_t mine = 0;
#pragma unroll
    for (int b = 0; b < 8; ++b) mine += h[b];
    uint32_t suf = mine;                          // candidates in this lane's bins and above
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t o = __shfl_down_sync(kFull, suf, d);
      if (lane + d < 32) suf += o;
    }
    const uint32_t vote = __ballot_sync(kFull, suf >= k);
    const int sel = 31 - __clz(vote);             // highest lane whose suffix still reaches k (C >= k: lane 0 does)
    uint32_t above = suf - mine, bin = (uint32_t)lane * 8u, in_bin = 0;
    bool found = false;
#pragma unroll
    for (int bb = 7; bb >= 0; --bb) {
      if (!found) {
        if (above + h[bb] >= k) { found = true; bin = (uint32_t)(lane * 8 + bb); in_bin = h[bb]; }
        else above += h[bb];
      }
    }
    bin = __shfl_sync(kFull, bin, sel);
    in_bin = __shfl_sync(kFull, in_bin, sel);
    cnt_hi = __shfl_sync(kFull, above, sel);      // candidates in the bins above: all kept, fewer than k
    lo = T1 + (bin << sh);                        // keys of the bin: lo <= key < lo + 2^sh
    hi = lo + (1u << sh);
    exact = cnt_hi + in_bin == k;                 // the whole bin is kept: threshold = its lower edge
  }
  uint32_t thr_ge = lo;                            // keep key >= thr_ge ...
  uint32_t thr_eq = 0xFFFFFFFFu, pos_le = 0;       // ... and key == thr_eq at position <= pos_le
  if (!exact) {
    while (hi - lo > 1u) {                         // count(key >= lo) > k > count(key >= hi) = cnt_hi
      const uint32_t mid = lo + ((hi - lo) >> 1);
      const uint32_t cnt = count_ge<NREG>(ck, cand_key, C, mid, lane);
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
    }
  }
  // ---- mark and compact the kept candidates
  uint32_t base = 0;
  if (NREG > 0) {
#pragma unroll
    for (int i = 0; i < NREG; ++i) {
      if (32u * (uint32_t)i < C) {
        const bool keep = ((uint32_t)lane + 32u * (uint32_t)i < C) &&
                          (ck[i] >= thr_ge || (ck[i] == thr_eq && cp[i] <= pos_le));
        const uint32_t bal = __ballot_sync(kFull, keep);
        if (keep && SL_CHECK(flags, cp[i] < (uint32_t)kC && base + __popc(bal & lanemask_lt()) < 128u)) {
          atomicOr(&bitmap[cp[i] >> 5], 1u << (cp[i] & 31u));
          kept_pos[base + __popc(bal & lanemask_lt())] = (uint16_t)cp[i];
        }
        base += __popc(bal);
      }
    }
  } else {
    for (uint32_t i0 = 0; i0 < C; i0 += 32) {
      const uint32_t i = i0 + lane;
      const uint32_t k_i = i < C ? cand_key[i] : 0u;
      const uint32_t p_i = i < C ? (uint32_t)cand_pos[i] : 0u;
      const bool keep = i < C && (k_i >= thr_ge || (k_i == thr_eq && p_i <= pos_le));
      const uint32_t bal = __ballot_sync(kFull, keep);
      if (keep && SL_CHECK(flags, p_i < (uint32_t)kC && base + __popc(bal & lanemask_lt()) < 128u)) {
        atomicOr(&bitmap[p_i >> 5], 1u << (p_i & 31u));
        kept_pos[base + __popc(bal & lanemask_lt())] = (uint16_t)p_i;
      }
      base += __popc(bal);
    }
  }
}

// Overflow path of the selector: exact radix select over the whole chunk by one warp; kept
// positions go to the bitmap (one ballot = one bitmap word) and to kept_pos.
__device__ __forceinline__ void warp_select_full(const float* ep, uint32_t k, uint32_t* hist, uint32_t* bitmap,
                                                 uint16_t* kept_pos, int lane, uint32_t* flags) {
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
#pragma unroll
  for (int b = 0; b < 8; ++b) hist[lane * 8 + b] = 0;     // leave the histogram clean for phase B
  const uint32_t kth = prefix;
  uint32_t eq_seen = 0, base = 0;
  for (int w = 0; w < kC / 32; ++w) {
    const uint32_t key = key_of(ep[w * 32 + lane]);
    const bool eq = key == kth;
    const uint32_t eqm = __ballot_sync(kFull, eq);
    const bool keep = key > kth || (eq && eq_seen + __popc(eqm & lanemask_lt()) < need);
    const uint32_t km = __ballot_sync(kFull, keep);
    if (lane == 0) bitmap[w] = km;
    if (keep && SL_CHECK(flags, base + __popc(km & lanemask_lt()) < 128u))
      kept_pos[base + __popc(km & lanemask_lt())] = (uint16_t)(w * 32 + lane);
    eq_seen += __popc(eqm);
    base += __popc(km);
  }
}

// One work item = one (full chunk, replica) pair.  CTA b of G owns the full chunks among
// b, b+G, b+2G, ... and walks their items in order: item w is replica w % R of its (w / R)-th chunk.
template <int T>
struct ItemCursor {
  uint32_t g;       // chunk number in the arena
  uint64_t base;    // element offset of the chunk's first element
  uint32_t stride;  // elements between the chunk's rows of 64: 64 for a consecutive chunk, the matrix's
                    // row length for a tile
  uint32_t t_lo;    // tensor of the chunk (lookup cache)
  int r;            // replica
  bool valid;

  // first full chunk at or after g0 (stepping by the grid size)
  __device__ __forceinline__ void seek(const Table<T>& tb, uint32_t g0, uint32_t step) {
    g = g0;
    valid = false;
    while (g < tb.n_chunks) {
      const ChunkRef c = locate_cached(tb, g, kC, t_lo);
      if (c.len == kC) { base = c.base; stride = c.stride ? c.stride : 64u; valid = true; return; }
      g += step;                                   // chunks that are not full belong to the tail launch
    }
  }
  __device__ __forceinline__ void start(const Table<T>& tb, uint32_t b, uint32_t step) { r = 0; t_lo = 0; seek(tb, b, step); }
  __device__ __forceinline__ void advance(const Table<T>& tb, int n, int R, uint32_t step) {
    r += n;
    while (valid && r >= R) { r -= R; seek(tb, g + step, step); }
  }
};

// TILED = false: every full chunk is 16 KB of consecutive memory and moves by TMA bulk copies as
// described above.  TILED = true (arenas with matrices cut into 64 x 64 tiles): a chunk is 64 rows
// of 256 bytes, `stride` elements apart.  Bulk copies of 256 bytes run at a third of the rate of
// 16 KB ones, so here the 256 producer threads fetch theta_local and e themselves with 16-byte
// cp.async copies, two items ahead, and write the residual back with 128-bit streaming stores;
// the selectors touch shared memory only.  Every thread copies exactly the float4s it will read
// in phase A, so completion is a per-thread cp.async.wait_group and needs no barrier (256
// per-thread arrivals on one mbarrier were tried first: they serialise and cost more than the
// copies).  In shared memory a tile is stored row after row, so everything between load and
// store is the same.
// BF = true (consecutive chunks only): theta_local and theta_global are bfloat16 arrays; a theta_local
// stage then holds 8 KB, and both are widened (exactly) as they are read.
template <int T, bool TILED, bool BF>
__global__ void __launch_bounds__(kFastThreads, 2)
compress_c4096_kernel(const __grid_constant__ CompressArgs<T> a) {
  static_assert(!(TILED && BF), "bfloat16 parameters take the tuned path for consecutive chunks only");
  extern __shared__ __align__(16) unsigned char smem_raw[];
  FastSmem& sm = *reinterpret_cast<FastSmem*>(smem_raw);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t G = gridDim.x;
  const int k = a.k, bits = a.bits, R = a.R;
  constexpr uint32_t kBytes = kC * 4;
  constexpr uint32_t kTlBytes = BF ? kC * 2 : kC * 4;        // bytes of theta_local per chunk
  // theta_local of replica r, `elems` elements in
  auto tl_src = [&](int r, uint64_t elems) -> const void* {
    const float* p = r < kPtrCache ? sm.p_tl[r] : a.p.theta_local[r];
    return BF ? (const void*)(reinterpret_cast<const uint16_t*>(p) + elems) : (const void*)(p + elems);
  };
  const uint64_t n_total = a.tb.offset[a.tb.n_tensors];      // debug build: the range every arena offset must stay in
  (void)n_total;

  for (int i = tid; i < kSel * (kC / 32); i += kFastThreads) (&sm.bitmap[0][0])[i] = 0;
  for (int i = tid; i < kSel * 256; i += kFastThreads) (&sm.hist[0][0])[i] = 0;
  for (int i = tid; i < kEeStages * 128; i += kFastThreads) (&sm.msg_codes[0][0])[i] = 0;
  if (tid < kPtrCache && tid < R) {
    sm.p_tl[tid] = a.p.theta_local[tid];
    sm.p_err[tid] = a.p.err[tid];
    sm.p_idx[tid] = a.p.idx[tid];
    sm.p_codes[tid] = a.p.codes[tid];
    sm.p_scales[tid] = a.p.scales[tid];
  }
  if (tid == 0) {
    sm.abort_item = 0;
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
  const uint32_t wait_limit = a.wait_polls == 0 ? kWaitLimit : a.wait_polls == 0xFFFFFFFFu ? 0u : a.wait_polls;

  if (warp < kWarps) {
    // ======================= producers =======================================
    ItemCursor<T> cur;                            // item w
    cur.start(a.tb, blockIdx.x, G);
    // This thread's float4s are number t4 + 256 j (j = 0..3) of the chunk, with
    // t4 = 64 (lane / 8) + 8 warp + lane % 8: every 8 lanes read 128 contiguous bytes (no bank
    // conflicts), and every warp samples each of the sixteen 256-element regions of the chunk
    // with 32 elements, so a row boundary inside the chunk (rows of very different scale) cannot
    // leave a warp with small values only, which would ruin the lower bound below.
    const int t4 = ((lane >> 3) << 6) + (warp << 3) + (lane & 7);
    ItemCursor<T> pf = cur;                       // the item whose theta_local (TILED: and e) is loaded next
    // TILED: float4 f of a chunk is columns 4 (f % 16) .. +3 of row f / 16; a thread copies the
    // float4s t4 + 256 j it will read itself (one group of copies per item)
    auto tile_load = [&](const ItemCursor<T>& it, int st_tl, int st_ee) {
      const float* src_tl = (it.r < kPtrCache ? sm.p_tl[it.r] : a.p.theta_local[it.r]) + it.base;
      const float* src_ee = (it.r < kPtrCache ? sm.p_err[it.r] : a.p.err[it.r]) + it.base;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int f = t4 + 256 * j;
        const size_t off = (size_t)(f >> 4) * it.stride + (size_t)((f & 15) << 2);
        if (!SL_CHECK(a.flags, it.base + off + 4 <= n_total)) continue;
        cp_async_16(reinterpret_cast<float4*>(sm.tl[st_tl]) + f, src_tl + off);
        cp_async_16(reinterpret_cast<float4*>(sm.ee[st_ee]) + f, src_ee + off);
      }
    };
    uint32_t tl_issued = 0;                       // thread 0: theta_local copies issued so far (the j-th goes to stage j % 2)
    for (int i = 0; i < kTlStages; ++i) {
      if (pf.valid) {
        if (TILED) {
          tile_load(pf, i, i);
        } else if (tid == 0 && SL_CHECK(a.flags, pf.base + kC <= n_total)) {
          ++tl_issued;
          mbar_expect_tx(&sm.full_tl[i], kTlBytes);
          tma_load_1d(sm.tl[i], tl_src(pf.r, pf.base), kTlBytes, &sm.full_tl[i]);
        }
        pf.advance(a.tb, 1, R, G);
      }
      if (TILED) cp_async_commit();               // one group per item, empty ones included, keeps the count uniform
    }
    const int cwords = bits == 32 ? k : (k * bits) >> 5;   // 32-bit words of codes per chunk
    const int jsel = 32 - (k + kWarps - 1) / kWarps;   // lane holding the ceil(k/8)-th largest after an ascending sort
    const float beta = a.beta;
    float4 G4[4];                                 // this thread's 16 elements of theta_global
    // theta_global of a chunk into this thread's registers (float4 f = t4 + 256 j; row f / 16 of a tile)
    auto load_theta = [&](const ItemCursor<T>& it) {
      const float* tg = a.theta_global + it.base;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int f = t4 + 256 * j;
        const size_t off = TILED ? (size_t)(f >> 4) * it.stride + (size_t)((f & 15) << 2) : (size_t)f * 4;
        if (SL_CHECK(a.flags, it.base + off + 4 <= n_total)) {
          if constexpr (BF)
            G4[j] = bf16x4_widen(__ldcs(reinterpret_cast<const uint2*>(reinterpret_cast<const uint16_t*>(a.theta_global) + it.base + off)));
          else
            G4[j] = __ldcs(reinterpret_cast<const float4*>(tg + off));
        }
      }
    };
    if (cur.valid) load_theta(cur);
    uint32_t g_m1 = 0, g_m2 = 0;                  // chunk, replica (TILED: and place) of items w-1 and w-2
    int r_m1 = 0, r_m2 = 0;
    uint64_t base_m1 = 0, base_m2 = 0;
    uint32_t stride_m1 = 64, stride_m2 = 64;
    // TILED: the residual of a finished item goes back to the error buffer from its stage
    auto tile_store = [&](int rp, uint64_t base, uint32_t stride, int st_ee) {
      float* dst = (rp < kPtrCache ? sm.p_err[rp] : a.p.err[rp]) + base;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int f = tid + 256 * j;
        const size_t off = (size_t)(f >> 4) * stride + (size_t)((f & 15) << 2);
        if (SL_CHECK(a.flags, base + off + 4 <= n_total))
          __stcs(reinterpret_cast<float4*>(dst + off), reinterpret_cast<const float4*>(sm.ee[st_ee])[f]);
      }
    };
    __syncwarp();

    uint32_t w = 0;
#pragma unroll 1
    for (; cur.valid; ++w) {
      const int st = w % kTlStages, se = w % kEeStages, q = w % kSel;
      if (TILED) {
        cp_async_wait_but_one();                  // this thread's copies for item w have landed (item w+1's may fly)
      } else if (!mbar_wait(&sm.full_tl[st], (w / kTlStages) & 1u, wait_limit, sm.abort_item) ||
                 !mbar_wait(&sm.full_ee[se], (w / kEeStages) & 1u, wait_limit, sm.abort_item)) {
        sm.abort_item = w + 1;                    // (any non-zero mark) phase A below then works on stale data: harmless
      }
      const float4* tl4 = reinterpret_cast<const float4*>(sm.tl[st]);
      float4* ee4 = reinterpret_cast<float4*>(sm.ee[se]);
      // ---- A ----
      uint32_t key[16];
      uint32_t tmax = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float4 L;
        if constexpr (BF) L = bf16x4_widen(reinterpret_cast<const uint2*>(sm.tl[st])[t4 + 256 * j]);
        else L = tl4[t4 + 256 * j];
        const float4 E = ee4[t4 + 256 * j];
        float4 v;
        v.x = __fmaf_rn(beta, E.x, __fsub_rn(G4[j].x, L.x));
        v.y = __fmaf_rn(beta, E.y, __fsub_rn(G4[j].y, L.y));
        v.z = __fmaf_rn(beta, E.z, __fsub_rn(G4[j].z, L.z));
        v.w = __fmaf_rn(beta, E.w, __fsub_rn(G4[j].w, L.w));
        ee4[t4 + 256 * j] = v;
        key[4 * j + 0] = key_of(v.x);
        key[4 * j + 1] = key_of(v.y);
        key[4 * j + 2] = key_of(v.z);
        key[4 * j + 3] = key_of(v.w);
        tmax = max(tmax, max(max(key[4 * j], key[4 * j + 1]), max(key[4 * j + 2], key[4 * j + 3])));
      }
      if (!TILED) fence_async_smem();             // e' must be visible to the bulk store that drains this stage
      // the next item: same chunk, or the next chunk, whose theta_global is requested now (the
      // registers are free) so that it arrives while this item is finished
      ItemCursor<T> nxt = cur;
      nxt.advance(a.tb, 1, R, G);
      if (nxt.valid && nxt.r == 0) load_theta(nxt);
      uint32_t v = tmax;
      if (TILED) {
        // In a tile every row of the matrix has its own scale and a warp's float4s cover only 16 of
        // the 64 rows, so the per-warp bound below could be taken over small rows only.  Regroup:
        // group `warp` takes the maxima of threads 8 lane + warp, one from every warp and every
        // row phase, so each group samples all 64 rows.
        sm.tmax_x[tid] = tmax;
        named_sync(1, kThreads);
        v = sm.tmax_x[8 * lane + warp];
      }
      // bitonic sort of the group's 32 thread maxima, ascending over lanes
#pragma unroll
      for (int size = 2; size <= 32; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
          const uint32_t o = __shfl_xor_sync(kFull, v, stride);
          const bool up = (lane & size) == 0, lower = (lane & stride) == 0;
          v = (up == lower) ? min(v, o) : max(v, o);
        }
      }
      const uint32_t wmin = __shfl_sync(kFull, v, jsel);     // this group's ceil(k/8)-th largest thread maximum
      const uint32_t wmax = __shfl_sync(kFull, v, 31);
      if (lane == 0) { sm.wmin[se][warp] = wmin; sm.wmax[se][warp] = wmax; }
      if (w >= (uint32_t)kSel) {
        __syncwarp();
        named_sync(4 + q, kPairThreads);          // selector q has finished item w-2
        // ---- E (item w-2): its message leaves shared memory (warp 0, three coalesced stores) ----
        if (warp == 0 && SL_CHECK(a.flags, g_m2 < a.tb.n_chunks && r_m2 < R)) {
          const int sp = (w - kSel) % kEeStages;
          const bool pc = r_m2 < kPtrCache;
          uint16_t* oidx = (pc ? sm.p_idx[r_m2] : a.p.idx[r_m2]) + (uint64_t)g_m2 * (uint64_t)k;
          uint32_t* ocodes = reinterpret_cast<uint32_t*>((pc ? sm.p_codes[r_m2] : a.p.codes[r_m2]) + (uint64_t)g_m2 * (uint64_t)a.stride);
          for (int i = lane; i < (k >> 1); i += 32)
            reinterpret_cast<uint32_t*>(oidx)[i] = reinterpret_cast<const uint32_t*>(sm.msg_idx[sp])[i];
          for (int i = lane; i < cwords; i += 32) {
            ocodes[i] = sm.msg_codes[sp][i];
            sm.msg_codes[sp][i] = 0;              // the next message in this stage ORs its codes into zeros
          }
          if (lane == 0) (pc ? sm.p_scales[r_m2] : a.p.scales[r_m2])[g_m2] = sm.msg_scale[sp];
        }
        if (TILED) tile_store(r_m2, base_m2, stride_m2, (w - kSel) % kEeStages);
      }
      named_sync(1, kThreads);
      // a wait of this item gave up (every such mark was written before the barrier above; a mark of a
      // later item, by a thread that has run ahead, is larger): all producers leave here
      if (pf.valid) {
        // every producer has read theta_local(w) (TILED: and written back the stage of e(w-2)):
        // the stages take item w+2's
        if (TILED) {
          tile_load(pf, st, (w + kTlStages) % kEeStages);
        } else if (tid == 0 && sm.abort_item == 0 && SL_CHECK(a.flags, pf.base + kC <= n_total)) {
          ++tl_issued;
          mbar_expect_tx(&sm.full_tl[st], kTlBytes);
          tma_load_1d(sm.tl[st], tl_src(pf.r, pf.base), kTlBytes, &sm.full_tl[st]);
        }
        pf.advance(a.tb, 1, R, G);
      }
      if (TILED) cp_async_commit();
      uint32_t T1, smax;
      {
        const uint4 m0 = reinterpret_cast<const uint4*>(sm.wmin[se])[0], m1 = reinterpret_cast<const uint4*>(sm.wmin[se])[1];
        const uint4 x0 = reinterpret_cast<const uint4*>(sm.wmax[se])[0], x1 = reinterpret_cast<const uint4*>(sm.wmax[se])[1];
        T1 = min(min(min(m0.x, m0.y), min(m0.z, m0.w)), min(min(m1.x, m1.y), min(m1.z, m1.w)));
        smax = max(max(max(x0.x, x0.y), max(x0.z, x0.w)), max(max(x1.x, x1.y), max(x1.z, x1.w)));
      }
      const int sh = hist_shift(T1, smax);
      // ---- B ----
      uint32_t mask = 0;
#pragma unroll
      for (int e = 0; e < 16; ++e) mask |= (key[e] >= T1 ? 1u : 0u) << e;
      if (mask) {
        uint32_t at = atomicAdd(&sm.count[q], (uint32_t)__popc(mask));
        uint32_t* ckey = sm.cand_key[q];
        uint16_t* cpos = sm.cand_pos[q];
        uint32_t* hist = sm.hist[q];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          if (mask & (1u << e)) {
            if (at < (uint32_t)kCandMax) {
              ckey[at] = key[e];
              cpos[at] = (uint16_t)(((e >> 2) << 10) + (t4 << 2) + (e & 3));
            }
            if (SL_CHECK(a.flags, ((key[e] - T1) >> sh) < 256u)) atomicAdd(&hist[(key[e] - T1) >> sh], 1u);
            ++at;
          }
        }
      }
      __syncwarp();                               // bar.* is warp-aligned: reconverge first
      named_arrive(2 + q, kPairThreads);          // candidate list q is ready (bar.arrive orders the shared-memory
                                                  // writes before it; a membar here would also wait for global stores)
      g_m2 = g_m1; r_m2 = r_m1; base_m2 = base_m1; stride_m2 = stride_m1;
      g_m1 = cur.g; r_m1 = cur.r; base_m1 = cur.base; stride_m1 = cur.stride;
      cur = nxt;
    }
    // the last kSel items' messages
    const uint32_t W = w;
    for (uint32_t wp = (W > (uint32_t)kSel ? W - kSel : 0); wp < W; ++wp) {
      const bool last = wp + 1 == W;
      const uint32_t gp = last ? g_m1 : g_m2;
      const int rp = last ? r_m1 : r_m2;
      __syncwarp();
      named_sync(4 + wp % kSel, kPairThreads);
      if (warp == 0 && SL_CHECK(a.flags, gp < a.tb.n_chunks && rp < R)) {
        const int sp = wp % kEeStages;
        const bool pc = rp < kPtrCache;
        uint16_t* oidx = (pc ? sm.p_idx[rp] : a.p.idx[rp]) + (uint64_t)gp * (uint64_t)k;
        uint32_t* ocodes = reinterpret_cast<uint32_t*>((pc ? sm.p_codes[rp] : a.p.codes[rp]) + (uint64_t)gp * (uint64_t)a.stride);
        for (int i = lane; i < (k >> 1); i += 32)
          reinterpret_cast<uint32_t*>(oidx)[i] = reinterpret_cast<const uint32_t*>(sm.msg_idx[sp])[i];
        for (int i = lane; i < cwords; i += 32) ocodes[i] = sm.msg_codes[sp][i];
        if (lane == 0) (pc ? sm.p_scales[rp] : a.p.scales[rp])[gp] = sm.msg_scale[sp];
      }
      if (TILED) tile_store(rp, last ? base_m1 : base_m2, last ? stride_m1 : stride_m2, wp % kEeStages);
    }
    if (!TILED && tid == 0 && sm.abort_item != 0)     // gave up somewhere: let this thread's copies in flight land
      giveup_drain(sm.full_tl, kTlStages, 1, tl_issued, kTlStages, a.flags);
  } else {
    // ======================= selectors =======================================
    const int q = warp - kWarps;
    ItemCursor<T> cur;                            // item w = q, q+2, q+4, ...
    cur.start(a.tb, blockIdx.x, G);
    cur.advance(a.tb, q, R, G);
    ItemCursor<T> pf = cur;                       // the item whose e is loaded next by this selector: w, w+2 at start, then w+4
    uint32_t ee_issued = 0;                       // lane 0: e copies issued so far (the j-th goes to stage q + kSel * (j % 2))
    if (TILED) {
      pf.valid = false;                           // the producers move all the data
    } else if (lane == 0) {
      for (int i = q; i < kEeStages && pf.valid; i += kSel) {
        if (SL_CHECK(a.flags, pf.base + kC <= n_total)) {
          ++ee_issued;
          mbar_expect_tx(&sm.full_ee[i], kBytes);
          tma_load_1d(sm.ee[i], (pf.r < kPtrCache ? sm.p_err[pf.r] : a.p.err[pf.r]) + pf.base, kBytes, &sm.full_ee[i]);
        }
        pf.advance(a.tb, kSel, R, G);
      }
    } else {
      for (int i = q; i < kEeStages && pf.valid; i += kSel) pf.advance(a.tb, kSel, R, G);
    }
    __syncwarp();
    uint32_t* bitmap = sm.bitmap[q];
    uint16_t* kept_pos = sm.kept_pos[q];
    uint8_t* prefix = sm.prefix[q];
    int pending_stage = -1;                       // stage whose bulk store is in flight
#pragma unroll 1
    for (uint32_t w = q; cur.valid; w += kSel) {
      const int se = w % kEeStages;
      float* ep = sm.ee[se];
      named_sync(2 + q, kPairThreads);            // candidate list q is ready
      if (!TILED && sm.abort_item != 0) {
        // a wait has given up: the stages may still be written by copies in flight, so nothing is selected
        // from them; only the hand-off is kept in step
        __syncwarp();
        named_arrive(4 + q, kPairThreads);
        cur.advance(a.tb, kSel, R, G);
        continue;
      }
      // The store of this selector's previous item was issued a whole hand-off ago; once it has
      // read its stage, e of the item four ahead is loaded into it.
      if (!TILED && pending_stage >= 0) {
        if (lane == 0) {
          tma_store_wait_read_all();
          if (pf.valid && sm.abort_item == 0 && SL_CHECK(a.flags, pf.base + kC <= n_total)) {
            ++ee_issued;
            mbar_expect_tx(&sm.full_ee[pending_stage], kBytes);
            tma_load_1d(sm.ee[pending_stage], (pf.r < kPtrCache ? sm.p_err[pf.r] : a.p.err[pf.r]) + pf.base, kBytes,
                        &sm.full_ee[pending_stage]);
          }
        }
        pf.advance(a.tb, kSel, R, G);
        __syncwarp();
      }
      const uint32_t C = sm.count[q];
      uint32_t T1, smax;
      {
        const uint4 m0 = reinterpret_cast<const uint4*>(sm.wmin[se])[0], m1 = reinterpret_cast<const uint4*>(sm.wmin[se])[1];
        const uint4 x0 = reinterpret_cast<const uint4*>(sm.wmax[se])[0], x1 = reinterpret_cast<const uint4*>(sm.wmax[se])[1];
        T1 = min(min(min(m0.x, m0.y), min(m0.z, m0.w)), min(min(m1.x, m1.y), min(m1.z, m1.w)));
        smax = max(max(max(x0.x, x0.y), max(x0.z, x0.w)), max(max(x1.x, x1.y), max(x1.z, x1.w)));
      }
      const float sc = __uint_as_float(smax);
      uint16_t* midx = sm.msg_idx[se];
      uint32_t* mcodes = sm.msg_codes[se];
      // ---- C ----
      if (C > (uint32_t)kCandMax) warp_select_full(ep, (uint32_t)k, sm.hist[q], bitmap, kept_pos, lane, a.flags);
      else if (C <= 32u * kCandReg)
        select_candidates<kCandReg>(sm.cand_key[q], sm.cand_pos[q], C, (uint32_t)k, T1, smax, sm.hist[q], bitmap, kept_pos, lane, a.flags);
      else if (C <= 32u * kCandRegBig)
        select_candidates<kCandRegBig>(sm.cand_key[q], sm.cand_pos[q], C, (uint32_t)k, T1, smax, sm.hist[q], bitmap, kept_pos, lane, a.flags);
      else
        select_candidates<0>(sm.cand_key[q], sm.cand_pos[q], C, (uint32_t)k, T1, smax, sm.hist[q], bitmap, kept_pos, lane, a.flags);
      __syncwarp();
      if (lane == 0) sm.count[q] = 0;
      // ---- D ----
      {
        const uint4 bm = reinterpret_cast<const uint4*>(bitmap)[lane];
        const uint32_t c0 = __popc(bm.x), c1 = __popc(bm.y), c2 = __popc(bm.z), c3 = __popc(bm.w);
        const uint32_t mine = c0 + c1 + c2 + c3;
        uint32_t incl = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const uint32_t o = __shfl_up_sync(kFull, incl, d);
          if (lane >= d) incl += o;
        }
        const uint32_t ex = incl - mine;           // kept positions before this lane's 128 positions (<= 128)
        reinterpret_cast<uint32_t*>(prefix)[lane] = ex | ((ex + c0) << 8) | ((ex + c0 + c1) << 16) | ((ex + c0 + c1 + c2) << 24);
      }
      __syncwarp();
      for (int t = lane; t < k; t += 32) {
        const uint32_t pos = kept_pos[t];
        if (!SL_CHECK(a.flags, t < 128 && pos < (uint32_t)kC)) continue;
        const uint32_t wd = pos >> 5;
        const uint32_t slot = (uint32_t)prefix[wd] + __popc(bitmap[wd] & ((1u << (pos & 31u)) - 1u));
        if (!SL_CHECK(a.flags, slot < (uint32_t)k && slot < 128u)) continue;
        const float v = ep[pos];
        midx[slot] = (uint16_t)pos;
        float sent;
        if (bits == 32) {
          mcodes[slot] = __float_as_uint(v);
          sent = v;
        } else {
          const uint32_t code = quant_code(v, sc, bits);
          atomicOr(&mcodes[(slot * (uint32_t)bits) >> 5], code << ((slot * (uint32_t)bits) & 31u));
          sent = dequant(code, sc, bits);
        }
        ep[pos] = __fsub_rn(v, sent);             // line 4: the residual
      }
      if (lane == 0) {
        sm.msg_scale[se] = sc;
        if (smax >= 0x7F800000u && a.flags) atomicOr(a.flags, (uint32_t)SL_FLAG_NONFINITE);
      }
      if (!TILED) fence_async_smem();             // the patched stage is read by a bulk store
      __syncwarp();
      reinterpret_cast<uint4*>(bitmap)[lane] = make_uint4(0, 0, 0, 0);
      // ---- E: the stage drains to the error buffer (TILED: the producers write it back) ----
      if (!TILED && lane == 0 && sm.abort_item == 0 && SL_CHECK(a.flags, cur.base + kC <= n_total && cur.r < R))
        tma_store_1d((cur.r < kPtrCache ? sm.p_err[cur.r] : a.p.err[cur.r]) + cur.base, ep, kBytes);
      pending_stage = se;
      __syncwarp();
      named_arrive(4 + q, kPairThreads);          // item w is finished: message final, candidate list free
      cur.advance(a.tb, kSel, R, G);
    }
    if (!TILED && lane == 0) {
      tma_store_wait_read_all();                  // shared memory must outlive the bulk stores' reads ...
      if (sm.abort_item != 0)                     // ... and, after a give-up, the copies still coming in
        giveup_drain(&sm.full_ee[q], kEeStages / kSel, kSel, ee_issued, kEeStages / kSel, nullptr);
    }
  }
}

}  // namespace

template <int T>
bool compress_is_tuned(const CompressArgs<T>& a, bool aligned16) {
  // even k: the message's positions leave shared memory as 32-bit words.  bfloat16 parameters: consecutive
  // chunks only, and every tensor must start on 16 bytes of the 2-byte arrays too (offsets multiples of 8)
  if (a.theta_bf16) {
    if (a.tb.side != 0) return false;
    for (uint32_t t = 0; t <= a.tb.n_tensors; ++t)
      if (a.tb.offset[t] % 8 != 0) return false;
  }
  return aligned16 && a.chunk == kC && a.k <= 128 && ((a.k * a.bits) % 32) == 0 && (a.k % 2) == 0;
}

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
  if (compress_is_tuned(a, aligned16)) {
    const int sms = sm_count(&e);
    if (e != cudaSuccess) return e;
    // persistent grid: two CTAs per SM, each walking its share of the chunks
    const unsigned grid = (unsigned)std::min<uint64_t>((uint64_t)a.tb.n_chunks, (uint64_t)sms * 2u);
    auto launch = [&](auto kernel) -> cudaError_t {
      const cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(FastSmem));
      if (err != cudaSuccess) return err;
      kernel<<<grid, kFastThreads, sizeof(FastSmem), st>>>(a);
      return cudaSuccess;
    };
    if (a.tb.side != 0) e = launch(compress_c4096_kernel<T, true, false>);
    else if (a.theta_bf16) e = launch(compress_c4096_kernel<T, false, true>);
    else e = launch(compress_c4096_kernel<T, false, false>);
    if (e != cudaSuccess) return e;
    if (a.tb.n_tails)
      compress_generic_kernel<T, true><<<a.tb.n_tails * (unsigned)a.R, kThreads, gsmem, st>>>(a);
    return cudaPeekAtLastError();
  }
  const uint64_t blocks = (uint64_t)a.tb.n_chunks * (uint64_t)a.R;
  if (blocks > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
  compress_generic_kernel<T, false><<<(unsigned)blocks, kThreads, gsmem, st>>>(a);
  return cudaPeekAtLastError();
}

template bool compress_is_tuned<256>(const CompressArgs<256>&, bool);
template bool compress_is_tuned<SL_MAX_TENSORS>(const CompressArgs<SL_MAX_TENSORS>&, bool);
template cudaError_t launch_compress<256>(const CompressArgs<256>&, bool, cudaStream_t);
template cudaError_t launch_compress<SL_MAX_TENSORS>(const CompressArgs<SL_MAX_TENSORS>&, bool, cudaStream_t);

}  // namespace sl
