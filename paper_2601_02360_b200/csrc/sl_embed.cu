// Token-embedding re-projection after an outer synchronisation (paper §2.4, Eqs. 3-4):
//     T_perp <- T_perp + (T_S - Pi_S(T_S)),   T_S <- Pi_S(T_S),   Pi_S(t) = t U U^T.
//
// The table's rows are dealt out in groups of 32, evenly over one CTA per SM; a CTA walks its
// rows in sub-tiles of up to 128 rows.  Both contractions of a sub-tile run on the
// 5th-generation tensor cores (tcgen05.mma, kind::tf32) with accumulators in tensor memory:
//
//   pass 1   P[128 x k]  = T_S[rows x d] . U[d x k]        K-loop over d in steps of 32 columns.
//            A = a T_S tile (K-major, 128-byte swizzle), B = 32 rows of U (U is stored with k
//            contiguous, so the operand is fed "MN-major", which for 32-bit elements exists only
//            in the 128-byte swizzle with 32-byte atoms).  P stays in tensor memory.
//   pass 2   O[128 x 128] = P[128 x k] . U[n0.., :]^T      for each block of 128 output columns.
//            A = P read straight from tensor memory, B = 128 rows of U (K-major).  O is double
//            buffered in tensor memory.  (An MMA of N = 64 costs as many cycles as one of
//            N = 128, so the blocks are 128 wide; the epilogue takes them in parts of 32.)
//
// The tensor cores cut (do not round) a float32 operand to TF32, which would shorten the result by
// about 1.5e-3 at every call; so the epilogue warps, idle during pass 1, round each T_S tile to the
// nearest TF32 value in shared memory before the MMA warp may use it, and round P in tensor memory
// between the passes.  U is used as given (the caller rounds it once: it never changes).
//
// All global traffic is bulk tensor copies (TMA): warp 0 loads the MMA operands; warp 6 loads,
// for pass 2, the T_S / T_perp tiles of each 32-column part into swizzled shared-memory buffers;
// warp 1 owns tensor memory and issues the MMAs; warps 2-5 (one thread per row) read O from
// tensor memory and apply Eqs. 3-4 in place in those buffers with explicitly rounded float32
// operations (the 128-byte swizzle makes the row-per-thread accesses conflict-free); warp 7
// stores the buffers back with bulk tensor stores, which clip at the table's edges.  The pass-1
// operand ring shares its shared memory with the pass-2 buffers.  Rows a sub-tile does not own
// (its height is a multiple of 32 below 128) are never stored.  Every wait is bounded; a wait
// that gives up raises SL_FLAG_TIMEOUT and all roles fall through to the common exit.
#include "sl_common.cuh"
#include "sl_tc.cuh"

namespace sl {
namespace {

using namespace tc;

constexpr int kRows = 128;        // rows per sub-tile (MMA M)
constexpr int kTileK = 32;        // floats per 128-byte swizzle row
constexpr int kBlockN = 128;      // output columns per pass-2 MMA block
constexpr int kPartN = 32;        // ... which the epilogue takes in four parts of one swizzle row each
constexpr int kRing1 = 4;         // pass-1 ring: T_S tile (16 KB) + 32 rows of U (up to 32 KB) per slot
constexpr int kSlotA = kRows * kTileK * 4;
constexpr int kSlot1 = kSlotA + 256 * kTileK * 4;
constexpr int kEBufs = 5;         // pass-2 tile buffers: 128 x 32 of T_S (16 KB) + the same of T_perp
constexpr int kEHalf = kRows * kTileK * 4;
constexpr int kESize = 2 * kEHalf;
constexpr int kRing2 = 4;         // pass-2 ring: 128 rows of U x 32 columns per slot
constexpr int kSlot2 = kBlockN * kTileK * 4;
constexpr int kRing2InX = 2;      // its first slots lie behind the tile buffers, the others in `y`
constexpr int kThreads = 320;      // ten warps, see the kernel
static_assert(kEBufs * kESize + kRing2InX * kSlot2 == kRing1 * kSlot1, "pass-2 buffers fill the pass-1 ring");

struct EmbedSmem {
  uint8_t x[kRing1 * kSlot1];                   // pass 1: operand ring; pass 2: tile buffers + ring slots
  uint8_t y[kRing2 - kRing2InX][kSlot2];
  uint64_t full1[kRing1], ready1[kRing1], empty1[kRing1], full2[kRing2], empty2[kRing2];
  uint64_t o_full[2], o_empty[2], e_full[kEBufs + 1], e_empty[kEBufs + 1], e_done[kEBufs + 1];
  uint64_t p_done, x_free;   // per sub-tile: pass 1 has read its ring / pass 2 has left the shared region
  uint64_t p_ready;          // per sub-tile: the coordinates in tensor memory have been rounded to TF32
  uint64_t mma_idle;         // after a give-up only: the MMAs issued so far have retired
  uint32_t tmem_base;
  WaitCtl ctl;
};

// bounded wait on one of this kernel's barriers (see tc::mbar_wait)
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, EmbedSmem& sm) {
  return tc::mbar_wait(b, parity, sm.ctl);
}

struct Maps {
  CUtensorMap ts128, ts32, tp128, tp32;   // T_S / T_perp, boxes of 128 and of 32 rows x 32 floats
  CUtensorMap u_n;                        // U, box 32 rows (d) x 32 floats (k), 32-byte-atom swizzle
  CUtensorMap u_k;                        // U, box 128 rows (d) x 32 floats (k)
};

// PAIR (k <= 128, more than one sub-tile per CTA): two sub-tiles A and B go through pass 1 together and share
// every slice of U - a slot holds their two T_S tiles and at most 16 KB of U, their coordinates lie side by
// side in tensor memory (columns [0, 128) and [128, 256)) - then pass 2 runs for A and for B.
template <bool PAIR>
__global__ void __launch_bounds__(kThreads, 1)
embed_reproject_kernel(const __grid_constant__ Maps maps, uint64_t V, uint32_t d, uint32_t kp, uint32_t* flags,
                       uint32_t wait_polls) {
  extern __shared__ uint8_t raw[];
  EmbedSmem& sm = *reinterpret_cast<EmbedSmem*>(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t k_tiles1 = (d + kTileK - 1) / kTileK;      // pass 1: steps over d
  const uint32_t k_tiles2 = kp / kTileK;                    // pass 2: steps over k (padded)
  const uint32_t n_blocks = (d + kBlockN - 1) / kBlockN;
  const uint32_t n_parts = (d + kPartN - 1) / kPartN;
  // this CTA's rows: groups [g0, g1) of 32 rows
  const uint64_t G = (V + 31) / 32;
  const uint64_t g0 = (uint64_t)blockIdx.x * G / gridDim.x, g1 = (uint64_t)(blockIdx.x + 1) * G / gridDim.x;
  // PAIR: the U blocks of pass 2 are half as large (k <= 128), two ring slots are enough and the shared region
  // holds a sixth tile buffer instead of the other two
  constexpr int kEB = PAIR ? kEBufs + 1 : kEBufs, kR2 = PAIR ? 2 : kRing2, kR2X = PAIR ? 0 : kRing2InX;
  static_assert(kEB * kESize + kR2X * kSlot2 == kRing1 * kSlot1, "pass-2 buffers fill the pass-1 ring");
  auto r2slot = [&](uint32_t s2) -> uint8_t* {
    if constexpr (kR2X == 0) return sm.y[s2];
    else return s2 < (uint32_t)kR2X ? sm.x + kEB * kESize + s2 * kSlot2 : sm.y[s2 - kR2X];
  };
  constexpr uint64_t kStep = PAIR ? 8 : 4;                  // groups of 32 rows per turn of the loops below
  constexpr uint32_t kUoff = PAIR ? 2 * kSlotA : kSlotA;    // where the slice of U lies in a pass-1 slot
  auto groups_a = [&](uint64_t g) { return (uint32_t)(g1 - g < 4 ? g1 - g : 4); };
  auto groups_b = [&](uint64_t g) { return !PAIR || g + 4 >= g1 ? 0u : (uint32_t)(g1 - g - 4 < 4 ? g1 - g - 4 : 4); };

  if (tid == 0) {
    for (int s = 0; s < kRing1; ++s) { mbar_init(&sm.full1[s], 3); mbar_init(&sm.ready1[s], 4); mbar_init(&sm.empty1[s], 1); }
    for (int s = 0; s < kR2; ++s) { mbar_init(&sm.full2[s], 1); mbar_init(&sm.empty2[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&sm.o_full[b], 1); mbar_init(&sm.o_empty[b], 4); }
    for (int b = 0; b < kEB; ++b) {
      mbar_init(&sm.e_full[b], 1); mbar_init(&sm.e_empty[b], 1); mbar_init(&sm.e_done[b], 4);
    }
    mbar_init(&sm.p_done, 1);
    mbar_init(&sm.p_ready, 4);
    mbar_init(&sm.x_free, 1);
    mbar_init(&sm.mma_idle, 1);
    sm.ctl.abort = 0;
    sm.ctl.polls = wait_polls;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tbase = sm.tmem_base;
  const uint32_t t_p = tbase;            // P: columns [0, kp)
  const uint32_t t_o = tbase + 256;      // O: two buffers of 128 columns

  // bounded wait for the last of `uses` uses of a barrier (nothing to wait for when it was never used)
  auto wait_last = [&](uint64_t* bar, uint32_t uses) { return uses == 0 || mbar_wait(bar, (uses - 1) & 1u, sm); };
  // pass 1: the boxes of a U slice are shared by three producer warps (issuing a tensor-map copy costs its
  // thread about 0.05 us, and a K step has up to nine): warp 0 takes [0, u_split1), warp 8 [u_split1, u_split2),
  // warp 9 the rest; each announces its own bytes on the slot's barrier
  const uint32_t u_boxes = kp / 32, u_split1 = (u_boxes + 1) / 3, u_split2 = (2 * u_boxes + 1) / 3;
  if (warp == 8 || warp == 9) {
    if (lane == 0) {
      const uint32_t lo = warp == 8 ? u_split1 : u_split2, hi = warp == 8 ? u_split2 : u_boxes;
      uint32_t it1 = 0, t = 0;
      bool ok = true;
      for (uint64_t g = g0; ok && g < g1; g += kStep, ++t) {
        if (t > 0) ok = mbar_wait(&sm.x_free, (t - 1) & 1u, sm);
        for (uint32_t kt = 0; ok && kt < k_tiles1; ++kt, ++it1) {
          const uint32_t s = it1 % kRing1;
          ok = mbar_wait(&sm.empty1[s], ((it1 / kRing1) & 1u) ^ 1u, sm);
          if (!ok) break;
          uint8_t* slot = sm.x + s * kSlot1;
          mbar_expect_tx(&sm.full1[s], (hi - lo) * 4096);
          for (uint32_t n = lo; n < hi; ++n)
            tma_load_2d(slot + kUoff + n * 4096, &maps.u_n, (int)(n * 32), (int)(kt * kTileK), &sm.full1[s]);
        }
      }
      if (!ok)
        for (uint32_t s = 0; s < (uint32_t)kRing1; ++s) landed(&sm.full1[s], ring_uses(it1, s, kRing1));
    }
  } else if (warp == 0) {
    if (lane == 0) {
      // ---- operand producer: T_S tiles and (its share of) U for pass 1, U for pass 2 ----
      uint32_t it1 = 0, it2 = 0, t = 0;
      bool ok = true;
      for (uint64_t g = g0; ok && g < g1; g += kStep, ++t) {
        const uint32_t hg = groups_a(g), hb = groups_b(g), h = (hg + hb) * 32;
        const int r0 = (int)(g * 32);
        // the pass-1 ring lies over the pass-2 buffers of the previous sub-tile: wait until its last tile
        // store has left shared memory (by then its MMAs have long read their ring slots).  Waits that
        // cross roles go through barriers with one phase per sub-tile, so that a waiter can never be
        // two phases away and be fooled by the parity.
        if (t > 0) ok = mbar_wait(&sm.x_free, (t - 1) & 1u, sm);
        for (uint32_t kt = 0; ok && kt < k_tiles1; ++kt, ++it1) {
          const uint32_t s = it1 % kRing1;
          ok = mbar_wait(&sm.empty1[s], ((it1 / kRing1) & 1u) ^ 1u, sm);
          if (!ok) break;
          uint8_t* slot = sm.x + s * kSlot1;
          mbar_expect_tx(&sm.full1[s], h * 128 + u_split1 * 4096);
          if (hg == 4) {
            tma_load_2d(slot, &maps.ts128, (int)(kt * kTileK), r0, &sm.full1[s]);
          } else {
            for (uint32_t i = 0; i < hg; ++i)
              tma_load_2d(slot + i * 4096, &maps.ts32, (int)(kt * kTileK), r0 + 32 * (int)i, &sm.full1[s]);
          }
          if (PAIR) {
            if (hb == 4) {
              tma_load_2d(slot + kSlotA, &maps.ts128, (int)(kt * kTileK), r0 + kRows, &sm.full1[s]);
            } else {
              for (uint32_t i = 0; i < hb; ++i)
                tma_load_2d(slot + kSlotA + i * 4096, &maps.ts32, (int)(kt * kTileK), r0 + kRows + 32 * (int)i, &sm.full1[s]);
            }
          }
          for (uint32_t n = 0; n < u_split1; ++n)      // the other boxes of the slice come from warps 8 and 9
            tma_load_2d(slot + kUoff + n * 4096, &maps.u_n, (int)(n * 32), (int)(kt * kTileK), &sm.full1[s]);
        }
        // ... and the pass-2 ring lies over the pass-1 ring: its last MMAs must have read it
        ok = ok && mbar_wait(&sm.p_done, t & 1u, sm);
        for (uint32_t c = 0; ok && c < n_blocks * (hb ? 2u : 1u); ++c)     // (PAIR: the blocks of A, then those of B)
          for (uint32_t kt = 0; kt < k_tiles2; ++kt, ++it2) {
            const uint32_t s = it2 % kR2;
            ok = mbar_wait(&sm.empty2[s], ((it2 / kR2) & 1u) ^ 1u, sm);
            if (!ok) break;
            mbar_expect_tx(&sm.full2[s], kSlot2);
            tma_load_2d(r2slot(s), &maps.u_k, (int)(kt * kTileK), (int)((c >= n_blocks ? c - n_blocks : c) * kBlockN), &sm.full2[s]);
          }
      }
      if (!ok) {
        for (uint32_t s = 0; s < (uint32_t)kRing1; ++s) landed(&sm.full1[s], ring_uses(it1, s, kRing1));
        for (uint32_t s = 0; s < (uint32_t)kR2; ++s) landed(&sm.full2[s], ring_uses(it2, s, kR2));
      }
    }
  } else if (warp == 6) {
    if (lane == 0) {
      // ---- tile producer: the T_S / T_perp tiles of each 32-column part of pass 2 ----
      uint32_t hcg = 0, t = 0;
      bool ok = true;
      for (uint64_t g = g0; ok && g < g1; g += kStep, ++t) {
        // the tile buffers lie over the pass-1 ring: wait until this sub-tile's pass 1 has read it
        ok = mbar_wait(&sm.p_done, t & 1u, sm);
       for (uint32_t sub = 0; ok && sub < (groups_b(g) ? 2u : 1u); ++sub) {
        const uint32_t hg = sub ? groups_b(g) : groups_a(g), h = hg * 32;
        const int r0 = (int)(g * 32) + (int)sub * kRows;
        for (uint32_t hb = 0; ok && hb < n_parts; ++hb, ++hcg) {
          const uint32_t b = hcg % kEB;
          ok = wait_last(&sm.e_empty[b], hcg / kEB);
          if (!ok) break;
          const int x = (int)(hb * kPartN);
          uint8_t* ets = sm.x + b * kESize;
          uint8_t* etp = ets + kEHalf;
          mbar_expect_tx(&sm.e_full[b], 2 * h * 128);
          if (hg == 4) {
            tma_load_2d(ets, &maps.ts128, x, r0, &sm.e_full[b]);
            tma_load_2d(etp, &maps.tp128, x, r0, &sm.e_full[b]);
          } else {
            for (uint32_t i = 0; i < hg; ++i) {
              tma_load_2d(ets + i * 4096, &maps.ts32, x, r0 + 32 * (int)i, &sm.e_full[b]);
              tma_load_2d(etp + i * 4096, &maps.tp32, x, r0 + 32 * (int)i, &sm.e_full[b]);
            }
          }
        }
       }
      }
      if (!ok)
        for (uint32_t b = 0; b < (uint32_t)kEB; ++b) landed(&sm.e_full[b], ring_uses(hcg, b, kEB));
    }
  } else if (warp == 7) {
    if (lane == 0) {
      // ---- tile store: writes each finished part back and frees its buffer ----
      uint32_t hcg = 0;
      bool ok = true;
      for (uint64_t g = g0; ok && g < g1; g += kStep) {
       for (uint32_t sub = 0; ok && sub < (groups_b(g) ? 2u : 1u); ++sub) {
        const uint32_t hg = sub ? groups_b(g) : groups_a(g);
        const int r0 = (int)(g * 32) + (int)sub * kRows;
        for (uint32_t hb = 0; ok && hb < n_parts; ++hb, ++hcg) {
          const uint32_t b = hcg % kEB;
          ok = mbar_wait(&sm.e_done[b], (hcg / kEB) & 1u, sm);
          if (!ok) break;
          const int x = (int)(hb * kPartN);
          const uint32_t e = smem_u32(sm.x + b * kESize);
          for (uint32_t i = 0; i < hg; ++i) {
            tma_store_2d(&maps.ts32, x, r0 + 32 * (int)i, e + i * 4096);
            tma_store_2d(&maps.tp32, x, r0 + 32 * (int)i, e + kEHalf + i * 4096);
          }
          bulk_commit();
          bulk_wait_read_all();          // the copies have read the buffer: the tile producer may refill it
          mbar_arrive(&sm.e_empty[b]);
        }
       }
        if (ok) mbar_arrive(&sm.x_free);  // the next sub-tile's operand ring may overwrite the buffers
      }
      bulk_wait_all();
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---- MMA issuer ----
      uint32_t it1 = 0, it2 = 0, cg = 0, t = 0;
      bool ok = true;
      const uint32_t idesc1 = instr_desc(kRows, (int)kp, 1);
      const uint32_t idesc2 = instr_desc(kRows, kBlockN, 0);
      const uint64_t desc_k = smem_desc(0, 16, 1024, 2);      // K-major tile, rows of 128 bytes
      const uint64_t desc_n = smem_desc(0, 4096, 512, 1);     // U rows as N-major operand
      for (uint64_t g = g0; ok && g < g1; g += kStep, ++t) {
        const bool two = groups_b(g) != 0;
        for (uint32_t kt = 0; ok && kt < k_tiles1; ++kt, ++it1) {
          const uint32_t s = it1 % kRing1;
          ok = mbar_wait(&sm.ready1[s], (it1 / kRing1) & 1u, sm);      // landed and rounded (see the epilogue warps)
          if (!ok) break;
          tc_fence_after();
          const uint32_t a0 = smem_u32(sm.x + s * kSlot1);
          const uint64_t da = desc_k | (uint64_t)((a0 >> 4) & 0x3FFF);
          const uint64_t db = desc_n | (uint64_t)(((a0 + kUoff) >> 4) & 0x3FFF);
#pragma unroll
          for (int j = 0; j < 4; ++j)   // K = 8 per instruction: 32 bytes along a swizzled row of A, 8 rows of U
            mma_ss(t_p, da + 2 * j, db + 64 * j, idesc1, (kt | (uint32_t)j) != 0);
          if (PAIR && two) {
            const uint64_t da2 = desc_k | (uint64_t)(((a0 + kSlotA) >> 4) & 0x3FFF);
#pragma unroll
            for (int j = 0; j < 4; ++j) mma_ss(t_p + 128, da2 + 2 * j, db + 64 * j, idesc1, (kt | (uint32_t)j) != 0);
          }
          mma_commit(&sm.empty1[s]);
        }
        if (ok) mma_commit(&sm.p_done);
        ok = ok && mbar_wait(&sm.p_ready, t & 1u, sm);   // the epilogue warps have rounded P in place
        for (uint32_t c = 0; ok && c < n_blocks * (two ? 2u : 1u); ++c, ++cg) {
          const uint32_t t_pa = t_p + (c >= n_blocks ? 128u : 0u);          // the coordinates of A, then of B
          const uint32_t buf = cg & 1u;
          ok = wait_last(&sm.o_empty[buf], cg >> 1);
          if (!ok) break;
          tc_fence_after();
          for (uint32_t kt = 0; kt < k_tiles2; ++kt, ++it2) {
            const uint32_t s = it2 % kR2;
            ok = mbar_wait(&sm.full2[s], (it2 / kR2) & 1u, sm);
            if (!ok) break;
            tc_fence_after();
            const uint64_t db = desc_k | (uint64_t)((smem_u32(r2slot(s)) >> 4) & 0x3FFF);
#pragma unroll
            for (int j = 0; j < 4; ++j)
              mma_ts(t_o + buf * kBlockN, t_pa + kt * kTileK + 8 * j, db + 2 * j, idesc2, (kt | (uint32_t)j) != 0);
            mma_commit(&sm.empty2[s]);
          }
          if (!ok) break;
          mma_commit(&sm.o_full[buf]);
        }
      }
      if (!ok) mma_quiesce(&sm.mma_idle);
    }
  } else {
    // ---- epilogue: one thread per row; warp w may read tensor-memory lanes 32*(w%4).. only ----
    const int q = warp & 3;
    const uint32_t row = (uint32_t)(32 * q + lane);
    const uint32_t sw = row & 7u;
    uint32_t cg = 0, hcg = 0, t = 0, it1 = 0;
    bool ok = true;
    for (uint64_t g = g0; ok && g < g1; g += kStep, ++t) {
      const uint32_t hgb = groups_b(g);
      // The tensor cores CUT a float32 operand to TF32, which would shorten every product; values that
      // are already TF32 pass through unchanged.  So during pass 1 these warps round every T_S tile to the
      // nearest TF32 value in place as soon as it has landed (element-wise: the swizzle is irrelevant) and
      // only then hand it to the MMA warp; between the passes they do the same to the coordinates P in
      // tensor memory.  (U is not touched: round it once with sl_round_tf32, it never changes.)
      for (uint32_t kt = 0; ok && kt < k_tiles1; ++kt, ++it1) {
        const uint32_t s = it1 % kRing1;
        ok = mbar_wait(&sm.full1[s], (it1 / kRing1) & 1u, sm);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const uint32_t a0 = smem_u32(sm.x + s * kSlot1) + (uint32_t)(tid - 64) * 16;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          float4 v = lds128(a0 + 2048 * i);
          v.x = __uint_as_float(round_tf32(__float_as_uint(v.x)));
          v.y = __uint_as_float(round_tf32(__float_as_uint(v.y)));
          v.z = __uint_as_float(round_tf32(__float_as_uint(v.z)));
          v.w = __uint_as_float(round_tf32(__float_as_uint(v.w)));
          sts128(a0 + 2048 * i, v);
        }
        if (PAIR && hgb) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            float4 v = lds128(a0 + kSlotA + 2048 * i);
            v.x = __uint_as_float(round_tf32(__float_as_uint(v.x)));
            v.y = __uint_as_float(round_tf32(__float_as_uint(v.y)));
            v.z = __uint_as_float(round_tf32(__float_as_uint(v.z)));
            v.w = __uint_as_float(round_tf32(__float_as_uint(v.w)));
            sts128(a0 + kSlotA + 2048 * i, v);
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.ready1[s]);
      }
      if (!ok) break;
      ok = mbar_wait(&sm.p_done, t & 1u, sm);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      for (uint32_t half = 0; half < (hgb ? 2u : 1u); ++half)
        for (uint32_t cb = 0; cb < kp; cb += 32) {
          uint32_t v[32];
          const uint32_t ta = t_p + 128 * half + cb + ((uint32_t)(32 * q) << 16);
          tmem_ld32(ta, v);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = round_tf32(v[i]);
          tmem_st32(ta, v);
        }
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.p_ready);
      for (uint32_t cc = 0; ok && cc < n_blocks * (hgb ? 2u : 1u); ++cc, ++cg) {
        const uint32_t c = cc >= n_blocks ? cc - n_blocks : cc;               // the blocks of A, then those of B
        const uint32_t h = (cc >= n_blocks ? hgb : groups_a(g)) * 32;
        const uint32_t buf = cg & 1u;
        const uint32_t left = (d - c * kBlockN + kPartN - 1) / kPartN;
        const uint32_t np = left < 4 ? left : 4;      // parts of this block that exist
        ok = mbar_wait(&sm.o_full[buf], (cg >> 1) & 1u, sm);
        for (uint32_t part = 0; part < np; ++part, ++hcg) {
          const uint32_t b = hcg % kEB;
          ok = ok && mbar_wait(&sm.e_full[b], (hcg / kEB) & 1u, sm);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          uint32_t o[32];
          tmem_ld32(t_o + buf * kBlockN + part * kPartN + ((uint32_t)(32 * q) << 16), o);
          tmem_ld_wait();
          if (part + 1 == np) {      // this warp has taken all it needs from the O buffer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.o_empty[buf]);
          }
          const uint32_t e = smem_u32(sm.x + b * kESize);
          if (row < h) {
#pragma unroll
            for (uint32_t ch = 0; ch < 8; ++ch) {
              const uint32_t a = e + row * 128 + ((ch ^ sw) << 4);
              const float4 ts = lds128(a);
              float4 tp = lds128(a + kEHalf);
              float4 pi;
              pi.x = __uint_as_float(o[ch * 4 + 0]);
              pi.y = __uint_as_float(o[ch * 4 + 1]);
              pi.z = __uint_as_float(o[ch * 4 + 2]);
              pi.w = __uint_as_float(o[ch * 4 + 3]);
              tp.x = __fadd_rn(tp.x, __fsub_rn(ts.x, pi.x));
              tp.y = __fadd_rn(tp.y, __fsub_rn(ts.y, pi.y));
              tp.z = __fadd_rn(tp.z, __fsub_rn(ts.z, pi.z));
              tp.w = __fadd_rn(tp.w, __fsub_rn(ts.w, pi.w));
              sts128(a, pi);
              sts128(a + kEHalf, tp);
            }
          }
          // hand the finished buffer to the storing warp
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.e_done[b]);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(512) : "memory");
  }
  if (tid == 0 && sm.ctl.abort && flags) atomicOr(flags, (uint32_t)SL_FLAG_TIMEOUT);
}


__global__ void __launch_bounds__(256) round_tf32_kernel(float* __restrict__ x, uint64_t n) {
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x)
    x[i] = __uint_as_float(round_tf32(__float_as_uint(x[i])));
}

// Shapes the tensor-core kernel does not take (k or d not a multiple of 4, k above 256, unaligned
// pointers): plain float32 fused multiply-adds, one CTA per kGenRows rows.  The coordinates
// P = T_S U of those rows sit in shared memory; then every column of the rows is rebuilt from
// them and Eqs. 3-4 are applied in place.  Slow (U is streamed from L2 for every CTA) but exact
// to float32 rounding; needs kGenRows * k floats of shared memory (k <= 4096).
constexpr int kGenRows = 8;
constexpr int kGenThreads = 256;

__global__ void __launch_bounds__(kGenThreads)
embed_reproject_generic_kernel(float* __restrict__ T_S, float* __restrict__ T_perp, const float* __restrict__ U,
                               uint64_t V, uint32_t d, uint32_t k) {
  extern __shared__ float coord[];              // [kGenRows][k]
  const uint64_t r0 = (uint64_t)blockIdx.x * kGenRows;
  const uint32_t rows = (uint32_t)(V - r0 < (uint64_t)kGenRows ? V - r0 : (uint64_t)kGenRows);
  // coordinates: thread -> (row, j); the row's elements are broadcast, U[i][j..] is read coalesced
  for (uint32_t t = threadIdx.x; t < rows * k; t += kGenThreads) {
    const uint32_t r = t / k, j = t - r * k;
    const float* ts = T_S + (r0 + r) * d;
    float acc = 0.0f;
    for (uint32_t i = 0; i < d; ++i) acc = __fmaf_rn(ts[i], U[(uint64_t)i * k + j], acc);
    coord[r * k + j] = acc;
  }
  __syncthreads();                              // every read of the old rows for the coordinates is done
  for (uint32_t t = threadIdx.x; t < rows * d; t += kGenThreads) {
    const uint32_t r = t / d, n = t - r * d;
    const float* u = U + (uint64_t)n * k;
    const float* c = coord + r * k;
    float pi = 0.0f;
    for (uint32_t j = 0; j < k; ++j) pi = __fmaf_rn(c[j], u[j], pi);
    const uint64_t at = (r0 + r) * d + n;
    T_perp[at] = __fadd_rn(T_perp[at], __fsub_rn(T_S[at], pi));
    T_S[at] = pi;
  }
}

}  // namespace

cudaError_t launch_round_tf32(float* x, uint64_t n, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  const uint64_t blocks = (n + 255) / 256;
  cudaError_t e;
  const uint64_t cap = (uint64_t)sm_count(&e) * 16u;
  if (e != cudaSuccess) return e;
  round_tf32_kernel<<<(unsigned)(blocks < cap ? blocks : cap), 256, 0, st>>>(x, n);
  return cudaGetLastError();
}

bool embed_is_tuned(const float* T_S, const float* T_perp, const float* U, uint32_t d, uint32_t k) {
  auto al16 = [](const void* p) { return ((uintptr_t)p & 15u) == 0; };
  return d % 4 == 0 && k % 4 == 0 && k >= 4 && k <= 256 && al16(T_S) && al16(T_perp) && al16(U);
}

cudaError_t launch_embed_reproject(float* T_S, float* T_perp, const float* U, uint64_t V, uint32_t d, uint32_t k,
                                   uint32_t* flags, cudaStream_t st) {
  if (!embed_is_tuned(T_S, T_perp, U, d, k)) {
    const size_t smem = (size_t)kGenRows * k * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(embed_reproject_generic_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    const uint64_t grid = (V + kGenRows - 1) / kGenRows;
    if (grid > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    embed_reproject_generic_kernel<<<(unsigned)grid, kGenThreads, smem, st>>>(T_S, T_perp, U, V, d, k);
    return cudaGetLastError();
  }
  // a box row of the tables is 128 bytes of a much longer row whose neighbouring 128 bytes are wanted
  // next (the next 32-column part, the next K step): fetch 256 bytes into L2 at a time
  constexpr CUtensorMapL2promotion kTablePromo = CU_TENSOR_MAP_L2_PROMOTION_L2_256B;
  Maps m;
  if (!make_map(&m.ts128, T_S, d, V, kRows, CU_TENSOR_MAP_SWIZZLE_128B, kTablePromo) ||
      !make_map(&m.ts32, T_S, d, V, 32, CU_TENSOR_MAP_SWIZZLE_128B, kTablePromo) ||
      !make_map(&m.tp128, T_perp, d, V, kRows, CU_TENSOR_MAP_SWIZZLE_128B, kTablePromo) ||
      !make_map(&m.tp32, T_perp, d, V, 32, CU_TENSOR_MAP_SWIZZLE_128B, kTablePromo) ||
      !make_map(&m.u_n, U, k, d, 32, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B) ||
      !make_map(&m.u_k, U, k, d, kBlockN, CU_TENSOR_MAP_SWIZZLE_128B))
    return cudaErrorInvalidValue;
  const int smem = (int)sizeof(EmbedSmem) + 1024;
  cudaError_t e;
  const int sms = sm_count(&e);
  if (e != cudaSuccess) return e;
  const uint32_t kp = (k + 31u) & ~31u;
  const uint64_t tiles = (V + kRows - 1) / kRows;          // never more CTAs than full sub-tiles
  const unsigned grid = (unsigned)(tiles < (uint64_t)sms ? tiles : (uint64_t)sms);
  // more than four groups of 32 rows for every CTA and room for two coordinate tiles: two sub-tiles share pass 1
  const bool pair = kp <= 128 && (V + 31) / 32 > 4ull * grid;
  auto kern = pair ? embed_reproject_kernel<true> : embed_reproject_kernel<false>;
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  kern<<<grid, kThreads, smem, st>>>(m, V, d, kp, flags, debug_wait_polls());
  return cudaGetLastError();
}

}  // namespace sl
