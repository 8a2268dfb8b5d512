// Subspace compression of stage-boundary activations (paper §2.3):
//     compress     Xt   = (X - T_perp[x] - Pos) U        n_tok x d  ->  n_tok x k  (what travels)
//     reconstruct  Xhat = Xt U^T + T_perp[x] + Pos       n_tok x k  ->  n_tok x d
//     gradients    Gt   = G U                            (compress without the embedding terms)
// Token t of the flattened batch sits at position t mod L.  Both directions are one tcgen05
// contraction (kind::tf32, accumulator in tensor memory) fused with the gather of the embedding
// rows, built from the same pieces as the embedding re-projection kernel:
//
//   compress     K-loop over d in steps of 32 columns.  The X tile arrives by TMA (K-major,
//                128-byte swizzle; three producer warps share a step's copies); eight warps (eight threads per token row, so that a gathered
//                128-byte segment is one request) then subtract the token's T_perp row and its Pos
//                row - fetched with plain loads two steps ahead - round to the nearest TF32 value
//                (the tensor cores would cut instead) and hand the tile to the MMA warp; B = 32
//                rows of U, N-major.  The same warps write the accumulator out as Xt.
//                Without embedding terms and with at least two sub-tiles per CTA, two sub-tiles
//                go through K together and share every U slice (see the dual kernel).
//   reconstruct  the Xt tile (all k columns) is rounded and moved to tensor memory once per
//                sub-tile and is the A operand of every 128-column block; B = 128 rows of U through
//                a ring; the accumulator is double buffered; the gathered rows wait in stages of
//                shared memory, the epilogue adds them and a tensor-map store writes the part.
//
// One CTA per SM.  Compression deals the tokens in groups of 32 evenly over the CTAs, sub-tiles of up to 128
// tokens; reconstruction deals the (sub-tile, 128-column block) pairs evenly, so a sub-tile may be shared.
// Every wait is bounded (SL_FLAG_TIMEOUT); a token id outside [0, V) gathers nothing and raises
// SL_FLAG_BAD_INDEX.  Other shapes (k or d not a multiple of 4, k above 256, unaligned pointers)
// take plain float32 kernels.
#include "sl_common.cuh"
#include "sl_tc.cuh"

namespace sl {
namespace {

using namespace tc;

constexpr int kRows = 128;
constexpr int kTileK = 32;
constexpr int kBlockN = 128;
constexpr int kRing = 4;
constexpr int kSlotA = kRows * kTileK * 4;            // 16 KB
constexpr int kSlotP = kSlotA + 256 * kTileK * 4;     // compress: X tile + 32 rows of U
constexpr int kRowWarps = 8;                          // two per 32-lane window of tensor memory
constexpr int kThreads = 128 + 32 * kRowWarps;        // producer warps 0, 2, 3, MMA warp 1, the row warps

struct SubParams {
  const float* T_perp;
  const float* pos;
  const int32_t* ids;       // NULL: no embedding terms (gradients)
  float* out;
  uint64_t n_tok, V;
  uint32_t L, d, k, kp;
  uint32_t* flags;
  uint32_t wait_polls;      // caller-set limit of the bounded waits in polls (0: the default)
};

// the token a row thread serves in a sub-tile: its embedding row and position row (or none)
struct RowInfo {
  bool valid, gather;
  const float* tp;
  const float* ps;
};
__device__ __forceinline__ RowInfo row_info(const SubParams& p, uint64_t r0, uint32_t h, uint32_t row, bool& bad) {
  RowInfo ri;
  const uint64_t t = r0 + row;
  ri.valid = row < h && t < p.n_tok;
  ri.gather = false;
  ri.tp = nullptr; ri.ps = nullptr;
  if (ri.valid && p.ids) {
    const int32_t id = p.ids[t];
    if (id < 0 || (uint64_t)id >= p.V) bad = true;
    else {
      ri.gather = true;
      ri.tp = p.T_perp + (uint64_t)id * p.d;
      ri.ps = p.pos + (t % p.L) * (uint64_t)p.d;
    }
  }
  return ri;
}

// A CTA's share of a reconstruction.  The sub-tiles of 128 tokens are dealt whole, q to every CTA; the
// remaining ones (fewer than there are CTAs) are cut by 128-column blocks, each among the same number of CTAs, so
// the last piece of a CTA is a range of blocks of a sub-tile it shares.  (Every sub-tile streams all of U,
// however few rows it has, and a piece costs its blocks plus the hand-over of the Xt tile: dealing whole
// sub-tiles only would leave most CTAs waiting for those that got one more.)
// The blocks of a piece are independent; CTA b walks them from the (b mod n)-th on, so that the CTAs do not
// all ask L2 for the same rows of U at the same time (no effect on the result).
struct Piece {
  uint64_t r0;              // first token of the sub-tile
  uint32_t hg, cb, n, rot;  // its groups of 32 tokens (1..4); first block and number of blocks; where the walk starts
  __device__ __forceinline__ uint32_t block(uint32_t i) const {
    const uint32_t c = i + rot;
    return cb + (c >= n ? c - n : c);
  }
};
struct Sched {
  uint64_t G, n_sub;
  uint32_t n_blocks, q, n_pieces, tail_cb, tail_n;
  uint64_t tail_st;
  __device__ __forceinline__ Sched(uint32_t n_blocks_, uint64_t G_) : G(G_), n_sub((G_ + 3) / 4), n_blocks(n_blocks_) {
    const uint64_t grid = gridDim.x, b = blockIdx.x;
    q = (uint32_t)(n_sub / grid);
    const uint64_t rem = n_sub - (uint64_t)q * grid;
    tail_cb = tail_n = 0;
    tail_st = 0;
    if (rem) {
      const uint64_t sh = grid / rem;                 // CTAs that share one of the remaining sub-tiles
      if (b < rem * sh) {
        const uint32_t j = (uint32_t)(b % sh);
        tail_st = (uint64_t)q * grid + b / sh;
        tail_cb = (uint32_t)((uint64_t)j * n_blocks / sh);
        tail_n = (uint32_t)((uint64_t)(j + 1) * n_blocks / sh) - tail_cb;
      }
    }
    n_pieces = q + (tail_n ? 1u : 0u);
  }
  __device__ __forceinline__ Piece piece(uint32_t i) const {
    Piece pc;
    const bool whole = i < q;
    const uint64_t st = whole ? (uint64_t)i * gridDim.x + blockIdx.x : tail_st;
    pc.cb = whole ? 0u : tail_cb;
    pc.n = whole ? n_blocks : tail_n;
    pc.rot = blockIdx.x % pc.n;
    pc.r0 = st * kRows;
    pc.hg = (uint32_t)(G - 4 * st < 4 ? G - 4 * st : 4);
    return pc;
  }
};

// ------------------------------------------------------------------------------------------ compress
struct ProjSmem {
  uint8_t ring[kRing * kSlotP];
  uint64_t full[kRing], ready[kRing], empty[kRing], p_done, p_free;
  uint64_t mma_idle;        // after a give-up only: the MMAs issued so far have retired
  uint32_t tmem_base;
  WaitCtl ctl;
};
struct ProjMaps { CUtensorMap x128, x32, u_n; };

__global__ void __launch_bounds__(kThreads, 1)
subspace_project_kernel(const __grid_constant__ ProjMaps maps, const __grid_constant__ SubParams p) {
  extern __shared__ uint8_t raw[];
  ProjSmem& sm = *reinterpret_cast<ProjSmem*>(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t k_tiles = (p.d + kTileK - 1) / kTileK;
  const uint64_t G = (p.n_tok + 31) / 32;
  const uint64_t g0 = (uint64_t)blockIdx.x * G / gridDim.x, g1 = (uint64_t)(blockIdx.x + 1) * G / gridDim.x;
  if (tid == 0) {
    for (int s = 0; s < kRing; ++s) { mbar_init(&sm.full[s], 3); mbar_init(&sm.ready[s], kRowWarps); mbar_init(&sm.empty[s], 1); }
    mbar_init(&sm.p_done, 1);
    mbar_init(&sm.p_free, kRowWarps);
    mbar_init(&sm.mma_idle, 1);
    sm.ctl.abort = 0;
    sm.ctl.polls = p.wait_polls;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)), "r"(256) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t t_p = sm.tmem_base;
  bool bad = false;

  if (warp == 0 || warp == 2 || warp == 3) {
    // ---- three producer warps share the copies of a K step (issuing a tensor-map copy costs its thread
    // about 0.05 us, and a step has up to nine): warp 0 the X tile and the first boxes of the U slice,
    // warps 2 and 3 the other boxes; each announces its own bytes on the slot's barrier ----
    if (lane == 0) {
      const uint32_t pi = warp == 0 ? 0u : (uint32_t)warp - 1u;          // 0, 1, 2
      const uint32_t nb = p.kp / 32;                                      // boxes of 32 columns in a U slice
      const uint32_t lo = pi == 0 ? 0u : (pi * nb + 1) / 3, hi = pi == 2 ? nb : ((pi + 1) * nb + 1) / 3;
      uint32_t it = 0;
      bool ok = true;
      for (uint64_t g = g0; ok && g < g1; g += 4) {
        const uint32_t hg = (uint32_t)(g1 - g < 4 ? g1 - g : 4), h = hg * 32;
        const int r0 = (int)(g * 32);
        for (uint32_t kt = 0; ok && kt < k_tiles; ++kt, ++it) {
          const uint32_t s = it % kRing;
          ok = mbar_wait(&sm.empty[s], ((it / kRing) & 1u) ^ 1u, sm.ctl);
          if (!ok) break;
          uint8_t* slot = sm.ring + s * kSlotP;
          mbar_expect_tx(&sm.full[s], (pi == 0 ? h * 128 : 0u) + (hi - lo) * 4096);
          if (pi == 0) {
            if (hg == 4) tma_load_2d(slot, &maps.x128, (int)(kt * kTileK), r0, &sm.full[s]);
            else
              for (uint32_t i = 0; i < hg; ++i)
                tma_load_2d(slot + i * 4096, &maps.x32, (int)(kt * kTileK), r0 + 32 * (int)i, &sm.full[s]);
          }
          for (uint32_t n = lo; n < hi; ++n)
            tma_load_2d(slot + kSlotA + n * 4096, &maps.u_n, (int)(n * 32), (int)(kt * kTileK), &sm.full[s]);
        }
      }
      if (!ok)                                       // gave up: let this thread's copies in flight land first
        for (uint32_t s = 0; s < (uint32_t)kRing; ++s) landed(&sm.full[s], ring_uses(it, s, kRing));
    }
  } else if (warp == 1) {
    if (lane == 0) {
      uint32_t it = 0, t = 0;
      bool ok = true;
      const uint32_t idesc = instr_desc(kRows, (int)p.kp, 1);
      const uint64_t desc_k = smem_desc(0, 16, 1024, 2), desc_n = smem_desc(0, 4096, 512, 1);
      for (uint64_t g = g0; ok && g < g1; g += 4, ++t) {
        if (t > 0) {                                 // the row warps have read the previous accumulator
          ok = mbar_wait(&sm.p_free, (t - 1) & 1u, sm.ctl);
          if (!ok) break;
          tc_fence_after();
        }
        for (uint32_t kt = 0; ok && kt < k_tiles; ++kt, ++it) {
          const uint32_t s = it % kRing;
          ok = mbar_wait(&sm.ready[s], (it / kRing) & 1u, sm.ctl);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a0 = smem_u32(sm.ring + s * kSlotP);
          const uint64_t da = desc_k | (uint64_t)((a0 >> 4) & 0x3FFF);
          const uint64_t db = desc_n | (uint64_t)(((a0 + kSlotA) >> 4) & 0x3FFF);
#pragma unroll
          for (int j = 0; j < 4; ++j) mma_ss(t_p, da + 2 * j, db + 64 * j, idesc, (kt | (uint32_t)j) != 0);
          mma_commit(&sm.empty[s]);
        }
        if (ok) mma_commit(&sm.p_done);
      }
      if (!ok) mma_quiesce(&sm.mma_idle);
    }
  } else {
    // ---- row warps.  Element-wise part: eight threads per token row, one 16-byte chunk each, so that a
    // gathered 128-byte segment is one request; thread j serves chunk j % 8 of rows j / 8 + 32 i.
    // Accumulator read-out: warp w reads tensor-memory lanes 32*(w%4).., the two warps of a window
    // alternate over blocks of 32 columns. ----
    const uint32_t q = (uint32_t)(warp & 3), half = (uint32_t)(warp - 4) >> 2;
    const uint32_t row = 32u * q + (uint32_t)lane;
    const uint32_t j = (uint32_t)(tid - 128), gch = j & 7u, grow = j >> 3;
    const uint32_t goff = grow * 128 + ((gch ^ (grow & 7u)) << 4);     // + 4096 i: the swizzle repeats every 8 rows
    const bool wide = p.k % 8 == 0 && ((uintptr_t)p.out & 31u) == 0;   // every row piece of Xt starts on 32 bytes
    uint32_t it = 0, t = 0;
    bool ok = true;
    // the token rows this thread gathers for, and the embedding and position values of two K steps in flight
    // while one is used; those of a sub-tile's first two steps are requested before the previous sub-tile's
    // accumulator is written out, so that they are there when its K loop starts
    const float* tp[4];
    const float* ps[4];
    uint32_t mask = 0;
    float4 et[2][4], ep[2][4];
    auto fetch = [&](uint32_t kt, float4 (&dt)[4], float4 (&dp)[4]) {
      const uint32_t col = kt * kTileK + 4u * gch;
      const bool in_col = kt < k_tiles && col < p.d;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const bool in = in_col && ((mask >> i) & 1u);
        dt[i] = in ? __ldg(reinterpret_cast<const float4*>(tp[i] + kt * kTileK)) : make_float4(0.f, 0.f, 0.f, 0.f);
        dp[i] = in ? __ldg(reinterpret_cast<const float4*>(ps[i] + kt * kTileK)) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    };
    auto open_tile = [&](uint64_t g) {
      const uint32_t h = (uint32_t)(g1 - g < 4 ? g1 - g : 4) * 32;
      mask = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const RowInfo ri = row_info(p, g * 32, h, grow + 32u * (uint32_t)i, bad);
        tp[i] = ri.gather ? ri.tp + 4 * gch : nullptr;
        ps[i] = ri.gather ? ri.ps + 4 * gch : nullptr;
        mask |= ri.gather ? 1u << i : 0u;
      }
      fetch(0, et[0], ep[0]);
      fetch(1, et[1], ep[1]);
    };
    if (g0 < g1) open_tile(g0);
    for (uint64_t g = g0; ok && g < g1; g += 4, ++t) {
      const uint32_t hg = (uint32_t)(g1 - g < 4 ? g1 - g : 4), h = hg * 32;
      const uint64_t r0 = g * 32;
      for (uint32_t kt = 0; ok && kt < k_tiles; kt += 2) {
#pragma unroll
        for (int par = 0; par < 2; ++par) {          // two K steps per trip so that the buffers keep static indices
          const uint32_t kk = kt + (uint32_t)par;
          if (kk < k_tiles) {
            float4 ct[4], cp[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { ct[i] = et[par][i]; cp[i] = ep[par][i]; }
            fetch(kk + 2, et[par], ep[par]);
            const uint32_t s = it % kRing;
            ok = ok && mbar_wait(&sm.full[s], (it / kRing) & 1u, sm.ctl);
            ok = __all_sync(0xffffffffu, ok);
            if (ok) {
              const uint32_t a0 = smem_u32(sm.ring + s * kSlotP) + goff;
#pragma unroll
              for (uint32_t i = 0; i < 4; ++i) {
                const uint32_t a = a0 + 4096u * i;
                float4 v = lds128(a);
                v.x = __fsub_rn(__fsub_rn(v.x, ct[i].x), cp[i].x);
                v.y = __fsub_rn(__fsub_rn(v.y, ct[i].y), cp[i].y);
                v.z = __fsub_rn(__fsub_rn(v.z, ct[i].z), cp[i].z);
                v.w = __fsub_rn(__fsub_rn(v.w, ct[i].w), cp[i].w);
                v.x = __uint_as_float(round_tf32(__float_as_uint(v.x)));
                v.y = __uint_as_float(round_tf32(__float_as_uint(v.y)));
                v.z = __uint_as_float(round_tf32(__float_as_uint(v.z)));
                v.w = __uint_as_float(round_tf32(__float_as_uint(v.w)));
                sts128(a, v);
              }
              asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
              __syncwarp();
              if (lane == 0) mbar_arrive(&sm.ready[s]);
              ++it;
            }
          }
        }
      }
      if (!ok) break;
      if (g + 4 < g1) open_tile(g + 4);
      // the coordinates of this sub-tile's tokens: out of tensor memory, into Xt (the two warps of a lane
      // window take alternate blocks of 32 columns)
      ok = mbar_wait(&sm.p_done, t & 1u, sm.ctl);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      for (uint32_t cb = 32u * half; cb < p.kp; cb += 64) {
        uint32_t v[32];
        tmem_ld32(t_p + cb + ((32u * q) << 16), v);
        tmem_ld_wait();
        if (row < h && r0 + row < p.n_tok) {
          float* dst = p.out + (r0 + row) * (uint64_t)p.k + cb;
          if (wide) {                                // 32-byte stores: half as many write transactions
#pragma unroll
            for (int i = 0; i < 32; i += 8)
              if (cb + (uint32_t)i < p.k) stg256(dst + i, v + i);
          } else {
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              if (cb + (uint32_t)i < p.k)
                *reinterpret_cast<float4*>(dst + i) = make_float4(__uint_as_float(v[i]), __uint_as_float(v[i + 1]),
                                                                  __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.p_free);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(t_p), "r"(256) : "memory");
  }
  if (bad && p.flags) atomicOr(p.flags, (uint32_t)SL_FLAG_BAD_INDEX);
  if (tid == 0 && sm.ctl.abort && p.flags) atomicOr(p.flags, (uint32_t)SL_FLAG_TIMEOUT);
}

// ------------------------------------------------------- compress without embedding terms, two sub-tiles
// Gt = G U for the activation gradients.  An SM takes in about 32 bytes per clock whatever the path, and of
// the 48 KB a K step of the kernel above takes in, 32 KB are the slice of U.  With nothing to gather there
// are registers and shared memory to spare, so two sub-tiles of 128 tokens advance through K together: they
// share every U slice (64 KB per step for 256 tokens instead of 96 KB) and accumulate in the two halves of
// tensor memory.  Used when every CTA has at least two sub-tiles anyway.
constexpr int kRingD = 3;
constexpr int kSlotD = 2 * kSlotA + 256 * kTileK * 4;   // two X tiles + 32 rows of U: 64 KB
struct DualSmem {
  uint8_t ring[kRingD * kSlotD];
  uint64_t full[kRingD], ready[kRingD], empty[kRingD], p_done, p_free;
  uint64_t mma_idle;        // after a give-up only: the MMAs issued so far have retired
  uint32_t tmem_base;
  WaitCtl ctl;
};

__global__ void __launch_bounds__(kThreads, 1)
subspace_project_dual_kernel(const __grid_constant__ ProjMaps maps, const __grid_constant__ SubParams p) {
  extern __shared__ uint8_t raw[];
  DualSmem& sm = *reinterpret_cast<DualSmem*>(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t k_tiles = (p.d + kTileK - 1) / kTileK;
  const uint64_t G = (p.n_tok + 31) / 32;
  const uint64_t g0 = (uint64_t)blockIdx.x * G / gridDim.x, g1 = (uint64_t)(blockIdx.x + 1) * G / gridDim.x;
  // 32-token groups of the two sub-tiles of the tile that starts at group g
  auto groups_a = [&](uint64_t g) { return (uint32_t)(g1 - g < 4 ? g1 - g : 4); };
  auto groups_b = [&](uint64_t g) { return g + 4 >= g1 ? 0u : (uint32_t)(g1 - g - 4 < 4 ? g1 - g - 4 : 4); };
  if (tid == 0) {
    for (int s = 0; s < kRingD; ++s) { mbar_init(&sm.full[s], 3); mbar_init(&sm.ready[s], kRowWarps); mbar_init(&sm.empty[s], 1); }
    mbar_init(&sm.p_done, 1);
    mbar_init(&sm.p_free, kRowWarps);
    mbar_init(&sm.mma_idle, 1);
    sm.ctl.abort = 0;
    sm.ctl.polls = p.wait_polls;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t t_p = sm.tmem_base;      // accumulator of sub-tile A; B is 256 columns further

  if (warp == 0 || warp == 2 || warp == 3) {
    // ---- three producer warps share the copies of a K step: warp 0 the two X tiles and the first boxes of
    // the U slice, warps 2 and 3 the other boxes ----
    if (lane == 0) {
      const uint32_t pi = warp == 0 ? 0u : (uint32_t)warp - 1u;
      const uint32_t nb = p.kp / 32;
      const uint32_t lo = pi == 0 ? 0u : (pi * nb + 1) / 3, hi = pi == 2 ? nb : ((pi + 1) * nb + 1) / 3;
      uint32_t it = 0;
      bool ok = true;
      for (uint64_t g = g0; ok && g < g1; g += 8) {
        const uint32_t ha = groups_a(g), hb = groups_b(g);
        const int r0 = (int)(g * 32);
        for (uint32_t kt = 0; ok && kt < k_tiles; ++kt, ++it) {
          const uint32_t s = it % kRingD;
          ok = mbar_wait(&sm.empty[s], ((it / kRingD) & 1u) ^ 1u, sm.ctl);
          if (!ok) break;
          uint8_t* slot = sm.ring + s * kSlotD;
          mbar_expect_tx(&sm.full[s], (pi == 0 ? (ha + hb) * 4096 : 0u) + (hi - lo) * 4096);
          if (pi == 0) {
            if (ha == 4) tma_load_2d(slot, &maps.x128, (int)(kt * kTileK), r0, &sm.full[s]);
            else
              for (uint32_t i = 0; i < ha; ++i)
                tma_load_2d(slot + i * 4096, &maps.x32, (int)(kt * kTileK), r0 + 32 * (int)i, &sm.full[s]);
            if (hb == 4) tma_load_2d(slot + kSlotA, &maps.x128, (int)(kt * kTileK), r0 + kRows, &sm.full[s]);
            else
              for (uint32_t i = 0; i < hb; ++i)
                tma_load_2d(slot + kSlotA + i * 4096, &maps.x32, (int)(kt * kTileK), r0 + kRows + 32 * (int)i, &sm.full[s]);
          }
          for (uint32_t n = lo; n < hi; ++n)
            tma_load_2d(slot + 2 * kSlotA + n * 4096, &maps.u_n, (int)(n * 32), (int)(kt * kTileK), &sm.full[s]);
        }
      }
      if (!ok)
        for (uint32_t s = 0; s < (uint32_t)kRingD; ++s) landed(&sm.full[s], ring_uses(it, s, kRingD));
    }
  } else if (warp == 1) {
    if (lane == 0) {
      uint32_t it = 0, t = 0;
      bool ok = true;
      const uint32_t idesc = instr_desc(kRows, (int)p.kp, 1);
      const uint64_t desc_k = smem_desc(0, 16, 1024, 2), desc_n = smem_desc(0, 4096, 512, 1);
      for (uint64_t g = g0; ok && g < g1; g += 8, ++t) {
        const bool two = groups_b(g) != 0;
        if (t > 0) {                                 // the row warps have read the previous accumulators
          ok = mbar_wait(&sm.p_free, (t - 1) & 1u, sm.ctl);
          if (!ok) break;
          tc_fence_after();
        }
        for (uint32_t kt = 0; ok && kt < k_tiles; ++kt, ++it) {
          const uint32_t s = it % kRingD;
          ok = mbar_wait(&sm.ready[s], (it / kRingD) & 1u, sm.ctl);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a0 = smem_u32(sm.ring + s * kSlotD);
          const uint64_t da = desc_k | (uint64_t)((a0 >> 4) & 0x3FFF);
          const uint64_t da2 = desc_k | (uint64_t)(((a0 + kSlotA) >> 4) & 0x3FFF);
          const uint64_t db = desc_n | (uint64_t)(((a0 + 2 * kSlotA) >> 4) & 0x3FFF);
#pragma unroll
          for (int j = 0; j < 4; ++j) mma_ss(t_p, da + 2 * j, db + 64 * j, idesc, (kt | (uint32_t)j) != 0);
          if (two) {
#pragma unroll
            for (int j = 0; j < 4; ++j) mma_ss(t_p + 256, da2 + 2 * j, db + 64 * j, idesc, (kt | (uint32_t)j) != 0);
          }
          mma_commit(&sm.empty[s]);
        }
        if (ok) mma_commit(&sm.p_done);
      }
      if (!ok) mma_quiesce(&sm.mma_idle);
    }
  } else {
    // ---- row warps: round the landed tiles to the nearest TF32 value in place (the tensor cores would cut),
    // eight threads per row; then write the accumulators out ----
    const uint32_t q = (uint32_t)(warp & 3), half = (uint32_t)(warp - 4) >> 2;
    const uint32_t row = 32u * q + (uint32_t)lane;
    const uint32_t j = (uint32_t)(tid - 128), gch = j & 7u, grow = j >> 3;
    const uint32_t goff = grow * 128 + ((gch ^ (grow & 7u)) << 4);
    const bool wide = p.k % 8 == 0 && ((uintptr_t)p.out & 31u) == 0;   // every row piece of Xt starts on 32 bytes
    uint32_t it = 0, t = 0;
    bool ok = true;
    for (uint64_t g = g0; ok && g < g1; g += 8, ++t) {
      const uint32_t ha = groups_a(g), hb = groups_b(g);
      const uint32_t chunks = hb ? 8u : 4u;          // 16-byte chunks per thread: rows grow + 32 i of A, then of B
      for (uint32_t kt = 0; ok && kt < k_tiles; ++kt, ++it) {
        const uint32_t s = it % kRingD;
        ok = mbar_wait(&sm.full[s], (it / kRingD) & 1u, sm.ctl);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const uint32_t a0 = smem_u32(sm.ring + s * kSlotD) + goff;
#pragma unroll
        for (uint32_t i = 0; i < 8; ++i) {
          if (i < chunks) {
            const uint32_t a = a0 + 4096u * i;        // the B tile follows the A tile: i = 4 .. 7 are its rows
            float4 v = lds128(a);
            v.x = __uint_as_float(round_tf32(__float_as_uint(v.x)));
            v.y = __uint_as_float(round_tf32(__float_as_uint(v.y)));
            v.z = __uint_as_float(round_tf32(__float_as_uint(v.z)));
            v.w = __uint_as_float(round_tf32(__float_as_uint(v.w)));
            sts128(a, v);
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.ready[s]);
      }
      if (!ok) break;
      ok = mbar_wait(&sm.p_done, t & 1u, sm.ctl);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      for (uint32_t tile = 0; tile < (hb ? 2u : 1u); ++tile) {
        const uint32_t h = (tile ? hb : ha) * 32;
        const uint64_t r0 = g * 32 + (uint64_t)tile * kRows;
        for (uint32_t cb = 32u * half; cb < p.kp; cb += 64) {
          uint32_t v[32];
          tmem_ld32(t_p + tile * 256 + cb + ((32u * q) << 16), v);
          tmem_ld_wait();
          if (row < h && r0 + row < p.n_tok) {
            float* dst = p.out + (r0 + row) * (uint64_t)p.k + cb;
            if (wide) {
#pragma unroll
              for (int i = 0; i < 32; i += 8)
                if (cb + (uint32_t)i < p.k) stg256(dst + i, v + i);
            } else {
#pragma unroll
              for (int i = 0; i < 32; i += 4)
                if (cb + (uint32_t)i < p.k)
                  *reinterpret_cast<float4*>(dst + i) = make_float4(__uint_as_float(v[i]), __uint_as_float(v[i + 1]),
                                                                    __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.p_free);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(t_p), "r"(512) : "memory");
  }
  if (tid == 0 && sm.ctl.abort && p.flags) atomicOr(p.flags, (uint32_t)SL_FLAG_TIMEOUT);
}

// ------------------------------------------------ compress with embedding terms, two sub-tiles per U slice
// The same pairing for the projection WITH embedding terms: two sub-tiles of 128 tokens share every U slice
// (128 KB instead of 160 KB taken in per K step and 256 tokens).  The gathered T_perp / position segments of
// 256 token rows do not fit the registers of eight row warps, so this form has sixteen: thread j serves the
// 16-byte chunk j % 8 of the rows j / 8 + 64 i (i = 0..3) of the 256-row pair - rows 0..127 are sub-tile A,
// 128..255 sub-tile B - and keeps the values of the next K step in registers while it applies the current
// ones.  Everything else (producers, MMA warp, ring, accumulators in the two halves of tensor memory) is the
// kernel above.
constexpr int kRowWarpsG = 16;
constexpr int kThreadsG = 128 + 32 * kRowWarpsG;

__global__ void __launch_bounds__(kThreadsG, 1)
subspace_project_dual_gather_kernel(const __grid_constant__ ProjMaps maps, const __grid_constant__ SubParams p) {
  extern __shared__ uint8_t raw[];
  DualSmem& sm = *reinterpret_cast<DualSmem*>(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t k_tiles = (p.d + kTileK - 1) / kTileK;
  const uint64_t G = (p.n_tok + 31) / 32;
  const uint64_t g0 = (uint64_t)blockIdx.x * G / gridDim.x, g1 = (uint64_t)(blockIdx.x + 1) * G / gridDim.x;
  auto groups_a = [&](uint64_t g) { return (uint32_t)(g1 - g < 4 ? g1 - g : 4); };
  auto groups_b = [&](uint64_t g) { return g + 4 >= g1 ? 0u : (uint32_t)(g1 - g - 4 < 4 ? g1 - g - 4 : 4); };
  if (tid == 0) {
    for (int s = 0; s < kRingD; ++s) { mbar_init(&sm.full[s], 3); mbar_init(&sm.ready[s], kRowWarpsG); mbar_init(&sm.empty[s], 1); }
    mbar_init(&sm.p_done, 1);
    mbar_init(&sm.p_free, kRowWarpsG);
    mbar_init(&sm.mma_idle, 1);
    sm.ctl.abort = 0;
    sm.ctl.polls = p.wait_polls;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t t_p = sm.tmem_base;      // accumulator of sub-tile A; B is 256 columns further
  bool bad = false;

  if (warp == 0 || warp == 2 || warp == 3) {
    if (lane == 0) {
      const uint32_t pi = warp == 0 ? 0u : (uint32_t)warp - 1u;
      const uint32_t nb = p.kp / 32;
      const uint32_t lo = pi == 0 ? 0u : (pi * nb + 1) / 3, hi = pi == 2 ? nb : ((pi + 1) * nb + 1) / 3;
      uint32_t it = 0;
      bool ok = true;
      for (uint64_t g = g0; ok && g < g1; g += 8) {
        const uint32_t ha = groups_a(g), hb = groups_b(g);
        const int r0 = (int)(g * 32);
        for (uint32_t kt = 0; ok && kt < k_tiles; ++kt, ++it) {
          const uint32_t s = it % kRingD;
          ok = mbar_wait(&sm.empty[s], ((it / kRingD) & 1u) ^ 1u, sm.ctl);
          if (!ok) break;
          uint8_t* slot = sm.ring + s * kSlotD;
          mbar_expect_tx(&sm.full[s], (pi == 0 ? (ha + hb) * 4096 : 0u) + (hi - lo) * 4096);
          if (pi == 0) {
            if (ha == 4) tma_load_2d(slot, &maps.x128, (int)(kt * kTileK), r0, &sm.full[s]);
            else
              for (uint32_t i = 0; i < ha; ++i)
                tma_load_2d(slot + i * 4096, &maps.x32, (int)(kt * kTileK), r0 + 32 * (int)i, &sm.full[s]);
            if (hb == 4) tma_load_2d(slot + kSlotA, &maps.x128, (int)(kt * kTileK), r0 + kRows, &sm.full[s]);
            else
              for (uint32_t i = 0; i < hb; ++i)
                tma_load_2d(slot + kSlotA + i * 4096, &maps.x32, (int)(kt * kTileK), r0 + kRows + 32 * (int)i, &sm.full[s]);
          }
          for (uint32_t n = lo; n < hi; ++n)
            tma_load_2d(slot + 2 * kSlotA + n * 4096, &maps.u_n, (int)(n * 32), (int)(kt * kTileK), &sm.full[s]);
        }
      }
      if (!ok)
        for (uint32_t s = 0; s < (uint32_t)kRingD; ++s) landed(&sm.full[s], ring_uses(it, s, kRingD));
    }
  } else if (warp == 1) {
    if (lane == 0) {
      uint32_t it = 0, t = 0;
      bool ok = true;
      const uint32_t idesc = instr_desc(kRows, (int)p.kp, 1);
      const uint64_t desc_k = smem_desc(0, 16, 1024, 2), desc_n = smem_desc(0, 4096, 512, 1);
      for (uint64_t g = g0; ok && g < g1; g += 8, ++t) {
        const bool two = groups_b(g) != 0;
        if (t > 0) {
          ok = mbar_wait(&sm.p_free, (t - 1) & 1u, sm.ctl);
          if (!ok) break;
          tc_fence_after();
        }
        for (uint32_t kt = 0; ok && kt < k_tiles; ++kt, ++it) {
          const uint32_t s = it % kRingD;
          ok = mbar_wait(&sm.ready[s], (it / kRingD) & 1u, sm.ctl);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a0 = smem_u32(sm.ring + s * kSlotD);
          const uint64_t da = desc_k | (uint64_t)((a0 >> 4) & 0x3FFF);
          const uint64_t da2 = desc_k | (uint64_t)(((a0 + kSlotA) >> 4) & 0x3FFF);
          const uint64_t db = desc_n | (uint64_t)(((a0 + 2 * kSlotA) >> 4) & 0x3FFF);
#pragma unroll
          for (int j = 0; j < 4; ++j) mma_ss(t_p, da + 2 * j, db + 64 * j, idesc, (kt | (uint32_t)j) != 0);
          if (two) {
#pragma unroll
            for (int j = 0; j < 4; ++j) mma_ss(t_p + 256, da2 + 2 * j, db + 64 * j, idesc, (kt | (uint32_t)j) != 0);
          }
          mma_commit(&sm.empty[s]);
        }
        if (ok) mma_commit(&sm.p_done);
      }
      if (!ok) mma_quiesce(&sm.mma_idle);
    }
  } else {
    // ---- sixteen row warps ----
    const uint32_t q = (uint32_t)(warp & 3), sub = (uint32_t)(warp - 4) >> 2;      // sub 0..3: tile sub & 1, column blocks sub >> 1
    const uint32_t row = 32u * q + (uint32_t)lane;
    const uint32_t j = (uint32_t)(tid - 128), gch = j & 7u, grow = j >> 3;          // grow 0..63
    const uint32_t goff = grow * 128 + ((gch ^ (grow & 7u)) << 4);                  // + 8192 i: row grow + 64 i of the pair
    const bool wide = p.k % 8 == 0 && ((uintptr_t)p.out & 31u) == 0;
    uint32_t it = 0, t = 0;
    bool ok = true;
    const float* tp[4];
    const float* ps[4];
    uint32_t mask = 0;
    float4 nt[4], np_[4];                           // the values of the K step after the current one
    auto fetch = [&](uint32_t kt) {
      const uint32_t col = kt * kTileK + 4u * gch;
      const bool in_col = kt < k_tiles && col < p.d;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const bool in = in_col && ((mask >> i) & 1u);
        nt[i] = in ? __ldg(reinterpret_cast<const float4*>(tp[i] + kt * kTileK)) : make_float4(0.f, 0.f, 0.f, 0.f);
        np_[i] = in ? __ldg(reinterpret_cast<const float4*>(ps[i] + kt * kTileK)) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    };
    auto open_tile = [&](uint64_t g) {
      const uint32_t ha = groups_a(g) * 32, hb = groups_b(g) * 32;
      mask = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t r = grow + 64u * (uint32_t)i;                                 // row of the pair
        const RowInfo ri = r < (uint32_t)kRows ? row_info(p, g * 32, ha, r, bad) : row_info(p, g * 32 + kRows, hb, r - kRows, bad);
        tp[i] = ri.gather ? ri.tp + 4 * gch : nullptr;
        ps[i] = ri.gather ? ri.ps + 4 * gch : nullptr;
        mask |= ri.gather ? 1u << i : 0u;
      }
      fetch(0);
    };
    if (g0 < g1) open_tile(g0);
    for (uint64_t g = g0; ok && g < g1; g += 8, ++t) {
      const uint32_t ha = groups_a(g), hb = groups_b(g);
      for (uint32_t kt = 0; ok && kt < k_tiles; ++kt, ++it) {
        float4 ct[4], cp[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) { ct[i] = nt[i]; cp[i] = np_[i]; }
        fetch(kt + 1);
        const uint32_t s = it % kRingD;
        ok = mbar_wait(&sm.full[s], (it / kRingD) & 1u, sm.ctl);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const uint32_t a0 = smem_u32(sm.ring + s * kSlotD) + goff;
#pragma unroll
        for (uint32_t i = 0; i < 4; ++i) {
          if (i < 2 || hb) {                        // rows 128.. exist only with a second sub-tile
            const uint32_t a = a0 + 8192u * i;
            float4 v = lds128(a);
            v.x = __fsub_rn(__fsub_rn(v.x, ct[i].x), cp[i].x);
            v.y = __fsub_rn(__fsub_rn(v.y, ct[i].y), cp[i].y);
            v.z = __fsub_rn(__fsub_rn(v.z, ct[i].z), cp[i].z);
            v.w = __fsub_rn(__fsub_rn(v.w, ct[i].w), cp[i].w);
            v.x = __uint_as_float(round_tf32(__float_as_uint(v.x)));
            v.y = __uint_as_float(round_tf32(__float_as_uint(v.y)));
            v.z = __uint_as_float(round_tf32(__float_as_uint(v.z)));
            v.w = __uint_as_float(round_tf32(__float_as_uint(v.w)));
            sts128(a, v);
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.ready[s]);
      }
      if (!ok) break;
      if (g + 8 < g1) open_tile(g + 8);
      ok = mbar_wait(&sm.p_done, t & 1u, sm.ctl);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      {
        const uint32_t tile = sub & 1u;
        const uint32_t h = (tile ? hb : ha) * 32;
        const uint64_t r0 = g * 32 + (uint64_t)tile * kRows;
        if (h) {
          for (uint32_t cb = 32u * (sub >> 1); cb < p.kp; cb += 64) {
            uint32_t v[32];
            tmem_ld32(t_p + tile * 256 + cb + ((32u * q) << 16), v);
            tmem_ld_wait();
            if (row < h && r0 + row < p.n_tok) {
              float* dst = p.out + (r0 + row) * (uint64_t)p.k + cb;
              if (wide) {
#pragma unroll
                for (int i = 0; i < 32; i += 8)
                  if (cb + (uint32_t)i < p.k) stg256(dst + i, v + i);
              } else {
#pragma unroll
                for (int i = 0; i < 32; i += 4)
                  if (cb + (uint32_t)i < p.k)
                    *reinterpret_cast<float4*>(dst + i) = make_float4(__uint_as_float(v[i]), __uint_as_float(v[i + 1]),
                                                                      __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.p_free);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(t_p), "r"(512) : "memory");
  }
  if (bad && p.flags) atomicOr(p.flags, (uint32_t)SL_FLAG_BAD_INDEX);
  if (tid == 0 && sm.ctl.abort && p.flags) atomicOr(p.flags, (uint32_t)SL_FLAG_TIMEOUT);
}

// --------------------------- the same when the batch is a whole number of PAIRS of sequences of L tokens
// (L a multiple of 32): sub-tile B is not the 128 tokens after sub-tile A but the same positions of the next
// sequence, L tokens on, so that row r of B has the position row of row r of A and a thread fetches it once
// for both (a quarter less to gather; 0.222 -> 0.213 ms at 64K tokens).  The work is dealt in units of 32
// positions x 2 sequences, up to four units to a pass; a pass may cross from one pair of sequences to the
// next, its tiles then come in as boxes of 32 rows.
struct PairPass {
  uint64_t c;               // where the pass starts in the CTA's range of units
  uint32_t h;               // its units: groups of 32 tokens in A and in B
};
struct PairSched {
  uint64_t lo, hi, L;
  uint32_t per;             // units in a sequence
  __device__ __forceinline__ PairSched(const SubParams& p) {
    L = p.L;
    per = p.L / 32;
    const uint64_t n = (p.n_tok / (2 * (uint64_t)p.L)) * per;
    lo = (uint64_t)blockIdx.x * n / gridDim.x;
    hi = (uint64_t)(blockIdx.x + 1) * n / gridDim.x;
  }
  // the pass that starts at c (false: none); next = where the one after it starts
  __device__ __forceinline__ bool at(uint64_t c, PairPass& ps, uint64_t& next) const {
    if (c >= hi) return false;
    const uint64_t left = hi - c;
    ps.c = c;
    ps.h = (uint32_t)(left < 4 ? left : 4);
    next = c + ps.h;
    return true;
  }
  // first token of group j of sub-tile A / B
  __device__ __forceinline__ uint64_t ta(uint64_t c, uint32_t j) const {
    const uint32_t u = (uint32_t)c + j, sp = u / per;              // (the host checks that the units fit 32 bits)
    return (uint64_t)sp * 2 * L + (uint64_t)(u - sp * per) * 32;
  }
  __device__ __forceinline__ uint64_t tb(uint64_t c, uint32_t j) const { return ta(c, j) + L; }
  // the four groups of a sub-tile are 128 consecutive tokens
  __device__ __forceinline__ bool whole(const PairPass& ps) const { return ps.h == 4 && (uint32_t)ps.c % per + 3 < per; }
};

__global__ void __launch_bounds__(kThreadsG, 1)
subspace_project_dual_samepos_kernel(const __grid_constant__ ProjMaps maps, const __grid_constant__ SubParams p) {
  extern __shared__ uint8_t raw[];
  DualSmem& sm = *reinterpret_cast<DualSmem*>(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t k_tiles = (p.d + kTileK - 1) / kTileK;
  const PairSched sc(p);
  if (tid == 0) {
    for (int s = 0; s < kRingD; ++s) { mbar_init(&sm.full[s], 3); mbar_init(&sm.ready[s], kRowWarpsG); mbar_init(&sm.empty[s], 1); }
    mbar_init(&sm.p_done, 1);
    mbar_init(&sm.p_free, kRowWarpsG);
    mbar_init(&sm.mma_idle, 1);
    sm.ctl.abort = 0;
    sm.ctl.polls = p.wait_polls;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t t_p = sm.tmem_base;      // accumulator of sub-tile A; B is 256 columns further
  bool bad = false;

  if (warp == 0 || warp == 2 || warp == 3) {
    if (lane == 0) {
      const uint32_t pi = warp == 0 ? 0u : (uint32_t)warp - 1u;
      const uint32_t nb = p.kp / 32;
      const uint32_t lo = pi == 0 ? 0u : (pi * nb + 1) / 3, hi = pi == 2 ? nb : ((pi + 1) * nb + 1) / 3;
      uint32_t it = 0;
      bool ok = true;
      PairPass ps;
      for (uint64_t c = sc.lo, cn; ok && sc.at(c, ps, cn); c = cn) {
        const uint32_t ha = ps.h, hb = ps.h;
        const bool wa = sc.whole(ps), wb = wa;
        int ra[4], rb[4];
#pragma unroll
        for (uint32_t i = 0; i < 4; ++i) { ra[i] = (int)sc.ta(ps.c, i); rb[i] = (int)sc.tb(ps.c, i); }
        for (uint32_t kt = 0; ok && kt < k_tiles; ++kt, ++it) {
          const uint32_t s = it % kRingD;
          ok = mbar_wait(&sm.empty[s], ((it / kRingD) & 1u) ^ 1u, sm.ctl);
          if (!ok) break;
          uint8_t* slot = sm.ring + s * kSlotD;
          mbar_expect_tx(&sm.full[s], (pi == 0 ? (ha + hb) * 4096 : 0u) + (hi - lo) * 4096);
          if (pi == 0) {
            if (wa) tma_load_2d(slot, &maps.x128, (int)(kt * kTileK), ra[0], &sm.full[s]);
            else {
#pragma unroll
              for (uint32_t i = 0; i < 4; ++i)
                if (i < ha) tma_load_2d(slot + i * 4096, &maps.x32, (int)(kt * kTileK), ra[i], &sm.full[s]);
            }
            if (wb) tma_load_2d(slot + kSlotA, &maps.x128, (int)(kt * kTileK), rb[0], &sm.full[s]);
            else {
#pragma unroll
              for (uint32_t i = 0; i < 4; ++i)
                if (i < hb) tma_load_2d(slot + kSlotA + i * 4096, &maps.x32, (int)(kt * kTileK), rb[i], &sm.full[s]);
            }
          }
          for (uint32_t n = lo; n < hi; ++n)
            tma_load_2d(slot + 2 * kSlotA + n * 4096, &maps.u_n, (int)(n * 32), (int)(kt * kTileK), &sm.full[s]);
        }
      }
      if (!ok)
        for (uint32_t s = 0; s < (uint32_t)kRingD; ++s) landed(&sm.full[s], ring_uses(it, s, kRingD));
    }
  } else if (warp == 1) {
    if (lane == 0) {
      uint32_t it = 0, t = 0;
      bool ok = true;
      const uint32_t idesc = instr_desc(kRows, (int)p.kp, 1);
      const uint64_t desc_k = smem_desc(0, 16, 1024, 2), desc_n = smem_desc(0, 4096, 512, 1);
      PairPass ps;
      for (uint64_t c = sc.lo, cn; ok && sc.at(c, ps, cn); c = cn, ++t) {
        if (t > 0) {
          ok = mbar_wait(&sm.p_free, (t - 1) & 1u, sm.ctl);
          if (!ok) break;
          tc_fence_after();
        }
        for (uint32_t kt = 0; ok && kt < k_tiles; ++kt, ++it) {
          const uint32_t s = it % kRingD;
          ok = mbar_wait(&sm.ready[s], (it / kRingD) & 1u, sm.ctl);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a0 = smem_u32(sm.ring + s * kSlotD);
          const uint64_t da = desc_k | (uint64_t)((a0 >> 4) & 0x3FFF);
          const uint64_t da2 = desc_k | (uint64_t)(((a0 + kSlotA) >> 4) & 0x3FFF);
          const uint64_t db = desc_n | (uint64_t)(((a0 + 2 * kSlotA) >> 4) & 0x3FFF);
#pragma unroll
          for (int j = 0; j < 4; ++j) mma_ss(t_p, da + 2 * j, db + 64 * j, idesc, (kt | (uint32_t)j) != 0);
#pragma unroll
          for (int j = 0; j < 4; ++j) mma_ss(t_p + 256, da2 + 2 * j, db + 64 * j, idesc, (kt | (uint32_t)j) != 0);
          mma_commit(&sm.empty[s]);
        }
        if (ok) mma_commit(&sm.p_done);
      }
      if (!ok) mma_quiesce(&sm.mma_idle);
    }
  } else {
    // ---- sixteen row warps ----
    const uint32_t q = (uint32_t)(warp & 3), sub = (uint32_t)(warp - 4) >> 2;      // sub 0..3: tile sub & 1, column blocks sub >> 1
    const uint32_t row = 32u * q + (uint32_t)lane;
    const uint32_t j = (uint32_t)(tid - 128), gch = j & 7u, grow = j >> 3;          // grow 0..63
    const uint32_t goff = grow * 128 + ((gch ^ (grow & 7u)) << 4);                  // + 8192 i: row grow + 64 i of the pair
    const bool wide = p.k % 8 == 0 && ((uintptr_t)p.out & 31u) == 0;
    uint32_t it = 0, t = 0;
    bool ok = true;
    const float* tp[4];
    const float* ps[2];
    uint32_t mask = 0;
    constexpr int kPosRows = 2;                     // rows i and i + 2 of a thread share their position row
    float4 nt[4], np_[kPosRows];                    // the values of the K step after the current one
    auto fetch = [&](uint32_t kt) {
      const uint32_t col = kt * kTileK + 4u * gch;
      const bool in_col = kt < k_tiles && col < p.d;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const bool in = in_col && ((mask >> i) & 1u);
        nt[i] = in ? __ldg(reinterpret_cast<const float4*>(tp[i] + kt * kTileK)) : make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < kPosRows) {
          const bool inp = in_col && ((mask >> (4 + i)) & 1u);
          np_[i] = inp ? __ldg(reinterpret_cast<const float4*>(ps[i] + kt * kTileK)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
    };
    // mask bit i: row i has terms.  The position row of rows i and i + 2 is fetched once, under bit 4 + i,
    // when either of them has terms (a token id out of range leaves only its own row without)
    auto open_tile = [&](const PairPass& pp) {
      mask = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t r = (grow + 64u * (uint32_t)i) & 127u, gj = r >> 5;             // row of its sub-tile, its group
        const bool in_b = i >= 2;
        const RowInfo ri = row_info(p, in_b ? sc.tb(pp.c, gj) : sc.ta(pp.c, gj), pp.h > gj ? 32u : 0u, r & 31u, bad);
        tp[i] = ri.gather ? ri.tp + 4 * gch : nullptr;
        mask |= ri.gather ? 1u << i : 0u;
        if (ri.gather) { ps[i & 1] = ri.ps + 4 * gch; mask |= 16u << (i & 1); }
      }
      fetch(0);
    };
    // only where the pass starts is carried through the loop; what it covers is worked out again where needed
    uint64_t c = sc.lo;
    {
      PairPass first;
      uint64_t cn;
      if (sc.at(c, first, cn)) open_tile(first);
    }
    for (; ok && c < sc.hi; ++t) {
      PairPass cur;
      uint64_t cn;
      sc.at(c, cur, cn);
      for (uint32_t kt = 0; ok && kt < k_tiles; ++kt, ++it) {
        float4 ct[4], cp[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          ct[i] = nt[i];
          cp[i] = (mask >> i) & 1u ? np_[i & 1] : make_float4(0.f, 0.f, 0.f, 0.f);       // (none for a row without terms)
        }
        fetch(kt + 1);
        const uint32_t s = it % kRingD;
        ok = mbar_wait(&sm.full[s], (it / kRingD) & 1u, sm.ctl);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const uint32_t a0 = smem_u32(sm.ring + s * kSlotD) + goff;
#pragma unroll
        for (uint32_t i = 0; i < 4; ++i) {
          {
            const uint32_t a = a0 + 8192u * i;
            float4 v = lds128(a);
            v.x = __fsub_rn(__fsub_rn(v.x, ct[i].x), cp[i].x);
            v.y = __fsub_rn(__fsub_rn(v.y, ct[i].y), cp[i].y);
            v.z = __fsub_rn(__fsub_rn(v.z, ct[i].z), cp[i].z);
            v.w = __fsub_rn(__fsub_rn(v.w, ct[i].w), cp[i].w);
            v.x = __uint_as_float(round_tf32(__float_as_uint(v.x)));
            v.y = __uint_as_float(round_tf32(__float_as_uint(v.y)));
            v.z = __uint_as_float(round_tf32(__float_as_uint(v.z)));
            v.w = __uint_as_float(round_tf32(__float_as_uint(v.w)));
            sts128(a, v);
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.ready[s]);
      }
      if (!ok) break;
      {
        PairPass nxt;
        uint64_t cnn;
        if (sc.at(cn, nxt, cnn)) open_tile(nxt);
      }
      ok = mbar_wait(&sm.p_done, t & 1u, sm.ctl);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      {
        const uint32_t tile = sub & 1u;
        const uint32_t h = cur.h * 32;
        const uint64_t tok = (tile ? sc.tb(cur.c, q) : sc.ta(cur.c, q)) + (uint64_t)lane;   // row = 32 q + lane: group q of the sub-tile
        if (h) {
          for (uint32_t cb = 32u * (sub >> 1); cb < p.kp; cb += 64) {
            uint32_t v[32];
            tmem_ld32(t_p + tile * 256 + cb + ((32u * q) << 16), v);
            tmem_ld_wait();
            if (row < h && tok < p.n_tok) {
              float* dst = p.out + tok * (uint64_t)p.k + cb;
              if (wide) {
#pragma unroll
                for (int i = 0; i < 32; i += 8)
                  if (cb + (uint32_t)i < p.k) stg256(dst + i, v + i);
              } else {
#pragma unroll
                for (int i = 0; i < 32; i += 4)
                  if (cb + (uint32_t)i < p.k)
                    *reinterpret_cast<float4*>(dst + i) = make_float4(__uint_as_float(v[i]), __uint_as_float(v[i + 1]),
                                                                      __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.p_free);
      c = cn;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(t_p), "r"(512) : "memory");
  }
  if (bad && p.flags) atomicOr(p.flags, (uint32_t)SL_FLAG_BAD_INDEX);
  if (tid == 0 && sm.ctl.abort && p.flags) atomicOr(p.flags, (uint32_t)SL_FLAG_TIMEOUT);
}

// --------------------------------------------------------------------------------------- reconstruct
// Per sub-tile of 128 tokens the Xt tile goes through a two-slot staging buffer into tensor memory
// (rounded to TF32 on the way) and is the A operand of every 128-column block.  The embedding and
// position rows of a 32-column part are gathered into a stage of shared memory by 16-byte
// asynchronous copies, several parts ahead of their use (whole 128-byte segments per row, so every
// line is fetched by one request); the epilogue adds them to the accumulator part in place and a
// tensor-map store writes the finished part.  Warps: 0 operand TMA, 1 MMA, 2 part store,
// 3..6 Xt staging -> tensor memory and the gathers, 7..10 epilogue.
constexpr int kSlotB = kBlockN * kTileK * 4;          // 16 KB: 128 rows of U x 32 columns
constexpr int kRingB = 4;                             // slots of the U ring (a power of two: the roles index it with % and /)
constexpr int kStages = 4;                            // gather / output stages
constexpr int kStageA = 2;                            // staging slots of the Xt tile
struct ReconSmem {
  uint8_t ring[kRingB][kSlotB];
  uint8_t st_t[kStages][kSlotA];                      // gathered T_perp segments of a part, then the finished part
  uint8_t st_p[kStages][kSlotA];                      // gathered position segments
  uint8_t a[kStageA][kSlotA];
  uint64_t full[kRingB], empty[kRingB], o_full[2], o_empty[2];
  uint64_t a_full[kStageA], a_empty[kStageA], a_ready, a_free;
  uint64_t g_full[kStages], g_done[kStages], g_empty[kStages];
  uint64_t t_free[kStages];                            // the epilogue has read the stage's T_perp segments
  uint64_t mma_idle;        // after a give-up only: the MMAs issued so far have retired
  uint32_t tmem_base;
  WaitCtl ctl;
};
struct ReconMaps { CUtensorMap xt128, xt32, u_k, o128, o32; };

constexpr int kReconThreads = 352;

__device__ __forceinline__ void cp_async_16z(uint32_t dst, const void* src, uint32_t bytes) {   // bytes 0: zero fill
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}

__global__ void __launch_bounds__(kReconThreads, 1)
subspace_reconstruct_kernel(const __grid_constant__ ReconMaps maps, const __grid_constant__ SubParams p) {
  extern __shared__ uint8_t raw[];
  ReconSmem& sm = *reinterpret_cast<ReconSmem*>(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t k_tiles = p.kp / kTileK;
  const uint32_t n_blocks = (p.d + kBlockN - 1) / kBlockN;
  const uint64_t G = (p.n_tok + 31) / 32;
  const Sched sc(n_blocks, G);
  if (tid == 0) {
    for (int s = 0; s < kRingB; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&sm.o_full[b], 1); mbar_init(&sm.o_empty[b], 4); }
    for (int s = 0; s < kStageA; ++s) { mbar_init(&sm.a_full[s], 1); mbar_init(&sm.a_empty[s], 4); }
    mbar_init(&sm.a_ready, 4);
    mbar_init(&sm.a_free, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.g_full[s], 128); mbar_init(&sm.g_done[s], 4); mbar_init(&sm.g_empty[s], 1); mbar_init(&sm.t_free[s], 4);
    }
    mbar_init(&sm.mma_idle, 1);
    sm.ctl.abort = 0;
    sm.ctl.polls = p.wait_polls;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t t_a = sm.tmem_base;            // the Xt tile: 128 lanes x kp columns
  const uint32_t t_o = sm.tmem_base + 256;      // two accumulators of 128 columns
  bool bad = false;
  // 32-column parts of block c that lie inside the matrix
  auto parts_of = [&](uint32_t c) { const uint32_t left = p.d - c * kBlockN; return left >= (uint32_t)kBlockN ? 4u : (left + 31u) / 32u; };

  if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 0, ia = 0;
      bool ok = true;
      for (uint32_t pi = 0; ok && pi < sc.n_pieces; ++pi) {
        const Piece pc = sc.piece(pi);
        const uint32_t hg = pc.hg, h = hg * 32;
        const int r0 = (int)pc.r0;
        for (uint32_t kt = 0; ok && kt < k_tiles; ++kt, ++ia) {
          const uint32_t s = ia % kStageA;
          ok = mbar_wait(&sm.a_empty[s], ((ia / kStageA) & 1u) ^ 1u, sm.ctl);
          if (!ok) break;
          mbar_expect_tx(&sm.a_full[s], h * 128);
          if (hg == 4) tma_load_2d(sm.a[s], &maps.xt128, (int)(kt * kTileK), r0, &sm.a_full[s]);
          else
            for (uint32_t i = 0; i < hg; ++i)
              tma_load_2d(sm.a[s] + i * 4096, &maps.xt32, (int)(kt * kTileK), r0 + 32 * (int)i, &sm.a_full[s]);
        }
        for (uint32_t ci = 0; ok && ci < pc.n; ++ci)
          for (uint32_t kt = 0; kt < k_tiles; ++kt, ++it) {
            const uint32_t s = it % kRingB;
            ok = mbar_wait(&sm.empty[s], ((it / kRingB) & 1u) ^ 1u, sm.ctl);
            if (!ok) break;
            mbar_expect_tx(&sm.full[s], kSlotB);
            tma_load_2d(sm.ring[s], &maps.u_k, (int)(kt * kTileK), (int)(pc.block(ci) * kBlockN), &sm.full[s]);
          }
      }
      if (!ok) {
        for (uint32_t s = 0; s < (uint32_t)kRingB; ++s) landed(&sm.full[s], ring_uses(it, s, kRingB));
        for (uint32_t s = 0; s < (uint32_t)kStageA; ++s) landed(&sm.a_full[s], ring_uses(ia, s, kStageA));
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      uint32_t it = 0, cg = 0, t = 0;
      bool ok = true;
      const uint32_t idesc = instr_desc(kRows, kBlockN, 0);
      const uint64_t desc_k = smem_desc(0, 16, 1024, 2);
      for (uint32_t pi = 0; ok && pi < sc.n_pieces; ++pi, ++t) {
        const Piece pc = sc.piece(pi);
        ok = mbar_wait(&sm.a_ready, t & 1u, sm.ctl);          // the tile is in tensor memory, rounded
        if (!ok) break;
        tc_fence_after();
        for (uint32_t c = 0; ok && c < pc.n; ++c, ++cg) {
          const uint32_t buf = cg & 1u, u = cg >> 1;
          if (u) {
            ok = mbar_wait(&sm.o_empty[buf], (u - 1) & 1u, sm.ctl);
            if (!ok) break;
            tc_fence_after();
          }
          for (uint32_t kt = 0; kt < k_tiles; ++kt, ++it) {
            const uint32_t s = it % kRingB;
            ok = mbar_wait(&sm.full[s], (it / kRingB) & 1u, sm.ctl);
            if (!ok) break;
            tc_fence_after();
            const uint64_t db = desc_k | (uint64_t)((smem_u32(sm.ring[s]) >> 4) & 0x3FFF);
#pragma unroll
            for (int j = 0; j < 4; ++j)
              mma_ts(t_o + buf * kBlockN, t_a + kt * kTileK + 8 * j, db + 2 * j, idesc, (kt | (uint32_t)j) != 0);
            mma_commit(&sm.empty[s]);
          }
          if (!ok) break;
          mma_commit(&sm.o_full[buf]);
        }
        if (ok) mma_commit(&sm.a_free);
      }
      if (!ok) mma_quiesce(&sm.mma_idle);
    }
  } else if (warp == 2) {
    // ---- part store: a finished part leaves by tensor-map store; its stage is free once the store has read it ----
    if (lane == 0) {
      uint32_t is = 0;
      bool ok = true;
      for (uint32_t pi = 0; ok && pi < sc.n_pieces; ++pi) {
        const Piece pc = sc.piece(pi);
        const uint32_t hg = pc.hg;
        const int r0 = (int)pc.r0;
        for (uint32_t ci = 0; ok && ci < pc.n; ++ci) {
          const uint32_t c = pc.block(ci), np = parts_of(c);
          for (uint32_t part = 0; part < np; ++part, ++is) {
            const uint32_t s = is % kStages;
            ok = mbar_wait(&sm.g_done[s], (is / kStages) & 1u, sm.ctl);
            if (!ok) break;
            const int col0 = (int)(c * kBlockN + part * 32);
            const uint32_t src = smem_u32(sm.st_p[s]);        // the finished part sits in the position stage
            if (hg == 4) tma_store_2d(&maps.o128, col0, r0, src);
            else
              for (uint32_t i = 0; i < hg; ++i) tma_store_2d(&maps.o32, col0, r0 + 32 * (int)i, src + i * 4096);
            bulk_commit();
            bulk_wait_read_all();
            mbar_arrive(&sm.g_empty[s]);
          }
        }
      }
      bulk_wait_all();
    }
  } else if (warp < 7) {
    // ---- staging warps: Xt tile -> tensor memory (thread = lane of its 32-lane window), then the gathers ----
    const uint32_t q = (uint32_t)(warp & 3);
    const uint32_t row = 32u * q + (uint32_t)lane;
    const uint32_t gt = (uint32_t)(tid - 96), gch = gt & 7u, grow = gt >> 3;   // gather: 8 threads per 128-byte segment
    uint32_t ia = 0, ig = 0, t = 0;
    bool ok = true;
    for (uint32_t pi = 0; ok && pi < sc.n_pieces; ++pi, ++t) {
      const Piece pc = sc.piece(pi);
      const uint32_t hg = pc.hg, h = hg * 32;
      const uint64_t r0 = pc.r0;
      // the eight rows this thread gathers for: row grow + 16 i
      const float* tp[8];
      const float* ps[8];
      uint32_t mask = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const RowInfo ri = row_info(p, r0, h, grow + 16u * (uint32_t)i, bad);
        tp[i] = ri.gather ? ri.tp + 4 * gch : p.T_perp;
        ps[i] = ri.gather ? ri.ps + 4 * gch : p.pos;
        mask |= ri.gather ? 1u << i : 0u;
      }
      if (t > 0) {                                   // the MMAs of the previous sub-tile have read the old tile
        ok = mbar_wait(&sm.a_free, (t - 1) & 1u, sm.ctl);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
      }
      for (uint32_t kt = 0; kt < k_tiles; ++kt, ++ia) {
        const uint32_t s = ia % kStageA;
        ok = mbar_wait(&sm.a_full[s], (ia / kStageA) & 1u, sm.ctl);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        uint32_t v[32];
        const uint32_t a0 = smem_u32(sm.a[s]) + row * 128;
#pragma unroll
        for (uint32_t ch = 0; ch < 8; ++ch) {
          const float4 f = lds128(a0 + ((ch ^ (row & 7u)) << 4));
          v[4 * ch + 0] = round_tf32(__float_as_uint(f.x));
          v[4 * ch + 1] = round_tf32(__float_as_uint(f.y));
          v[4 * ch + 2] = round_tf32(__float_as_uint(f.z));
          v[4 * ch + 3] = round_tf32(__float_as_uint(f.w));
        }
        tmem_st32(t_a + kt * kTileK + ((32u * q) << 16), v);
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.a_empty[s]);
      }
      if (!ok) break;
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.a_ready);
      for (uint32_t ci = 0; ok && ci < pc.n; ++ci) {
        const uint32_t c = pc.block(ci), np = parts_of(c);
        for (uint32_t part = 0; part < np; ++part, ++ig) {
          const uint32_t s = ig % kStages;
          const uint32_t col0 = c * kBlockN + part * 32;
          const bool in_col = col0 + 4 * gch < p.d;
          const uint32_t dt = smem_u32(sm.st_t[s]), dp = smem_u32(sm.st_p[s]);
          // the T_perp half of the stage is free as soon as the epilogue has read it - the finished part waits
          // for its store in the position half - so the gathers that come from DRAM start one store earlier
          ok = mbar_wait(&sm.t_free[s], ((ig / kStages) & 1u) ^ 1u, sm.ctl);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          if (p.ids) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const uint32_t r = grow + 16u * (uint32_t)i;
              const uint32_t off = r * 128 + ((gch ^ (r & 7u)) << 4);
              const bool in = in_col && ((mask >> i) & 1u);
              cp_async_16z(dt + off, in ? (const void*)(tp[i] + col0) : (const void*)p.T_perp, in ? 16u : 0u);
            }
          }
          ok = mbar_wait(&sm.g_empty[s], ((ig / kStages) & 1u) ^ 1u, sm.ctl);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          if (p.ids) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const uint32_t r = grow + 16u * (uint32_t)i;
              const uint32_t off = r * 128 + ((gch ^ (r & 7u)) << 4);
              const bool in = in_col && ((mask >> i) & 1u);
              cp_async_16z(dp + off, in ? (const void*)(ps[i] + col0) : (const void*)p.pos, in ? 16u : 0u);
            }
          }
          asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(&sm.g_full[s])) : "memory");
        }
      }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
  } else {
    // ---- epilogue warps: accumulator part + gathered rows, in place in the stage ----
    const uint32_t q = (uint32_t)(warp & 3);
    const uint32_t row = 32u * q + (uint32_t)lane;
    const uint32_t roff = row * 128, sw = row & 7u;
    const bool add = p.ids != nullptr;
    uint32_t cg = 0, ie = 0;
    bool ok = true;
    for (uint32_t pi = 0; ok && pi < sc.n_pieces; ++pi) {
      const Piece pc = sc.piece(pi);
      for (uint32_t ci = 0; ok && ci < pc.n; ++ci, ++cg) {
        const uint32_t buf = cg & 1u;
        ok = mbar_wait(&sm.o_full[buf], (cg >> 1) & 1u, sm.ctl);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const uint32_t np = parts_of(pc.block(ci));
        for (uint32_t part = 0; part < np; ++part, ++ie) {
          const uint32_t s = ie % kStages;
          uint32_t v[32];
          tmem_ld32(t_o + buf * kBlockN + part * 32 + ((32u * q) << 16), v);
          ok = mbar_wait(&sm.g_full[s], (ie / kStages) & 1u, sm.ctl);
          ok = __all_sync(0xffffffffu, ok);
          tmem_ld_wait();
          if (!ok) break;
          const uint32_t bt = smem_u32(sm.st_t[s]) + roff, bp = smem_u32(sm.st_p[s]) + roff;
#pragma unroll
          for (uint32_t ch = 0; ch < 8; ++ch) {
            const uint32_t o = (ch ^ sw) << 4;
            float4 r = make_float4(__uint_as_float(v[4 * ch]), __uint_as_float(v[4 * ch + 1]), __uint_as_float(v[4 * ch + 2]),
                                   __uint_as_float(v[4 * ch + 3]));
            if (add) {
              const float4 e = lds128(bt + o), f = lds128(bp + o);
              r.x = __fadd_rn(__fadd_rn(r.x, e.x), f.x);
              r.y = __fadd_rn(__fadd_rn(r.y, e.y), f.y);
              r.z = __fadd_rn(__fadd_rn(r.z, e.z), f.z);
              r.w = __fadd_rn(__fadd_rn(r.w, e.w), f.w);
            }
            sts128(bp + o, r);                     // the finished part replaces the position segment it used
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) { mbar_arrive(&sm.t_free[s]); mbar_arrive(&sm.g_done[s]); }
        }
        if (!ok) break;
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.o_empty[buf]);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(sm.tmem_base), "r"(512) : "memory");
  }
  if (bad && p.flags) atomicOr(p.flags, (uint32_t)SL_FLAG_BAD_INDEX);
  if (tid == 0 && sm.ctl.abort && p.flags) atomicOr(p.flags, (uint32_t)SL_FLAG_TIMEOUT);
}

// ------------------------------------------------------------ reconstruct without embedding terms
// Ghat = Gt U^T (activation gradients on their way back).  With nothing to gather, the launch above is bound
// by the pace at which ONE thread can wait for a slot of U, issue its four MMAs and commit (a TF32 MMA covers
// K = 8 only), and the shared memory of the position stages lies idle.  So this form has two MMA-issuing
// warps, each with its own four-slot ring of U (the second ring in the idle stages), its own producer warp
// and its own accumulator: warp m takes the 128-column blocks whose running number is m modulo 2 and writes
// accumulator m, so the double buffer of the accumulators is also the split of the work.  The epilogue
// takes the blocks in their order, as before.  Warps: 0 Xt tiles + ring 0, 1 MMA (even blocks), 2 part
// store, 3..6 Xt staging -> tensor memory, 7..10 epilogue, 11 MMA (odd blocks), 12 ring 1.
struct GradSmem {
  uint8_t ring[2][kRingB][kSlotB];
  uint8_t st[kStages][kSlotA];                        // finished parts on their way out
  uint8_t a[kStageA][kSlotA];
  uint64_t full[2][kRingB], empty[2][kRingB], o_full[2], o_empty[2];
  uint64_t a_full[kStageA], a_empty[kStageA], a_ready, a_free;
  uint64_t g_done[kStages], g_empty[kStages];
  uint64_t mma_idle[2];
  uint32_t tmem_base;
  WaitCtl ctl;
};
constexpr int kGradThreads = 416;

__global__ void __launch_bounds__(kGradThreads, 1)
subspace_reconstruct_grad_kernel(const __grid_constant__ ReconMaps maps, const __grid_constant__ SubParams p) {
  extern __shared__ uint8_t raw[];
  GradSmem& sm = *reinterpret_cast<GradSmem*>(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t k_tiles = p.kp / kTileK;
  const uint32_t n_blocks = (p.d + kBlockN - 1) / kBlockN;
  const uint64_t G = (p.n_tok + 31) / 32;
  const Sched sc(n_blocks, G);
  if (tid == 0) {
    for (int m = 0; m < 2; ++m)
      for (int s = 0; s < kRingB; ++s) { mbar_init(&sm.full[m][s], 1); mbar_init(&sm.empty[m][s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&sm.o_full[b], 1); mbar_init(&sm.o_empty[b], 4); mbar_init(&sm.mma_idle[b], 1); }
    for (int s = 0; s < kStageA; ++s) { mbar_init(&sm.a_full[s], 1); mbar_init(&sm.a_empty[s], 4); }
    mbar_init(&sm.a_ready, 4);
    mbar_init(&sm.a_free, 2);                         // both MMA warps are through with the tile
    for (int s = 0; s < kStages; ++s) { mbar_init(&sm.g_done[s], 4); mbar_init(&sm.g_empty[s], 1); }
    sm.ctl.abort = 0;
    sm.ctl.polls = p.wait_polls;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t t_a = sm.tmem_base;            // the Xt tile: 128 lanes x kp columns
  const uint32_t t_o = sm.tmem_base + 256;      // two accumulators of 128 columns
  auto parts_of = [&](uint32_t c) { const uint32_t left = p.d - c * kBlockN; return left >= (uint32_t)kBlockN ? 4u : (left + 31u) / 32u; };

  if (warp == 0 || warp == 12) {
    // ---- producers: warp 0 the Xt tiles and the U slots of the even blocks, warp 12 those of the odd blocks ----
    if (lane == 0) {
      const uint32_t m = warp == 0 ? 0u : 1u;
      uint32_t it = 0, ia = 0, cg = 0;
      bool ok = true;
      for (uint32_t pi = 0; ok && pi < sc.n_pieces; ++pi) {
        const Piece pc = sc.piece(pi);
        const uint32_t hg = pc.hg, h = hg * 32;
        const int r0 = (int)pc.r0;
        if (m == 0) {
          for (uint32_t kt = 0; ok && kt < k_tiles; ++kt, ++ia) {
            const uint32_t s = ia % kStageA;
            ok = mbar_wait(&sm.a_empty[s], ((ia / kStageA) & 1u) ^ 1u, sm.ctl);
            if (!ok) break;
            mbar_expect_tx(&sm.a_full[s], h * 128);
            if (hg == 4) tma_load_2d(sm.a[s], &maps.xt128, (int)(kt * kTileK), r0, &sm.a_full[s]);
            else
              for (uint32_t i = 0; i < hg; ++i)
                tma_load_2d(sm.a[s] + i * 4096, &maps.xt32, (int)(kt * kTileK), r0 + 32 * (int)i, &sm.a_full[s]);
          }
        }
        for (uint32_t ci = 0; ok && ci < pc.n; ++ci, ++cg) {
          if ((cg & 1u) != m) continue;
          for (uint32_t kt = 0; kt < k_tiles; ++kt, ++it) {
            const uint32_t s = it % kRingB;
            ok = mbar_wait(&sm.empty[m][s], ((it / kRingB) & 1u) ^ 1u, sm.ctl);
            if (!ok) break;
            mbar_expect_tx(&sm.full[m][s], kSlotB);
            tma_load_2d(sm.ring[m][s], &maps.u_k, (int)(kt * kTileK), (int)(pc.block(ci) * kBlockN), &sm.full[m][s]);
          }
        }
      }
      if (!ok) {
        for (uint32_t s = 0; s < (uint32_t)kRingB; ++s) landed(&sm.full[m][s], ring_uses(it, s, kRingB));
        if (m == 0)
          for (uint32_t s = 0; s < (uint32_t)kStageA; ++s) landed(&sm.a_full[s], ring_uses(ia, s, kStageA));
      }
    }
  } else if (warp == 1 || warp == 11) {
    // ---- two MMA issuers: warp 1 the blocks with an even running number (accumulator 0), warp 11 the odd ones ----
    if (lane == 0) {
      const uint32_t m = warp == 1 ? 0u : 1u;
      uint32_t it = 0, cg = 0, t = 0, mine = 0;
      bool ok = true;
      const uint32_t idesc = instr_desc(kRows, kBlockN, 0);
      const uint64_t desc_k = smem_desc(0, 16, 1024, 2);
      for (uint32_t pi = 0; ok && pi < sc.n_pieces; ++pi, ++t) {
        const Piece pc = sc.piece(pi);
        ok = mbar_wait(&sm.a_ready, t & 1u, sm.ctl);          // the tile is in tensor memory, rounded
        if (!ok) break;
        tc_fence_after();
        for (uint32_t c = 0; ok && c < pc.n; ++c, ++cg) {
          if ((cg & 1u) != m) continue;
          if (mine) {                                          // the epilogue has read this accumulator's previous block
            ok = mbar_wait(&sm.o_empty[m], (mine - 1) & 1u, sm.ctl);
            if (!ok) break;
            tc_fence_after();
          }
          ++mine;
          for (uint32_t kt = 0; kt < k_tiles; ++kt, ++it) {
            const uint32_t s = it % kRingB;
            ok = mbar_wait(&sm.full[m][s], (it / kRingB) & 1u, sm.ctl);
            if (!ok) break;
            tc_fence_after();
            const uint64_t db = desc_k | (uint64_t)((smem_u32(sm.ring[m][s]) >> 4) & 0x3FFF);
#pragma unroll
            for (int j = 0; j < 4; ++j)
              mma_ts(t_o + m * kBlockN, t_a + kt * kTileK + 8 * j, db + 2 * j, idesc, (kt | (uint32_t)j) != 0);
            mma_commit(&sm.empty[m][s]);
          }
          if (!ok) break;
          mma_commit(&sm.o_full[m]);
        }
        if (ok) mma_commit(&sm.a_free);
      }
      if (!ok) mma_quiesce(&sm.mma_idle[m]);
    }
  } else if (warp == 2) {
    // ---- part store ----
    if (lane == 0) {
      uint32_t is = 0, held = kStages;          // held: the stage whose store was issued last (kStages: none)
      bool ok = true;
      for (uint32_t pi = 0; ok && pi < sc.n_pieces; ++pi) {
        const Piece pc = sc.piece(pi);
        const uint32_t hg = pc.hg;
        const int r0 = (int)pc.r0;
        for (uint32_t ci = 0; ok && ci < pc.n; ++ci) {
          const uint32_t c = pc.block(ci), np = parts_of(c);
          for (uint32_t part = 0; part < np; ++part, ++is) {
            const uint32_t s = is % kStages;
            ok = mbar_wait(&sm.g_done[s], (is / kStages) & 1u, sm.ctl);
            if (!ok) break;
            const int col0 = (int)(c * kBlockN + part * 32);
            const uint32_t src = smem_u32(sm.st[s]);
            if (hg == 4) tma_store_2d(&maps.o128, col0, r0, src);
            else
              for (uint32_t i = 0; i < hg; ++i) tma_store_2d(&maps.o32, col0, r0 + 32 * (int)i, src + i * 4096);
            bulk_commit();
            // the store just issued is not waited for: the stage of the store BEFORE it is released once that
            // one has read its source, so that the wait never sits between two stores
            bulk_wait_read_but_one();
            if (held != kStages) mbar_arrive(&sm.g_empty[held]);
            held = s;
          }
        }
      }
      bulk_wait_read_all();
      if (held != kStages) mbar_arrive(&sm.g_empty[held]);
      bulk_wait_all();
    }
  } else if (warp < 7) {
    // ---- staging warps: Xt tile -> tensor memory, rounded to TF32 (thread = lane of its 32-lane window) ----
    const uint32_t q = (uint32_t)(warp & 3);
    const uint32_t row = 32u * q + (uint32_t)lane;
    uint32_t ia = 0, t = 0;
    bool ok = true;
    for (uint32_t pi = 0; ok && pi < sc.n_pieces; ++pi, ++t) {
      const Piece pc = sc.piece(pi);
      if (t > 0) {                                   // both MMA warps have read the old tile
        ok = mbar_wait(&sm.a_free, (t - 1) & 1u, sm.ctl);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
      }
      for (uint32_t kt = 0; kt < k_tiles; ++kt, ++ia) {
        const uint32_t s = ia % kStageA;
        ok = mbar_wait(&sm.a_full[s], (ia / kStageA) & 1u, sm.ctl);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        uint32_t v[32];
        const uint32_t a0 = smem_u32(sm.a[s]) + row * 128;
#pragma unroll
        for (uint32_t ch = 0; ch < 8; ++ch) {
          const float4 f = lds128(a0 + ((ch ^ (row & 7u)) << 4));
          v[4 * ch + 0] = round_tf32(__float_as_uint(f.x));
          v[4 * ch + 1] = round_tf32(__float_as_uint(f.y));
          v[4 * ch + 2] = round_tf32(__float_as_uint(f.z));
          v[4 * ch + 3] = round_tf32(__float_as_uint(f.w));
        }
        tmem_st32(t_a + kt * kTileK + ((32u * q) << 16), v);
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.a_empty[s]);
      }
      if (!ok) break;
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.a_ready);
    }
  } else if (warp < 11) {
    // ---- epilogue warps: accumulator part -> stage (swizzled like the store's box) ----
    const uint32_t q = (uint32_t)(warp & 3);
    const uint32_t row = 32u * q + (uint32_t)lane;
    const uint32_t roff = row * 128, sw = row & 7u;
    uint32_t cg = 0, ie = 0;
    bool ok = true;
    for (uint32_t pi = 0; ok && pi < sc.n_pieces; ++pi) {
      const Piece pc = sc.piece(pi);
      for (uint32_t ci = 0; ok && ci < pc.n; ++ci, ++cg) {
        const uint32_t buf = cg & 1u;
        ok = mbar_wait(&sm.o_full[buf], (cg >> 1) & 1u, sm.ctl);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const uint32_t np = parts_of(pc.block(ci));
        for (uint32_t part = 0; part < np; ++part, ++ie) {
          const uint32_t s = ie % kStages;
          uint32_t v[32];
          tmem_ld32(t_o + buf * kBlockN + part * 32 + ((32u * q) << 16), v);
          ok = mbar_wait(&sm.g_empty[s], ((ie / kStages) & 1u) ^ 1u, sm.ctl);   // the store has read the stage's last part
          ok = __all_sync(0xffffffffu, ok);
          tmem_ld_wait();
          if (!ok) break;
          const uint32_t bt = smem_u32(sm.st[s]) + roff;
#pragma unroll
          for (uint32_t ch = 0; ch < 8; ++ch)
            sts128(bt + ((ch ^ sw) << 4), make_float4(__uint_as_float(v[4 * ch]), __uint_as_float(v[4 * ch + 1]),
                                                      __uint_as_float(v[4 * ch + 2]), __uint_as_float(v[4 * ch + 3])));
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.g_done[s]);
        }
        if (!ok) break;
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.o_empty[buf]);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(sm.tmem_base), "r"(512) : "memory");
  }
  if (tid == 0 && sm.ctl.abort && p.flags) atomicOr(p.flags, (uint32_t)SL_FLAG_TIMEOUT);
}

// --------------------------------------------------------------------- plain float32 kernels (any shape)
__global__ void __launch_bounds__(256) subspace_project_generic_kernel(const float* __restrict__ X, const float* __restrict__ U,
                                                                       SubParams p) {
  const uint64_t n = p.n_tok * (uint64_t)p.k;
  bool bad = false;
  for (uint64_t e = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (uint64_t)gridDim.x * blockDim.x) {
    const uint64_t t = e / p.k;
    const uint32_t j = (uint32_t)(e - t * p.k);
    const float* x = X + t * p.d;
    const float* tp = nullptr;
    const float* ps = nullptr;
    if (p.ids) {
      const int32_t id = p.ids[t];
      if (id < 0 || (uint64_t)id >= p.V) bad = true;
      else { tp = p.T_perp + (uint64_t)id * p.d; ps = p.pos + (t % p.L) * (uint64_t)p.d; }
    }
    float acc = 0.0f;
    for (uint32_t i = 0; i < p.d; ++i) {
      float a = x[i];
      if (tp) a = __fsub_rn(__fsub_rn(a, tp[i]), ps[i]);
      acc = __fmaf_rn(a, U[(uint64_t)i * p.k + j], acc);
    }
    p.out[e] = acc;
  }
  if (bad && p.flags) atomicOr(p.flags, (uint32_t)SL_FLAG_BAD_INDEX);
}

__global__ void __launch_bounds__(256) subspace_reconstruct_generic_kernel(const float* __restrict__ Xt,
                                                                           const float* __restrict__ U, SubParams p) {
  const uint64_t n = p.n_tok * (uint64_t)p.d;
  bool bad = false;
  for (uint64_t e = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (uint64_t)gridDim.x * blockDim.x) {
    const uint64_t t = e / p.d;
    const uint32_t c = (uint32_t)(e - t * p.d);
    const float* xt = Xt + t * p.k;
    const float* u = U + (uint64_t)c * p.k;
    float acc = 0.0f;
    for (uint32_t j = 0; j < p.k; ++j) acc = __fmaf_rn(xt[j], u[j], acc);
    if (p.ids) {
      const int32_t id = p.ids[t];
      if (id < 0 || (uint64_t)id >= p.V) bad = true;
      else acc = __fadd_rn(__fadd_rn(acc, p.T_perp[(uint64_t)id * p.d + c]), p.pos[(t % p.L) * (uint64_t)p.d + c]);
    }
    p.out[e] = acc;
  }
  if (bad && p.flags) atomicOr(p.flags, (uint32_t)SL_FLAG_BAD_INDEX);
}

bool al16(const void* q) { return ((uintptr_t)q & 15u) == 0; }

unsigned persistent_grid(uint64_t n_tok, cudaError_t* e) {
  const int sms = sm_count(e);
  if (*e != cudaSuccess) return 0;
  const uint64_t tiles = (n_tok + kRows - 1) / kRows;
  return (unsigned)(tiles < (uint64_t)sms ? tiles : (uint64_t)sms);
}

}  // namespace

cudaError_t launch_subspace_project(const float* X, const int32_t* ids, const float* T_perp, const float* pos,
                                    const float* U, uint64_t n_tok, uint32_t L, uint64_t V, uint32_t d, uint32_t k,
                                    float* Xt, uint32_t* flags, cudaStream_t st) {
  SubParams p{T_perp, pos, ids, Xt, n_tok, V, L, d, k, (k + 31u) & ~31u, flags, debug_wait_polls()};
  const bool tuned = d % 4 == 0 && k % 4 == 0 && k >= 4 && k <= 256 && al16(X) && al16(U) && al16(Xt) &&
                     (!ids || (al16(T_perp) && al16(pos)));
  if (!tuned) {
    const uint64_t blocks = (n_tok * (uint64_t)k + 255) / 256;
    cudaError_t e;
    const uint64_t cap = (uint64_t)sm_count(&e) * 32u;
    if (e != cudaSuccess) return e;
    subspace_project_generic_kernel<<<(unsigned)(blocks < cap ? blocks : cap), 256, 0, st>>>(X, U, p);
    return cudaGetLastError();
  }
  ProjMaps m;
  constexpr CUtensorMapL2promotion promo = CU_TENSOR_MAP_L2_PROMOTION_L2_256B;
  if (!make_map(&m.x128, X, d, n_tok, kRows, CU_TENSOR_MAP_SWIZZLE_128B, promo) ||
      !make_map(&m.x32, X, d, n_tok, 32, CU_TENSOR_MAP_SWIZZLE_128B, promo) ||
      !make_map(&m.u_n, U, k, d, 32, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B))
    return cudaErrorInvalidValue;
  cudaError_t e;
  const unsigned grid = persistent_grid(n_tok, &e);
  if (e != cudaSuccess) return e;
  if ((n_tok + kRows - 1) / kRows >= 2ull * grid) {
    // at least two sub-tiles for every CTA: two sub-tiles share every U slice
    const int smem = (int)sizeof(DualSmem) + 1024;
    if (ids) {
      // a whole number of pairs of sequences: the two sub-tiles of a pass are the same positions of two sequences
      const bool same_pos = L >= 32 && L % 32 == 0 && n_tok % (2ull * L) == 0 && n_tok / 32 < 0xFFFFFFF0ull;
      auto kern = same_pos ? subspace_project_dual_samepos_kernel : subspace_project_dual_gather_kernel;
      e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      if (e != cudaSuccess) return e;
      kern<<<grid, kThreadsG, smem, st>>>(m, p);
      return cudaGetLastError();
    }
    e = cudaFuncSetAttribute(subspace_project_dual_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    subspace_project_dual_kernel<<<grid, kThreads, smem, st>>>(m, p);
    return cudaGetLastError();
  }
  const int smem = (int)sizeof(ProjSmem) + 1024;
  e = cudaFuncSetAttribute(subspace_project_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  subspace_project_kernel<<<grid, kThreads, smem, st>>>(m, p);
  return cudaGetLastError();
}

cudaError_t launch_subspace_reconstruct(const float* Xt, const int32_t* ids, const float* T_perp, const float* pos,
                                        const float* U, uint64_t n_tok, uint32_t L, uint64_t V, uint32_t d, uint32_t k,
                                        float* Xhat, uint32_t* flags, cudaStream_t st) {
  SubParams p{T_perp, pos, ids, Xhat, n_tok, V, L, d, k, (k + 31u) & ~31u, flags, debug_wait_polls()};
  const bool tuned = d % 4 == 0 && k % 4 == 0 && k >= 4 && k <= 256 && al16(Xt) && al16(U) && al16(Xhat) &&
                     (!ids || (al16(T_perp) && al16(pos)));
  if (!tuned) {
    const uint64_t blocks = (n_tok * (uint64_t)d + 255) / 256;
    cudaError_t e;
    const uint64_t cap = (uint64_t)sm_count(&e) * 32u;
    if (e != cudaSuccess) return e;
    subspace_reconstruct_generic_kernel<<<(unsigned)(blocks < cap ? blocks : cap), 256, 0, st>>>(Xt, U, p);
    return cudaGetLastError();
  }
  ReconMaps m;
  if (!make_map(&m.xt128, Xt, k, n_tok, kRows, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !make_map(&m.xt32, Xt, k, n_tok, 32, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !make_map(&m.u_k, U, k, d, kBlockN, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !make_map(&m.o128, Xhat, d, n_tok, kRows, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !make_map(&m.o32, Xhat, d, n_tok, 32, CU_TENSOR_MAP_SWIZZLE_128B))
    return cudaErrorInvalidValue;
  cudaError_t e;
  const uint64_t sms = (uint64_t)sm_count(&e);
  if (e != cudaSuccess) return e;
  const uint64_t units = ((n_tok + kRows - 1) / kRows) * ((d + kBlockN - 1) / kBlockN);   // (sub-tile, block) pairs
  const unsigned grid = (unsigned)(units < sms ? units : sms);
  if (!ids) {                                        // no embedding terms: two MMA-issuing warps, two rings of U
    const int gsmem = (int)sizeof(GradSmem) + 1024;
    e = cudaFuncSetAttribute(subspace_reconstruct_grad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, gsmem);
    if (e != cudaSuccess) return e;
    subspace_reconstruct_grad_kernel<<<grid, kGradThreads, gsmem, st>>>(m, p);
    return cudaGetLastError();
  }
  const int smem = (int)sizeof(ReconSmem) + 1024;
  e = cudaFuncSetAttribute(subspace_reconstruct_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  subspace_reconstruct_kernel<<<grid, kReconThreads, smem, st>>>(m, p);
  return cudaGetLastError();
}

}  // namespace sl
