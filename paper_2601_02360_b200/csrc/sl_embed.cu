// Token-embedding re-projection after an outer synchronisation (paper §2.4, Eqs. 3-4):
//     T_perp <- T_perp + (T_S - Pi_S(T_S)),   T_S <- Pi_S(T_S),   Pi_S(t) = t U U^T.
//
// One CTA owns 128 rows of the table.  Both contractions run on the 5th-generation tensor
// cores (tcgen05.mma, kind::tf32) with their accumulators in tensor memory:
//
//   pass 1   P[128 x k]  = T_S[128 x d] . U[d x k]        K-loop over d in steps of 32 columns.
//            A = a T_S tile (K-major, 128-byte swizzle), B = 32 rows of U (N-major: U is stored
//            with k contiguous, so the operand is fed "MN-major", which for 32-bit elements
//            exists only in the 128-byte swizzle with 32-byte atoms).  P stays in tensor memory.
//   pass 2   O[128 x 128] = P[128 x k] . U[n0.., :]^T      for each block of 128 output columns.
//            A = P read straight from tensor memory (no round trip through shared memory),
//            B = 128 rows of U (K-major).  O is double buffered in tensor memory, so the
//            element-wise update of block c overlaps the contraction of block c+1.
//
// Warp roles: warp 0 issues the bulk tensor copies (TMA) into a 3-slot ring, warp 1 owns tensor
// memory and issues the MMAs, warps 2-9 are the epilogue: each reads 32 lanes x 64 columns of O
// from tensor memory, turns them through a padded shared-memory tile so that global accesses are
// whole 256-byte row segments (a batch of 16 rows in flight per warp), and applies Eqs. 3-4 with explicitly rounded float32 operations.
// Out-of-range rows and columns (V, d, k not multiples of the tile) are zero-filled by the
// copies and masked in the epilogue.  Every wait is bounded; a wait that gives up raises
// SL_FLAG_TIMEOUT and all roles fall through to the common exit, which frees tensor memory.
#include <cuda.h>   // CUtensorMap and its enums only: the encoder is fetched through the runtime
#include <mutex>

#include "sl_common.cuh"

namespace sl {
namespace {

constexpr int kRows = 128;        // rows of the table per CTA (MMA M)
constexpr int kTileK = 32;        // floats per 128-byte swizzle row
constexpr int kBlockN = 128;      // output columns per pass-2 block
constexpr int kStages = 3;
constexpr int kSlotA = kRows * kTileK * 4;          // 16 KB
constexpr int kSlotB = 256 * kTileK * 4;            // 32 KB
constexpr int kSlot = kSlotA + kSlotB;
constexpr int kEpiWarps = 8;      // two warps per 32-lane window of tensor memory, 64 columns each
constexpr int kStageStride = 64 + 4;                // floats; 272-byte rows keep 16-byte stores conflict-free
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr long long kWaitClocks = 2000000000ll;     // about a second

struct EmbedSmem {
  uint8_t slot[kStages][kSlot];
  float stage[kEpiWarps][32][kStageStride];
  uint64_t full[kStages], empty[kStages], o_full[2], o_empty[2];
  uint32_t tmem_base;
  volatile uint32_t abort;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* b, int n) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(n));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
// bounded wait: false when the phase did not complete within kWaitClocks or another role gave up
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, EmbedSmem& sm) {
  const long long t0 = clock64();
  for (;;) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
    if (ok) return true;
    if (sm.abort || clock64() - t0 > kWaitClocks) { sm.abort = 1; return false; }
    __nanosleep(32);
  }
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(smem_u32(bar)), "r"(x), "r"(y) : "memory");
}

// shared-memory matrix descriptor of tcgen05.mma: start address, leading and stride byte offsets
// (all in 16-byte units), descriptor version 1, swizzle mode (2: 128-byte, 1: 128-byte with 32-byte atoms)
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t swizzle) {
  return (uint64_t)((saddr >> 4) & 0x3FFF) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32) | ((uint64_t)1 << 46) | ((uint64_t)swizzle << 61);
}
// instruction descriptor, kind::tf32: float32 accumulator, TF32 A and B, A K-major, M x N tile
__device__ __forceinline__ uint32_t instr_desc(int M, int N, int b_mn_major) {
  return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}"
               ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t db, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n}"
               ::"r"(d_tmem), "r"(a_tmem), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,"
      "%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
embed_reproject_kernel(const __grid_constant__ CUtensorMap map_ts, const __grid_constant__ CUtensorMap map_u_n,
                       const __grid_constant__ CUtensorMap map_u_k, float* __restrict__ T_S,
                       float* __restrict__ T_perp, uint64_t V, uint32_t d, uint32_t kp, uint32_t* flags) {
  extern __shared__ uint8_t raw[];
  EmbedSmem& sm = *reinterpret_cast<EmbedSmem*>(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint64_t m0 = (uint64_t)blockIdx.x * kRows;
  const uint32_t k_tiles1 = (d + kTileK - 1) / kTileK;      // pass 1: steps over d
  const uint32_t k_tiles2 = kp / kTileK;                    // pass 2: steps over k (padded)
  const uint32_t n_blocks = (d + kBlockN - 1) / kBlockN;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&sm.o_full[b], 1); mbar_init(&sm.o_empty[b], kEpiWarps); }
    sm.abort = 0;
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

  if (warp == 0) {
    if (lane == 0) {
      // ---- producer: one ring over both passes ----
      uint32_t it = 0;
      bool ok = true;
      for (uint32_t kt = 0; ok && kt < k_tiles1; ++kt, ++it) {
        const uint32_t s = it % kStages;
        ok = mbar_wait(&sm.empty[s], ((it / kStages) & 1u) ^ 1u, sm);
        if (!ok) break;
        mbar_expect_tx(&sm.full[s], kSlotA + kp * kTileK * 4);
        tma_load_2d(sm.slot[s], &map_ts, (int)(kt * kTileK), (int)m0, &sm.full[s]);
        for (uint32_t g = 0; g < kp / 32; ++g)
          tma_load_2d(sm.slot[s] + kSlotA + g * 4096, &map_u_n, (int)(g * 32), (int)(kt * kTileK), &sm.full[s]);
      }
      for (uint32_t c = 0; ok && c < n_blocks; ++c)
        for (uint32_t kt = 0; kt < k_tiles2; ++kt, ++it) {
          const uint32_t s = it % kStages;
          ok = mbar_wait(&sm.empty[s], ((it / kStages) & 1u) ^ 1u, sm);
          if (!ok) break;
          mbar_expect_tx(&sm.full[s], kBlockN * kTileK * 4);
          tma_load_2d(sm.slot[s] + kSlotA, &map_u_k, (int)(kt * kTileK), (int)(c * kBlockN), &sm.full[s]);
        }
      // no copy of this CTA may still be in flight when it exits
      const uint32_t last = it < (uint32_t)kStages ? it : (uint32_t)kStages;
      for (uint32_t b = 0; b < last; ++b) {
        const uint32_t j = it - 1 - b;
        const long long t0 = clock64();
        for (;;) {
          uint32_t done;
          asm volatile("{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                       : "=r"(done) : "r"(smem_u32(&sm.full[j % kStages])), "r"((j / kStages) & 1u) : "memory");
          if (done || clock64() - t0 > kWaitClocks) break;
          __nanosleep(64);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---- MMA issuer ----
      uint32_t it = 0;
      bool ok = true;
      const uint32_t idesc1 = instr_desc(kRows, (int)kp, 1);
      const uint32_t idesc2 = instr_desc(kRows, kBlockN, 0);
      for (uint32_t kt = 0; ok && kt < k_tiles1; ++kt, ++it) {
        const uint32_t s = it % kStages;
        ok = mbar_wait(&sm.full[s], (it / kStages) & 1u, sm);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a0 = smem_u32(sm.slot[s]), b0 = a0 + kSlotA;
#pragma unroll
        for (int j = 0; j < 4; ++j)   // K = 8 per instruction: 32 bytes along a swizzled row of A, 8 rows of U
          mma_ss(t_p, smem_desc(a0 + 32 * j, 16, 1024, 2), smem_desc(b0 + 1024 * j, 4096, 512, 1), idesc1,
                 (kt | (uint32_t)j) != 0);
        mma_commit(&sm.empty[s]);
      }
      for (uint32_t c = 0; ok && c < n_blocks; ++c) {
        const uint32_t buf = c & 1u;
        if (c >= 2) {
          ok = mbar_wait(&sm.o_empty[buf], ((c >> 1) - 1u) & 1u, sm);
          if (!ok) break;
          tc_fence_after();
        }
        for (uint32_t kt = 0; kt < k_tiles2; ++kt, ++it) {
          const uint32_t s = it % kStages;
          ok = mbar_wait(&sm.full[s], (it / kStages) & 1u, sm);
          if (!ok) break;
          tc_fence_after();
          const uint32_t b0 = smem_u32(sm.slot[s]) + kSlotA;
#pragma unroll
          for (int j = 0; j < 4; ++j)
            mma_ts(t_o + buf * kBlockN, t_p + kt * kTileK + 8 * j, smem_desc(b0 + 32 * j, 16, 1024, 2), idesc2,
                   (kt | (uint32_t)j) != 0);
          mma_commit(&sm.empty[s]);
        }
        if (!ok) break;
        mma_commit(&sm.o_full[buf]);
      }
    }
  } else {
    // ---- epilogue: warp w may read tensor-memory lanes 32*(w%4).. only (the hardware's lane window
    // of a warp); the two warps of a window take 64 columns of the block each ----
    const int q = warp & 3, h = (warp - 2) >> 2;
    float (*st)[kStageStride] = sm.stage[warp - 2];
    const int sub = lane >> 4, c4 = (lane & 15) * 4;   // read-back: half a warp per row
    bool ok = true;
    for (uint32_t c = 0; ok && c < n_blocks; ++c) {
      const uint32_t buf = c & 1u;
      ok = mbar_wait(&sm.o_full[buf], (c >> 1) & 1u, sm);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int cb = 0; cb < 2; ++cb) {
        uint32_t r[32];
        tmem_ld32(t_o + buf * kBlockN + 64 * h + cb * 32 + ((uint32_t)(32 * q) << 16), r);
#pragma unroll
        for (int i = 0; i < 32; i += 4)
          *reinterpret_cast<uint4*>(&st[lane][cb * 32 + i]) = make_uint4(r[i], r[i + 1], r[i + 2], r[i + 3]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.o_empty[buf]);
      const uint32_t col = c * kBlockN + 64 * h + c4;
      if (col < d) {
#pragma unroll 1
        for (int rb = 0; rb < 32; rb += 16) {
          float4 ts[8], tp[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {      // all loads of the batch first: 8 KB in flight per warp
            const uint64_t row = m0 + (uint64_t)(32 * q + rb + 2 * i + sub);
            if (row < V) {
              ts[i] = __ldcs(reinterpret_cast<const float4*>(T_S + row * d + col));
              tp[i] = __ldcs(reinterpret_cast<const float4*>(T_perp + row * d + col));
            }
          }
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int rr = rb + 2 * i + sub;
            const uint64_t row = m0 + (uint64_t)(32 * q + rr);
            if (row < V) {
              const float4 o = *reinterpret_cast<const float4*>(&st[rr][c4]);
              float4 t = tp[i];
              t.x = __fadd_rn(t.x, __fsub_rn(ts[i].x, o.x));
              t.y = __fadd_rn(t.y, __fsub_rn(ts[i].y, o.y));
              t.z = __fadd_rn(t.z, __fsub_rn(ts[i].z, o.z));
              t.w = __fadd_rn(t.w, __fsub_rn(ts[i].w, o.w));
              __stcs(reinterpret_cast<float4*>(T_S + row * d + col), o);
              __stcs(reinterpret_cast<float4*>(T_perp + row * d + col), t);
            }
          }
        }
      }
      __syncwarp();
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(512) : "memory");
  }
  if (tid == 0 && sm.abort && flags) atomicOr(flags, (uint32_t)SL_FLAG_TIMEOUT);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encoder() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// row-major float32 matrix [outer][inner] -> a map whose box is box_outer rows of 32 floats
bool make_map(CUtensorMap* m, const float* p, uint64_t inner, uint64_t outer, uint32_t box_outer, CUtensorMapSwizzle sw) {
  EncodeTiledFn enc = encoder();
  if (!enc) return false;
  const cuuint64_t dims[2] = {inner, outer};
  const cuuint64_t strides[1] = {inner * 4};
  const cuuint32_t box[2] = {(cuuint32_t)kTileK, box_outer};
  const cuuint32_t es[2] = {1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(p), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t launch_embed_reproject(float* T_S, float* T_perp, const float* U, uint64_t V, uint32_t d, uint32_t k,
                                   uint32_t* flags, cudaStream_t st) {
  CUtensorMap map_ts, map_u_n, map_u_k;
  if (!make_map(&map_ts, T_S, d, V, kRows, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !make_map(&map_u_n, U, k, d, 32, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B) ||
      !make_map(&map_u_k, U, k, d, kBlockN, CU_TENSOR_MAP_SWIZZLE_128B))
    return cudaErrorInvalidValue;
  const int smem = (int)sizeof(EmbedSmem) + 1024;
  const cudaError_t attr =
      cudaFuncSetAttribute(embed_reproject_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (attr != cudaSuccess) return attr;
  const uint32_t kp = (k + 31u) & ~31u;
  const uint64_t grid = (V + kRows - 1) / kRows;
  if (grid > 0x7FFFFFFFull) return cudaErrorInvalidValue;
  embed_reproject_kernel<<<(unsigned)grid, kThreads, smem, st>>>(map_ts, map_u_n, map_u_k, T_S, T_perp, V, d, kp, flags);
  return cudaGetLastError();
}

}  // namespace sl
