// 12-bit wire form of the message positions (Eq. 2 line 3 sends indices and values; a position
// of a chunk of at most 4096 elements fits 12 bits).  Slot j of a chunk occupies bits
// [12 j, 12 j + 12) of the chunk's ceil(12 k / 8) bytes, least-significant bits first; the
// padding 0xFFFF travels as 0xFFF and is told from position 4095 on the way back by the chunk's
// length (a chunk with all 4096 positions has no padding).  Two small element-wise kernels: the
// messages are about 1 % of the step's traffic, so nothing here is tuned beyond coalescing.
#include "sl_common.cuh"

namespace sl {
namespace {

__device__ __forceinline__ uint32_t to12(uint32_t v, uint32_t* flags) {
  if (v == 0xFFFFu) return 0xFFFu;
  if (v > 0xFFFu) {
    if (flags) atomicOr(flags, (uint32_t)SL_FLAG_BAD_INDEX);
    return v & 0xFFFu;
  }
  return v;
}

// one thread per pair of slots: 24 bits = 3 bytes (the odd last slot of a chunk: 2 bytes)
__global__ void pack_idx12_kernel(const uint16_t* __restrict__ idx, uint8_t* __restrict__ out, uint64_t n_chunks,
                                  uint32_t k, uint32_t stride, uint32_t* flags) {
  const uint32_t pairs = (k + 1) / 2;
  const uint64_t n = n_chunks * pairs;
  for (uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; t < n; t += (uint64_t)gridDim.x * blockDim.x) {
    const uint64_t g = t / pairs;
    const uint32_t j = (uint32_t)(t - g * pairs);
    const uint16_t* src = idx + g * k + 2 * j;
    uint8_t* dst = out + g * stride + 3 * j;
    const uint32_t a = to12(src[0], flags);
    if (2 * j + 1 < k) {
      const uint32_t w = a | (to12(src[1], flags) << 12);
      dst[0] = (uint8_t)w; dst[1] = (uint8_t)(w >> 8); dst[2] = (uint8_t)(w >> 16);
    } else {
      dst[0] = (uint8_t)a; dst[1] = (uint8_t)(a >> 8);
    }
  }
}

// one thread per slot
template <int T>
__global__ void unpack_idx12_kernel(const __grid_constant__ Table<T> tb, const uint8_t* __restrict__ in,
                                    uint16_t* __restrict__ idx, uint32_t k, uint32_t stride, int chunk) {
  const uint64_t n = (uint64_t)tb.n_chunks * k;
  for (uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; t < n; t += (uint64_t)gridDim.x * blockDim.x) {
    const uint32_t g = (uint32_t)(t / k);
    const uint32_t j = (uint32_t)(t - (uint64_t)g * k);
    const uint8_t* src = in + (uint64_t)g * stride + 3 * (j >> 1);
    const uint32_t v = (j & 1u) ? ((uint32_t)(src[1] >> 4) | ((uint32_t)src[2] << 4))
                                : ((uint32_t)src[0] | (((uint32_t)src[1] & 0xFu) << 8));
    uint32_t o = v;
    if (v == 0xFFFu && locate(tb, g, chunk).len != 4096) o = 0xFFFFu;
    idx[t] = (uint16_t)o;
  }
}

// grid-stride launch: enough CTAs for the work, at most 32 per SM
unsigned grid_for(uint64_t n, int block) {
  const uint64_t b = (n + block - 1) / block;
  cudaError_t e;
  const int sms = sm_count(&e);
  const uint64_t cap = (uint64_t)(sms > 0 ? sms : 1) * 32u;
  return (unsigned)(b < 1 ? 1 : (b > cap ? cap : b));
}

}  // namespace

cudaError_t launch_pack_idx12(const uint16_t* idx, uint64_t n_chunks, int k, uint8_t* packed, uint32_t* flags,
                              cudaStream_t st) {
  if (n_chunks == 0) return cudaSuccess;
  const uint32_t stride = (uint32_t)((12u * (uint32_t)k + 7u) / 8u);
  pack_idx12_kernel<<<grid_for(n_chunks * ((k + 1) / 2), 256), 256, 0, st>>>(idx, packed, n_chunks, (uint32_t)k, stride,
                                                                          flags);
  return cudaGetLastError();
}

template <int T>
cudaError_t launch_unpack_idx12(const Table<T>& tb, const uint8_t* packed, int chunk, int k, uint16_t* idx,
                                cudaStream_t st) {
  if (tb.n_chunks == 0) return cudaSuccess;
  const uint32_t stride = (uint32_t)((12u * (uint32_t)k + 7u) / 8u);
  unpack_idx12_kernel<T><<<grid_for((uint64_t)tb.n_chunks * k, 256), 256, 0, st>>>(tb, packed, idx, (uint32_t)k, stride,
                                                                                 chunk);
  return cudaGetLastError();
}

template cudaError_t launch_unpack_idx12<256>(const Table<256>&, const uint8_t*, int, int, uint16_t*, cudaStream_t);
template cudaError_t launch_unpack_idx12<SL_MAX_TENSORS>(const Table<SL_MAX_TENSORS>&, const uint8_t*, int, int,
                                                         uint16_t*, cudaStream_t);

}  // namespace sl
