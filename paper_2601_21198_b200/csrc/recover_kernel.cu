// The paper's own GPU step in isolation: re-assembly of already decompressed
// exponent bytes and sign+mantissa bytes into bf16 (Section 3.3, "Memory-Coalesced
// Tensor Recovery Kernel": each thread fetches contiguous segments of both streams
// with vector loads, rebuilds the values in registers and writes them back with
// vector stores).  2 bytes read and 2 bytes written per element: the pure-bandwidth
// reference point for the fused decode kernel, and the recovery step for callers
// that keep E-chunks decompressed.
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <cstdint>

#include "zipmoe.h"

namespace zipmoe_dev {

__device__ __forceinline__ uint32_t merge2(uint32_t exp_pair, uint32_t sm_pair) {
  // two elements: byte i of each input -> bf16 i = sign << 15 | exp << 7 | mantissa
  const uint32_t e = __byte_perm(exp_pair, 0, 0x4140);   // [e0, 0, e1, 0]
  const uint32_t s = __byte_perm(sm_pair, 0, 0x1100);    // [s0, s0, s1, s1]
  return (s & 0x807F807Fu) | (e << 7);
}

__global__ void __launch_bounds__(256) recover_kernel(const uint8_t *__restrict__ exp, const uint8_t *__restrict__ sm,
                                                      uint64_t n, uint16_t *__restrict__ out) {
  const uint64_t n16 = n / 16;
  const uint4 *e4 = reinterpret_cast<const uint4 *>(exp), *s4 = reinterpret_cast<const uint4 *>(sm);
  uint4 *o4 = reinterpret_cast<uint4 *>(out);
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  auto merge16 = [&](const uint4 &e, const uint4 &s, uint64_t i) {
    const uint32_t ew[4] = {e.x, e.y, e.z, e.w}, sw[4] = {s.x, s.y, s.z, s.w};
    uint32_t o[8];
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      o[2 * w] = merge2(ew[w], sw[w]);
      o[2 * w + 1] = merge2(ew[w] >> 16, sw[w] >> 16);
    }
    __stcs(o4 + 2 * i, make_uint4(o[0], o[1], o[2], o[3]));
    __stcs(o4 + 2 * i + 1, make_uint4(o[4], o[5], o[6], o[7]));
  };
  uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  // four independent 16-element groups per thread and trip: 128 bytes of loads in flight per thread
  for (; i + 3 * stride < n16; i += 4 * stride) {
    uint4 e[4], s[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      e[u] = __ldcs(e4 + i + u * stride);
      s[u] = __ldcs(s4 + i + u * stride);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) merge16(e[u], s[u], i + u * stride);
  }
  for (; i < n16; i += stride) merge16(__ldcs(e4 + i), __ldcs(s4 + i), i);
  // the last n % 16 elements, one per thread of the first block
  const uint64_t tail = n16 * 16 + threadIdx.x;
  if (blockIdx.x == 0 && threadIdx.x < 16 && tail < n) {
    const uint32_t e = exp[tail], s = sm[tail];
    out[tail] = (uint16_t)(((s & 0x80u) << 8) | (e << 7) | (s & 0x7Fu));
  }
}

}  // namespace zipmoe_dev

extern "C" zipmoe_status zipmoe_recover(const uint8_t *exp, const uint8_t *sm, uint64_t n_elems, uint16_t *out_bf16,
                                        zipmoe_stream stream) {
  nvtxRangePushA("zipmoe_recover");
  struct Pop { ~Pop() { nvtxRangePop(); } } pop;
  if (n_elems == 0) return ZIPMOE_OK;
  if (!exp || !sm || !out_bf16) return ZIPMOE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(exp) | reinterpret_cast<uintptr_t>(sm) | reinterpret_cast<uintptr_t>(out_bf16)) & 15)
    return ZIPMOE_ERR_INVALID_ARG;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return ZIPMOE_ERR_CUDA;
  uint64_t blocks = (n_elems / 16 + 255) / 256;
  const uint64_t cap = (uint64_t)sms * 8;
  if (blocks > cap) blocks = cap;
  if (blocks == 0) blocks = 1;
  zipmoe_dev::recover_kernel<<<(unsigned)blocks, 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(exp, sm, n_elems,
                                                                                                  out_bf16);
  return cudaGetLastError() == cudaSuccess ? ZIPMOE_OK : ZIPMOE_ERR_CUDA;
}
