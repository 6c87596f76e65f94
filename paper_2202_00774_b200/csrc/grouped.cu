// Grouped convolutions (the 3x3 convolutions of RegNetX, Section 4) on the kernels of the ordinary data
// gradient: the filters of the groups are written once per call as the block-diagonal filters of an ordinary
// convolution, with the channel counts brought up to the multiples of 64 the tensor-core kernels tile by.
#include <cuda_runtime.h>
#include <stdint.h>

#include "sdgp_internal.cuh"

namespace sdgp {
namespace {

// One thread per 8 consecutive input channels of one (output channel, tap) of the expanded filters.
__global__ void __launch_bounds__(256) expand_grouped_kernel(const uint4* __restrict__ Wg, uint4* __restrict__ Wfull, int Cout,
                                                             int taps, int cin_g, int cout_g, int cin_pad, int64_t vectors) {
  const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= vectors) return;
  const int per_row = cin_pad >> 3;
  const int c8 = (int)(v % per_row);
  const int64_t row = v / per_row;  // co * taps + tap
  const int co = (int)(row / taps);
  uint4 out = make_uint4(0u, 0u, 0u, 0u);
  if (co < Cout) {
    const int cj = c8 * 8 - (co / cout_g) * cin_g;  // channel within the group of `co`, if this vector lies in its block
    if (cj >= 0 && cj < cin_g) out = Wg[(row * cin_g + cj) >> 3];
  }
  Wfull[v] = out;
}

}  // namespace

cudaError_t launch_expand_grouped_weights(const void* Wg, int Cout, int taps, int Cin, int groups, int cout_pad, int cin_pad,
                                          void* Wfull, cudaStream_t stream) {
  const int64_t vectors = (int64_t)cout_pad * taps * (cin_pad >> 3);
  if (vectors == 0) return cudaSuccess;
  const int64_t blocks = (vectors + 255) / 256;
  if (blocks > 0x7FFFFFFF) return cudaErrorInvalidValue;
  expand_grouped_kernel<<<(unsigned)blocks, 256, 0, stream>>>((const uint4*)Wg, (uint4*)Wfull, Cout, taps, Cin / groups,
                                                              Cout / groups, cin_pad, vectors);
  return cudaGetLastError();
}

}  // namespace sdgp
