// Internal declarations shared by the translation units of the SDGP library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sdgp.h"

namespace sdgp {

cudaError_t launch_prune(const void* dO, int64_t rows, int64_t K, int n, int m, int scheme,
                         uint64_t seed, void* dense, void* values, void* meta, void* mask,
                         cudaStream_t stream);

// Stride-1 data gradient on the tensor cores. sparse == false: A is dense dL/dO [B,P,Q,Cout];
// sparse == true: A is the compressed values [B,P,Q,Cout/2] and meta [B,P,Q,Cout/16].
// Wt [Cout,R,S,Cin], dD [B,H,W,Cin]. A fully connected layer is B = H = 1, W = rows, R = S = 1.
sdgp_status launch_dgrad(bool sparse, const void* A, const void* meta, const void* Wt, void* dD, int B,
                         int H, int W, int Cin, int Cout, int R, int S, int pad, cudaStream_t stream);

// Synchronises the device, then reads and clears the kernels' error word.
sdgp_status read_device_error();

}  // namespace sdgp
