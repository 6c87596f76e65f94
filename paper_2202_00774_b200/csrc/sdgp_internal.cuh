// Internal declarations shared by the translation units of the SDGP library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sdgp.h"

namespace sdgp {

// k_pad (0 = none): row pitch, in elements, of the compressed outputs. When k_pad > K the extra
// chunks of every row are written as zero values with the position pair (0,1), so a consumer can
// treat the row as k_pad channels (used to bring a channel count up to a whole 128-channel block).
cudaError_t launch_prune(const void* dO, int64_t rows, int64_t K, int n, int m, int scheme,
                         uint64_t seed, void* dense, void* values, void* meta, void* mask,
                         cudaStream_t stream, int64_t k_pad = 0, int dtype = SDGP_BF16);

// The producer of dL/dO below a ReLU fused with its pruning: the gradient above the ReLU (dY) passes where the
// activation `act` is positive; `grad` (optional) receives that unpruned dL/dO, the other outputs are
// launch_prune's. n <= 2, or n == m (nothing pruned: only `grad` and the mask make sense then). skip (optional): a second
// gradient of the same shape, added to dY (fp32 sum, rounded to the 16-bit type) before the gate.
cudaError_t launch_relu_backward_prune(const void* dY, const void* act, int64_t rows, int64_t K, int n, int m, int scheme,
                                       uint64_t seed, void* grad, void* dense, void* values, void* meta, void* mask,
                                       cudaStream_t stream, int dtype = SDGP_BF16, const void* skip = nullptr);

// The same producer below a ReLU that is followed by 2 x 2 max pooling of stride 2: dYp is the pooled gradient
// [B, H/2, W/2, K], act the activation [B, H, W, K]; each pooled gradient goes to the first largest activation of its
// window if that is positive. skip_pooled (optional): a second gradient of the pooled shape, added to dYp first.
// B * H * W * K / 32 must fit 31 bits; H and W even.
cudaError_t launch_maxpool_relu_backward_prune(const void* dYp, const void* act, int B, int H, int W, int64_t K, int n, int m,
                                               int scheme, uint64_t seed, void* grad, void* dense, void* values, void* meta,
                                               void* mask, cudaStream_t stream, int dtype = SDGP_BF16,
                                               const void* skip_pooled = nullptr);

// Per-channel reading of the L1 rescale (channel.cu). sums: 2 * K floats (cleared by the call): the
// column sums of |x| over all rows, then the same over the survivors of the magnitude function.
cudaError_t launch_channel_sums(const void* dO, int64_t rows, int64_t K, int n, int m, int dtype, float* sums,
                                cudaStream_t stream);
// scales[k] = sums[k] / sums[K + k] (1 where the denominator is 0)
cudaError_t launch_channel_scales(const float* sums, int64_t K, float* scales, cudaStream_t stream);
// Wout[k, :] = W[k, :] * scale[k] rounded to the element type (row_elems elements per row, a multiple of 8); also
// writes the K scales.
cudaError_t launch_scale_weights(const void* W, const float* sums, int64_t K, int64_t row_elems, int dtype, void* Wout,
                                 float* scales, cudaStream_t stream);

// Data gradient on the tensor cores (stride 1 or 2). sparse == false: A is dense dL/dO
// [B,P,Q,Cout]; sparse == true: A is the compressed values [B,P,Q,Cp/2] and meta [B,P,Q,Cp/16]
// with Cp = Cout rounded up to a multiple of 128 (see launch_prune's k_pad).
// Wt [Cout,R,S,Cin], dD [B,H,W,Cin]. A fully connected layer is B = H = 1, W = rows, R = S = 1.
// fused != nullptr: A is the dense dL/dO and the kernel prunes it on the fly (n <= 2).
struct FusedPrune {
  int n;
  int m;  // group size: 4, 8, 16 (32 in the whole-filter-reuse kernel only)
  int scheme;
  uint64_t seed;
};
// dtype: element type of A, Wt and dD (SDGP_BF16 or SDGP_FP16; accumulation is fp32 either way).
// Fused pruning with the rescaled scheme exists for bf16 only.
// stored != nullptr: Cin and Cout are the channel counts the kernels tile by (multiples of 64; Wt has that
// many rows and columns, the extra ones zero) while the tensors in global memory hold fewer channels per
// pixel: `a` for a dense A (0 = Cout; a compressed A is always padded to whole 128-channel blocks), `d` for dD
// (0 = Cin), both multiples of 8. TMA reads the missing channels of A as zeros and clips the stores of dD.
struct StoredChannels {
  int a;
  int d;
};
// conv_groups != nullptr: Wt is block-diagonal - input channels [g * cin_g, (g + 1) * cin_g) are connected to output
// channels [g * cout_g, (g + 1) * cout_g) only, everything else in Wt is zero - so a tile of input channels skips
// the channel blocks of dL/dO that only meet zeros.
struct ConvGroups {
  int cin_g;
  int cout_g;
};
sdgp_status launch_dgrad(bool sparse, const void* A, const void* meta, const void* Wt, void* dD, int B,
                         int H, int W, int Cin, int Cout, int R, int S, int stride, int pad, cudaStream_t stream,
                         const FusedPrune* fused = nullptr, int dtype = SDGP_BF16, const StoredChannels* stored = nullptr,
                         const ConvGroups* conv_groups = nullptr);

// Filters of a grouped convolution, Wg [Cout, R*S, Cin/groups], written as the block-diagonal filters of an
// ordinary one, Wfull [cout_pad, R*S, cin_pad] (zeros outside each group's block and in the padding).
cudaError_t launch_expand_grouped_weights(const void* Wg, int Cout, int taps, int Cin, int groups, int cout_pad, int cin_pad,
                                          void* Wfull, cudaStream_t stream);

// Launches a one-CTA kernel whose only wait can never be satisfied (50 ms limit).
sdgp_status launch_bounded_wait_selftest(cudaStream_t stream);

// Synchronises the device, then reads and clears the kernels' error word.
sdgp_status read_device_error();

}  // namespace sdgp
