/*
 * sdgp.h - C ABI of the Structured Data Gradient Pruning (SDGP) GPU library.
 *
 * During back-propagation SDGP prunes the output data gradient dL/dO of a layer to an N:M
 * pattern along the output-channel dimension (keep n of every m consecutive elements) and
 * then computes the input data gradient dL/dD = prune(dL/dO) . W from the pruned tensor
 * (Algorithm 1; Section 2.1, Fig. 2 and Fig. 3; Section 3.2 for the pruning functions).
 *
 * Conventions common to every entry point
 *   - All tensor pointers are DEVICE pointers (global memory of the current CUDA device),
 *     caller-owned, 16-byte aligned, contiguous, row-major; bf16 unless stated.
 *   - Inputs are never written (dL/dO is still needed for the weight gradient, Section 3.1).
 *     Outputs are fully overwritten.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream). Work is enqueued
 *     asynchronously; the call returns before it finishes.
 *   - The library allocates no device memory; scratch is the caller's `workspace`.
 *   - Argument errors are found on the host and returned BEFORE anything is launched.
 *     Nothing aborts, throws or traps. A kernel whose internal wait runs out raises a flag
 *     that sdgp_last_device_error() reports.
 *   - n == m is legal and prunes nothing (the dense data gradient).
 *
 * Pruning functions P (Section 3.2), applied to each group of m consecutive elements:
 *   SDGP_RANDOM              keep the n elements with the smallest 16-bit random keys. Keys come
 *                            from Philox4x32-10 (Salmon et al., SC'11): key = seed, counter =
 *                            (e >> 3) with e the element's linear index row*K + k, element e taking
 *                            little-endian half-word (e & 7) of the 128-bit output. Equal keys:
 *                            lower index wins.
 *   SDGP_MAGNITUDE           keep the n largest magnitudes (order of the bf16 bit pattern with the
 *                            sign cleared); equal magnitudes: lower index wins; survivors keep
 *                            their exact bits.
 *   SDGP_RESCALED_MAGNITUDE  same survivors, each multiplied by sum|group| / sum|survivors| so the
 *                            group's L1 norm is preserved: fp32 magnitudes, balanced pairwise
 *                            summation in index order, IEEE division, fp32 multiply, round to
 *                            nearest-even bf16; a zero denominator gives scale 1; a NaN result is
 *                            stored as 0x7FC0.
 *   Pruned positions hold +0.0.
 *
 * Compressed form (for patterns with n <= 2 and m % 4 == 0, where every aligned 4-element chunk
 * holds at most two survivors - the form a 2:4 sparse tensor core consumes):
 *   values [rows, K/2]  two slots per 4-chunk: the chunk's survivor positions, padded with the
 *                       lowest unused positions up to two and sorted ascending (p0 < p1); slot i
 *                       holds the pruned tensor's value at p_i (a pad slot therefore holds +0.0).
 *   meta   [rows, K/16] uint16; chunk c of a row sits in bits [4*(c%4), 4*(c%4)+3] of word c/4 and
 *                       is p0 | p1 << 2.
 */
#ifndef SDGP_H_
#define SDGP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SDGP_OK = 0,
  SDGP_ERR_INVALID_ARG = 1, /* null pointer, negative size, n/m out of range, K % m != 0, ... */
  SDGP_ERR_UNSUPPORTED = 2, /* legal request this build has no kernel for */
  SDGP_ERR_ALIGNMENT = 3,   /* pointer not 16-byte aligned / extent not a multiple the layout needs */
  SDGP_ERR_WORKSPACE = 4,   /* workspace missing or smaller than sdgp_workspace_size_*() */
  SDGP_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed (launch, tensor-map encode, ...) */
  SDGP_ERR_TIMEOUT = 6,     /* a bounded wait inside a kernel ran out (see sdgp_last_device_error) */
  SDGP_ERR_TOO_LARGE = 7    /* problem exceeds the fixed scratch of sdgp_dgrad_linear_static */
} sdgp_status;

typedef enum { SDGP_RANDOM = 0, SDGP_MAGNITUDE = 1, SDGP_RESCALED_MAGNITUDE = 2 } sdgp_scheme;

/* Element type of the 16-bit tensors of the *_typed entry points (the un-suffixed ones are bf16). */
typedef enum {
  SDGP_BF16 = 0, /* bfloat16 */
  SDGP_FP16 = 1  /* IEEE binary16, the precision the paper's experiments trained in (Section 4) */
} sdgp_dtype;

/* `flags` of the dgrad entry points. */
enum {
  SDGP_FLAG_TWO_PASS = 0, /* prune kernel writes compressed dL/dO into the workspace, sparse GEMM reads it */
  SDGP_FLAG_FUSED = 1,    /* pruning happens inside the dgrad kernel (n <= 2; m = 4, 8 or 16, also 32 for convolutions
                             that run on the whole-filter-reuse kernel); no workspace, no compressed tensor in
                             global memory */
  SDGP_FLAG_DENSE = 2,    /* no pruning: dense tensor-core data gradient of dL/dO itself (n, m, scheme ignored) */
  SDGP_FLAG_MASKED = 3,   /* prune kernel writes the pruned tensor as a dense copy (pruned positions +0.0, the tensor
                             Algorithm 1 returns) into the workspace and the dense tensor-core kernel contracts it:
                             for every 1 <= n <= m, m in {4, 8, 16, 32}, in particular the patterns of Section 4.2
                             that leave more than two survivors in some aligned 4-chunk (3:4, 4:8, 4:16, 8:16,
                             16:32, ...), which a 2:4 sparse tensor core cannot take; no speed-up over dense */
  SDGP_FLAG_CHANNEL = 4   /* two-pass under the OTHER reading of the L1 rescale (Section 3.3, caption of Fig. 4: the
                             norm is preserved "per channel" over batch and spatial positions): survivors of the
                             magnitude function, one factor per output channel k for the whole tensor,
                             sum_rows |dO[.,k]| / sum_rows |kept dO[.,k]| (1 if nothing of the channel is kept), applied
                             inside the contraction by scaling row k of W (a scaled copy of W in the workspace).
                             `scheme` must be SDGP_RESCALED_MAGNITUDE, n <= 2. Costs one more read of dL/dO. */
};

/* Algorithm 1 with pruning function `scheme` on dO viewed as [rows, K], groups of m along K.
 * Requirements: 1 <= n <= m <= 32, m in {4, 8, 16, 32}, K % m == 0, K % 16 == 0 (K % 32 == 0 when
 * `mask` is requested). Any of the four outputs may be NULL; values/meta additionally need
 * n <= 2 (else SDGP_ERR_UNSUPPORTED).
 *   dOp_dense [rows, K]    bf16  pruned copy (the tensor the paper's implementation produces)
 *   values    [rows, K/2]  bf16  compressed survivors      (see file header)
 *   meta      [rows, K/16] u16   survivor positions        (see file header)
 *   mask      [rows, K/32] u32   bit k%32 of word k/32 set iff element k is kept
 * rows == 0 or K == 0 is a no-op returning SDGP_OK. */
sdgp_status sdgp_prune(const void* dO, int64_t rows, int64_t K, int n, int m, sdgp_scheme scheme,
                       uint64_t seed, void* dOp_dense, void* values, void* meta, void* mask,
                       void* stream);

/* Fully connected data gradient (Section 2.1, Fig. 2): dD[r, c] = sum_k prune(dO)[r, k] * W[k, c].
 *   dO [rows, K] bf16, W [K, N] bf16 (output channels x input channels), dD [rows, N] bf16,
 *   fp32 accumulation, round-to-nearest-even bf16 result.
 * Requirements: K % 64 == 0, N % 64 == 0 (any rows >= 0); m in {4,8,16,32} dividing K; the sparse
 * modes (two-pass, fused) need n <= 2 (or n == m, which prunes nothing), SDGP_FLAG_MASKED takes any
 * n <= m. Workspace: sdgp_workspace_size_linear() bytes, 256-byte aligned (two-pass: the compressed
 * rows, padded to whole blocks of 128 channels; masked: the pruned dense copy, rows * K * 2 bytes). */
sdgp_status sdgp_dgrad_linear(const void* dO, const void* W, void* dD, int64_t rows, int64_t K,
                              int64_t N, int n, int m, sdgp_scheme scheme, uint64_t seed,
                              void* workspace, size_t workspace_bytes, uint32_t flags, void* stream);

/* Convolution data gradient (Section 3.1, Fig. 3), NHWC, for the forward cross-correlation
 *   O[b,p,q,co] = sum_{r,s,ci} D[b, p*stride - pad + r, q*stride - pad + s, ci] * W[co,r,s,ci]:
 *   dD[b,h,w,ci] = sum over r, s, co and the (p, q) with p*stride - pad + r == h and
 *                  q*stride - pad + s == w of prune(dO)[b,p,q,co] * W[co,r,s,ci].
 *   dO [B,P,Q,Cout] with P = (H + 2*pad - R)/stride + 1, Q likewise; W [Cout,R,S,Cin];
 *   dD [B,H,Wd,Cin]. Groups of m run along Cout at a fixed (b,p,q).
 * Requirements: stride 1 or 2 (other strides: SDGP_ERR_UNSUPPORTED), Cout % 64 == 0, Cin % 64 == 0,
 * pad <= R-1 and pad <= S-1. Workspace: sdgp_workspace_size_conv2d() bytes, 256-byte aligned. */
sdgp_status sdgp_dgrad_conv2d(const void* dO, const void* W, void* dD, int B, int H, int Wd, int Cin,
                              int Cout, int R, int S, int stride, int pad, int n, int m,
                              sdgp_scheme scheme, uint64_t seed, void* workspace,
                              size_t workspace_bytes, uint32_t flags, void* stream);

/* The contraction of Section 2.1 (Fig. 2, fully connected) / Section 3.1 (Fig. 3, convolution) alone, from
 * an already compressed dL/dO (output of sdgp_prune):
 * values [rows, K/2] bf16 and meta [rows, K/16] u16 in place of dO. No workspace. Needs
 * K % 128 == 0 (Cout % 128 == 0 for the convolution), N % 64 == 0, stride 1 or 2. */
sdgp_status sdgp_spmm_linear(const void* values, const void* meta, const void* W, void* dD,
                             int64_t rows, int64_t K, int64_t N, void* stream);
sdgp_status sdgp_spmm_conv2d(const void* values, const void* meta, const void* W, void* dD, int B,
                             int H, int Wd, int Cin, int Cout, int R, int S, int stride, int pad,
                             void* stream);

/* The same five operations for tensors of element type `dtype` (dO, W, dD, the dense pruned copy and
 * the compressed values alike); SDGP_BF16 is exactly the un-suffixed entry point. With SDGP_FP16:
 *   - ranking and selection are unchanged (the binary16 pattern with the sign cleared orders
 *     magnitudes just as the bf16 pattern does; NaN > Inf > finite), random keys likewise;
 *   - SDGP_RESCALED_MAGNITUDE widens binary16 to fp32 exactly, sums, divides and multiplies in fp32
 *     as above and rounds to nearest-even binary16 (overflow gives infinity; a NaN result is
 *     stored as 0x7E00);
 *   - the contraction multiplies binary16 operands on the tensor cores with fp32 accumulation and
 *     rounds dD to nearest-even binary16;
 *   - SDGP_FLAG_FUSED with SDGP_RESCALED_MAGNITUDE returns SDGP_ERR_UNSUPPORTED (the in-kernel
 *     prune of that scheme exists for bf16 only).
 * Any other dtype value: SDGP_ERR_INVALID_ARG. */
sdgp_status sdgp_prune_typed(const void* dO, int64_t rows, int64_t K, int n, int m, sdgp_scheme scheme,
                             uint64_t seed, sdgp_dtype dtype, void* dOp_dense, void* values, void* meta,
                             void* mask, void* stream);
sdgp_status sdgp_dgrad_linear_typed(const void* dO, const void* W, void* dD, int64_t rows, int64_t K,
                                    int64_t N, int n, int m, sdgp_scheme scheme, uint64_t seed,
                                    sdgp_dtype dtype, void* workspace, size_t workspace_bytes,
                                    uint32_t flags, void* stream);
sdgp_status sdgp_dgrad_conv2d_typed(const void* dO, const void* W, void* dD, int B, int H, int Wd, int Cin,
                                    int Cout, int R, int S, int stride, int pad, int n, int m,
                                    sdgp_scheme scheme, uint64_t seed, sdgp_dtype dtype, void* workspace,
                                    size_t workspace_bytes, uint32_t flags, void* stream);
sdgp_status sdgp_spmm_linear_typed(const void* values, const void* meta, const void* W, void* dD,
                                   int64_t rows, int64_t K, int64_t N, sdgp_dtype dtype, void* stream);
sdgp_status sdgp_spmm_conv2d_typed(const void* values, const void* meta, const void* W, void* dD, int B,
                                   int H, int Wd, int Cin, int Cout, int R, int S, int stride, int pad,
                                   sdgp_dtype dtype, void* stream);

/* The producer of the pruned dL/dO (Section 2.1, Fig. 2: in the backward pass a layer's dL/dO is what the layer above
 * hands down; Section 3.1: the pruned tensor is a copy, the unpruned one still feeds the weight gradient; Section 3.3: its
 * many exact zeros come from the ReLU). One pass over the gradient dY above a ReLU and that ReLU's activation `act`
 * (its output or its input, [rows, K] each, element type `dtype`) forms
 *     dL/dO[r, k] = dY[r, k] if act[r, k] > 0 (a number greater than zero; NaN passes nothing), else +0.0
 * and applies Algorithm 1 to it, so that no separate pass has to read dL/dO again before the sparse contraction
 * (sdgp_spmm_*) can run:
 *   grad      [rows, K]   the unpruned dL/dO (survivors keep the bits of dY)           - optional
 *   dOp_dense, values, meta, mask: as sdgp_prune, computed from that dL/dO            - each optional
 * Requirements as sdgp_prune; groups of 8, 16 and 32 need n <= 2 (n == m is allowed for m == 4: nothing is pruned and
 * the call is a plain ReLU backward). */
sdgp_status sdgp_relu_backward_prune(const void* dY, const void* act, int64_t rows, int64_t K, int n, int m,
                                     sdgp_scheme scheme, uint64_t seed, sdgp_dtype dtype, void* grad, void* dOp_dense,
                                     void* values, void* meta, void* mask, void* stream);

/* The same producer below the ReLU that FOLLOWS A RESIDUAL ADDITION, y = ReLU(x + F(x)) (the ResNets of Section 4): two
 * consumers of y hand down a data gradient each (Section 2.1, Fig. 2) - the next block's branch and its skip path - and the
 * gradient that reaches the ReLU is their sum. One pass reads both gradients and the activation and forms
 *     dL/dO[r, k] = round16(dY[r, k] + dSkip[r, k]) if act[r, k] > 0, else +0.0
 * (one IEEE single-precision addition of the two 16-bit values, rounded to `dtype` to nearest-even; a NaN sum is stored as
 * the canonical quiet NaN 0x7FC0 / 0x7E00), then applies Algorithm 1 to it. dSkip: [rows, K], element type `dtype`,
 * 16-byte aligned, never written; everything else as sdgp_relu_backward_prune. A null dSkip is SDGP_ERR_INVALID_ARG
 * (unless rows * K == 0). */
sdgp_status sdgp_residual_relu_backward_prune(const void* dY, const void* dSkip, const void* act, int64_t rows, int64_t K,
                                              int n, int m, sdgp_scheme scheme, uint64_t seed, sdgp_dtype dtype, void* grad,
                                              void* dOp_dense, void* values, void* meta, void* mask, void* stream);

/* The same producer below a ReLU that is FOLLOWED BY A 2 x 2 MAX POOLING of stride 2 (the blocks of ResNet-9, Section 4:
 * convolution, normalisation, ReLU, pooling): the gradient handed down (Section 2.1, Fig. 2) has the pooled shape
 * dYp [B, H/2, Wd/2, K]; `act` [B, H, Wd, K] is the ReLU's activation (output or input), NHWC, element type `dtype`.
 * One pass forms dL/dO [B, H, Wd, K]: in every window and channel the pooled gradient goes to the window's largest
 * activation - the first one in the order (0,0), (0,1), (1,0), (1,1) if several are equal, as the usual pooling backward
 * does - provided that activation is a number greater than zero; every other position is +0.0 (a NaN is never the
 * maximum). Algorithm 1 then runs along K on that tensor viewed as [B*H*Wd, K]; grad, dOp_dense, values, meta, mask as
 * sdgp_relu_backward_prune. dSkipP (optional, may be null): a second gradient of the pooled shape - in ResNet-9 a residual
 * block follows the pooling, so two gradients reach the pooling's output - added to dYp first, with the arithmetic of
 * sdgp_residual_relu_backward_prune. H and Wd must be even (else SDGP_ERR_INVALID_ARG); B*H*Wd*K / 32 must be below 2^31. */
sdgp_status sdgp_maxpool_relu_backward_prune(const void* dYp, const void* dSkipP, const void* act, int B, int H, int Wd, int64_t K, int n, int m,
                                             sdgp_scheme scheme, uint64_t seed, sdgp_dtype dtype, void* grad, void* dOp_dense,
                                             void* values, void* meta, void* mask, void* stream);

/* Data gradient of a GROUPED convolution (the 3x3 convolutions of RegNetX, one of the networks of Section 4; the
 * contraction is Section 2.1 / Fig. 2 and Section 3.1 / Fig. 3 with the sum over output channels restricted to the
 * group of the input channel): output channel co belongs to group co / (Cout/groups) and is connected to the
 * Cin/groups input channels of that group only, so
 *   dD[b,h,w,ci] = sum over r, s, the (p, q) with p*stride - pad + r == h and q*stride - pad + s == w, and the co of
 *                  group ci / (Cin/groups), of prune(dO)[b,p,q,co] * W[co,r,s, ci % (Cin/groups)].
 *   dO [B,P,Q,Cout], W [Cout,R,S,Cin/groups], dD [B,H,Wd,Cin], element type `dtype`. Algorithm 1 runs along Cout as
 *   for any layer (the groups of m know nothing of the convolution's groups).
 * groups == 1 is an ordinary convolution; unlike sdgp_dgrad_conv2d this entry point also takes channel counts that
 * are not multiples of 64 (RegNetX-400MF has 32 and 160): Cout % 16 == 0 when anything is pruned (% 8 otherwise),
 * (Cin/groups) % 8 == 0. flags: SDGP_FLAG_TWO_PASS, SDGP_FLAG_DENSE, SDGP_FLAG_MASKED, and SDGP_FLAG_FUSED where both
 * channel counts are multiples of 64 (SDGP_ERR_UNSUPPORTED otherwise). Other requirements as sdgp_dgrad_conv2d.
 * The call first writes the filters as the block-diagonal filters of an ordinary convolution, channel counts
 * rounded up to multiples of 64, into the workspace (read again by the contraction on `stream`), then runs the
 * ordinary kernels on them; dL/dO and dD are used as stored, without padded copies.
 * Workspace: sdgp_workspace_size_conv2d_grouped() bytes (every mode needs one), 256-byte aligned, owned by the caller. */
size_t sdgp_workspace_size_conv2d_grouped(int B, int H, int Wd, int Cin, int Cout, int R, int S, int stride, int pad,
                                          int groups, uint32_t flags);
sdgp_status sdgp_dgrad_conv2d_grouped(const void* dO, const void* W, void* dD, int B, int H, int Wd, int Cin, int Cout,
                                      int R, int S, int stride, int pad, int groups, int n, int m, sdgp_scheme scheme,
                                      uint64_t seed, sdgp_dtype dtype, void* workspace, size_t workspace_bytes,
                                      uint32_t flags, void* stream);

/* The factors of SDGP_FLAG_CHANNEL on their own: dO [rows, K] of element type `dtype`, groups of m along K,
 * magnitude function with n survivors (any 1 <= n <= m, m in {4, 8, 16, 32}, K % m == 0, K % 8 == 0).
 * `out` is a device array of 3 * K floats: [0, K) the factors, [K, 2K) the column sums of |dO| over all rows,
 * [2K, 3K) the same sums over the survivors. fp32 sums (partial sums per thread, combined with atomic adds:
 * the last bits depend on the order). */
sdgp_status sdgp_channel_scales(const void* dO, int64_t rows, int64_t K, int n, int m, sdgp_dtype dtype, float* out,
                                void* stream);

/* No counterpart in the paper: a convenience variant of sdgp_dgrad_linear (two-pass mode) that
 * takes no workspace and allocates nothing - for callers that cannot call cudaMalloc where
 * the gradient is computed (inside another runtime's no-allocation region, in a plugin whose
 * host owns all device memory, in a latency-critical loop). The compressed dL/dO goes into a
 * 9 MiB array that is part of the library image in device memory, so every GPU that loads the
 * library holds those 9 MiB until the process exits.
 *   Limit: rows * K <= 8,388,608 elements (e.g. 4096 x 2048); larger -> SDGP_ERR_TOO_LARGE.
 *   Requirements: K % 128 == 0, N % 64 == 0, m in {4, 8, 16, 32} dividing K, n <= 2 or n == m
 *   (n == m prunes nothing: the dense kernel reads dO directly and the array is not used),
 *   16-byte aligned pointers; violations are reported before anything is launched.
 *   The first call on each device looks up the array's device address (one host-side runtime
 *   query, no allocation); make that first call outside any stream capture. First calls made
 *   from several host threads at once are safe: each stores the same address.
 *   All calls on a device share the one array: two calls whose kernels may overlap on the GPU
 *   (different streams, no dependency) race on it and give wrong results - serialise them.
 *   Nothing in the array has to be cleared between calls: each call rewrites what it reads. */
sdgp_status sdgp_dgrad_linear_static(const void* dO, const void* W, void* dD, int64_t rows, int64_t K,
                                     int64_t N, int n, int m, sdgp_scheme scheme, uint64_t seed,
                                     void* stream);

/* Bytes of workspace the matching dgrad call needs for these shapes and flags (0 for
 * SDGP_FLAG_DENSE and SDGP_FLAG_FUSED; the size of dL/dO for SDGP_FLAG_MASKED; the compressed tensor,
 * 3 * K floats and a copy of W for SDGP_FLAG_CHANNEL). */
size_t sdgp_workspace_size_linear(int64_t rows, int64_t K, int64_t N, uint32_t flags);
size_t sdgp_workspace_size_conv2d(int B, int H, int Wd, int Cin, int Cout, int R, int S, int stride,
                                  int pad, uint32_t flags);

/* Reads and clears the device-side error word of the current device (synchronises the device).
 * SDGP_OK, or SDGP_ERR_TIMEOUT if a kernel gave up on a bounded wait since the last call. */
sdgp_status sdgp_last_device_error(void);

/* Self-test of the failure path (no counterpart in the paper): enqueues a one-CTA kernel that waits,
 * with a 50 ms limit, on a barrier nothing signals. The kernel must end by itself and leave
 * SDGP_ERR_TIMEOUT for the next sdgp_last_device_error() call; the context stays usable. */
sdgp_status sdgp_selftest_bounded_wait(void* stream);

/* Static, NUL-terminated description of a status code. */
const char* sdgp_status_string(sdgp_status status);

#ifdef __cplusplus
}
#endif
#endif /* SDGP_H_ */
