// extern "C" entry points: argument validation, workspace carving, dispatch.
#include "sdgp_internal.cuh"

namespace {

bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

bool valid_dtype(sdgp_dtype d) { return d == SDGP_BF16 || d == SDGP_FP16; }

size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// The sparse contraction works on whole blocks of 128 channels; the compressed workspace rows are
// padded up to that.
int64_t pad128(int64_t k) { return (k + 127) / 128 * 128; }

sdgp_status check_prune_args(int64_t rows, int64_t K, int n, int m, int scheme) {
  if (rows < 0 || K < 0) return SDGP_ERR_INVALID_ARG;
  if (scheme < 0 || scheme > 2) return SDGP_ERR_INVALID_ARG;
  if (m < 1 || m > 32 || n < 1 || n > m) return SDGP_ERR_INVALID_ARG;
  if (m != 4 && m != 8 && m != 16 && m != 32) return SDGP_ERR_UNSUPPORTED;
  if (K % m != 0) return SDGP_ERR_INVALID_ARG;
  return SDGP_OK;
}

struct Carve {
  void* values;
  void* meta;
  size_t bytes;
};

Carve carve_compressed(void* workspace, int64_t elements) {
  Carve c;
  const size_t values_bytes = round_up((size_t)elements, 256);      // elements/2 bf16
  const size_t meta_bytes = round_up((size_t)elements / 8, 256);    // elements/16 uint16
  c.values = workspace;
  c.meta = workspace ? (void*)((uint8_t*)workspace + values_bytes) : nullptr;
  c.bytes = values_bytes + meta_bytes;
  return c;
}

}  // namespace

extern "C" {

const char* sdgp_status_string(sdgp_status status) {
  switch (status) {
    case SDGP_OK: return "ok";
    case SDGP_ERR_INVALID_ARG: return "invalid argument";
    case SDGP_ERR_UNSUPPORTED: return "unsupported configuration";
    case SDGP_ERR_ALIGNMENT: return "misaligned pointer or extent";
    case SDGP_ERR_WORKSPACE: return "workspace missing or too small";
    case SDGP_ERR_CUDA: return "CUDA call failed";
    case SDGP_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case SDGP_ERR_TOO_LARGE: return "problem exceeds the library's fixed scratch capacity";
  }
  return "unknown status";
}

sdgp_status sdgp_prune(const void* dO, int64_t rows, int64_t K, int n, int m, sdgp_scheme scheme,
                       uint64_t seed, void* dOp_dense, void* values, void* meta, void* mask,
                       void* stream) {
  return sdgp_prune_typed(dO, rows, K, n, m, scheme, seed, SDGP_BF16, dOp_dense, values, meta, mask, stream);
}

sdgp_status sdgp_prune_typed(const void* dO, int64_t rows, int64_t K, int n, int m, sdgp_scheme scheme,
                             uint64_t seed, sdgp_dtype dtype, void* dOp_dense, void* values, void* meta,
                             void* mask, void* stream) {
  if (!valid_dtype(dtype)) return SDGP_ERR_INVALID_ARG;
  sdgp_status st = check_prune_args(rows, K, n, m, (int)scheme);
  if (st != SDGP_OK) return st;
  if (rows == 0 || K == 0) return SDGP_OK;
  if (!dO) return SDGP_ERR_INVALID_ARG;
  if ((values || meta) && n > 2) return SDGP_ERR_UNSUPPORTED;
  if (K % 16 != 0 || (mask && K % 32 != 0)) return SDGP_ERR_ALIGNMENT;
  if (!aligned16(dO) || !aligned16(dOp_dense) || !aligned16(values) || !aligned16(meta) || !aligned16(mask))
    return SDGP_ERR_ALIGNMENT;
  cudaError_t e = sdgp::launch_prune(dO, rows, K, n, m, (int)scheme, seed, dOp_dense, values, meta, mask,
                                     (cudaStream_t)stream, 0, (int)dtype);
  return e == cudaSuccess ? SDGP_OK : SDGP_ERR_CUDA;
}

static sdgp_status relu_backward_prune(const void* dY, const void* dSkip, const void* act, int64_t rows, int64_t K, int n,
                                       int m, sdgp_scheme scheme, uint64_t seed, sdgp_dtype dtype, void* grad,
                                       void* dOp_dense, void* values, void* meta, void* mask, void* stream) {
  if (!valid_dtype(dtype)) return SDGP_ERR_INVALID_ARG;
  sdgp_status st = check_prune_args(rows, K, n, m, (int)scheme);
  if (st != SDGP_OK) return st;
  if (n > 2 && !(m == 4)) return SDGP_ERR_UNSUPPORTED;   // groups of 8, 16, 32: the threshold selection keeps one or two
  if (rows == 0 || K == 0) return SDGP_OK;
  if (!dY || !act) return SDGP_ERR_INVALID_ARG;
  if ((values || meta) && n > 2) return SDGP_ERR_UNSUPPORTED;
  if (K % 16 != 0 || (mask && K % 32 != 0)) return SDGP_ERR_ALIGNMENT;
  if (!aligned16(dY) || !aligned16(act) || !aligned16(grad) || !aligned16(dOp_dense) || !aligned16(values) ||
      !aligned16(meta) || !aligned16(mask))
    return SDGP_ERR_ALIGNMENT;
  if (!aligned16(dSkip)) return SDGP_ERR_ALIGNMENT;
  cudaError_t e = sdgp::launch_relu_backward_prune(dY, act, rows, K, n, m, (int)scheme, seed, grad, dOp_dense, values, meta,
                                                   mask, (cudaStream_t)stream, (int)dtype, dSkip);
  return e == cudaSuccess ? SDGP_OK : SDGP_ERR_CUDA;
}

sdgp_status sdgp_relu_backward_prune(const void* dY, const void* act, int64_t rows, int64_t K, int n, int m,
                                     sdgp_scheme scheme, uint64_t seed, sdgp_dtype dtype, void* grad, void* dOp_dense,
                                     void* values, void* meta, void* mask, void* stream) {
  return relu_backward_prune(dY, nullptr, act, rows, K, n, m, scheme, seed, dtype, grad, dOp_dense, values, meta, mask, stream);
}

sdgp_status sdgp_maxpool_relu_backward_prune(const void* dYp, const void* dSkipP, const void* act, int B, int H, int Wd, int64_t K, int n, int m,
                                             sdgp_scheme scheme, uint64_t seed, sdgp_dtype dtype, void* grad, void* dOp_dense,
                                             void* values, void* meta, void* mask, void* stream) {
  if (!valid_dtype(dtype)) return SDGP_ERR_INVALID_ARG;
  if (B < 0 || H < 0 || Wd < 0 || (H & 1) || (Wd & 1)) return SDGP_ERR_INVALID_ARG;
  const int64_t rows = (int64_t)B * H * Wd;
  sdgp_status st = check_prune_args(rows, K, n, m, (int)scheme);
  if (st != SDGP_OK) return st;
  if (n > 2 && !(m == 4)) return SDGP_ERR_UNSUPPORTED;
  if (rows == 0 || K == 0) return SDGP_OK;
  if (!dYp || !act) return SDGP_ERR_INVALID_ARG;
  if ((values || meta) && n > 2) return SDGP_ERR_UNSUPPORTED;
  if (K % 16 != 0 || (mask && K % 32 != 0)) return SDGP_ERR_ALIGNMENT;
  if (!aligned16(dYp) || !aligned16(dSkipP) || !aligned16(act) || !aligned16(grad) || !aligned16(dOp_dense) || !aligned16(values) ||
      !aligned16(meta) || !aligned16(mask))
    return SDGP_ERR_ALIGNMENT;
  if (rows * (K / 8) / 4 > 0x7FFFFFFF) return SDGP_ERR_UNSUPPORTED;   // the kernel numbers the pooled vectors in 32 bits
  cudaError_t e = sdgp::launch_maxpool_relu_backward_prune(dYp, act, B, H, Wd, K, n, m, (int)scheme, seed, grad, dOp_dense, values,
                                                           meta, mask, (cudaStream_t)stream, (int)dtype, dSkipP);
  return e == cudaSuccess ? SDGP_OK : SDGP_ERR_CUDA;
}

sdgp_status sdgp_residual_relu_backward_prune(const void* dY, const void* dSkip, const void* act, int64_t rows, int64_t K,
                                              int n, int m, sdgp_scheme scheme, uint64_t seed, sdgp_dtype dtype, void* grad,
                                              void* dOp_dense, void* values, void* meta, void* mask, void* stream) {
  if (!dSkip && rows != 0 && K != 0) return SDGP_ERR_INVALID_ARG;
  return relu_backward_prune(dY, dSkip, act, rows, K, n, m, scheme, seed, dtype, grad, dOp_dense, values, meta, mask, stream);
}

// SDGP_FLAG_CHANNEL: behind the compressed tensor, 3 * K floats (factors, two column sums) and the scaled copy of W
static size_t channel_floats_bytes(int64_t K) { return round_up((size_t)K * 3 * sizeof(float), 256); }
static size_t channel_extra_bytes(int64_t K, int64_t w_row_elems) {
  return channel_floats_bytes(K) + round_up((size_t)K * (size_t)w_row_elems * 2, 256);
}

size_t sdgp_workspace_size_linear(int64_t rows, int64_t K, int64_t N, uint32_t flags) {
  if (rows <= 0 || K <= 0) return 0;
  if (flags == SDGP_FLAG_MASKED) return round_up((size_t)rows * (size_t)K * 2, 256);
  if (flags != SDGP_FLAG_TWO_PASS && flags != SDGP_FLAG_CHANNEL) return 0;
  return carve_compressed(nullptr, rows * pad128(K)).bytes + (flags == SDGP_FLAG_CHANNEL ? channel_extra_bytes(K, N) : 0);
}

size_t sdgp_workspace_size_conv2d(int B, int H, int Wd, int Cin, int Cout, int R, int S, int stride,
                                  int pad, uint32_t flags) {
  if ((flags != SDGP_FLAG_TWO_PASS && flags != SDGP_FLAG_MASKED && flags != SDGP_FLAG_CHANNEL) || stride < 1) return 0;
  const int64_t P = (H + 2 * pad - R) / stride + 1, Q = (Wd + 2 * pad - S) / stride + 1;
  if (B <= 0 || P <= 0 || Q <= 0 || Cout <= 0) return 0;
  if (flags == SDGP_FLAG_MASKED) return round_up((size_t)B * P * Q * Cout * 2, 256);
  return carve_compressed(nullptr, (int64_t)B * P * Q * pad128(Cout)).bytes +
         (flags == SDGP_FLAG_CHANNEL ? channel_extra_bytes(Cout, (int64_t)R * S * Cin) : 0);
}

sdgp_status sdgp_spmm_conv2d(const void* values, const void* meta, const void* W, void* dD, int B,
                             int H, int Wd, int Cin, int Cout, int R, int S, int stride, int pad,
                             void* stream) {
  return sdgp_spmm_conv2d_typed(values, meta, W, dD, B, H, Wd, Cin, Cout, R, S, stride, pad, SDGP_BF16, stream);
}

sdgp_status sdgp_spmm_conv2d_typed(const void* values, const void* meta, const void* W, void* dD, int B,
                                   int H, int Wd, int Cin, int Cout, int R, int S, int stride, int pad,
                                   sdgp_dtype dtype, void* stream) {
  if (!valid_dtype(dtype)) return SDGP_ERR_INVALID_ARG;
  if (B < 0 || H < 0 || Wd < 0 || Cin < 1 || Cout < 1 || R < 1 || S < 1 || stride < 1 || pad < 0)
    return SDGP_ERR_INVALID_ARG;
  if (stride > 2) return SDGP_ERR_UNSUPPORTED;
  if (pad > R - 1 || pad > S - 1) return SDGP_ERR_UNSUPPORTED;
  if (Cout % 128 != 0) return SDGP_ERR_UNSUPPORTED;  // caller-supplied compressed rows are not padded
  if ((int64_t)B * H * Wd == 0) return SDGP_OK;
  if (!values || !meta || !W || !dD) return SDGP_ERR_INVALID_ARG;
  if (!aligned16(values) || !aligned16(meta) || !aligned16(W) || !aligned16(dD)) return SDGP_ERR_ALIGNMENT;
  return sdgp::launch_dgrad(true, values, meta, W, dD, B, H, Wd, Cin, Cout, R, S, stride, pad, (cudaStream_t)stream,
                            nullptr, (int)dtype);
}

sdgp_status sdgp_spmm_linear(const void* values, const void* meta, const void* W, void* dD,
                             int64_t rows, int64_t K, int64_t N, void* stream) {
  return sdgp_spmm_linear_typed(values, meta, W, dD, rows, K, N, SDGP_BF16, stream);
}

sdgp_status sdgp_spmm_linear_typed(const void* values, const void* meta, const void* W, void* dD,
                                   int64_t rows, int64_t K, int64_t N, sdgp_dtype dtype, void* stream) {
  if (rows < 0 || K < 1 || N < 1) return SDGP_ERR_INVALID_ARG;
  if (rows > 0x7FFFFFFF || K > 0x7FFFFFFF || N > 0x7FFFFFFF) return SDGP_ERR_UNSUPPORTED;
  return sdgp_spmm_conv2d_typed(values, meta, W, dD, 1, 1, (int)rows, (int)N, (int)K, 1, 1, 1, 0, dtype, stream);
}

sdgp_status sdgp_dgrad_conv2d(const void* dO, const void* W, void* dD, int B, int H, int Wd, int Cin,
                              int Cout, int R, int S, int stride, int pad, int n, int m,
                              sdgp_scheme scheme, uint64_t seed, void* workspace,
                              size_t workspace_bytes, uint32_t flags, void* stream) {
  return sdgp_dgrad_conv2d_typed(dO, W, dD, B, H, Wd, Cin, Cout, R, S, stride, pad, n, m, scheme, seed, SDGP_BF16,
                                 workspace, workspace_bytes, flags, stream);
}

sdgp_status sdgp_dgrad_conv2d_typed(const void* dO, const void* W, void* dD, int B, int H, int Wd, int Cin,
                                    int Cout, int R, int S, int stride, int pad, int n, int m,
                                    sdgp_scheme scheme, uint64_t seed, sdgp_dtype dtype, void* workspace,
                                    size_t workspace_bytes, uint32_t flags, void* stream) {
  if (!valid_dtype(dtype)) return SDGP_ERR_INVALID_ARG;
  if (B < 0 || H < 0 || Wd < 0 || Cin < 1 || Cout < 1 || R < 1 || S < 1 || stride < 1 || pad < 0)
    return SDGP_ERR_INVALID_ARG;
  if (flags > SDGP_FLAG_CHANNEL) return SDGP_ERR_INVALID_ARG;
  if (stride > 2) return SDGP_ERR_UNSUPPORTED;
  if (pad > R - 1 || pad > S - 1) return SDGP_ERR_UNSUPPORTED;
  if (flags != SDGP_FLAG_DENSE) {
    sdgp_status st = check_prune_args(0, Cout, n, m, (int)scheme);
    if (st != SDGP_OK) return st;
    if (n > 2 && n != m && flags != SDGP_FLAG_MASKED) return SDGP_ERR_UNSUPPORTED;  // not 2:4-compatible
  }
  if ((int64_t)B * H * Wd == 0) return SDGP_OK;
  const int64_t P = (H + 2 * pad - R) / stride + 1, Q = (Wd + 2 * pad - S) / stride + 1;
  if (P < 1 || Q < 1) return SDGP_ERR_INVALID_ARG;
  if (!dO || !W || !dD) return SDGP_ERR_INVALID_ARG;
  if (!aligned16(dO) || !aligned16(W) || !aligned16(dD)) return SDGP_ERR_ALIGNMENT;
  cudaStream_t s = (cudaStream_t)stream;
  const int dt = (int)dtype;
  if (flags == SDGP_FLAG_DENSE || n == m)
    return sdgp::launch_dgrad(false, dO, nullptr, W, dD, B, H, Wd, Cin, Cout, R, S, stride, pad, s, nullptr, dt);
  if (Cin % 64 != 0 || Cout % 64 != 0) return SDGP_ERR_UNSUPPORTED;
  if (flags == SDGP_FLAG_MASKED) {
    // Algorithm 1 as printed: a pruned dense copy, then the dense contraction
    const size_t need = round_up((size_t)B * P * Q * Cout * 2, 256);
    if (!workspace || workspace_bytes < need) return SDGP_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255u) != 0) return SDGP_ERR_ALIGNMENT;
    cudaError_t e = sdgp::launch_prune(dO, (int64_t)B * P * Q, Cout, n, m, (int)scheme, seed, workspace, nullptr,
                                       nullptr, nullptr, s, 0, dt);
    if (e != cudaSuccess) return SDGP_ERR_CUDA;
    return sdgp::launch_dgrad(false, workspace, nullptr, W, dD, B, H, Wd, Cin, Cout, R, S, stride, pad, s, nullptr, dt);
  }
  if (flags == SDGP_FLAG_FUSED) {
    if (dtype == SDGP_FP16 && scheme == SDGP_RESCALED_MAGNITUDE) return SDGP_ERR_UNSUPPORTED;  // bf16 arithmetic only
    const sdgp::FusedPrune fp = {n, m, (int)scheme, seed};
    return sdgp::launch_dgrad(true, dO, nullptr, W, dD, B, H, Wd, Cin, Cout, R, S, stride, pad, s, &fp, dt);
  }
  const int64_t Cpad = pad128(Cout);
  const Carve c = carve_compressed(workspace, (int64_t)B * P * Q * Cpad);
  if (flags == SDGP_FLAG_CHANNEL) {
    // per-channel reading of the rescale: magnitude survivors, factors folded into a scaled copy of W
    if (scheme != SDGP_RESCALED_MAGNITUDE) return SDGP_ERR_INVALID_ARG;
    const int64_t w_row = (int64_t)R * S * Cin, rows = (int64_t)B * P * Q;
    if (!workspace || workspace_bytes < c.bytes + channel_extra_bytes(Cout, w_row)) return SDGP_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255u) != 0) return SDGP_ERR_ALIGNMENT;
    float* floats = (float*)((uint8_t*)workspace + c.bytes);       // [0,K) factors, [K,3K) the two sums
    void* w_scaled = (uint8_t*)floats + channel_floats_bytes(Cout);
    if (sdgp::launch_channel_sums(dO, rows, Cout, n, m, dt, floats + Cout, s) != cudaSuccess) return SDGP_ERR_CUDA;
    if (sdgp::launch_scale_weights(W, floats + Cout, Cout, w_row, dt, w_scaled, floats, s) != cudaSuccess) return SDGP_ERR_CUDA;
    if (sdgp::launch_prune(dO, rows, Cout, n, m, SDGP_MAGNITUDE, seed, nullptr, c.values, c.meta, nullptr, s, Cpad, dt) !=
        cudaSuccess)
      return SDGP_ERR_CUDA;
    return sdgp::launch_dgrad(true, c.values, c.meta, w_scaled, dD, B, H, Wd, Cin, Cout, R, S, stride, pad, s, nullptr, dt);
  }
  if (!workspace || workspace_bytes < c.bytes) return SDGP_ERR_WORKSPACE;
  if (((uintptr_t)workspace & 255u) != 0) return SDGP_ERR_ALIGNMENT;
  cudaError_t e = sdgp::launch_prune(dO, (int64_t)B * P * Q, Cout, n, m, (int)scheme, seed, nullptr, c.values,
                                     c.meta, nullptr, s, Cpad, dt);
  if (e != cudaSuccess) return SDGP_ERR_CUDA;
  return sdgp::launch_dgrad(true, c.values, c.meta, W, dD, B, H, Wd, Cin, Cout, R, S, stride, pad, s, nullptr, dt);
}

// Grouped convolution: the expanded (block-diagonal, channel-padded) filters sit at the start of the workspace
static int round64(int c) { return (c + 63) / 64 * 64; }
static size_t grouped_weights_bytes(int Cin, int Cout, int R, int S) {
  return round_up((size_t)round64(Cout) * R * S * round64(Cin) * 2, 256);
}

size_t sdgp_workspace_size_conv2d_grouped(int B, int H, int Wd, int Cin, int Cout, int R, int S, int stride, int pad,
                                          int groups, uint32_t flags) {
  if (flags > SDGP_FLAG_MASKED || stride < 1 || groups < 1 || Cin < 1 || Cout < 1 || R < 1 || S < 1) return 0;
  const int64_t P = (H + 2 * pad - R) / stride + 1, Q = (Wd + 2 * pad - S) / stride + 1;
  if (B <= 0 || P <= 0 || Q <= 0) return 0;
  const size_t w = grouped_weights_bytes(Cin, Cout, R, S);
  if (flags == SDGP_FLAG_MASKED) return w + round_up((size_t)B * P * Q * Cout * 2, 256);
  if (flags == SDGP_FLAG_TWO_PASS) return w + carve_compressed(nullptr, (int64_t)B * P * Q * pad128(Cout)).bytes;
  return w;
}

sdgp_status sdgp_dgrad_conv2d_grouped(const void* dO, const void* W, void* dD, int B, int H, int Wd, int Cin, int Cout,
                                      int R, int S, int stride, int pad, int groups, int n, int m, sdgp_scheme scheme,
                                      uint64_t seed, sdgp_dtype dtype, void* workspace, size_t workspace_bytes,
                                      uint32_t flags, void* stream) {
  if (!valid_dtype(dtype)) return SDGP_ERR_INVALID_ARG;
  if (B < 0 || H < 0 || Wd < 0 || Cin < 1 || Cout < 1 || R < 1 || S < 1 || stride < 1 || pad < 0 || groups < 1)
    return SDGP_ERR_INVALID_ARG;
  if (Cin % groups != 0 || Cout % groups != 0) return SDGP_ERR_INVALID_ARG;
  if (flags > SDGP_FLAG_MASKED) return SDGP_ERR_INVALID_ARG;
  if (stride > 2) return SDGP_ERR_UNSUPPORTED;
  if (pad > R - 1 || pad > S - 1) return SDGP_ERR_UNSUPPORTED;
  if ((Cin / groups) % 8 != 0 || Cout % 8 != 0) return SDGP_ERR_UNSUPPORTED;  // 16-byte vectors and tensor-map strides
  const bool prunes = flags != SDGP_FLAG_DENSE && n != m;
  if (flags != SDGP_FLAG_DENSE) {
    sdgp_status st = check_prune_args(0, Cout, n, m, (int)scheme);
    if (st != SDGP_OK) return st;
    if (n > 2 && n != m && flags != SDGP_FLAG_MASKED) return SDGP_ERR_UNSUPPORTED;  // not 2:4-compatible
    if (prunes && Cout % 16 != 0) return SDGP_ERR_ALIGNMENT;
  }
  if ((int64_t)B * H * Wd == 0) return SDGP_OK;
  const int64_t P = (H + 2 * pad - R) / stride + 1, Q = (Wd + 2 * pad - S) / stride + 1;
  if (P < 1 || Q < 1) return SDGP_ERR_INVALID_ARG;
  if (!dO || !W || !dD) return SDGP_ERR_INVALID_ARG;
  if (!aligned16(dO) || !aligned16(W) || !aligned16(dD)) return SDGP_ERR_ALIGNMENT;
  const int cin_k = round64(Cin), cout_k = round64(Cout);  // the channel counts the kernels tile by
  const size_t w_bytes = grouped_weights_bytes(Cin, Cout, R, S);
  if (!workspace || workspace_bytes < sdgp_workspace_size_conv2d_grouped(B, H, Wd, Cin, Cout, R, S, stride, pad, groups,
                                                                          prunes ? flags : SDGP_FLAG_DENSE))
    return SDGP_ERR_WORKSPACE;
  if (((uintptr_t)workspace & 255u) != 0) return SDGP_ERR_ALIGNMENT;
  cudaStream_t s = (cudaStream_t)stream;
  const int dt = (int)dtype;
  const void* w_full = W;  // one group and whole 64-channel blocks: the filters are already in the kernels' form
  void* rest = (uint8_t*)workspace + w_bytes;
  if (groups > 1 || Cin != cin_k || Cout != cout_k) {
    if (sdgp::launch_expand_grouped_weights(W, Cout, R * S, Cin, groups, cout_k, cin_k, workspace, s) != cudaSuccess)
      return SDGP_ERR_CUDA;
    w_full = workspace;
  }
  const sdgp::StoredChannels dense_view = {Cout != cout_k ? Cout : 0, Cin != cin_k ? Cin : 0};
  const sdgp::StoredChannels sparse_view = {0, dense_view.d};  // a compressed dL/dO is padded by the prune kernel
  const bool padded = dense_view.a != 0 || dense_view.d != 0;
  const sdgp::ConvGroups cg = {Cin / groups, Cout / groups};
  const sdgp::ConvGroups* cgp = groups > 1 ? &cg : nullptr;
  if (!prunes)
    return sdgp::launch_dgrad(false, dO, nullptr, w_full, dD, B, H, Wd, cin_k, cout_k, R, S, stride, pad, s, nullptr, dt,
                              padded ? &dense_view : nullptr, cgp);
  const int64_t rows = (int64_t)B * P * Q;
  if (flags == SDGP_FLAG_MASKED) {
    if (sdgp::launch_prune(dO, rows, Cout, n, m, (int)scheme, seed, rest, nullptr, nullptr, nullptr, s, 0, dt) != cudaSuccess)
      return SDGP_ERR_CUDA;
    return sdgp::launch_dgrad(false, rest, nullptr, w_full, dD, B, H, Wd, cin_k, cout_k, R, S, stride, pad, s, nullptr, dt,
                              padded ? &dense_view : nullptr, cgp);
  }
  if (flags == SDGP_FLAG_FUSED) {
    if (padded) return SDGP_ERR_UNSUPPORTED;  // the in-kernel prune reads dL/dO by the channel count it tiles by
    if (dtype == SDGP_FP16 && scheme == SDGP_RESCALED_MAGNITUDE) return SDGP_ERR_UNSUPPORTED;
    const sdgp::FusedPrune fp = {n, m, (int)scheme, seed};
    return sdgp::launch_dgrad(true, dO, nullptr, w_full, dD, B, H, Wd, cin_k, cout_k, R, S, stride, pad, s, &fp, dt, nullptr, cgp);
  }
  const int64_t Cpad = pad128(Cout);
  const Carve c = carve_compressed(rest, rows * Cpad);
  if (sdgp::launch_prune(dO, rows, Cout, n, m, (int)scheme, seed, nullptr, c.values, c.meta, nullptr, s, Cpad, dt) != cudaSuccess)
    return SDGP_ERR_CUDA;
  return sdgp::launch_dgrad(true, c.values, c.meta, w_full, dD, B, H, Wd, cin_k, cout_k, R, S, stride, pad, s, nullptr, dt,
                            sparse_view.d ? &sparse_view : nullptr, cgp);
}

sdgp_status sdgp_dgrad_linear(const void* dO, const void* W, void* dD, int64_t rows, int64_t K,
                              int64_t N, int n, int m, sdgp_scheme scheme, uint64_t seed,
                              void* workspace, size_t workspace_bytes, uint32_t flags, void* stream) {
  return sdgp_dgrad_linear_typed(dO, W, dD, rows, K, N, n, m, scheme, seed, SDGP_BF16, workspace, workspace_bytes,
                                 flags, stream);
}

sdgp_status sdgp_dgrad_linear_typed(const void* dO, const void* W, void* dD, int64_t rows, int64_t K,
                                    int64_t N, int n, int m, sdgp_scheme scheme, uint64_t seed,
                                    sdgp_dtype dtype, void* workspace, size_t workspace_bytes,
                                    uint32_t flags, void* stream) {
  if (rows < 0 || K < 1 || N < 1) return SDGP_ERR_INVALID_ARG;
  if (rows > 0x7FFFFFFF || K > 0x7FFFFFFF || N > 0x7FFFFFFF) return SDGP_ERR_UNSUPPORTED;
  return sdgp_dgrad_conv2d_typed(dO, W, dD, 1, 1, (int)rows, (int)N, (int)K, 1, 1, 1, 0, n, m, scheme, seed, dtype,
                                 workspace, workspace_bytes, flags, stream);
}

sdgp_status sdgp_channel_scales(const void* dO, int64_t rows, int64_t K, int n, int m, sdgp_dtype dtype, float* out,
                                void* stream) {
  if (!valid_dtype(dtype)) return SDGP_ERR_INVALID_ARG;
  sdgp_status st = check_prune_args(rows, K, n, m, SDGP_MAGNITUDE);
  if (st != SDGP_OK) return st;
  if (K == 0) return SDGP_OK;
  if (!out || (rows > 0 && !dO)) return SDGP_ERR_INVALID_ARG;
  if (K % 8 != 0 || !aligned16(dO) || ((uintptr_t)out & 3u) != 0) return SDGP_ERR_ALIGNMENT;
  cudaStream_t s = (cudaStream_t)stream;
  if (sdgp::launch_channel_sums(dO, rows, K, n, m, (int)dtype, out + K, s) != cudaSuccess) return SDGP_ERR_CUDA;
  return sdgp::launch_channel_scales(out + K, K, out, s) == cudaSuccess ? SDGP_OK : SDGP_ERR_CUDA;
}

sdgp_status sdgp_last_device_error(void) { return sdgp::read_device_error(); }

sdgp_status sdgp_selftest_bounded_wait(void* stream) { return sdgp::launch_bounded_wait_selftest((cudaStream_t)stream); }

}  // extern "C"
