// The per-channel reading of the L1 rescale (Section 3.3 and the caption of Fig. 4: the norm is
// preserved "per channel" over batch and spatial positions; Section 3.2 words it per group).
// Survivors are those of the magnitude function; channel k of the whole [rows, K] tensor gets one
// factor scale[k] = sum_r |x[r,k]| / sum_r |kept x[r,k]| (1 when nothing of the channel is kept).
// Because the factor is the same for every row, it is folded into row k of W
// (dD = (A diag(s)) W = A (diag(s) W)): the pruned tensor itself is never rescaled, and the sparse
// contraction runs unchanged on the scaled copy of W.
//
// Cost: one more read of dL/dO (column sums cannot be known before the whole tensor has been seen)
// and one pass over W.
#include "prune_core.cuh"
#include "sdgp_internal.cuh"

namespace sdgp {
namespace {

constexpr int kChThreads = 256;

constexpr int kChSlots = 4096;  // channels one block pass accumulates in shared memory (2 x 16 KB)

// Chunk columns a block handles side by side: as many as there are threads, chunks in a row, or
// shared-memory slots.
template <int CH>
__host__ __device__ constexpr int chunk_columns(int cpr) {
  int ct = cpr < kChThreads ? cpr : kChThreads;
  return ct < kChSlots / CH ? ct : kChSlots / CH;
}

// sums[0..K) += sum over rows of |x|, sums[K..2K) += the same over kept elements only. A thread owns
// one chunk of whole groups (8 elements, or m when m > 8) of a set of rows and keeps the chunk's
// partial sums in registers; the mask is the prune kernels' (larger magnitude wins, equal
// magnitudes: lower position), found by counting. The threads of a block that share a chunk column
// combine their sums in shared memory, so that a block adds to each global sum once.
template <int M, bool F16>
__global__ void __launch_bounds__(kChThreads)
channel_sums_kernel(const uint4* __restrict__ dO, int64_t rows, int K, int n, float* __restrict__ sums) {
  constexpr int CH = M < 8 ? 8 : M;
  constexpr int VEC = CH / 8;
  __shared__ float sh_t[kChSlots], sh_s[kChSlots];
  const int cpr = K / CH;                                  // chunks per row
  const int ct = chunk_columns<CH>(cpr);
  const int lanes = kChThreads / ct;                       // rows handled side by side
  const int cc0 = threadIdx.x % ct, lane = threadIdx.x / ct;
  for (int cbase = 0; cbase < cpr; cbase += ct) {
    for (int i = threadIdx.x; i < ct * CH; i += kChThreads) sh_t[i] = sh_s[i] = 0.0f;
    __syncthreads();
    const int cc = cbase + cc0;
    if (lane < lanes && cc < cpr) {
      float t[CH], s[CH];
#pragma unroll
      for (int i = 0; i < CH; ++i) t[i] = s[i] = 0.0f;
      for (int64_t r = (int64_t)blockIdx.x * lanes + lane; r < rows; r += (int64_t)gridDim.x * lanes) {
        const uint4* src = dO + (r * K + (int64_t)cc * CH) / 8;
        uint32_t x[CH];
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
          const uint4 w = __ldg(src + v);
          const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
          for (int i = 0; i < 8; ++i) x[8 * v + i] = (i & 1) ? (ww[i >> 1] >> 16) : (ww[i >> 1] & 0xFFFFu);
        }
        if (M == 4) {
          // groups of four: the packed-lane selection of the prune kernel (register i = elements i and i + 4)
          const uint4 w = make_uint4(x[0] | (x[1] << 16), x[2] | (x[3] << 16), x[4] | (x[5] << 16), x[6] | (x[7] << 16));
          uint32_t y[4], km[4];
          switch (n) {
            case 1: m4_prune_vector<1, SDGP_MAGNITUDE, F16>(w, 0, 0u, 0u, y[0], y[1], y[2], y[3], km[0], km[1], km[2], km[3]); break;
            case 2: m4_prune_vector<2, SDGP_MAGNITUDE, F16>(w, 0, 0u, 0u, y[0], y[1], y[2], y[3], km[0], km[1], km[2], km[3]); break;
            case 3: m4_prune_vector<3, SDGP_MAGNITUDE, F16>(w, 0, 0u, 0u, y[0], y[1], y[2], y[3], km[0], km[1], km[2], km[3]); break;
            default: m4_prune_vector<4, SDGP_MAGNITUDE, F16>(w, 0, 0u, 0u, y[0], y[1], y[2], y[3], km[0], km[1], km[2], km[3]); break;
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            t[i] += lane_lo<F16>(x[i] & 0x7FFFu);
            t[4 + i] += lane_lo<F16>(x[4 + i] & 0x7FFFu);
            s[i] += lane_lo_abs<F16>(y[i]);          // pruned lanes are +0
            s[4 + i] += lane_hi_abs<F16>(y[i]);
          }
          continue;
        }
        uint32_t c[CH];
#pragma unroll
        for (int i = 0; i < CH; ++i) c[i] = ((x[i] & 0x7FFFu) << 5) | (uint32_t)(31 - (i % M));
#pragma unroll
        for (int i = 0; i < CH; ++i) {
          int above = 0;
#pragma unroll
          for (int o = 0; o < CH; ++o)
            if (o != i && (o / M) == (i / M)) above += (c[o] > c[i]) ? 1 : 0;
          const float a = lane_lo<F16>(x[i] & 0x7FFFu);
          t[i] += a;
          if (above < n) s[i] += a;
        }
      }
#pragma unroll
      for (int i = 0; i < CH; ++i) {
        atomicAdd(&sh_t[cc0 * CH + i], t[i]);
        atomicAdd(&sh_s[cc0 * CH + i], s[i]);
      }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < ct * CH; i += kChThreads) {
      const int64_t k = (int64_t)cbase * CH + i;
      if (k < K) {
        atomicAdd(sums + k, sh_t[i]);
        atomicAdd(sums + K + k, sh_s[i]);
      }
    }
    __syncthreads();
  }
}

__device__ __forceinline__ float channel_scale(const float* sums, int K, int k) {
  const float t = sums[k], s = sums[K + k];
  return s == 0.0f ? 1.0f : __fdiv_rn(t, s);
}

__global__ void channel_scales_kernel(const float* __restrict__ sums, int K, float* __restrict__ scales) {
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k < K) scales[k] = channel_scale(sums, K, k);
}

// Wout[k, :] = round(W[k, :] * scale[k]); one thread per 8 elements, row length a multiple of 8.
template <bool F16>
__global__ void scale_weights_kernel(const uint4* __restrict__ W, const float* __restrict__ sums, int K, int64_t row_vecs,
                                     uint4* __restrict__ Wout, float* __restrict__ scales) {
  const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= (int64_t)K * row_vecs) return;
  const int k = (int)(v / row_vecs);
  const float sc = channel_scale(sums, K, k);
  if (v == (int64_t)k * row_vecs) scales[k] = sc;
  const uint4 w = __ldg(W + v);
  uint4 o;
  o.x = pack_pair_rn<F16>(__fmul_rn(lane_lo<F16>(w.x), sc), __fmul_rn(lane_hi<F16>(w.x), sc));
  o.y = pack_pair_rn<F16>(__fmul_rn(lane_lo<F16>(w.y), sc), __fmul_rn(lane_hi<F16>(w.y), sc));
  o.z = pack_pair_rn<F16>(__fmul_rn(lane_lo<F16>(w.z), sc), __fmul_rn(lane_hi<F16>(w.z), sc));
  o.w = pack_pair_rn<F16>(__fmul_rn(lane_lo<F16>(w.w), sc), __fmul_rn(lane_hi<F16>(w.w), sc));
  Wout[v] = o;
}

template <int M>
cudaError_t launch_sums_m(bool f16, const void* dO, int64_t rows, int K, int n, float* sums, cudaStream_t stream) {
  constexpr int CH = M < 8 ? 8 : M;
  const int cpr = K / CH;
  const int ct = chunk_columns<CH>(cpr);
  const int lanes = kChThreads / ct;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    return cudaErrorUnknown;
  int64_t blocks = (rows + lanes - 1) / lanes;
  // measured: twice as many blocks cost more in the closing adds than they gain in loads in flight, half as many the reverse
  if (blocks > 4 * (int64_t)sms) blocks = 4 * (int64_t)sms;
  if (blocks < 1) return cudaSuccess;
  if (f16) channel_sums_kernel<M, true><<<(unsigned)blocks, kChThreads, 0, stream>>>((const uint4*)dO, rows, K, n, sums);
  else channel_sums_kernel<M, false><<<(unsigned)blocks, kChThreads, 0, stream>>>((const uint4*)dO, rows, K, n, sums);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_channel_sums(const void* dO, int64_t rows, int64_t K, int n, int m, int dtype, float* sums,
                                cudaStream_t stream) {
  if (K > 0x7FFFFFFF || K % 8 != 0 || K % m != 0) return cudaErrorInvalidValue;
  if (cudaMemsetAsync(sums, 0, (size_t)K * 2 * sizeof(float), stream) != cudaSuccess) return cudaErrorUnknown;
  const bool f16 = dtype == SDGP_FP16;
  switch (m) {
    case 4: return launch_sums_m<4>(f16, dO, rows, (int)K, n, sums, stream);
    case 8: return launch_sums_m<8>(f16, dO, rows, (int)K, n, sums, stream);
    case 16: return launch_sums_m<16>(f16, dO, rows, (int)K, n, sums, stream);
    case 32: return launch_sums_m<32>(f16, dO, rows, (int)K, n, sums, stream);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_channel_scales(const float* sums, int64_t K, float* scales, cudaStream_t stream) {
  if (K < 1) return cudaSuccess;
  channel_scales_kernel<<<(unsigned)((K + 255) / 256), 256, 0, stream>>>(sums, (int)K, scales);
  return cudaGetLastError();
}

cudaError_t launch_scale_weights(const void* W, const float* sums, int64_t K, int64_t row_elems, int dtype, void* Wout,
                                 float* scales, cudaStream_t stream) {
  if (row_elems % 8 != 0 || K < 1) return cudaErrorInvalidValue;
  const int64_t row_vecs = row_elems / 8, total = K * row_vecs;
  const int64_t blocks = (total + 255) / 256;
  if (blocks > 0x7FFFFFFF) return cudaErrorInvalidValue;
  if (dtype == SDGP_FP16)
    scale_weights_kernel<true><<<(unsigned)blocks, 256, 0, stream>>>((const uint4*)W, sums, (int)K, row_vecs, (uint4*)Wout, scales);
  else
    scale_weights_kernel<false><<<(unsigned)blocks, 256, 0, stream>>>((const uint4*)W, sums, (int)K, row_vecs, (uint4*)Wout, scales);
  return cudaGetLastError();
}

}  // namespace sdgp
