// N:M pruning of the output data gradient (Algorithm 1, Section 3.2), sm_100a.
//
// One thread owns one aligned run of 8 bf16 elements (a single 128-bit load). Groups of
// m = 4 (two per thread) and m = 8 (one per thread) are ranked inside the thread; groups of
// 16 and 32 span 2 and 4 neighbouring lanes, which trade their keys with warp shuffles.
// The kernel is a pure stream: 2 B read per element, 1 B of compressed values, 1/8 B of
// position metadata (+ 1/8 B mask, + 2 B dense copy when asked for), every output indexed by
// the same 8-element vector number so all stores coalesce.
#include <cuda_bf16.h>

#include "prune_core.cuh"
#include "ptx.cuh"
#include "sdgp_internal.cuh"

namespace sdgp {
namespace {

constexpr int kThreads = 256;
constexpr int kVecPerThread = 4;
// Resident blocks per SM the compiler is asked to make room for. Six (at most 40 registers per thread instead of the 42-46
// it takes unasked, which round up to five blocks) measured 7 % more bytes per second for the magnitude function, 6 % for
// groups of 8 and 3 % for the random function; the rescaled function and the producers below a ReLU spill at 40 registers
// and measured slower, so they keep the compiler's own choice. Eight blocks (32 registers, 64-72 bytes spilled per thread)
// measured 9 % fewer bytes per second than six.
template <int SCHEME, bool RELU>
constexpr int kBlocksPerSm = (!RELU && SCHEME != SDGP_RESCALED_MAGNITUDE) ? 6 : 0;

// Survivor positions of a 4-chunk from its 4-bit keep mask: pad with the lowest unused
// positions up to two, ascending; entry = p0 | p1 << 2 (16 nibbles packed in 64 bits).
__device__ __forceinline__ uint32_t chunk_nibble(uint32_t keep4) {
  return (uint32_t)(0x444E4DCC49884444ull >> (4 * keep4)) & 0xFu;
}

// Launch with programmatic stream serialisation: the kernel may be scheduled while the previous
// kernel of the stream is still draining; it waits for that kernel before its first load.
template <typename... Params, typename... Args>
cudaError_t launch_after_previous(void (*kernel)(Params...), dim3 grid, dim3 block, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, Params(args)...);
}

// The producer of dL/dO below a ReLU (Section 2.1, Fig. 2): the 8 gradients g above the ReLU pass where the
// ReLU's activation a is positive (a number greater than zero: sign clear, magnitude between 1 and the
// pattern of infinity) and become +0.0 elsewhere. nan_add = 0x7FFF - (pattern of infinity) in both half-words:
// adding it to a magnitude sets the half-word's top bit exactly for the NaN patterns.
struct ReluSource {
  const uint4* act;   // the ReLU's activation, same shape as the gradient; nullptr: no ReLU, the input is dL/dO itself
  uint4* grad;        // optional: the unpruned dL/dO (kept for the weight gradient, Section 3.1)
  uint32_t nan_add;
  const uint4* skip;  // optional: the second gradient that reaches the ReLU where a residual connection joins its
                      // branch; the two are added before the gate
  int f16;            // element type of the sum (only read when skip is set)
  // 2 x 2 max pooling of stride 2 above the ReLU (pool_k8 != 0): the input gradient has the pooled shape
  // [B, H/2, W/2, K] and `act` the full one [B, H, W, K]; pool_k8 = K / 8, pool_hp = H / 2, pool_wp = W / 2.
  int pool_k8, pool_hp, pool_wp;
};

// Two 16-bit elements of each gradient, added in fp32 (one rounding) and rounded to the 16-bit type to nearest-even;
// a NaN sum becomes the canonical quiet NaN.
template <bool F16>
__device__ __forceinline__ uint32_t add_pair(uint32_t g, uint32_t s) {
  const float lo = __fadd_rn(lane_lo<F16>(g), lane_lo<F16>(s)), hi = __fadd_rn(lane_hi<F16>(g), lane_hi<F16>(s));
  return f32_to_elem_bits<F16>(lo) | (f32_to_elem_bits<F16>(hi) << 16);
}

__device__ __forceinline__ uint32_t relu_pass2(uint32_t g, uint32_t a, uint32_t nan_add) {
  const uint32_t mag = a & 0x7FFF7FFFu;
  const uint32_t nonzero = mag + 0x7FFF7FFFu, nan = mag + nan_add;   // top bit of each half-word
  const uint32_t ok = nonzero & ~nan & ~a;
  return g & prmt(ok, 0u, 0xBB99);  // top bits replicated over their half-words
}

template <bool RELU>
__device__ __forceinline__ uint4 load_gradient(const uint4* __restrict__ dO, int64_t v, const ReluSource& src) {
  uint4 g = __ldg(dO + v);
  if (RELU) {
    const uint4 a = __ldg(src.act + v);
    if (src.skip) {
      const uint4 k = __ldg(src.skip + v);
      g = src.f16 ? make_uint4(add_pair<true>(g.x, k.x), add_pair<true>(g.y, k.y), add_pair<true>(g.z, k.z), add_pair<true>(g.w, k.w))
                  : make_uint4(add_pair<false>(g.x, k.x), add_pair<false>(g.y, k.y), add_pair<false>(g.z, k.z),
                               add_pair<false>(g.w, k.w));
    }
    g = make_uint4(relu_pass2(g.x, a.x, src.nan_add), relu_pass2(g.y, a.y, src.nan_add), relu_pass2(g.z, a.z, src.nan_add),
                   relu_pass2(g.w, a.w, src.nan_add));
    if (src.grad) src.grad[v] = g;
  }
  return g;
}

// Pooling backward for one 32-bit word (two channels) of a window: a[0..3] are the activation words at the window's
// four positions in the order (0,0), (0,1), (1,0), (1,1), g the pooled gradient's word. Per channel the gradient goes
// to the first largest activation if that is a number greater than zero. Both channels at once, in 16-bit lanes:
// key = the pattern where it is a positive number, else 0 (15 bits; patterns of positive numbers order like the
// numbers); (key_a | 0x8000) - key_b keeps the lane's top bit exactly when key_a >= key_b, and no borrow leaves the
// lane. Position t wins when its key is strictly above every earlier one and not below any later one; position 0
// must also be non-zero (a later winner is above a key that is at least zero).
__device__ __forceinline__ void pool_select2(const uint32_t (&a)[4], uint32_t g, uint32_t nan_add, uint32_t (&out)[4]) {
  constexpr uint32_t H = 0x80008000u;
  uint32_t k[4];
#pragma unroll
  for (int t = 0; t < 4; ++t) k[t] = relu_pass2(a[t], a[t], nan_add);
  const uint32_t ge01 = (k[0] | H) - k[1], ge02 = (k[0] | H) - k[2], ge03 = (k[0] | H) - k[3];
  const uint32_t ge12 = (k[1] | H) - k[2], ge13 = (k[1] | H) - k[3], ge23 = (k[2] | H) - k[3];
  const uint32_t nz0 = k[0] + 0x7FFF7FFFu;  // top bit of a lane: its key is not zero
  uint32_t win[4];
  win[0] = (ge01 & ge02 & ge03) & (nz0 & H);
  win[1] = (~ge01 & ge12 & ge13) & H;
  win[2] = (~ge02 & ~ge12 & ge23) & H;
  win[3] = (~ge03 & ~ge13 & ~ge23) & H;
#pragma unroll
  for (int t = 0; t < 4; ++t) out[t] = g & prmt(win[t], 0u, 0xBB99);  // top bits replicated over their half-words
}

// The four vectors a thread prunes and their numbers in dL/dO (>= nvec: none). Without pooling they are the thread's
// slots of four consecutive 256-vector stripes (every load of a warp is one contiguous 512 bytes). With pooling a
// thread owns the four pixels of one window for one 8-channel vector: it reads the pooled gradient once and the four
// activation vectors, and its lanes still hold neighbouring channel vectors of the same pixel.
template <bool RELU>
__device__ __forceinline__ void load_unit(const uint4* __restrict__ dO, int64_t nvec, const ReluSource& src,
                                          int64_t (&vi)[kVecPerThread], uint4 (&in)[kVecPerThread]) {
  if (RELU && src.pool_k8 != 0) {
    const int64_t u = (int64_t)blockIdx.x * kThreads + threadIdx.x;  // number of the pooled gradient's vector
    const bool live = u < (nvec >> 2);
    int64_t pix00 = 0;
    int cv = 0;
    if (live) {  // (the host checked that the number of pooled vectors fits 32 bits)
      const uint32_t window = (uint32_t)u / (uint32_t)src.pool_k8;
      cv = (int)((uint32_t)u - window * (uint32_t)src.pool_k8);
      const uint32_t t = window / (uint32_t)src.pool_wp;
      const uint32_t j = window - t * (uint32_t)src.pool_wp;
      const uint32_t b = t / (uint32_t)src.pool_hp;
      const uint32_t i = t - b * (uint32_t)src.pool_hp;
      pix00 = (((int64_t)b * src.pool_hp * 2 + 2 * i) * src.pool_wp + j) * 2;  // pixel (2i, 2j) of image b
    }
    uint4 a[4];
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      vi[it] = live ? (pix00 + (it >> 1) * (2 * src.pool_wp) + (it & 1)) * src.pool_k8 + cv : nvec;
      a[it] = live ? __ldg(src.act + vi[it]) : make_uint4(0u, 0u, 0u, 0u);
    }
    uint4 g = live ? __ldg(dO + u) : make_uint4(0u, 0u, 0u, 0u);
    if (live && src.skip) {  // a second gradient of the pooled shape (a residual connection joins below the pooling)
      const uint4 k = __ldg(src.skip + u);
      g = src.f16 ? make_uint4(add_pair<true>(g.x, k.x), add_pair<true>(g.y, k.y), add_pair<true>(g.z, k.z), add_pair<true>(g.w, k.w))
                  : make_uint4(add_pair<false>(g.x, k.x), add_pair<false>(g.y, k.y), add_pair<false>(g.z, k.z),
                               add_pair<false>(g.w, k.w));
    }
    uint32_t ox[4], oy[4], oz[4], ow[4];
    const uint32_t ax[4] = {a[0].x, a[1].x, a[2].x, a[3].x}, ay[4] = {a[0].y, a[1].y, a[2].y, a[3].y},
                   az[4] = {a[0].z, a[1].z, a[2].z, a[3].z}, aw[4] = {a[0].w, a[1].w, a[2].w, a[3].w};
    pool_select2(ax, g.x, src.nan_add, ox);
    pool_select2(ay, g.y, src.nan_add, oy);
    pool_select2(az, g.z, src.nan_add, oz);
    pool_select2(aw, g.w, src.nan_add, ow);
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      in[it] = make_uint4(ox[it], oy[it], oz[it], ow[it]);
      if (live && src.grad) src.grad[vi[it]] = in[it];
    }
    return;
  }
  const int64_t base = (int64_t)blockIdx.x * (kThreads * kVecPerThread) + threadIdx.x;
#pragma unroll
  for (int it = 0; it < kVecPerThread; ++it) {
    vi[it] = base + (int64_t)it * kThreads;
    in[it] = (vi[it] < nvec) ? load_gradient<RELU>(dO, vi[it], src) : make_uint4(0, 0, 0, 0);
  }
}

// M: group size; LANES = lanes that share a group (1, 2 or 4).
template <int M, int SCHEME, bool F16>
__global__ void __launch_bounds__(kThreads)
prune_kernel(const uint4* __restrict__ dO, int64_t nvec, int n, uint32_t seed_lo, uint32_t seed_hi,
             uint4* __restrict__ dense, uint2* __restrict__ values, uint8_t* __restrict__ meta,
             uint8_t* __restrict__ mask) {
  ptx::wait_for_previous_grid();
  ptx::launch_dependents();  // only once this grid's own predecessor is done: at most one grid ever waits behind a running one
  constexpr int LANES = (M <= 8) ? 1 : M / 8;
  constexpr int SUB = (M == 4) ? 4 : 8;  // elements of this thread that share a group
  const int64_t base = (int64_t)blockIdx.x * (kThreads * kVecPerThread) + threadIdx.x;

  uint4 in[kVecPerThread];
#pragma unroll
  for (int it = 0; it < kVecPerThread; ++it) {
    const int64_t v = base + (int64_t)it * kThreads;
    in[it] = (v < nvec) ? __ldg(dO + v) : make_uint4(0, 0, 0, 0);
  }

#pragma unroll
  for (int it = 0; it < kVecPerThread; ++it) {
    const int64_t v = base + (int64_t)it * kThreads;
    const uint32_t w[4] = {in[it].x, in[it].y, in[it].z, in[it].w};
    uint32_t x[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = (i & 1) ? (w[i >> 1] >> 16) : (w[i >> 1] & 0xFFFFu);

    // ---- ranking key: larger composite = better; unique inside a group ----
    uint32_t key16[8];
    if (SCHEME == SDGP_RANDOM) {
      const uint4 o = philox4x32_10((uint32_t)v, (uint32_t)((uint64_t)v >> 32), 0u, 0u, seed_lo, seed_hi);
      const uint32_t r[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const uint32_t r16 = (i & 1) ? (r[i >> 1] >> 16) : (r[i >> 1] & 0xFFFFu);
        key16[i] = 0xFFFFu - r16;  // smallest random key ranks first
      }
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) key16[i] = x[i] & 0x7FFFu;  // |x| as an integer
    }
    const int lane_in_group = (LANES == 1) ? 0 : (threadIdx.x & (LANES - 1));
    uint32_t c[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int j = (M == 4) ? (i & 3) : (lane_in_group * 8 + i);  // position inside the group
      c[i] = (key16[i] << 5) | (uint32_t)(31 - j);                 // ties: lower position wins
    }

    // ---- keep <=> fewer than n elements of the group rank above ----
    int above[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      int cnt = 0;
#pragma unroll
      for (int o = 0; o < 8; ++o)
        if (o != i && (o / SUB) == (i / SUB)) cnt += (c[o] > c[i]) ? 1 : 0;
      above[i] = cnt;
    }
    if (LANES > 1) {
#pragma unroll
      for (int d = 1; d < LANES; ++d) {
#pragma unroll
        for (int o = 0; o < 8; ++o) {
          const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, c[o], d);
#pragma unroll
          for (int i = 0; i < 8; ++i) above[i] += (other > c[i]) ? 1 : 0;
        }
      }
    }
    uint32_t keep8 = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) keep8 |= (above[i] < n ? 1u : 0u) << i;

    // ---- survivor values ----
    uint32_t y[8];
    if (SCHEME == SDGP_RESCALED_MAGNITUDE && n < M) {  // n == m: nothing pruned, nothing rescaled
      float a[8], t[8], s[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        a[i] = lane_lo<F16>(x[i] & 0x7FFFu);
        t[i] = a[i];
        s[i] = ((keep8 >> i) & 1u) ? a[i] : 0.0f;
      }
      // balanced pairwise sums in index order; every add rounds once
#pragma unroll
      for (int width = 8; width > (8 / SUB); width >>= 1) {
#pragma unroll
        for (int i = 0; i < width / 2; ++i) {
          t[i] = __fadd_rn(t[2 * i], t[2 * i + 1]);
          s[i] = __fadd_rn(s[2 * i], s[2 * i + 1]);
        }
      }
      // M == 4: t[0], t[1] are the two groups' sums; otherwise t[0] is this lane's partial
      if (LANES > 1) {
#pragma unroll
        for (int d = 1; d < LANES; d <<= 1) {
          t[0] = __fadd_rn(t[0], __shfl_xor_sync(0xFFFFFFFFu, t[0], d));
          s[0] = __fadd_rn(s[0], __shfl_xor_sync(0xFFFFFFFFu, s[0], d));
        }
      }
      float scale[2];
#pragma unroll
      for (int g = 0; g < 2; ++g) {
        const int src = (M == 4) ? g : 0;
        scale[g] = (s[src] == 0.0f) ? 1.0f : __fdiv_rn(t[src], s[src]);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float xf = lane_lo<F16>(x[i]);
        y[i] = ((keep8 >> i) & 1u) ? f32_to_elem_bits<F16>(__fmul_rn(xf, scale[i >> 2])) : 0u;
      }
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) y[i] = ((keep8 >> i) & 1u) ? x[i] : 0u;
    }

    if (v >= nvec) continue;

    // ---- emit ----
    if (dense) dense[v] = make_uint4(y[0] | (y[1] << 16), y[2] | (y[3] << 16), y[4] | (y[5] << 16), y[6] | (y[7] << 16));
    if (mask) mask[v] = (uint8_t)keep8;
    if (values || meta) {
      uint32_t slots[4];
      uint32_t nib2 = 0;
#pragma unroll
      for (int ch = 0; ch < 2; ++ch) {
        const uint32_t nib = chunk_nibble((keep8 >> (4 * ch)) & 0xFu);
        const uint64_t quad = (uint64_t)(y[4 * ch] | (y[4 * ch + 1] << 16)) |
                              ((uint64_t)(y[4 * ch + 2] | (y[4 * ch + 3] << 16)) << 32);
        slots[2 * ch] = (uint32_t)(quad >> (16 * (nib & 3u))) & 0xFFFFu;
        slots[2 * ch + 1] = (uint32_t)(quad >> (16 * (nib >> 2))) & 0xFFFFu;
        nib2 |= nib << (4 * ch);
      }
      if (values) values[v] = make_uint2(slots[0] | (slots[1] << 16), slots[2] | (slots[3] << 16));
      if (meta) meta[v] = (uint8_t)nib2;
    }
  }
}

// ------------------------------------------------------------------------------------------
// m = 4 fast path. The two groups of a vector are processed as 16-bit SIMD lanes of one
// register: p_i = (element i of group A, element i of group B). Pairwise "i beats j" flags
// come from one packed subtraction each, the keep decision is one 3-input logic op per
// element (a threshold on the number of wins), and the compressed slots / position nibbles
// are computed on both lanes at once. About a quarter of the instructions of the generic path.

// Row pitch of the compressed outputs, in 8-element vectors: k8 per input row, kpad8 per output
// row (kpad8 == 0: same as the input). The extra vectors of a padded row are written as zero
// values with the position pair (0,1), by the thread that owns the row's last real vector.
struct OutPitch {
  int k8, kpad8;
};

// Writes one vector's outputs from the lane-paired form (see m4_prune_vector). COMPRESS: every
// 4-chunk holds at most two survivors, so values / meta can be produced.
// Output position of vector v's compressed outputs; writes the padding of a padded row when v is the row's last vector.
__device__ __forceinline__ int64_t compressed_index(int64_t v, uint2* __restrict__ values, uint8_t* __restrict__ meta,
                                                    OutPitch pitch) {
  if (pitch.kpad8 == 0) return v;
  const int64_t row = v / pitch.k8;
  const int kv = (int)(v - row * pitch.k8);
  const int64_t vo = row * pitch.kpad8 + kv;
  if (kv == pitch.k8 - 1) {
    for (int t = 1; t <= pitch.kpad8 - pitch.k8; ++t) {
      if (values) values[vo + t] = make_uint2(0u, 0u);
      if (meta) meta[vo + t] = (uint8_t)0x44;
    }
  }
  return vo;
}

__device__ __forceinline__ void emit_mask(int64_t v, uint32_t km0, uint32_t km1, uint32_t km2, uint32_t km3,
                                          uint8_t* __restrict__ mask) {
  const uint32_t t = (km0 & 0x00010001u) | (km1 & 0x00020002u) | (km2 & 0x00040004u) | (km3 & 0x00080008u);
  mask[v] = (uint8_t)((t & 0xFu) | (t >> 12));
}

// Writes one vector's outputs from the lane-paired form (see m4_prune_vector). COMPRESS: every
// 4-chunk holds at most two survivors, so values / meta can be produced.
template <bool COMPRESS>
__device__ __forceinline__ void emit_packed(int64_t v, uint32_t y0, uint32_t y1, uint32_t y2, uint32_t y3,
                                            uint32_t km0, uint32_t km1, uint32_t km2, uint32_t km3,
                                            uint4* __restrict__ dense, uint2* __restrict__ values,
                                            uint8_t* __restrict__ meta, uint8_t* __restrict__ mask,
                                            OutPitch pitch) {
  const int64_t vo = COMPRESS ? compressed_index(v, values, meta, pitch) : v;
  if (dense)
    dense[v] = make_uint4(prmt(y0, y1, 0x5410), prmt(y2, y3, 0x5410), prmt(y0, y1, 0x7632), prmt(y2, y3, 0x7632));
  if (mask) emit_mask(v, km0, km1, km2, km3, mask);
  if (COMPRESS && (values || meta)) {
    uint32_t slot0, slot1, nib2;
    compressed_slots(y0, y1, y2, y3, km0, km1, km2, km3, slot0, slot1, nib2);
    if (values) values[vo] = make_uint2(prmt(slot0, slot1, 0x5410), prmt(slot0, slot1, 0x7632));
    if (meta) meta[vo] = (uint8_t)nib2;
  }
}

template <int N, int SCHEME, bool F16, bool RELU>
__global__ void __launch_bounds__(kThreads, kBlocksPerSm<SCHEME, RELU>)
prune_m4_kernel(const uint4* __restrict__ dO, int64_t nvec, uint32_t seed_lo, uint32_t seed_hi,
                uint4* __restrict__ dense, uint2* __restrict__ values, uint8_t* __restrict__ meta,
                uint8_t* __restrict__ mask, OutPitch pitch, ReluSource src) {
  ptx::wait_for_previous_grid();
  ptx::launch_dependents();  // only once this grid's own predecessor is done: at most one grid ever waits behind a running one
  uint4 in[kVecPerThread];
  int64_t vi[kVecPerThread];
  load_unit<RELU>(dO, nvec, src, vi, in);
#pragma unroll
  for (int it = 0; it < kVecPerThread; ++it) {
    const int64_t v = vi[it];
    if (v >= nvec) continue;
    const uint4 w = in[it];
    uint32_t y0, y1, y2, y3, km0, km1, km2, km3;
    if constexpr (SCHEME == SDGP_RESCALED_MAGNITUDE && N <= 2) {
      if (!dense) {  // only the compressed form is wanted: rescale the two slots instead of the eight lanes
        uint32_t slot0, slot1, nib2;
        m4_rescaled_compressed<N, F16>(w, slot0, slot1, nib2, km0, km1, km2, km3);
        const int64_t vo = compressed_index(v, values, meta, pitch);
        if (mask) emit_mask(v, km0, km1, km2, km3, mask);
        if (values) values[vo] = make_uint2(prmt(slot0, slot1, 0x5410), prmt(slot0, slot1, 0x7632));
        if (meta) meta[vo] = (uint8_t)nib2;
        continue;
      }
    }
    m4_prune_vector<N, SCHEME, F16>(w, v, seed_lo, seed_hi, y0, y1, y2, y3, km0, km1, km2, km3);
    emit_packed<(N <= 2)>(v, y0, y1, y2, y3, km0, km1, km2, km3, dense, values, meta, mask, pitch);
  }
}

// Only the rescaled scheme reads values as numbers: the other two run the same (bf16-named)
// instantiation for both element types.
template <int N, bool RELU>
cudaError_t launch_m4_n(int scheme, bool f16, const void* dO, int64_t nvec, uint64_t seed, void* dense, void* values,
                        void* meta, void* mask, OutPitch pitch, cudaStream_t stream, ReluSource src) {
  const int64_t per_block = (int64_t)kThreads * kVecPerThread;
  const int64_t blocks = (nvec + per_block - 1) / per_block;
  if (blocks == 0) return cudaSuccess;
  if (blocks > 0x7FFFFFFF) return cudaErrorInvalidValue;
  const dim3 grid((unsigned)blocks), block(kThreads);
  const uint32_t lo = (uint32_t)seed, hi = (uint32_t)(seed >> 32);
#define SDGP_LAUNCH4(S, F)                                                                      \
  launch_after_previous(prune_m4_kernel<N, S, F, RELU>, grid, block, stream, (const uint4*)dO, nvec, lo, hi, (uint4*)dense, \
                                                    (uint2*)values, (uint8_t*)meta, (uint8_t*)mask, pitch, src)
  switch (scheme) {
    case SDGP_RANDOM: SDGP_LAUNCH4(SDGP_RANDOM, false); break;
    case SDGP_MAGNITUDE: SDGP_LAUNCH4(SDGP_MAGNITUDE, false); break;
    default:
      if (f16) SDGP_LAUNCH4(SDGP_RESCALED_MAGNITUDE, true);
      else SDGP_LAUNCH4(SDGP_RESCALED_MAGNITUDE, false);
      break;
  }
#undef SDGP_LAUNCH4
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Groups of 8, 16 or 32 with n <= 2: the survivors are the elements whose composite key
// (rank key << 5 | 31 - position, unique inside a group) reaches the group's n-th largest key.
// Each thread finds the two largest keys of its 8 elements with a max/min network, groups that
// span 2 or 4 lanes merge their pairs through xor-shuffles, and the outputs are written from the
// same lane-paired form as the m = 4 path.

template <int M, int N, int SCHEME, bool F16, bool RELU>
__global__ void __launch_bounds__(kThreads, kBlocksPerSm<SCHEME, RELU>)
prune_top2_kernel(const uint4* __restrict__ dO, int64_t nvec, uint32_t seed_lo, uint32_t seed_hi,
                  uint4* __restrict__ dense, uint2* __restrict__ values, uint8_t* __restrict__ meta,
                  uint8_t* __restrict__ mask, OutPitch pitch, ReluSource src) {
  ptx::wait_for_previous_grid();
  ptx::launch_dependents();  // only once this grid's own predecessor is done: at most one grid ever waits behind a running one
  constexpr int LANES = M / 8;
  static_assert(N == 1 || N == 2, "threshold selection keeps one or two elements");
  uint4 in[kVecPerThread];
  int64_t vi[kVecPerThread];
  load_unit<RELU>(dO, nvec, src, vi, in);
#pragma unroll
  for (int it = 0; it < kVecPerThread; ++it) {
    const int64_t v = vi[it];
    uint32_t y0, y1, y2, y3, km0, km1, km2, km3;
    if constexpr (SCHEME == SDGP_RESCALED_MAGNITUDE) {
      if (!dense) {  // (uniform over the grid: every lane of a group takes the same branch and meets in the shuffles)
        uint32_t slot0, slot1, nib2;
        top2_rescaled_compressed<M, F16>(in[it], N, (int)(threadIdx.x & (LANES - 1)), 0xFFFFFFFFu, slot0, slot1, nib2, km0, km1,
                                         km2, km3);
        if (v < nvec) {
          const int64_t vo = compressed_index(v, values, meta, pitch);
          if (mask) emit_mask(v, km0, km1, km2, km3, mask);
          if (values) values[vo] = make_uint2(prmt(slot0, slot1, 0x5410), prmt(slot0, slot1, 0x7632));
          if (meta) meta[vo] = (uint8_t)nib2;
        }
        continue;
      }
    }
    top2_prune_vector<M, SCHEME, F16>(in[it], v, seed_lo, seed_hi, N, (int)(threadIdx.x & (LANES - 1)), 0xFFFFFFFFu, y0, y1, y2,
                                      y3, km0, km1, km2, km3);
    if (v < nvec) emit_packed<true>(v, y0, y1, y2, y3, km0, km1, km2, km3, dense, values, meta, mask, pitch);
  }
}

template <int M, int N, bool RELU>
cudaError_t launch_top2(int scheme, bool f16, const void* dO, int64_t nvec, uint64_t seed, void* dense, void* values,
                        void* meta, void* mask, OutPitch pitch, cudaStream_t stream, ReluSource src) {
  const int64_t per_block = (int64_t)kThreads * kVecPerThread;
  const int64_t blocks = (nvec + per_block - 1) / per_block;
  if (blocks == 0) return cudaSuccess;
  if (blocks > 0x7FFFFFFF) return cudaErrorInvalidValue;
  const dim3 grid((unsigned)blocks), block(kThreads);
  const uint32_t lo = (uint32_t)seed, hi = (uint32_t)(seed >> 32);
#define SDGP_LAUNCH_T2(S, F)                                                                         \
  launch_after_previous(prune_top2_kernel<M, N, S, F, RELU>, grid, block, stream, (const uint4*)dO, nvec, lo, hi, (uint4*)dense, \
                                                         (uint2*)values, (uint8_t*)meta, (uint8_t*)mask, pitch, src)
  switch (scheme) {
    case SDGP_RANDOM: SDGP_LAUNCH_T2(SDGP_RANDOM, false); break;
    case SDGP_MAGNITUDE: SDGP_LAUNCH_T2(SDGP_MAGNITUDE, false); break;
    default:
      if (f16) SDGP_LAUNCH_T2(SDGP_RESCALED_MAGNITUDE, true);
      else SDGP_LAUNCH_T2(SDGP_RESCALED_MAGNITUDE, false);
      break;
  }
#undef SDGP_LAUNCH_T2
  return cudaGetLastError();
}

template <int M>
cudaError_t launch_m(int scheme, bool f16, const void* dO, int64_t nvec, int n, uint64_t seed, void* dense,
                     void* values, void* meta, void* mask, cudaStream_t stream) {
  const int64_t per_block = (int64_t)kThreads * kVecPerThread;
  const int64_t blocks = (nvec + per_block - 1) / per_block;
  if (blocks == 0) return cudaSuccess;
  if (blocks > 0x7FFFFFFF) return cudaErrorInvalidValue;
  const dim3 grid((unsigned)blocks), block(kThreads);
  const uint32_t lo = (uint32_t)seed, hi = (uint32_t)(seed >> 32);
  // Plain launch, without programmatic stream serialisation (the kernel's griddepcontrol
  // instructions then do nothing). With the attribute, a stream of back-to-back masked-mode steps
  // (this kernel, dense data-gradient kernel, this kernel, ...) stopped making progress on B200 after
  // a few steps, at 4:8, 8:16 and 4:32 alike; the m = 4 and top-2 kernels run thousands of such steps
  // with it. The cause was not found; the overlap it would buy on this slower path is small.
#define SDGP_LAUNCH(S, F)                                                                           \
  prune_kernel<M, S, F><<<grid, block, 0, stream>>>((const uint4*)dO, nvec, n, lo, hi, (uint4*)dense,       \
                                                    (uint2*)values, (uint8_t*)meta, (uint8_t*)mask)
  switch (scheme) {
    case SDGP_RANDOM: SDGP_LAUNCH(SDGP_RANDOM, false); break;
    case SDGP_MAGNITUDE: SDGP_LAUNCH(SDGP_MAGNITUDE, false); break;
    default:
      if (f16) SDGP_LAUNCH(SDGP_RESCALED_MAGNITUDE, true);
      else SDGP_LAUNCH(SDGP_RESCALED_MAGNITUDE, false);
      break;
  }
#undef SDGP_LAUNCH
  return cudaGetLastError();
}

template <bool RELU>
cudaError_t launch_prune_src(const void* dO, int64_t rows, int64_t K, int n, int m, int scheme, uint64_t seed, void* dense,
                             void* values, void* meta, void* mask, cudaStream_t stream, int64_t k_pad, int dtype,
                             ReluSource src) {
  const bool f16 = dtype == SDGP_FP16;
  const int64_t nvec = rows * (K / 8);
  OutPitch pitch = {(int)(K / 8), 0};
  if (k_pad != 0 && k_pad != K) {
    if (k_pad < K || k_pad % 8 != 0 || n > 2) return cudaErrorInvalidValue;  // padded rows exist only for compressed outputs
    pitch.kpad8 = (int)(k_pad / 8);
  }
  switch (m) {
    case 4:
      switch (n) {
        case 1: return launch_m4_n<1, RELU>(scheme, f16, dO, nvec, seed, dense, values, meta, mask, pitch, stream, src);
        case 2: return launch_m4_n<2, RELU>(scheme, f16, dO, nvec, seed, dense, values, meta, mask, pitch, stream, src);
        case 3: return launch_m4_n<3, RELU>(scheme, f16, dO, nvec, seed, dense, values, meta, mask, pitch, stream, src);
        default: return launch_m4_n<4, RELU>(scheme, f16, dO, nvec, seed, dense, values, meta, mask, pitch, stream, src);
      }
#define SDGP_M_CASE(M)                                                                                     \
  case M:                                                                                                  \
    if (n == 1) return launch_top2<M, 1, RELU>(scheme, f16, dO, nvec, seed, dense, values, meta, mask, pitch, stream, src); \
    if (n == 2) return launch_top2<M, 2, RELU>(scheme, f16, dO, nvec, seed, dense, values, meta, mask, pitch, stream, src); \
    if (RELU) return cudaErrorInvalidValue; /* the generic kernel reads dL/dO itself */                      \
    return launch_m<M>(scheme, f16, dO, nvec, n, seed, dense, values, meta, mask, stream);
    SDGP_M_CASE(8)
    SDGP_M_CASE(16)
    SDGP_M_CASE(32)
#undef SDGP_M_CASE
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

cudaError_t launch_prune(const void* dO, int64_t rows, int64_t K, int n, int m, int scheme,
                         uint64_t seed, void* dense, void* values, void* meta, void* mask,
                         cudaStream_t stream, int64_t k_pad, int dtype) {
  return launch_prune_src<false>(dO, rows, K, n, m, scheme, seed, dense, values, meta, mask, stream, k_pad, dtype,
                                 ReluSource{nullptr, nullptr, 0u, nullptr, 0, 0, 0, 0});
}

cudaError_t launch_relu_backward_prune(const void* dY, const void* act, int64_t rows, int64_t K, int n, int m, int scheme,
                                       uint64_t seed, void* grad, void* dense, void* values, void* meta, void* mask,
                                       cudaStream_t stream, int dtype, const void* skip) {
  const ReluSource src = {(const uint4*)act, (uint4*)grad, dtype == SDGP_FP16 ? 0x03FF03FFu : 0x007F007Fu,
                          (const uint4*)skip, dtype == SDGP_FP16 ? 1 : 0, 0, 0, 0};
  return launch_prune_src<true>(dY, rows, K, n, m, scheme, seed, dense, values, meta, mask, stream, 0, dtype, src);
}

cudaError_t launch_maxpool_relu_backward_prune(const void* dYp, const void* act, int B, int H, int W, int64_t K, int n, int m,
                                               int scheme, uint64_t seed, void* grad, void* dense, void* values, void* meta,
                                               void* mask, cudaStream_t stream, int dtype, const void* skip_pooled) {
  const ReluSource src = {(const uint4*)act, (uint4*)grad, dtype == SDGP_FP16 ? 0x03FF03FFu : 0x007F007Fu,
                          (const uint4*)skip_pooled, dtype == SDGP_FP16 ? 1 : 0, (int)(K / 8), H / 2, W / 2};
  return launch_prune_src<true>(dYp, (int64_t)B * H * W, K, n, m, scheme, seed, dense, values, meta, mask, stream, 0, dtype, src);
}

}  // namespace sdgp
