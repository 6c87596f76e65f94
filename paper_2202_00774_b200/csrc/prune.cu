// N:M pruning of the output data gradient (Algorithm 1, Section 3.2), sm_100a.
//
// One thread owns one aligned run of 8 bf16 elements (a single 128-bit load). Groups of
// m = 4 (two per thread) and m = 8 (one per thread) are ranked inside the thread; groups of
// 16 and 32 span 2 and 4 neighbouring lanes, which trade their keys with warp shuffles.
// The kernel is a pure stream: 2 B read per element, 1 B of compressed values, 1/8 B of
// position metadata (+ 1/8 B mask, + 2 B dense copy when asked for), every output indexed by
// the same 8-element vector number so all stores coalesce.
#include <cuda_bf16.h>

#include "sdgp_internal.cuh"

namespace sdgp {
namespace {

constexpr int kThreads = 256;
constexpr int kVecPerThread = 4;

// Philox4x32-10 (Salmon et al., SC'11): ten rounds, Weyl key schedule.
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return make_uint4(c0, c1, c2, c3);
}

// fp32 -> bf16 bits, round to nearest even; any NaN becomes 0x7FC0.
__device__ __forceinline__ uint32_t f32_to_bf16_bits(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FC0u;
  u += 0x7FFFu + ((u >> 16) & 1u);
  return u >> 16;
}

// Survivor positions of a 4-chunk from its 4-bit keep mask: pad with the lowest unused
// positions up to two, ascending; entry = p0 | p1 << 2 (16 nibbles packed in 64 bits).
__device__ __forceinline__ uint32_t chunk_nibble(uint32_t keep4) {
  return (uint32_t)(0x444E4DCC49884444ull >> (4 * keep4)) & 0xFu;
}

// M: group size; LANES = lanes that share a group (1, 2 or 4).
template <int M, int SCHEME>
__global__ void __launch_bounds__(kThreads)
prune_kernel(const uint4* __restrict__ dO, int64_t nvec, int n, uint32_t seed_lo, uint32_t seed_hi,
             uint4* __restrict__ dense, uint2* __restrict__ values, uint8_t* __restrict__ meta,
             uint8_t* __restrict__ mask) {
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
    if (SCHEME == SDGP_RESCALED_MAGNITUDE) {
      float a[8], t[8], s[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        a[i] = __uint_as_float((x[i] & 0x7FFFu) << 16);
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
        const float xf = __uint_as_float(x[i] << 16);
        y[i] = ((keep8 >> i) & 1u) ? f32_to_bf16_bits(__fmul_rn(xf, scale[i >> 2])) : 0u;
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

template <int LUT>
__device__ __forceinline__ uint32_t lop3(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, %4;" : "=r"(d) : "r"(a), "r"(b), "r"(c), "n"(LUT));
  return d;
}

// prmt.b32, default mode: result byte n = byte (sel nibble n & 7) of {b,a}; a nibble with its
// top bit set replicates that byte's sign bit over the whole result byte instead.
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

// Truth-table byte of "at least NEED of the three inputs are true", with optional input negation.
template <int NEED>
__host__ __device__ constexpr int threshold_lut(bool na, bool nb, bool nc) {
  int lut = 0;
  for (int idx = 0; idx < 8; ++idx) {
    const int a = ((idx >> 2) & 1) ^ (na ? 1 : 0), b = ((idx >> 1) & 1) ^ (nb ? 1 : 0), c = (idx & 1) ^ (nc ? 1 : 0);
    if (a + b + c >= NEED) lut |= 1 << idx;
  }
  return lut;
}


// Survivors of both lanes times their group's scale, rounded to bf16 (nearest even). When both
// group sums are finite every product is finite and the hardware's packed conversion applies;
// otherwise (Inf or NaN in the group) each value goes through the explicit rounding, which
// stores any NaN as 0x7FC0.
__device__ __forceinline__ void rescale_packed(uint32_t& y0, uint32_t& y1, uint32_t& y2, uint32_t& y3, uint32_t km0,
                                               uint32_t km1, uint32_t km2, uint32_t km3, float scA, float scB,
                                               float tA, float tB) {
  const bool finite = (__float_as_uint(tA) & 0x7F800000u) != 0x7F800000u &&
                      (__float_as_uint(tB) & 0x7F800000u) != 0x7F800000u;
  if (finite) {
#define SDGP_RESCALE_FAST(y, km)                                                                    \
  {                                                                                                 \
    const __nv_bfloat162 h = __floats2bfloat162_rn(__fmul_rn(__uint_as_float(y << 16), scA),        \
                                                   __fmul_rn(__uint_as_float(y & 0xFFFF0000u), scB)); \
    y = (*(const uint32_t*)&h) & km;                                                                \
  }
    SDGP_RESCALE_FAST(y0, km0) SDGP_RESCALE_FAST(y1, km1) SDGP_RESCALE_FAST(y2, km2) SDGP_RESCALE_FAST(y3, km3)
#undef SDGP_RESCALE_FAST
  } else {
#define SDGP_RESCALE_SLOW(y, km)                                                                    \
  y = (f32_to_bf16_bits(__fmul_rn(__uint_as_float(y << 16), scA)) |                                 \
       (f32_to_bf16_bits(__fmul_rn(__uint_as_float(y & 0xFFFF0000u), scB)) << 16)) & km;
    SDGP_RESCALE_SLOW(y0, km0) SDGP_RESCALE_SLOW(y1, km1) SDGP_RESCALE_SLOW(y2, km2) SDGP_RESCALE_SLOW(y3, km3)
#undef SDGP_RESCALE_SLOW
  }
}

// Writes one vector's outputs from the lane-paired form: y_i = (element i, element i + 4) after
// pruning, km_i = 0xFFFF in the lanes of kept elements. COMPRESS: every 4-chunk holds at most two
// survivors, so values / meta can be produced.
// Row pitch of the compressed outputs, in 8-element vectors: k8 per input row, kpad8 per output
// row (kpad8 == 0: same as the input). The extra vectors of a padded row are written as zero
// values with the position pair (0,1), by the thread that owns the row's last real vector.
struct OutPitch {
  int k8, kpad8;
};

template <bool COMPRESS>
__device__ __forceinline__ void emit_packed(int64_t v, uint32_t y0, uint32_t y1, uint32_t y2, uint32_t y3,
                                            uint32_t km0, uint32_t km1, uint32_t km2, uint32_t km3,
                                            uint4* __restrict__ dense, uint2* __restrict__ values,
                                            uint8_t* __restrict__ meta, uint8_t* __restrict__ mask,
                                            OutPitch pitch) {
  int64_t vo = v;
  if (pitch.kpad8 != 0) {
    const int64_t row = v / pitch.k8;
    const int kv = (int)(v - row * pitch.k8);
    vo = row * pitch.kpad8 + kv;
    if (COMPRESS && kv == pitch.k8 - 1) {
      for (int t = 1; t <= pitch.kpad8 - pitch.k8; ++t) {
        if (values) values[vo + t] = make_uint2(0u, 0u);
        if (meta) meta[vo + t] = (uint8_t)0x44;
      }
    }
  }
  if (dense)
    dense[v] = make_uint4(prmt(y0, y1, 0x5410), prmt(y2, y3, 0x5410), prmt(y0, y1, 0x7632), prmt(y2, y3, 0x7632));
  if (mask) {
    const uint32_t t = (km0 & 0x00010001u) | (km1 & 0x00020002u) | (km2 & 0x00040004u) | (km3 & 0x00080008u);
    mask[v] = (uint8_t)((t & 0xFu) | (t >> 12));
  }
  if (COMPRESS && (values || meta)) {
    // At most two survivors per chunk. Positions: p1 = last survivor, but at least 1;
    // p0 = first survivor if there are two, else 0 (the pad takes the lowest free position).
    const uint32_t k23 = km2 | km3;
    const uint32_t slot0 = y0 | (y1 & k23) | (y2 & km3);
    const uint32_t slot1 = y3 | (~km3 & (y2 | (~km2 & y1)));
    if (values) values[vo] = make_uint2(prmt(slot0, slot1, 0x5410), prmt(slot0, slot1, 0x7632));
    if (meta) {
      const uint32_t pos0 = (km1 & k23 & 0x00010001u) | (km2 & km3 & 0x00020002u);
      const uint32_t pos1 = 0x00010001u + (k23 & 0x00010001u) + (km3 & 0x00010001u);
      const uint32_t nib = pos0 + 4u * pos1;
      meta[vo] = (uint8_t)((nib & 0xFu) | (nib >> 12));
    }
  }
}

template <int N, int SCHEME>
__global__ void __launch_bounds__(kThreads)
prune_m4_kernel(const uint4* __restrict__ dO, int64_t nvec, uint32_t seed_lo, uint32_t seed_hi,
                uint4* __restrict__ dense, uint2* __restrict__ values, uint8_t* __restrict__ meta,
                uint8_t* __restrict__ mask, OutPitch pitch) {
  constexpr int NEED = 4 - N;  // an element is kept iff it beats at least 4 - n of the other three
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
    if (v >= nvec) continue;
    const uint4 w = in[it];
    // lanes: low half = group A (elements 0..3), high half = group B (elements 4..7)
    const uint32_t p0 = prmt(w.x, w.z, 0x5410), p1 = prmt(w.x, w.z, 0x7632);
    const uint32_t p2 = prmt(w.y, w.w, 0x5410), p3 = prmt(w.y, w.w, 0x7632);

    uint32_t km0, km1, km2, km3;  // 0xFFFF in a lane whose element is kept
    if (N == 4) {
      km0 = km1 = km2 = km3 = 0xFFFFFFFFu;
    } else if (SCHEME == SDGP_RANDOM) {
      const uint4 o = philox4x32_10((uint32_t)v, (uint32_t)((uint64_t)v >> 32), 0u, 0u, seed_lo, seed_hi);
      // 16-bit keys; smaller ranks first, equal keys: lower index. e(i,j) = r_j - r_i has its
      // sign bit set iff j ranks before i (j < i in key), i.e. iff i loses against j (for i < j).
      const uint32_t rA0 = o.x & 0xFFFFu, rA1 = o.x >> 16, rA2 = o.y & 0xFFFFu, rA3 = o.y >> 16;
      const uint32_t rB0 = o.z & 0xFFFFu, rB1 = o.z >> 16, rB2 = o.w & 0xFFFFu, rB3 = o.w >> 16;
#define SDGP_KEEP4(r0, r1, r2, r3, k0, k1, k2, k3)                                                \
  {                                                                                                \
    const uint32_t e01 = r1 - r0, e02 = r2 - r0, e03 = r3 - r0, e12 = r2 - r1, e13 = r3 - r1,      \
                   e23 = r3 - r2;                                                                  \
    k0 = lop3<threshold_lut<NEED>(true, true, true)>(e01, e02, e03);                               \
    k1 = lop3<threshold_lut<NEED>(false, true, true)>(e01, e12, e13);                              \
    k2 = lop3<threshold_lut<NEED>(false, false, true)>(e02, e12, e23);                             \
    k3 = lop3<threshold_lut<NEED>(false, false, false)>(e03, e13, e23);                            \
  }
      uint32_t a0, a1, a2, a3, b0, b1, b2, b3;  // keep flags in bit 31
      SDGP_KEEP4(rA0, rA1, rA2, rA3, a0, a1, a2, a3)
      SDGP_KEEP4(rB0, rB1, rB2, rB3, b0, b1, b2, b3)
#undef SDGP_KEEP4
      // replicate the two sign bits over their 16-bit lanes
      km0 = prmt(a0, b0, 0xFFBB); km1 = prmt(a1, b1, 0xFFBB);
      km2 = prmt(a2, b2, 0xFFBB); km3 = prmt(a3, b3, 0xFFBB);
    } else {
      // |x| as 15-bit integers. d(i,j) = (a_i | 0x8000) - a_j per lane never borrows across lanes
      // and has bit 15 of the lane set iff a_i >= a_j, i.e. iff i beats j (i < j: ties to i).
      constexpr uint32_t H = 0x80008000u;
      const uint32_t h0 = p0 | H, h1 = p1 | H, h2 = p2 | H;
      const uint32_t l1 = p1 & ~H, l2 = p2 & ~H, l3 = p3 & ~H;
      const uint32_t d01 = h0 - l1, d02 = h0 - l2, d03 = h0 - l3, d12 = h1 - l2, d13 = h1 - l3, d23 = h2 - l3;
      const uint32_t k0 = lop3<threshold_lut<NEED>(false, false, false)>(d01, d02, d03);
      const uint32_t k1 = lop3<threshold_lut<NEED>(true, false, false)>(d01, d12, d13);
      const uint32_t k2 = lop3<threshold_lut<NEED>(true, true, false)>(d02, d12, d23);
      const uint32_t k3 = lop3<threshold_lut<NEED>(true, true, true)>(d03, d13, d23);
      km0 = prmt(k0, 0, 0xBB99); km1 = prmt(k1, 0, 0xBB99);
      km2 = prmt(k2, 0, 0xBB99); km3 = prmt(k3, 0, 0xBB99);
    }

    uint32_t y0 = p0 & km0, y1 = p1 & km1, y2 = p2 & km2, y3 = p3 & km3;  // pruned lanes are +0.0
    if (SCHEME == SDGP_RESCALED_MAGNITUDE && N != 4) {
      // per group: scale = sum|x| / sum|kept x|, balanced pairwise sums in index order
      const float tA = __fadd_rn(__fadd_rn(__uint_as_float((p0 << 16) & 0x7FFF0000u), __uint_as_float((p1 << 16) & 0x7FFF0000u)),
                                 __fadd_rn(__uint_as_float((p2 << 16) & 0x7FFF0000u), __uint_as_float((p3 << 16) & 0x7FFF0000u)));
      const float tB = __fadd_rn(__fadd_rn(__uint_as_float(p0 & 0x7FFF0000u), __uint_as_float(p1 & 0x7FFF0000u)),
                                 __fadd_rn(__uint_as_float(p2 & 0x7FFF0000u), __uint_as_float(p3 & 0x7FFF0000u)));
      const float sA = __fadd_rn(__fadd_rn(__uint_as_float((y0 << 16) & 0x7FFF0000u), __uint_as_float((y1 << 16) & 0x7FFF0000u)),
                                 __fadd_rn(__uint_as_float((y2 << 16) & 0x7FFF0000u), __uint_as_float((y3 << 16) & 0x7FFF0000u)));
      const float sB = __fadd_rn(__fadd_rn(__uint_as_float(y0 & 0x7FFF0000u), __uint_as_float(y1 & 0x7FFF0000u)),
                                 __fadd_rn(__uint_as_float(y2 & 0x7FFF0000u), __uint_as_float(y3 & 0x7FFF0000u)));
      const float scA = (sA == 0.0f) ? 1.0f : __fdiv_rn(tA, sA);
      const float scB = (sB == 0.0f) ? 1.0f : __fdiv_rn(tB, sB);
      rescale_packed(y0, y1, y2, y3, km0, km1, km2, km3, scA, scB, tA, tB);
    }

    emit_packed<(N <= 2)>(v, y0, y1, y2, y3, km0, km1, km2, km3, dense, values, meta, mask, pitch);
  }
}

template <int N>
cudaError_t launch_m4_n(int scheme, const void* dO, int64_t nvec, uint64_t seed, void* dense, void* values,
                        void* meta, void* mask, OutPitch pitch, cudaStream_t stream) {
  const int64_t per_block = (int64_t)kThreads * kVecPerThread;
  const int64_t blocks = (nvec + per_block - 1) / per_block;
  if (blocks == 0) return cudaSuccess;
  if (blocks > 0x7FFFFFFF) return cudaErrorInvalidValue;
  const dim3 grid((unsigned)blocks), block(kThreads);
  const uint32_t lo = (uint32_t)seed, hi = (uint32_t)(seed >> 32);
#define SDGP_LAUNCH4(S)                                                                         \
  prune_m4_kernel<N, S><<<grid, block, 0, stream>>>((const uint4*)dO, nvec, lo, hi, (uint4*)dense, \
                                                    (uint2*)values, (uint8_t*)meta, (uint8_t*)mask, pitch)
  switch (scheme) {
    case SDGP_RANDOM: SDGP_LAUNCH4(SDGP_RANDOM); break;
    case SDGP_MAGNITUDE: SDGP_LAUNCH4(SDGP_MAGNITUDE); break;
    default: SDGP_LAUNCH4(SDGP_RESCALED_MAGNITUDE); break;
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

__device__ __forceinline__ void merge_top2(uint32_t& hi, uint32_t& lo, uint32_t hi2, uint32_t lo2) {
  const uint32_t h = max(hi, hi2);
  lo = max(min(hi, hi2), max(lo, lo2));
  hi = h;
}

template <int M, int N, int SCHEME>
__global__ void __launch_bounds__(kThreads)
prune_top2_kernel(const uint4* __restrict__ dO, int64_t nvec, uint32_t seed_lo, uint32_t seed_hi,
                  uint4* __restrict__ dense, uint2* __restrict__ values, uint8_t* __restrict__ meta,
                  uint8_t* __restrict__ mask, OutPitch pitch) {
  constexpr int LANES = M / 8;
  static_assert(N == 1 || N == 2, "threshold selection keeps one or two elements");
  const int64_t base = (int64_t)blockIdx.x * (kThreads * kVecPerThread) + threadIdx.x;
  const uint32_t pos0 = 31u - 8u * (uint32_t)(threadIdx.x & (LANES - 1));  // tie-break bits of element 0
  uint4 in[kVecPerThread];
#pragma unroll
  for (int it = 0; it < kVecPerThread; ++it) {
    const int64_t v = base + (int64_t)it * kThreads;
    in[it] = (v < nvec) ? __ldg(dO + v) : make_uint4(0, 0, 0, 0);
  }
#pragma unroll
  for (int it = 0; it < kVecPerThread; ++it) {
    const int64_t v = base + (int64_t)it * kThreads;
    const uint4 w = in[it];
    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
    uint32_t c[8];
    if (SCHEME == SDGP_RANDOM) {
      const uint4 o = philox4x32_10((uint32_t)v, (uint32_t)((uint64_t)v >> 32), 0u, 0u, seed_lo, seed_hi);
      const uint32_t r[4] = {~o.x, ~o.y, ~o.z, ~o.w};  // smallest random key ranks first
#pragma unroll
      for (int i = 0; i < 8; ++i)
        c[i] = (((i & 1) ? (r[i >> 1] >> 11) : (r[i >> 1] << 5)) & 0x1FFFE0u) | (pos0 - i);
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i)
        c[i] = (((i & 1) ? (ww[i >> 1] >> 11) : (ww[i >> 1] << 5)) & 0xFFFE0u) | (pos0 - i);  // |x| << 5 | tie-break
    }
    uint32_t hi, lo = 0;
    if (N == 1) {
      hi = max(max(max(c[0], c[1]), max(c[2], c[3])), max(max(c[4], c[5]), max(c[6], c[7])));
#pragma unroll
      for (int d = 1; d < LANES; d <<= 1) hi = max(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, d));
    } else {
      uint32_t h1 = max(c[2], c[3]), l1 = min(c[2], c[3]), h2 = max(c[4], c[5]), l2 = min(c[4], c[5]),
               h3 = max(c[6], c[7]), l3 = min(c[6], c[7]);
      hi = max(c[0], c[1]);
      lo = min(c[0], c[1]);
      merge_top2(hi, lo, h1, l1);
      merge_top2(h2, l2, h3, l3);
      merge_top2(hi, lo, h2, l2);
#pragma unroll
      for (int d = 1; d < LANES; d <<= 1) {
        const uint32_t oh = __shfl_xor_sync(0xFFFFFFFFu, hi, d), ol = __shfl_xor_sync(0xFFFFFFFFu, lo, d);
        merge_top2(hi, lo, oh, ol);
      }
    }
    const uint32_t t1 = ((N == 1) ? hi : lo) - 1u;  // keep <=> key > t1; (t1 - key) is then negative
    const uint32_t p0 = prmt(w.x, w.z, 0x5410), p1 = prmt(w.x, w.z, 0x7632);
    const uint32_t p2 = prmt(w.y, w.w, 0x5410), p3 = prmt(w.y, w.w, 0x7632);
    const uint32_t km0 = prmt(t1 - c[0], t1 - c[4], 0xFFBB), km1 = prmt(t1 - c[1], t1 - c[5], 0xFFBB);
    const uint32_t km2 = prmt(t1 - c[2], t1 - c[6], 0xFFBB), km3 = prmt(t1 - c[3], t1 - c[7], 0xFFBB);
    uint32_t y0 = p0 & km0, y1 = p1 & km1, y2 = p2 & km2, y3 = p3 & km3;
    if (SCHEME == SDGP_RESCALED_MAGNITUDE) {
      // balanced pairwise sums in index order: elements 0..3 are the low lanes, 4..7 the high lanes
#define SDGP_SUM8(q0, q1, q2, q3)                                                                                 \
  __fadd_rn(__fadd_rn(__fadd_rn(__uint_as_float((q0 << 16) & 0x7FFF0000u), __uint_as_float((q1 << 16) & 0x7FFF0000u)), \
                      __fadd_rn(__uint_as_float((q2 << 16) & 0x7FFF0000u), __uint_as_float((q3 << 16) & 0x7FFF0000u))), \
            __fadd_rn(__fadd_rn(__uint_as_float(q0 & 0x7FFF0000u), __uint_as_float(q1 & 0x7FFF0000u)),             \
                      __fadd_rn(__uint_as_float(q2 & 0x7FFF0000u), __uint_as_float(q3 & 0x7FFF0000u))))
      float tsum = SDGP_SUM8(p0, p1, p2, p3);
      float ssum = SDGP_SUM8(y0, y1, y2, y3);
#undef SDGP_SUM8
#pragma unroll
      for (int d = 1; d < LANES; d <<= 1) {
        tsum = __fadd_rn(tsum, __shfl_xor_sync(0xFFFFFFFFu, tsum, d));
        ssum = __fadd_rn(ssum, __shfl_xor_sync(0xFFFFFFFFu, ssum, d));
      }
      const float sc = (ssum == 0.0f) ? 1.0f : __fdiv_rn(tsum, ssum);
      rescale_packed(y0, y1, y2, y3, km0, km1, km2, km3, sc, sc, tsum, tsum);
    }
    if (v < nvec) emit_packed<true>(v, y0, y1, y2, y3, km0, km1, km2, km3, dense, values, meta, mask, pitch);
  }
}

template <int M, int N>
cudaError_t launch_top2(int scheme, const void* dO, int64_t nvec, uint64_t seed, void* dense, void* values,
                        void* meta, void* mask, OutPitch pitch, cudaStream_t stream) {
  const int64_t per_block = (int64_t)kThreads * kVecPerThread;
  const int64_t blocks = (nvec + per_block - 1) / per_block;
  if (blocks == 0) return cudaSuccess;
  if (blocks > 0x7FFFFFFF) return cudaErrorInvalidValue;
  const dim3 grid((unsigned)blocks), block(kThreads);
  const uint32_t lo = (uint32_t)seed, hi = (uint32_t)(seed >> 32);
#define SDGP_LAUNCH_T2(S)                                                                            \
  prune_top2_kernel<M, N, S><<<grid, block, 0, stream>>>((const uint4*)dO, nvec, lo, hi, (uint4*)dense, \
                                                         (uint2*)values, (uint8_t*)meta, (uint8_t*)mask, pitch)
  switch (scheme) {
    case SDGP_RANDOM: SDGP_LAUNCH_T2(SDGP_RANDOM); break;
    case SDGP_MAGNITUDE: SDGP_LAUNCH_T2(SDGP_MAGNITUDE); break;
    default: SDGP_LAUNCH_T2(SDGP_RESCALED_MAGNITUDE); break;
  }
#undef SDGP_LAUNCH_T2
  return cudaGetLastError();
}

template <int M>
cudaError_t launch_m(int scheme, const void* dO, int64_t nvec, int n, uint64_t seed, void* dense,
                     void* values, void* meta, void* mask, cudaStream_t stream) {
  const int64_t per_block = (int64_t)kThreads * kVecPerThread;
  const int64_t blocks = (nvec + per_block - 1) / per_block;
  if (blocks == 0) return cudaSuccess;
  if (blocks > 0x7FFFFFFF) return cudaErrorInvalidValue;
  const dim3 grid((unsigned)blocks), block(kThreads);
  const uint32_t lo = (uint32_t)seed, hi = (uint32_t)(seed >> 32);
#define SDGP_LAUNCH(S)                                                                              \
  prune_kernel<M, S><<<grid, block, 0, stream>>>((const uint4*)dO, nvec, n, lo, hi, (uint4*)dense, \
                                                 (uint2*)values, (uint8_t*)meta, (uint8_t*)mask)
  switch (scheme) {
    case SDGP_RANDOM: SDGP_LAUNCH(SDGP_RANDOM); break;
    case SDGP_MAGNITUDE: SDGP_LAUNCH(SDGP_MAGNITUDE); break;
    default: SDGP_LAUNCH(SDGP_RESCALED_MAGNITUDE); break;
  }
#undef SDGP_LAUNCH
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_prune(const void* dO, int64_t rows, int64_t K, int n, int m, int scheme,
                         uint64_t seed, void* dense, void* values, void* meta, void* mask,
                         cudaStream_t stream, int64_t k_pad) {
  const int64_t nvec = rows * (K / 8);
  OutPitch pitch = {(int)(K / 8), 0};
  if (k_pad != 0 && k_pad != K) {
    if (k_pad < K || k_pad % 8 != 0 || n > 2) return cudaErrorInvalidValue;  // padded rows exist only for compressed outputs
    pitch.kpad8 = (int)(k_pad / 8);
  }
  switch (m) {
    case 4:
      switch (n) {
        case 1: return launch_m4_n<1>(scheme, dO, nvec, seed, dense, values, meta, mask, pitch, stream);
        case 2: return launch_m4_n<2>(scheme, dO, nvec, seed, dense, values, meta, mask, pitch, stream);
        case 3: return launch_m4_n<3>(scheme, dO, nvec, seed, dense, values, meta, mask, pitch, stream);
        default: return launch_m4_n<4>(scheme, dO, nvec, seed, dense, values, meta, mask, pitch, stream);
      }
#define SDGP_M_CASE(M)                                                                                     \
  case M:                                                                                                  \
    if (n == 1) return launch_top2<M, 1>(scheme, dO, nvec, seed, dense, values, meta, mask, pitch, stream); \
    if (n == 2) return launch_top2<M, 2>(scheme, dO, nvec, seed, dense, values, meta, mask, pitch, stream); \
    return launch_m<M>(scheme, dO, nvec, n, seed, dense, values, meta, mask, stream);
    SDGP_M_CASE(8)
    SDGP_M_CASE(16)
    SDGP_M_CASE(32)
#undef SDGP_M_CASE
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace sdgp
