// Device code shared by the stand-alone prune kernels and the prune stage fused into the
// data-gradient kernel: the Philox generator, bf16 rounding, packed-lane helpers and the
// per-vector m = 4 pruning function (Algorithm 1, Section 3.2).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sdgp.h"

namespace sdgp {
namespace {

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


// Element type of the 16-bit tensors. Ranking and selection only read bit patterns (the pattern
// with the sign cleared orders bf16 and IEEE binary16 alike); the type matters where the rescale
// of Section 3.2 reads values as numbers and rounds the survivors. F16 = false: bf16, true: binary16.

// fp32 -> binary16 bits, round to nearest even (hardware conversion); any NaN becomes 0x7E00.
__device__ __forceinline__ uint32_t f32_to_f16_bits(float f) {
  const uint32_t h = __half_as_ushort(__float2half_rn(f));
  return ((h & 0x7FFFu) > 0x7C00u) ? 0x7E00u : h;
}

template <bool F16>
__device__ __forceinline__ uint32_t f32_to_elem_bits(float f) {
  return F16 ? f32_to_f16_bits(f) : f32_to_bf16_bits(f);
}

// The element in the low / high half of a lane-paired register as fp32 (exact).
template <bool F16>
__device__ __forceinline__ float lane_lo(uint32_t p) {
  return F16 ? __half2float(__ushort_as_half((unsigned short)(p & 0xFFFFu))) : __uint_as_float(p << 16);
}
template <bool F16>
__device__ __forceinline__ float lane_hi(uint32_t p) {
  return F16 ? __half2float(__ushort_as_half((unsigned short)(p >> 16))) : __uint_as_float(p & 0xFFFF0000u);
}
// ... and their magnitudes
// (the absolute value of the fp32 number clears the same sign bit, NaN payloads included, and rides on the add that
// consumes it instead of costing an integer instruction)
template <bool F16>
__device__ __forceinline__ float lane_lo_abs(uint32_t p) { return fabsf(lane_lo<F16>(p)); }
template <bool F16>
__device__ __forceinline__ float lane_hi_abs(uint32_t p) { return fabsf(lane_hi<F16>(p)); }

// Two fp32 values rounded to nearest even and packed (low, high): hardware conversion, finite inputs.
template <bool F16>
__device__ __forceinline__ uint32_t pack_pair_rn(float lo, float hi) {
  if (F16) {
    const __half2 h = __floats2half2_rn(lo, hi);
    return *(const uint32_t*)&h;
  }
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *(const uint32_t*)&h;
}

// Balanced pairwise sum, in index order, of the magnitudes in the low (high) halves of four
// lane-paired registers: (|e0| + |e1|) + (|e2| + |e3|), every add rounded once.
template <bool F16>
__device__ __forceinline__ float sum4_lo_abs(uint32_t q0, uint32_t q1, uint32_t q2, uint32_t q3) {
  return __fadd_rn(__fadd_rn(lane_lo_abs<F16>(q0), lane_lo_abs<F16>(q1)), __fadd_rn(lane_lo_abs<F16>(q2), lane_lo_abs<F16>(q3)));
}
template <bool F16>
__device__ __forceinline__ float sum4_hi_abs(uint32_t q0, uint32_t q1, uint32_t q2, uint32_t q3) {
  return __fadd_rn(__fadd_rn(lane_hi_abs<F16>(q0), lane_hi_abs<F16>(q1)), __fadd_rn(lane_hi_abs<F16>(q2), lane_hi_abs<F16>(q3)));
}

// Survivors of both lanes times their group's scale, rounded to the element type (nearest even).
// When both group sums are finite every fp32 product is finite and the hardware's packed
// conversion applies (a product beyond the binary16 range rounds to infinity, as IEEE says);
// otherwise (Inf or NaN in the group) each value goes through the explicit rounding, which
// stores any NaN as the one canonical quiet NaN.
template <bool F16>
__device__ __forceinline__ void rescale_packed(uint32_t& y0, uint32_t& y1, uint32_t& y2, uint32_t& y3, uint32_t km0,
                                               uint32_t km1, uint32_t km2, uint32_t km3, float scA, float scB,
                                               float tA, float tB) {
  const bool finite = (__float_as_uint(tA) & 0x7F800000u) != 0x7F800000u &&
                      (__float_as_uint(tB) & 0x7F800000u) != 0x7F800000u;
  if (finite) {
#define SDGP_RESCALE_FAST(y, km) \
  y = pack_pair_rn<F16>(__fmul_rn(lane_lo<F16>(y), scA), __fmul_rn(lane_hi<F16>(y), scB)) & km;
    SDGP_RESCALE_FAST(y0, km0) SDGP_RESCALE_FAST(y1, km1) SDGP_RESCALE_FAST(y2, km2) SDGP_RESCALE_FAST(y3, km3)
#undef SDGP_RESCALE_FAST
  } else {
#define SDGP_RESCALE_SLOW(y, km)                                                 \
  y = (f32_to_elem_bits<F16>(__fmul_rn(lane_lo<F16>(y), scA)) |                  \
       (f32_to_elem_bits<F16>(__fmul_rn(lane_hi<F16>(y), scB)) << 16)) & km;
    SDGP_RESCALE_SLOW(y0, km0) SDGP_RESCALE_SLOW(y1, km1) SDGP_RESCALE_SLOW(y2, km2) SDGP_RESCALE_SLOW(y3, km3)
#undef SDGP_RESCALE_SLOW
  }
}

// The two m = 4 groups of one 8-element vector w (vector number v of the tensor, which fixes the
// random keys). Lane-paired form: register i holds (element i, element i + 4) in its low / high
// 16 bits. Out: y_i = pruned (and, for the rescaled scheme, rescaled) values, km_i = 0xFFFF in
// the lanes of kept elements.
template <int N, int SCHEME, bool F16 = false>
__device__ __forceinline__ void m4_prune_vector(const uint4& w, int64_t v, uint32_t seed_lo, uint32_t seed_hi,
                                                uint32_t& y0, uint32_t& y1, uint32_t& y2, uint32_t& y3,
                                                uint32_t& km0, uint32_t& km1, uint32_t& km2, uint32_t& km3) {
  constexpr int NEED = 4 - N;  // an element is kept iff it beats at least 4 - n of the other three
  // lanes: low half = group A (elements 0..3), high half = group B (elements 4..7)
  const uint32_t p0 = prmt(w.x, w.z, 0x5410), p1 = prmt(w.x, w.z, 0x7632);
  const uint32_t p2 = prmt(w.y, w.w, 0x5410), p3 = prmt(w.y, w.w, 0x7632);

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

  y0 = p0 & km0; y1 = p1 & km1; y2 = p2 & km2; y3 = p3 & km3;  // pruned lanes are +0.0
  if (SCHEME == SDGP_RESCALED_MAGNITUDE && N != 4) {
    // per group: scale = sum|x| / sum|kept x|, balanced pairwise sums in index order
    const float tA = sum4_lo_abs<F16>(p0, p1, p2, p3), tB = sum4_hi_abs<F16>(p0, p1, p2, p3);
    const float sA = sum4_lo_abs<F16>(y0, y1, y2, y3), sB = sum4_hi_abs<F16>(y0, y1, y2, y3);
    const float scA = (sA == 0.0f) ? 1.0f : __fdiv_rn(tA, sA);
    const float scB = (sB == 0.0f) ? 1.0f : __fdiv_rn(tB, sB);
    rescale_packed<F16>(y0, y1, y2, y3, km0, km1, km2, km3, scA, scB, tA, tB);
  }

}

// Compressed form of both 4-chunks of a vector (at most two survivors per chunk): slot0 / slot1 =
// lane-paired values at the chunk's survivor positions p0 < p1 (p1 = last survivor, at least 1;
// p0 = first survivor if there are two, else 0: the pad takes the lowest free position), and
// nib2 = the two position nibbles p0 | p1 << 2 (chunk A in bits 0-3, chunk B in bits 4-7).
__device__ __forceinline__ void compressed_slots(uint32_t y0, uint32_t y1, uint32_t y2, uint32_t y3, uint32_t km0,
                                                 uint32_t km1, uint32_t km2, uint32_t km3, uint32_t& slot0,
                                                 uint32_t& slot1, uint32_t& nib2) {
  const uint32_t k23 = km2 | km3;
  slot0 = y0 | (y1 & k23) | (y2 & km3);
  slot1 = y3 | (~km3 & (y2 | (~km2 & y1)));
  const uint32_t pos0 = (km1 & k23 & 0x00010001u) | (km2 & km3 & 0x00020002u);
  const uint32_t pos1 = 0x00010001u + (k23 & 0x00010001u) + (km3 & 0x00010001u);
  const uint32_t nib = pos0 + 4u * pos1;
  nib2 = (nib & 0xFu) | ((nib >> 12) & 0xF0u);
}

// Magnitude function with the L1 rescale of Section 3.2 for callers that want only the compressed form (n <= 2):
// the same survivors, sums, divisions and roundings as m4_prune_vector, but the survivors are gathered into their two
// slots first, so that the sum over the kept elements is one addition of the slots' magnitudes (the other terms of
// the tree are +0, which changes nothing) and only the slots are multiplied and rounded: half the conversions,
// products and roundings of the lane-by-lane form. A slot that holds the pad of a chunk with one survivor is +0 and
// stays +0 (its product with a finite positive scale is +0; where the scale is not finite it is masked out: with one
// survivor the pad is slot 1 if the survivor is element 0 and slot 0 otherwise).
// km_i: keep masks as m4_prune_vector returns them (for the bit mask output).
template <int N, bool F16>
__device__ __forceinline__ void m4_rescaled_compressed(const uint4& w, uint32_t& slot0, uint32_t& slot1, uint32_t& nib2,
                                                       uint32_t& km0, uint32_t& km1, uint32_t& km2, uint32_t& km3) {
  static_assert(N == 1 || N == 2, "a compressed form exists for one or two survivors");
  uint32_t y0, y1, y2, y3;
  m4_prune_vector<N, SDGP_MAGNITUDE, F16>(w, 0, 0u, 0u, y0, y1, y2, y3, km0, km1, km2, km3);  // survivors, not yet rescaled
  const uint32_t p0 = prmt(w.x, w.z, 0x5410), p1 = prmt(w.x, w.z, 0x7632);
  const uint32_t p2 = prmt(w.y, w.w, 0x5410), p3 = prmt(w.y, w.w, 0x7632);
  const float tA = sum4_lo_abs<F16>(p0, p1, p2, p3), tB = sum4_hi_abs<F16>(p0, p1, p2, p3);
  compressed_slots(y0, y1, y2, y3, km0, km1, km2, km3, slot0, slot1, nib2);
  const float a0 = lane_lo<F16>(slot0), b0 = lane_hi<F16>(slot0), a1 = lane_lo<F16>(slot1), b1 = lane_hi<F16>(slot1);
  const float sA = __fadd_rn(fabsf(a0), fabsf(a1)), sB = __fadd_rn(fabsf(b0), fabsf(b1));
  const float scA = (sA == 0.0f) ? 1.0f : __fdiv_rn(tA, sA);
  const float scB = (sB == 0.0f) ? 1.0f : __fdiv_rn(tB, sB);
  const bool finite = (__float_as_uint(tA) & 0x7F800000u) != 0x7F800000u &&
                      (__float_as_uint(tB) & 0x7F800000u) != 0x7F800000u;
  if (finite) {  // every product is finite: the hardware's packed rounding applies (see rescale_packed)
    slot0 = pack_pair_rn<F16>(__fmul_rn(a0, scA), __fmul_rn(b0, scB));
    slot1 = pack_pair_rn<F16>(__fmul_rn(a1, scA), __fmul_rn(b1, scB));
  } else {
    const uint32_t keep0 = N == 2 ? 0xFFFFFFFFu : km0, keep1 = N == 2 ? 0xFFFFFFFFu : ~km0;
    slot0 = (f32_to_elem_bits<F16>(__fmul_rn(a0, scA)) | (f32_to_elem_bits<F16>(__fmul_rn(b0, scB)) << 16)) & keep0;
    slot1 = (f32_to_elem_bits<F16>(__fmul_rn(a1, scA)) | (f32_to_elem_bits<F16>(__fmul_rn(b1, scB)) << 16)) & keep1;
  }
}

// Groups of 8, 16 or 32 with n <= 2 (Algorithm 1 with the same three pruning functions): the survivors are the
// elements whose composite key (rank key << 5 | 31 - position, unique inside a group) reaches the group's n-th
// largest. The M / 8 vectors of a group are held by M / 8 neighbouring lanes (lane bits 0 and up; `part` = this
// lane's number among them, i.e. which eighth of the group the vector is); each lane finds the two largest keys
// of its 8 elements with a max/min network and the lanes merge their pairs through xor-shuffles, which every
// lane named in `lanes` must execute together. Output in the lane-paired form of m4_prune_vector.
__device__ __forceinline__ void merge_top2(uint32_t& hi, uint32_t& lo, uint32_t hi2, uint32_t lo2) {
  const uint32_t h = max(hi, hi2);
  lo = max(min(hi, hi2), max(lo, lo2));
  hi = h;
}

// Composite keys of the 8 elements of vector w (number v in the tensor); pos0 = tie-break bits of element 0.
template <int SCHEME>
__device__ __forceinline__ void top2_keys(const uint4& w, int64_t v, uint32_t seed_lo, uint32_t seed_hi, uint32_t pos0,
                                          uint32_t (&c)[8]) {
  const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
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
}

// The two largest of eight keys.
__device__ __forceinline__ void top2_of_8(const uint32_t (&c)[8], uint32_t& hi, uint32_t& lo) {
  uint32_t h1 = max(c[2], c[3]), l1 = min(c[2], c[3]), h2 = max(c[4], c[5]), l2 = min(c[4], c[5]),
           h3 = max(c[6], c[7]), l3 = min(c[6], c[7]);
  hi = max(c[0], c[1]);
  lo = min(c[0], c[1]);
  merge_top2(hi, lo, h1, l1);
  merge_top2(h2, l2, h3, l3);
  merge_top2(hi, lo, h2, l2);
}

// Lane-paired values and keep masks of a vector whose elements with key > t1 survive.
__device__ __forceinline__ void top2_apply(const uint4& w, const uint32_t (&c)[8], uint32_t t1, uint32_t& p0, uint32_t& p1,
                                           uint32_t& p2, uint32_t& p3, uint32_t& y0, uint32_t& y1, uint32_t& y2, uint32_t& y3,
                                           uint32_t& km0, uint32_t& km1, uint32_t& km2, uint32_t& km3) {
  p0 = prmt(w.x, w.z, 0x5410); p1 = prmt(w.x, w.z, 0x7632);
  p2 = prmt(w.y, w.w, 0x5410); p3 = prmt(w.y, w.w, 0x7632);
  km0 = prmt(t1 - c[0], t1 - c[4], 0xFFBB); km1 = prmt(t1 - c[1], t1 - c[5], 0xFFBB);  // (t1 - key) negative <=> kept
  km2 = prmt(t1 - c[2], t1 - c[6], 0xFFBB); km3 = prmt(t1 - c[3], t1 - c[7], 0xFFBB);
  y0 = p0 & km0; y1 = p1 & km1; y2 = p2 & km2; y3 = p3 & km3;
}

template <int M, int SCHEME, bool F16 = false>
__device__ __forceinline__ void top2_prune_vector(const uint4& w, int64_t v, uint32_t seed_lo, uint32_t seed_hi, int n,
                                                  int part, unsigned lanes, uint32_t& y0, uint32_t& y1, uint32_t& y2,
                                                  uint32_t& y3, uint32_t& km0, uint32_t& km1, uint32_t& km2,
                                                  uint32_t& km3) {
  constexpr int LANES = M / 8;
  uint32_t c[8], hi, lo;
  top2_keys<SCHEME>(w, v, seed_lo, seed_hi, 31u - 8u * (uint32_t)part, c);
  top2_of_8(c, hi, lo);
#pragma unroll
  for (int d = 1; d < LANES; d <<= 1) {
    const uint32_t oh = __shfl_xor_sync(lanes, hi, d), ol = __shfl_xor_sync(lanes, lo, d);
    merge_top2(hi, lo, oh, ol);
  }
  uint32_t p0, p1, p2, p3;
  top2_apply(w, c, ((n == 1) ? hi : lo) - 1u, p0, p1, p2, p3, y0, y1, y2, y3, km0, km1, km2, km3);
  if (SCHEME == SDGP_RESCALED_MAGNITUDE) {
    // balanced pairwise sums in index order: elements 0..3 are the low lanes, 4..7 the high lanes
    float tsum = __fadd_rn(sum4_lo_abs<F16>(p0, p1, p2, p3), sum4_hi_abs<F16>(p0, p1, p2, p3));
    float ssum = __fadd_rn(sum4_lo_abs<F16>(y0, y1, y2, y3), sum4_hi_abs<F16>(y0, y1, y2, y3));
#pragma unroll
    for (int d = 1; d < LANES; d <<= 1) {
      tsum = __fadd_rn(tsum, __shfl_xor_sync(lanes, tsum, d));
      ssum = __fadd_rn(ssum, __shfl_xor_sync(lanes, ssum, d));
    }
    const float sc = (ssum == 0.0f) ? 1.0f : __fdiv_rn(tsum, ssum);
    rescale_packed<F16>(y0, y1, y2, y3, km0, km1, km2, km3, sc, sc, tsum, tsum);
  }
}

// top2_prune_vector for the magnitude function with the L1 rescale, for callers that want only the compressed form:
// as m4_rescaled_compressed, the survivors of the vector's two chunks are gathered into the slots first; a chunk's share of
// the sum over the kept elements is then one addition of its slots' magnitudes (a group keeps at most two elements, so
// every other term of the oracle's tree is +0) and only the slots are scaled and rounded.
template <int M, bool F16>
__device__ __forceinline__ void top2_rescaled_compressed(const uint4& w, int n, int part, unsigned lanes, uint32_t& slot0,
                                                         uint32_t& slot1, uint32_t& nib2, uint32_t& km0, uint32_t& km1,
                                                         uint32_t& km2, uint32_t& km3) {
  constexpr int LANES = M / 8;
  uint32_t y0, y1, y2, y3;
  top2_prune_vector<M, SDGP_MAGNITUDE, F16>(w, 0, 0u, 0u, n, part, lanes, y0, y1, y2, y3, km0, km1, km2, km3);  // not yet rescaled
  const uint32_t p0 = prmt(w.x, w.z, 0x5410), p1 = prmt(w.x, w.z, 0x7632);
  const uint32_t p2 = prmt(w.y, w.w, 0x5410), p3 = prmt(w.y, w.w, 0x7632);
  float tsum = __fadd_rn(sum4_lo_abs<F16>(p0, p1, p2, p3), sum4_hi_abs<F16>(p0, p1, p2, p3));
  compressed_slots(y0, y1, y2, y3, km0, km1, km2, km3, slot0, slot1, nib2);
  const float a0 = lane_lo<F16>(slot0), b0 = lane_hi<F16>(slot0), a1 = lane_lo<F16>(slot1), b1 = lane_hi<F16>(slot1);
  float ssum = __fadd_rn(__fadd_rn(fabsf(a0), fabsf(a1)), __fadd_rn(fabsf(b0), fabsf(b1)));
#pragma unroll
  for (int d = 1; d < LANES; d <<= 1) {
    tsum = __fadd_rn(tsum, __shfl_xor_sync(lanes, tsum, d));
    ssum = __fadd_rn(ssum, __shfl_xor_sync(lanes, ssum, d));
  }
  const float sc = (ssum == 0.0f) ? 1.0f : __fdiv_rn(tsum, ssum);
  if ((__float_as_uint(tsum) & 0x7F800000u) != 0x7F800000u) {  // finite sums: finite scale, a +0 pad stays +0
    slot0 = pack_pair_rn<F16>(__fmul_rn(a0, sc), __fmul_rn(b0, sc));
    slot1 = pack_pair_rn<F16>(__fmul_rn(a1, sc), __fmul_rn(b1, sc));
  } else {
    // which slots hold survivors: slot 1 if anything but element 0 of the chunk is kept, slot 0 if element 0 is kept or two are
    const uint32_t keep1 = km1 | km2 | km3, keep0 = km0 | (km1 & km2) | (km3 & (km1 | km2));
    slot0 = (f32_to_elem_bits<F16>(__fmul_rn(a0, sc)) | (f32_to_elem_bits<F16>(__fmul_rn(b0, sc)) << 16)) & keep0;
    slot1 = (f32_to_elem_bits<F16>(__fmul_rn(a1, sc)) | (f32_to_elem_bits<F16>(__fmul_rn(b1, sc)) << 16)) & keep1;
  }
}

// One group of 16 whose two vectors (numbers v and v + 1) are held by the same thread.
template <int SCHEME, bool F16 = false>
__device__ __forceinline__ void top2_prune_group16(const uint4& wa, const uint4& wb, int64_t v, uint32_t seed_lo,
                                                   uint32_t seed_hi, int n, uint32_t (&ya)[4], uint32_t (&kma)[4],
                                                   uint32_t (&yb)[4], uint32_t (&kmb)[4]) {
  uint32_t ca[8], cb[8], hi, lo, hb, lb;
  top2_keys<SCHEME>(wa, v, seed_lo, seed_hi, 31u, ca);
  top2_keys<SCHEME>(wb, v + 1, seed_lo, seed_hi, 23u, cb);
  top2_of_8(ca, hi, lo);
  top2_of_8(cb, hb, lb);
  merge_top2(hi, lo, hb, lb);
  const uint32_t t1 = ((n == 1) ? hi : lo) - 1u;
  uint32_t pa[4], pb[4];
  top2_apply(wa, ca, t1, pa[0], pa[1], pa[2], pa[3], ya[0], ya[1], ya[2], ya[3], kma[0], kma[1], kma[2], kma[3]);
  top2_apply(wb, cb, t1, pb[0], pb[1], pb[2], pb[3], yb[0], yb[1], yb[2], yb[3], kmb[0], kmb[1], kmb[2], kmb[3]);
  if (SCHEME == SDGP_RESCALED_MAGNITUDE) {
    // the same tree as across two lanes: (sum of elements 0..7) + (sum of elements 8..15)
    const float ta = __fadd_rn(sum4_lo_abs<F16>(pa[0], pa[1], pa[2], pa[3]), sum4_hi_abs<F16>(pa[0], pa[1], pa[2], pa[3]));
    const float tb = __fadd_rn(sum4_lo_abs<F16>(pb[0], pb[1], pb[2], pb[3]), sum4_hi_abs<F16>(pb[0], pb[1], pb[2], pb[3]));
    const float sa = __fadd_rn(sum4_lo_abs<F16>(ya[0], ya[1], ya[2], ya[3]), sum4_hi_abs<F16>(ya[0], ya[1], ya[2], ya[3]));
    const float sb = __fadd_rn(sum4_lo_abs<F16>(yb[0], yb[1], yb[2], yb[3]), sum4_hi_abs<F16>(yb[0], yb[1], yb[2], yb[3]));
    const float tsum = __fadd_rn(ta, tb), ssum = __fadd_rn(sa, sb);
    const float sc = (ssum == 0.0f) ? 1.0f : __fdiv_rn(tsum, ssum);
    rescale_packed<F16>(ya[0], ya[1], ya[2], ya[3], kma[0], kma[1], kma[2], kma[3], sc, sc, tsum, tsum);
    rescale_packed<F16>(yb[0], yb[1], yb[2], yb[3], kmb[0], kmb[1], kmb[2], kmb[3], sc, sc, tsum, tsum);
  }
}

}  // namespace
}  // namespace sdgp
