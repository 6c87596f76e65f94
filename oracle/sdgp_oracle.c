/*
 * CPU oracle for Structured Data Gradient Pruning (SDGP).
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, plain, obviously-correct
 * statement of what the GPU library computes. It shares no code, header,
 * table or helper with the CUDA path and is never called from it; only the
 * tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * What follows the paper directly:
 *   - Algorithm 1 (group loop over the last, stride-1 dimension, zero-initialised
 *     copy, pruning function P applied to each m-element group);
 *   - Section 3.2 pruning functions (random / magnitude / rescaled magnitude) and
 *     the worked example there (rank by magnitude, prune the smallest m-n,
 *     restore survivors to their original positions);
 *   - Section 2.1 / Fig. 2-3 data-gradient contraction (the reduction runs over the
 *     output-channel dimension, which is the pruned one).
 *   - Section 2.1 / Fig. 2 (backward pass: a layer's dL/dO is what the layer above hands down), Section 3.1
 *     (the pruned tensor is a copy: the unpruned dL/dO still feeds the weight gradient) and Section 3.3
 *     (the many exact zeros of dL/dO come from the ReLU): oracle_relu_backward forms dL/dO from the
 *     gradient above a ReLU and that ReLU's activation; pruning it is then Algorithm 1 unchanged.
 *
 * Readings taken where the paper is silent (each is listed in the design notes):
 *   - ties between equal magnitudes go to the lower index;
 *   - magnitude order is the order of the bf16 bit pattern with the sign cleared;
 *   - the L1 rescale is per group, in fp32, with a fixed balanced summation tree; a group
 *     from which nothing is pruned (n == m) is returned unchanged; the per-channel reading of
 *     the same sentence is offered beside it (oracle_channel_scales);
 *   - "random" ranks elements by 16-bit keys drawn from Philox4x32-10
 *     (Salmon et al., SC'11) at a counter fixed by the element's linear index;
 *   - pruned positions hold +0.0.
 *
 * Parity status: prune (magnitude, rescaled), compressed format, dgrad linear and
 * dgrad conv are pinned by tests/ (paper's worked example, brute force,
 * invariants, library fp64 matmul / transposed convolution). The Philox round
 * function is pinned against an independent open-source engine at test time;
 * agreement with the authors' published known-answer vectors: parity unpinned.
 *
 * Storage: 16-bit floating-point tensors travel as uint16_t bit patterns, row-major.
 * Element type: bf16 (ORACLE_BF16, the default of the un-suffixed entry points) or IEEE
 * binary16 (ORACLE_FP16, the precision the paper trained in, Section 4). The type only
 * enters where a value is read as a number: the rescale of Section 3.2 and the contraction.
 * Ranking by the bit pattern with the sign cleared orders both formats by magnitude.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_ARG 1

enum { ORACLE_RANDOM = 0, ORACLE_MAGNITUDE = 1, ORACLE_RESCALED = 2 };
enum { ORACLE_BF16 = 0, ORACLE_FP16 = 1 };
#define ORACLE_MAX_M 32 /* Section 3.1: the implementation supports groups up to m = 32 */

/* ------------------------------------------------------------------ bf16 */

static float bf16_to_f32(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

double oracle_bf16_to_f64(uint16_t h) { return (double)bf16_to_f32(h); }

/* fp32 -> bf16, round to nearest, ties to even. A NaN result is stored as the one
 * canonical quiet NaN 0x7FC0: which payload an fp32 multiply by NaN returns differs
 * between processors, so the stored pattern is fixed here (a reading; the paper does
 * not discuss non-finite gradients). */
uint16_t oracle_f32_to_bf16(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)0x7FC0u;
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  return (uint16_t)(u >> 16);
}

/* ------------------------------------------------------------------ fp16 */

/* IEEE binary16 -> fp32, exact: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
static float f16_to_f32(uint16_t h) {
  int exp = (h >> 10) & 0x1F;
  int man = h & 0x3FF;
  float mag;
  if (exp == 0)
    mag = ldexpf((float)man, -24); /* zero and subnormals: man * 2^-24 */
  else if (exp == 31)
    mag = man ? NAN : INFINITY;
  else
    mag = ldexpf((float)(man + 1024), exp - 25); /* (1 + man/1024) * 2^(exp-15) */
  return (h & 0x8000u) ? -mag : mag;
}

/* fp32 -> binary16, round to nearest, ties to even: |f| is rounded to a whole multiple of
 * the binary16 spacing at its magnitude (2^(e-10) for 2^e <= |f| < 2^(e+1), e >= -14; 2^-24
 * below 2^-14), then packed. Overflow gives infinity; a NaN is stored as 0x7E00 (same
 * reading as for bf16: one canonical quiet NaN). */
uint16_t oracle_f32_to_f16(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
  uint32_t a = u & 0x7FFFFFFFu;
  if (a > 0x7F800000u) return (uint16_t)0x7E00u;
  if (a == 0x7F800000u) return (uint16_t)(sign | 0x7C00u);
  if (a == 0) return sign;
  float x = fabsf(f);
  int e;
  (void)frexpf(x, &e); /* x = frac * 2^e with frac in [0.5, 1): 2^(e-1) <= x < 2^e */
  int ue = e - 1;
  int q = (ue < -14 ? -14 : ue) - 10;      /* exponent of the spacing */
  float r = nearbyintf(ldexpf(x, -q));    /* exact scaling, then nearest-even (default rounding mode) */
  if (r == 0.0f) return sign;
  if (ue < -14) return (uint16_t)(sign | (uint16_t)r); /* subnormal; r == 1024 is the smallest normal */
  if (r == 2048.0f) {
    r = 1024.0f;
    ++ue;
  }
  if (ue > 15) return (uint16_t)(sign | 0x7C00u);
  return (uint16_t)(sign | (uint16_t)((ue + 15) << 10) | (uint16_t)((int)r - 1024));
}

double oracle_f16_to_f64(uint16_t h) { return (double)f16_to_f32(h); }

static float elem_to_f32(uint16_t bits, int dtype) { return dtype == ORACLE_FP16 ? f16_to_f32(bits) : bf16_to_f32(bits); }
static uint16_t elem_from_f32(float f, int dtype) { return dtype == ORACLE_FP16 ? oracle_f32_to_f16(f) : oracle_f32_to_bf16(f); }
static double elem_to_f64(uint16_t bits, int dtype) { return (double)elem_to_f32(bits, dtype); }

/* ---------------------------------------------------------------- Philox */

/* Philox4x32-10, Salmon et al. SC'11: ten rounds of two 32x32->64 multiplies
 * with a Weyl-sequence key schedule. */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
  const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    if (round > 0) {
      k0 += W0;
      k1 += W1;
    }
    uint64_t p0 = (uint64_t)M0 * c0;
    uint64_t p1 = (uint64_t)M1 * c2;
    uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    uint32_t n0 = hi1 ^ c1 ^ k0;
    uint32_t n1 = lo1;
    uint32_t n2 = hi0 ^ c3 ^ k1;
    uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* 16-bit random key of the element with linear index e = row*K + k.
 * One Philox block serves 8 consecutive elements: block number e>>3 is the
 * counter, the seed is the key, and element e takes half-word (e & 7) of the
 * 128-bit output (little-endian half-words of words 0..3). */
uint16_t oracle_random_key16(uint64_t seed, uint64_t e) {
  uint64_t q = e >> 3;
  uint32_t ctr[4] = {(uint32_t)q, (uint32_t)(q >> 32), 0u, 0u};
  uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t o[4];
  oracle_philox4x32_10(ctr, key, o);
  uint32_t w = o[(e >> 1) & 3];
  return (uint16_t)((e & 1) ? (w >> 16) : (w & 0xFFFFu));
}

/* ----------------------------------------------------------------- prune */

/* Balanced-tree fp32 sum: level l adds aligned neighbours of width 2^l, the
 * input padded with +0.0f up to the next power of two. */
static float tree_sum_f32(const float* a, int m) {
  float buf[ORACLE_MAX_M];
  int p = 1;
  while (p < m) p <<= 1;
  for (int j = 0; j < p; ++j) buf[j] = (j < m) ? a[j] : 0.0f;
  for (int width = p; width > 1; width >>= 1)
    for (int j = 0; j < width / 2; ++j) {
      volatile float s = buf[2 * j] + buf[2 * j + 1]; /* one rounding per add */
      buf[j] = s;
    }
  return buf[0];
}

/* P(group, n): Section 3.2. Fills keep[j] in {0,1} and out[j] (bf16 bits).
 * e0 is the linear index of the group's first element (random scheme only). */
static void prune_group(const uint16_t* x, int n, int m, int scheme, int dtype, uint64_t seed, uint64_t e0,
                        uint8_t* keep, uint16_t* out) {
  /* Rank: an index permutation ordered best-first, by a stable insertion sort
   * so that equal keys stay in index order (the lower index wins a tie). */
  int order[ORACLE_MAX_M];
  uint32_t rank_key[ORACLE_MAX_M];
  for (int j = 0; j < m; ++j) {
    order[j] = j;
    if (scheme == ORACLE_RANDOM)
      rank_key[j] = oracle_random_key16(seed, e0 + (uint64_t)j); /* smaller key ranks first */
    else
      rank_key[j] = (uint32_t)(x[j] & 0x7FFFu); /* |x| as an integer; larger ranks first */
  }
  for (int i = 1; i < m; ++i) {
    int idx = order[i];
    int pos = i;
    while (pos > 0) {
      int prev = order[pos - 1];
      int prev_is_worse = (scheme == ORACLE_RANDOM) ? (rank_key[prev] > rank_key[idx])
                                                    : (rank_key[prev] < rank_key[idx]);
      if (!prev_is_worse) break;
      order[pos] = prev;
      --pos;
    }
    order[pos] = idx;
  }
  /* Keep the first n of the ranking; restore them to their original positions. */
  for (int j = 0; j < m; ++j) {
    keep[j] = 0;
    out[j] = 0x0000u; /* zeros_like: pruned slots are +0.0 */
  }
  for (int i = 0; i < n; ++i) {
    keep[order[i]] = 1;
    out[order[i]] = x[order[i]];
  }
  if (scheme == ORACLE_RESCALED && n < m) {
    /* Rescale the survivors so that the group's L1 norm is preserved. With n == m nothing was
     * pruned, the norm is preserved as it stands and the group is returned unchanged (no
     * division takes place, so a group holding Inf or NaN is not turned into NaNs). */
    float mag_all[ORACLE_MAX_M], mag_kept[ORACLE_MAX_M];
    for (int j = 0; j < m; ++j) {
      float a = fabsf(elem_to_f32(x[j], dtype));
      mag_all[j] = a;
      mag_kept[j] = keep[j] ? a : 0.0f;
    }
    float T = tree_sum_f32(mag_all, m);
    float S = tree_sum_f32(mag_kept, m);
    volatile float scale = (S == 0.0f) ? 1.0f : T / S;
    for (int j = 0; j < m; ++j)
      if (keep[j]) {
        volatile float y = elem_to_f32(x[j], dtype) * scale;
        out[j] = elem_from_f32(y, dtype);
      }
  }
}

static int compressible(int n, int m) { return n <= 2 && (m % 4) == 0; }

/* Algorithm 1 over a [rows, K] tensor, groups of m along K.
 * Outputs (each may be NULL):
 *   dense  [rows, K]     bf16  pruned copy
 *   values [rows, K/2]   bf16  two slots per aligned 4-chunk, ascending position
 *   meta   [rows, K/16]  u16   one nibble per 4-chunk: pos0 | pos1 << 2
 *   mask   [rows, K/32]  u32   bit k%32 of word k/32 set iff element k is kept
 * values/meta need every 4-chunk to hold at most two survivors (n <= 2, m % 4 == 0)
 * and K % 16 == 0; mask needs K % 32 == 0. */
int oracle_prune_t(const uint16_t* dO, int64_t rows, int64_t K, int n, int m, int scheme, int dtype,
                   uint64_t seed, uint16_t* dense, uint16_t* values, uint16_t* meta, uint32_t* mask) {
  if (dtype != ORACLE_BF16 && dtype != ORACLE_FP16) return ORACLE_ERR_ARG;
  if (!dO || rows < 0 || K < 0 || m < 1 || m > ORACLE_MAX_M || n < 1 || n > m) return ORACLE_ERR_ARG;
  if (K % m != 0) return ORACLE_ERR_ARG;
  if (scheme < 0 || scheme > 2) return ORACLE_ERR_ARG;
  if ((values || meta) && (!compressible(n, m) || K % 16 != 0)) return ORACLE_ERR_ARG;
  if (mask && K % 32 != 0) return ORACLE_ERR_ARG;
  if (mask) memset(mask, 0, (size_t)(rows * (K / 32)) * sizeof(uint32_t));
  if (meta) memset(meta, 0, (size_t)(rows * (K / 16)) * sizeof(uint16_t));

#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r) {
    uint16_t* row_out = (uint16_t*)malloc((size_t)(K > 0 ? K : 1) * sizeof(uint16_t));
    uint8_t* row_keep = (uint8_t*)malloc((size_t)(K > 0 ? K : 1));
    for (int64_t g = 0; g < K / m; ++g) {
      uint64_t e0 = (uint64_t)r * (uint64_t)K + (uint64_t)(g * m);
      prune_group(dO + r * K + g * m, n, m, scheme, dtype, seed, e0, row_keep + g * m, row_out + g * m);
    }
    if (dense) memcpy(dense + r * K, row_out, (size_t)K * sizeof(uint16_t));
    if (mask)
      for (int64_t k = 0; k < K; ++k)
        if (row_keep[k]) mask[r * (K / 32) + k / 32] |= (1u << (k % 32));
    if (values || meta)
      for (int64_t c = 0; c < K / 4; ++c) {
        /* survivor positions of this 4-chunk, padded with the lowest free
         * positions up to two, then sorted ascending */
        int pos[2], cnt = 0;
        uint8_t taken[4] = {0, 0, 0, 0};
        for (int j = 0; j < 4; ++j)
          if (row_keep[4 * c + j]) {
            if (cnt < 2) pos[cnt] = j;
            ++cnt;
            taken[j] = 1;
          }
        for (int j = 0; j < 4 && cnt < 2; ++j)
          if (!taken[j]) {
            pos[cnt++] = j;
            taken[j] = 1;
          }
        if (pos[0] > pos[1]) {
          int t = pos[0];
          pos[0] = pos[1];
          pos[1] = t;
        }
        if (values) {
          values[r * (K / 2) + 2 * c + 0] = row_keep[4 * c + pos[0]] ? row_out[4 * c + pos[0]] : 0;
          values[r * (K / 2) + 2 * c + 1] = row_keep[4 * c + pos[1]] ? row_out[4 * c + pos[1]] : 0;
        }
        if (meta) {
          uint16_t nib = (uint16_t)(pos[0] | (pos[1] << 2));
          meta[r * (K / 16) + c / 4] |= (uint16_t)(nib << (4 * (c % 4)));
        }
      }
    free(row_out);
    free(row_keep);
  }
  return ORACLE_OK;
}

int oracle_prune(const uint16_t* dO, int64_t rows, int64_t K, int n, int m, int scheme,
                 uint64_t seed, uint16_t* dense, uint16_t* values, uint16_t* meta, uint32_t* mask) {
  return oracle_prune_t(dO, rows, K, n, m, scheme, ORACLE_BF16, seed, dense, values, meta, mask);
}

/* The other reading of the L1 rescale (Section 3.3 and the caption of Fig. 4 speak of the norm
 * being "preserved ... per channel" across batch and spatial positions, where Section 3.2 speaks
 * of the group): the survivors are those of the magnitude function, and every channel k gets one
 * scale for the whole tensor,
 *   scale[k] = sum_r |x[r,k]| / sum_r |x[r,k]| * kept[r,k]      (1 where the denominator is 0),
 * so that each channel's L1 norm over all rows is preserved. Sums in fp64, rows in ascending order.
 * The scaled tensor is never rounded to 16 bits: the scale multiplies the survivor inside the
 * contraction (see the k_scale argument of the data-gradient functions). */
int oracle_channel_scales(const uint16_t* dO, int64_t rows, int64_t K, int n, int m, int dtype, double* scale) {
  if (dtype != ORACLE_BF16 && dtype != ORACLE_FP16) return ORACLE_ERR_ARG;
  if (!dO || !scale || rows < 0 || K < 0 || m < 1 || m > ORACLE_MAX_M || n < 1 || n > m || K % m != 0)
    return ORACLE_ERR_ARG;
  double* total = (double*)calloc((size_t)(K > 0 ? K : 1), sizeof(double));
  double* kept = (double*)calloc((size_t)(K > 0 ? K : 1), sizeof(double));
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t g = 0; g < K / m; ++g) {
      uint8_t keep[ORACLE_MAX_M];
      uint16_t out[ORACLE_MAX_M];
      const uint16_t* x = dO + r * K + g * m;
      prune_group(x, n, m, ORACLE_MAGNITUDE, dtype, 0, 0, keep, out);
      for (int j = 0; j < m; ++j) {
        double a = fabs(elem_to_f64(x[j], dtype));
        total[g * m + j] += a;
        if (keep[j]) kept[g * m + j] += a;
      }
    }
  for (int64_t k = 0; k < K; ++k) scale[k] = (kept[k] == 0.0) ? 1.0 : total[k] / kept[k];
  free(total);
  free(kept);
  return ORACLE_OK;
}

/* Inverse of the compressed format: rebuild the dense [rows, K] tensor. */
int oracle_expand(const uint16_t* values, const uint16_t* meta, int64_t rows, int64_t K,
                  uint16_t* dense) {
  if (!values || !meta || !dense || K % 16 != 0) return ORACLE_ERR_ARG;
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t c = 0; c < K / 4; ++c) {
      uint16_t word = meta[r * (K / 16) + c / 4];
      int nib = (word >> (4 * (c % 4))) & 0xF;
      int p0 = nib & 3, p1 = (nib >> 2) & 3;
      for (int j = 0; j < 4; ++j) dense[r * K + 4 * c + j] = 0;
      dense[r * K + 4 * c + p0] = values[r * (K / 2) + 2 * c + 0];
      dense[r * K + 4 * c + p1] = values[r * (K / 2) + 2 * c + 1];
    }
  return ORACLE_OK;
}

/* ----------------------------------------------------------------- dgrad */

/* k_scale (nullable) in the two functions below: one factor per output channel k that multiplies
 * dOp[., k] inside the sum (the per-channel reading of the rescale, oracle_channel_scales). */

/* Fully connected data gradient (Fig. 2): dD[r, c] = sum_k dOp[r, k] * W[k, c],
 * dOp [rows, K], W [K, N] (output channels x input channels), fp64 accumulation
 * in ascending k. Rows may be a subset: row_index (nullable) lists which rows
 * of dOp to evaluate; dD then has n_rows rows in that order. */
int oracle_dgrad_linear_t(const uint16_t* dOp, const uint16_t* W, double* dD, int64_t rows, int64_t K,
                          int64_t N, const int64_t* row_index, int64_t n_rows, int dtype, const double* k_scale) {
  if (dtype != ORACLE_BF16 && dtype != ORACLE_FP16) return ORACLE_ERR_ARG;
  if (!dOp || !W || !dD || rows < 0 || K < 0 || N < 0) return ORACLE_ERR_ARG;
  int64_t count = row_index ? n_rows : rows;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < count; ++i) {
    int64_t r = row_index ? row_index[i] : i;
    for (int64_t c = 0; c < N; ++c) {
      double acc = 0.0;
      for (int64_t k = 0; k < K; ++k)
        acc += elem_to_f64(dOp[r * K + k], dtype) * (k_scale ? k_scale[k] : 1.0) * elem_to_f64(W[k * N + c], dtype);
      dD[i * N + c] = acc;
    }
  }
  return ORACLE_OK;
}

int oracle_dgrad_linear(const uint16_t* dOp, const uint16_t* W, double* dD, int64_t rows, int64_t K,
                        int64_t N, const int64_t* row_index, int64_t n_rows) {
  return oracle_dgrad_linear_t(dOp, W, dD, rows, K, N, row_index, n_rows, ORACLE_BF16, NULL);
}

/* Convolution data gradient (Fig. 3). Forward layer: cross-correlation
 *   O[b,p,q,co] = sum_{r,s,ci} D[b, p*stride - pad + r, q*stride - pad + s, ci] * W[co,r,s,ci]
 * so the gradient w.r.t. the input is
 *   dD[b,h,w,ci] = sum over (r,s,co) and the (p,q) with p*stride - pad + r == h,
 *                  q*stride - pad + s == w of dOp[b,p,q,co] * W[co,r,s,ci].
 * dOp NHWC [B,P,Q,Cout], W [Cout,R,S,Cin], dD NHWC [B,H,Wd,Cin] in fp64.
 * pixel_index (nullable) lists flattened (b*H + h)*Wd + w positions to evaluate. */
int oracle_dgrad_conv2d_t(const uint16_t* dOp, const uint16_t* W, double* dD, int B, int H, int Wd,
                          int Cin, int Cout, int R, int S, int stride, int pad,
                          const int64_t* pixel_index, int64_t n_pixels, int dtype, const double* k_scale) {
  if (dtype != ORACLE_BF16 && dtype != ORACLE_FP16) return ORACLE_ERR_ARG;
  if (!dOp || !W || !dD || stride < 1 || pad < 0 || R < 1 || S < 1) return ORACLE_ERR_ARG;
  int P = (H + 2 * pad - R) / stride + 1;
  int Q = (Wd + 2 * pad - S) / stride + 1;
  if (P < 1 || Q < 1) return ORACLE_ERR_ARG;
  int64_t count = pixel_index ? n_pixels : (int64_t)B * H * Wd;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < count; ++i) {
    int64_t pix = pixel_index ? pixel_index[i] : i;
    int w = (int)(pix % Wd);
    int h = (int)((pix / Wd) % H);
    int b = (int)(pix / ((int64_t)Wd * H));
    for (int ci = 0; ci < Cin; ++ci) {
      double acc = 0.0;
      for (int r = 0; r < R; ++r) {
        int hp = h + pad - r;
        if (hp < 0 || hp % stride != 0) continue;
        int p = hp / stride;
        if (p >= P) continue;
        for (int s = 0; s < S; ++s) {
          int wq = w + pad - s;
          if (wq < 0 || wq % stride != 0) continue;
          int q = wq / stride;
          if (q >= Q) continue;
          const uint16_t* g = dOp + (((int64_t)b * P + p) * Q + q) * Cout;
          for (int co = 0; co < Cout; ++co)
            acc += elem_to_f64(g[co], dtype) * (k_scale ? k_scale[co] : 1.0) *
                   elem_to_f64(W[(((int64_t)co * R + r) * S + s) * Cin + ci], dtype);
        }
      }
      dD[i * Cin + ci] = acc;
    }
  }
  return ORACLE_OK;
}

int oracle_dgrad_conv2d(const uint16_t* dOp, const uint16_t* W, double* dD, int B, int H, int Wd,
                        int Cin, int Cout, int R, int S, int stride, int pad,
                        const int64_t* pixel_index, int64_t n_pixels) {
  return oracle_dgrad_conv2d_t(dOp, W, dD, B, H, Wd, Cin, Cout, R, S, stride, pad, pixel_index, n_pixels, ORACLE_BF16,
                               NULL);
}

/* Grouped convolution (the 3x3 convolutions of RegNetX, Section 4): the channels fall into `groups` groups;
 * output channel co belongs to group co / (Cout / groups) and sees only the Cin / groups input channels of
 * its group, so W is [Cout, R, S, Cin / groups] and
 *   O[b,p,q,co] = sum_{r,s,cj} D[b, p*stride - pad + r, q*stride - pad + s, g(co) * Cin/groups + cj] * W[co,r,s,cj].
 * The gradient w.r.t. the input therefore sums, for input channel ci of group g = ci / (Cin / groups), over
 * the output channels of that group only:
 *   dD[b,h,w,ci] = sum over (r,s), the (p,q) with p*stride - pad + r == h, q*stride - pad + s == w, and the
 *                  co of group g, of dOp[b,p,q,co] * W[co,r,s, ci - g * Cin/groups].
 * Pruning (Algorithm 1) runs along the output channels of dL/dO as for any other layer; it does not know
 * about the convolution's groups. groups == 1 is oracle_dgrad_conv2d_t. */
int oracle_dgrad_conv2d_grouped_t(const uint16_t* dOp, const uint16_t* W, double* dD, int B, int H, int Wd,
                                  int Cin, int Cout, int R, int S, int stride, int pad, int groups,
                                  const int64_t* pixel_index, int64_t n_pixels, int dtype) {
  if (dtype != ORACLE_BF16 && dtype != ORACLE_FP16) return ORACLE_ERR_ARG;
  if (!dOp || !W || !dD || stride < 1 || pad < 0 || R < 1 || S < 1 || groups < 1) return ORACLE_ERR_ARG;
  if (Cin % groups != 0 || Cout % groups != 0) return ORACLE_ERR_ARG;
  int P = (H + 2 * pad - R) / stride + 1;
  int Q = (Wd + 2 * pad - S) / stride + 1;
  if (P < 1 || Q < 1) return ORACLE_ERR_ARG;
  const int cin_g = Cin / groups, cout_g = Cout / groups;
  int64_t count = pixel_index ? n_pixels : (int64_t)B * H * Wd;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < count; ++i) {
    int64_t pix = pixel_index ? pixel_index[i] : i;
    int w = (int)(pix % Wd);
    int h = (int)((pix / Wd) % H);
    int b = (int)(pix / ((int64_t)Wd * H));
    for (int ci = 0; ci < Cin; ++ci) {
      const int g = ci / cin_g, cj = ci - g * cin_g;
      double acc = 0.0;
      for (int r = 0; r < R; ++r) {
        int hp = h + pad - r;
        if (hp < 0 || hp % stride != 0) continue;
        int p = hp / stride;
        if (p >= P) continue;
        for (int s = 0; s < S; ++s) {
          int wq = w + pad - s;
          if (wq < 0 || wq % stride != 0) continue;
          int q = wq / stride;
          if (q >= Q) continue;
          const uint16_t* grad = dOp + (((int64_t)b * P + p) * Q + q) * Cout;
          for (int co = g * cout_g; co < (g + 1) * cout_g; ++co)
            acc += elem_to_f64(grad[co], dtype) * elem_to_f64(W[(((int64_t)co * R + r) * S + s) * cin_g + cj], dtype);
        }
      }
      dD[i * Cin + ci] = acc;
    }
  }
  return ORACLE_OK;
}

/* Direct forward convolution in fp64 on fp64 inputs; used only by the adjoint
 * identity test <conv(D), G> == <D, dgrad(G)>. */
int oracle_conv2d_forward_f64(const double* D, const uint16_t* W, double* O, int B, int H, int Wd,
                              int Cin, int Cout, int R, int S, int stride, int pad) {
  int P = (H + 2 * pad - R) / stride + 1;
  int Q = (Wd + 2 * pad - S) / stride + 1;
  if (P < 1 || Q < 1) return ORACLE_ERR_ARG;
  for (int b = 0; b < B; ++b)
    for (int p = 0; p < P; ++p)
      for (int q = 0; q < Q; ++q)
        for (int co = 0; co < Cout; ++co) {
          double acc = 0.0;
          for (int r = 0; r < R; ++r)
            for (int s = 0; s < S; ++s) {
              int h = p * stride - pad + r, w = q * stride - pad + s;
              if (h < 0 || h >= H || w < 0 || w >= Wd) continue;
              for (int ci = 0; ci < Cin; ++ci)
                acc += D[(((int64_t)b * H + h) * Wd + w) * Cin + ci] *
                       oracle_bf16_to_f64(W[(((int64_t)co * R + r) * S + s) * Cin + ci]);
            }
          O[(((int64_t)b * P + p) * Q + q) * Cout + co] = acc;
        }
  return ORACLE_OK;
}

/* ---------------------------------------------------------------- the producer of dL/dO
 *
 * Section 2.1 / Fig. 2: in the backward pass a layer's dL/dO is the gradient handed down by what follows
 * it. For a ReLU that is dO[e] = dY[e] where the ReLU's activation is positive and +0.0 elsewhere (its
 * derivative is 1 for positive inputs and 0 otherwise; the ReLU's output is positive exactly where its
 * input is, so either may be passed as `act`). An activation that is not a number passes nothing.
 * The survivors keep the exact bits of dY. */
int oracle_relu_backward(const uint16_t* dY, const uint16_t* act, int64_t count, int dtype, uint16_t* dO) {
  if (!dY || !act || !dO || count < 0 || (dtype != ORACLE_BF16 && dtype != ORACLE_FP16)) return ORACLE_ERR_ARG;
  for (int64_t e = 0; e < count; ++e) {
    const float a = elem_to_f32(act[e], dtype);
    dO[e] = (a > 0.0f) ? dY[e] : (uint16_t)0; /* a NaN compares false */
  }
  return ORACLE_OK;
}

/* Where a residual connection joins its branch (the ResNets of Section 4: y = ReLU(x + F(x))), the gradient
 * that reaches the ReLU is the SUM of what the two consumers of y hand down (Section 2.1 / Fig. 2: each
 * hands down its own data gradient). The producer of dL/dO below such a ReLU therefore adds the two
 * gradients first: s[e] = dY[e] + dSkip[e], one IEEE single-precision addition of the two 16-bit values
 * (both exact in single precision), rounded to the tensors' 16-bit type to nearest-even (a NaN sum is stored
 * as the canonical quiet NaN, as everywhere in this file); then dO[e] = s[e] where the activation is
 * positive and +0.0 elsewhere. */
int oracle_residual_relu_backward(const uint16_t* dY, const uint16_t* dSkip, const uint16_t* act, int64_t count, int dtype,
                                  uint16_t* dO) {
  if (!dY || !dSkip || !act || !dO || count < 0 || (dtype != ORACLE_BF16 && dtype != ORACLE_FP16)) return ORACLE_ERR_ARG;
  for (int64_t e = 0; e < count; ++e) {
    const float a = elem_to_f32(act[e], dtype);
    volatile float s = elem_to_f32(dY[e], dtype) + elem_to_f32(dSkip[e], dtype); /* one rounding, to single precision */
    dO[e] = (a > 0.0f) ? elem_from_f32(s, dtype) : (uint16_t)0;
  }
  return ORACLE_OK;
}

/* Where the ReLU is followed by a 2 x 2 max pooling of stride 2 (the convolution blocks of ResNet-9, Section 4:
 * convolution, normalisation, ReLU, pooling), the gradient handed down (Section 2.1 / Fig. 2) has the POOLED shape
 * [B, H/2, W/2, K]. Pooling backward sends each of its elements to the position of its window's maximum, the first
 * one in the order (0,0), (0,1), (1,0), (1,1) when several are equal, and the ReLU below passes it only where its
 * activation is positive. Both rules together: in every window and channel the gradient goes to the first largest
 * activation if that activation is a number greater than zero; every other position of dL/dO, and the whole window
 * if nothing in it is positive, is +0.0. `act` is the ReLU's output or input, [B, H, W, K]; H and W are even. The
 * survivor keeps the exact bits of the pooled gradient. */
int oracle_maxpool_relu_backward(const uint16_t* dYp, const uint16_t* act, int B, int H, int W, int K, int dtype,
                                 uint16_t* dO) {
  if (!dYp || !act || !dO || B < 0 || H < 0 || W < 0 || K < 0 || (H & 1) || (W & 1) ||
      (dtype != ORACLE_BF16 && dtype != ORACLE_FP16))
    return ORACLE_ERR_ARG;
  const int Hp = H / 2, Wp = W / 2;
  for (int b = 0; b < B; ++b)
    for (int i = 0; i < Hp; ++i)
      for (int j = 0; j < Wp; ++j)
        for (int k = 0; k < K; ++k) {
          int best = -1;
          float best_a = 0.0f;
          for (int pos = 0; pos < 4; ++pos) {
            const int h = 2 * i + (pos >> 1), w = 2 * j + (pos & 1);
            const int64_t e = (((int64_t)b * H + h) * W + w) * K + k;
            const float a = elem_to_f32(act[e], dtype);
            dO[e] = 0;
            if (a > 0.0f && (best < 0 || a > best_a)) { /* a NaN compares false: it is never the maximum */
              best = pos;
              best_a = a;
            }
          }
          if (best >= 0) {
            const int h = 2 * i + (best >> 1), w = 2 * j + (best & 1);
            dO[(((int64_t)b * H + h) * W + w) * K + k] = dYp[(((int64_t)b * Hp + i) * Wp + j) * K + k];
          }
        }
  return ORACLE_OK;
}

/* Section 4.3 estimator: removing a fraction (1 - n/m) of a pass that takes
 * share f of the runtime reduces the total by f * (1 - n/m). */
double oracle_runtime_reduction(double share, int n, int m) {
  return share * (1.0 - (double)n / (double)m);
}
