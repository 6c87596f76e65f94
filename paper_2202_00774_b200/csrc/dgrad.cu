// Data-gradient contraction dD = dOp . W on the sm_100a tensor cores (Section 2.1, Fig. 2/3).
//
// One persistent, warp-specialised kernel serves the fully connected layer and the stride-1
// convolution (an implicit GEMM whose K axis runs tap-major, output-channel-minor, so a
// 4-element pruning chunk never straddles two filter taps), with A either dense dL/dO
// (tcgen05.mma) or 2:4-compressed dL/dO plus position metadata (tcgen05.mma.sp):
//
//   warp 0      TMA producer: per K-block one 4-D box of A (a TW x TH x TB patch of pixels,
//               shifted by the filter tap; out-of-image pixels arrive as zeros), the matching
//               box of metadata, and BN/64 boxes of W.
//   warp 1      MMA issuer: copies the stage's metadata into TMEM (tcgen05.cp), issues four
//               MMAs per stage into a TMEM accumulator, commits to the stage's "empty" barrier.
//   warps 2-5   (sparse only) rearrange the stages' row-major metadata into the lane/column
//               order the tensor core reads from TMEM, one warp per stage, four stages at once.
//   warps 6-9   epilogue: TMEM -> registers -> bf16 -> swizzled staging tile -> TMA store,
//               overlapped with the next tile's main loop through a second accumulator.
//
// Every mbarrier wait is bounded; a wait that runs out records a code in g_device_error and
// the kernel still runs to completion and frees its TMEM.
#include <cuda.h>
#include <cuda_bf16.h>

#include "ptx.cuh"
#include "sdgp_internal.cuh"

namespace sdgp {

__device__ unsigned int g_device_error = 0;

namespace {

constexpr int kBM = 128;           // output pixels (rows) per tile = TMEM lanes
constexpr int kThreadsGemm = 320;  // 10 warps
constexpr int kABytes = kBM * 128; // one A stage: 128 rows x 128 B (64 bf16, dense or compressed)
constexpr int kEBytes = kBM * 16;  // one metadata stage: 128 rows x 8 uint16
constexpr uint32_t kTmemCols = 512;
constexpr int kOutBytes = kBM * 128;  // epilogue staging: 128 rows x 64 bf16 columns

struct DgradParams {
  int B, H, W;          // dD pixel grid (fully connected: B = H = 1, W = rows)
  int Cin, Cout;
  int R, S, pad;
  int TW, TH, TB;       // pixel patch of one tile, TW * TH * TB <= 128
  int tiles_w, tiles_h, tiles_b, tiles_n;
  int total_tiles;
  int k_blocks_per_tap; // ceil(Cout / channels per stage)
  int m_tiles;          // tiles_w * tiles_h * tiles_b
  int pair_tiles;       // CTA-pair kernel: ceil(m_tiles / 2) * tiles_n
  int meta_merged;      // metadata box spans whole pixel rows (8*TW uint16 per TMA request)
  uint16_t* dD;
};

template <bool SPARSE, int BN>
struct Cfg {
  static constexpr int kKB = SPARSE ? 128 : 64;           // W rows (output channels) per stage
  static constexpr int kBBytes = kKB * BN * 2;
  static constexpr int kStageBytes = kABytes + kBBytes + (SPARSE ? 2 * kEBytes : 0);
  static constexpr int kSmemBudget = 232448 - 2048;       // max dynamic smem minus barriers/alignment slack
  static constexpr int kOutBufs = ((kSmemBudget - 2 * kOutBytes) / kStageBytes >= 4) ? 2 : 1;
  static constexpr int kStagesFit = (kSmemBudget - kOutBufs * kOutBytes) / kStageBytes;
  static constexpr int kStages = kStagesFit > 8 ? 8 : kStagesFit;
  static constexpr int kAcc = (2 * BN + (SPARSE ? 4 * kStages : 0) <= (int)kTmemCols) ? 2 : 1;
  static constexpr int kMetaCol = kAcc * BN;              // first TMEM column of the metadata slots
  static constexpr int kSmemBytes = kStages * kStageBytes + kOutBufs * kOutBytes + 2048;
  static_assert(kStages >= 2, "pipeline needs at least two stages");
};

// Instruction descriptor: fp32 accumulate, bf16 A and B, A K-major, B MN-major, M = 128.
__host__ __device__ constexpr uint32_t make_idesc(int n, bool sparse) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(kBM >> 4) << 24) | (sparse ? (1u << 2) : 0u);
}


// One row of a stage's metadata: from the row-major order TMA delivers (8 uint16 per pixel,
// one per 16 channels) to the order tcgen05.cp moves into TMEM. For the MMA covering channels
// [32*k2, 32*k2+32) of the stage the tensor core reads one 32-bit TMEM column: lane
// (row%8) + 8*half + 16*(row/16) holds in its low 16 bits the four position nibbles of channels
// 32*k2 + 16*half + [0,16) of the row with bit 3 clear and in its high 16 bits those of row + 8.
__device__ __forceinline__ void rearrange_metadata_row(const uint8_t* raw_stage, uint8_t* hw_stage, int row,
                                                       int rows_used) {
  const uint4 raw = *(const uint4*)(raw_stage + row * 16);
  const uint32_t w4[4] = {raw.x, raw.y, raw.z, raw.w};
  uint16_t* hw = (uint16_t*)hw_stage;
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    uint32_t v = (u & 1) ? (w4[u >> 1] >> 16) : (w4[u >> 1] & 0xFFFFu);
    // rows outside the patch or outside the image carry no data: give them the well-formed
    // position pair (0,1) in every chunk
    if (row >= rows_used || v == 0u) v = 0x4444u;
    const int tl = (row & 7) + 8 * (u & 1) + 16 * (row >> 4);
    hw[tl * 8 + 2 * (u >> 1) + ((row >> 3) & 1)] = (uint16_t)v;
  }
}

// One warp rearranges a whole stage (lane l takes rows l, l+32, l+64, l+96); the four
// rearranger warps work on four different stages at once, so the per-stage latency of
// wait -> shuffle -> proxy fence -> arrive is overlapped four ways.
__device__ __forceinline__ void rearrange_metadata_stage(const uint8_t* raw_stage, uint8_t* hw_stage, int lane,
                                                         int rows_used) {
#pragma unroll
  for (int i = 0; i < 4; ++i) rearrange_metadata_row(raw_stage, hw_stage, lane + 32 * i, rows_used);
}

// The four epilogue warps move one 128-row x BN accumulator to global memory in 64-column
// slabs: TMEM -> registers -> bf16 -> a 128-byte-swizzled staging tile in shared memory -> one
// TMA store of the whole pixel patch (full-line writes; rows and pixels outside the tensor are
// clipped by the TMA unit). With NBUF = 2 the store of one slab overlaps the packing of the next.
// `chunk` counts slabs over the kernel's lifetime and picks the staging buffer.
template <int BN, int NBUF>
__device__ __forceinline__ void store_accumulator(uint32_t taddr, uint8_t* staging, const CUtensorMap* tmD,
                                                  int n0, int w0, int h0, int b0, bool tile_in_range, int row,
                                                  bool issuer, uint32_t& chunk) {
#pragma unroll 1
  for (int c0 = 0; c0 < BN; c0 += 64, ++chunk) {
    uint32_t packed[32];
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      uint32_t v[32];
      ptx::tmem_ld_32x32(taddr + (uint32_t)(c0 + 32 * half), v);
      ptx::tmem_ld_wait();
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(v[2 * e]), __uint_as_float(v[2 * e + 1]));
        packed[16 * half + e] = *(const uint32_t*)&h2;
      }
    }
    uint8_t* buf = staging + (chunk % NBUF) * kOutBytes;
    if (issuer) ptx::bulk_wait_group_read<NBUF - 1>();  // the store that last used this buffer has read it
    ptx::named_bar_sync(1, 128);
#pragma unroll
    for (int c = 0; c < 8; ++c)
      *(uint4*)(buf + row * 128 + ((c ^ (row & 7)) << 4)) =
          make_uint4(packed[4 * c], packed[4 * c + 1], packed[4 * c + 2], packed[4 * c + 3]);
    ptx::fence_proxy_async_smem();
    ptx::named_bar_sync(1, 128);
    if (issuer && tile_in_range) {
      ptx::tma_store_4d(tmD, buf, n0 + c0, w0, h0, b0);
      ptx::bulk_commit_group();
    }
  }
}

template <bool SPARSE, int BN>
__global__ void __launch_bounds__(kThreadsGemm, 1)
dgrad_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmE,
             const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmD,
             const DgradParams p) {
  using C = Cfg<SPARSE, BN>;
  constexpr int STAGES = C::kStages;
  constexpr int NACC = C::kAcc;

  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment: required by the 128-byte swizzle of the A and B stages
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = smem;
  uint8_t* sB = sA + STAGES * kABytes;
  uint8_t* sEraw = sB + STAGES * C::kBBytes;
  uint8_t* sEhw = sEraw + (SPARSE ? STAGES * kEBytes : 0);
  uint8_t* sOut = sEhw + (SPARSE ? STAGES * kEBytes : 0);
  uint64_t* bars = (uint64_t*)(sOut + C::kOutBufs * kOutBytes);
  uint64_t* full = bars;
  uint64_t* empty = full + STAGES;
  uint64_t* meta_ready = empty + STAGES;
  uint64_t* acc_full = meta_ready + STAGES;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = (uint32_t*)(acc_empty + 2);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  unsigned int* err = &g_device_error;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(&full[s], 1);
      ptx::mbar_init(&empty[s], 1);
      ptx::mbar_init(&meta_ready[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&acc_full[a], 1);
      ptx::mbar_init(&acc_empty[a], 4);
    }
    ptx::fence_mbar_init();
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmB);
    ptx::prefetch_tensormap(&tmD);
    if (SPARSE) ptx::prefetch_tensormap(&tmE);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  const int rows_used = p.TW * p.TH * p.TB;
  const int taps = p.R * p.S;
  const int k_iters = taps * p.k_blocks_per_tap;
  const uint32_t tx_bytes = (uint32_t)(rows_used * 128 + C::kBBytes + (SPARSE ? rows_used * 16 : 0));

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    if (ptx::elect_one()) {
      uint32_t it = 0;
      for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x) {
        int t = tile;
        const int nt = t % p.tiles_n; t /= p.tiles_n;
        const int wt = t % p.tiles_w; t /= p.tiles_w;
        const int ht = t % p.tiles_h; t /= p.tiles_h;
        const int bt = t;
        const int n0 = nt * BN, w0 = wt * p.TW, h0 = ht * p.TH, b0 = bt * p.TB;
        for (int tap = 0; tap < taps; ++tap) {
          const int r = tap / p.S, s = tap - r * p.S;
          const int q0 = w0 + p.pad - s, p0 = h0 + p.pad - r;  // dO pixel of the patch's corner
          for (int cb = 0; cb < p.k_blocks_per_tap; ++cb, ++it) {
            const int st = it % STAGES;
            const uint32_t ph = (it / STAGES) & 1u;
            ptx::mbar_wait(&empty[st], ph ^ 1u, err, 0x100u + st);
            ptx::mbar_arrive_expect_tx(&full[st], tx_bytes);
            ptx::tma_load_4d(sA + st * kABytes, &tmA, &full[st], cb * 64, q0, p0, b0);
            if (SPARSE) {
              if (p.meta_merged) ptx::tma_load_4d(sEraw + st * kEBytes, &tmE, &full[st], 8 * q0, p0, b0, 0);
              else ptx::tma_load_4d(sEraw + st * kEBytes, &tmE, &full[st], cb * 8, q0, p0, b0);
            }
#pragma unroll
            for (int j = 0; j < BN / 64; ++j)
              ptx::tma_load_2d(sB + st * C::kBBytes + j * (C::kKB * 128), &tmB, &full[st],
                               tap * p.Cin + n0 + 64 * j, cb * C::kKB);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------- MMA issuer
    if (ptx::elect_one()) {
      constexpr uint32_t idesc = make_idesc(BN, SPARSE);
      uint32_t it = 0, lt = 0;
      for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x, ++lt) {
        const int acc = lt % NACC;
        const uint32_t aph = (lt / NACC) & 1u;
        ptx::mbar_wait(&acc_empty[acc], aph ^ 1u, err, 0x200u + acc);
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < k_iters; ++kb, ++it) {
          const int st = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          ptx::mbar_wait(&full[st], ph, err, 0x300u + st);
          if (SPARSE) ptx::mbar_wait(&meta_ready[st], ph, err, 0x400u + st);
          ptx::tc_fence_after_sync();
          const uint64_t adesc = ptx::make_smem_desc(ptx::smem_u32(sA + st * kABytes), 16, 1024, 2);
          const uint64_t bdesc =
              ptx::make_smem_desc(ptx::smem_u32(sB + st * C::kBBytes), C::kKB * 128, 1024, 2);
          if (SPARSE) {
            const uint64_t edesc = ptx::make_smem_desc(ptx::smem_u32(sEhw + st * kEBytes), 128, 128, 0);
            ptx::tc_cp_128x128b(tmem_base + (uint32_t)(C::kMetaCol + 4 * st), edesc);
          }
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t accumulate = (kb > 0 || j > 0) ? 1u : 0u;
            // A: 32 bytes of a 128-byte swizzled row per MMA; B: 16 (dense) or 32 (sparse) rows of 128 B
            const uint64_t a_j = adesc + (uint64_t)(j * 2);
            const uint64_t b_j = bdesc + (uint64_t)(j * (C::kKB / 4) * 128 / 16);
            if (SPARSE) {
              const uint32_t col = (uint32_t)(C::kMetaCol + 4 * st + j);
              ptx::mma_sp_f16_ss(d_tmem, a_j, b_j, tmem_base + (col & ~1u), idesc | (col & 1u), accumulate);
            } else {
              ptx::mma_f16_ss(d_tmem, a_j, b_j, idesc, accumulate);
            }
          }
          ptx::tc_commit(&empty[st]);
        }
        ptx::tc_commit(&acc_full[acc]);
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------- metadata rearranger
    if (SPARSE) {
      uint32_t it = 0;
      for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x) {
        for (int kb = 0; kb < k_iters; ++kb, ++it) {
          if ((int)(it & 3u) != warp - 2) continue;  // this warp's turn: every fourth stage use
          const int st = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          ptx::mbar_wait(&full[st], ph, err, 0x500u + st);
          rearrange_metadata_stage(sEraw + st * kEBytes, sEhw + st * kEBytes, lane, rows_used);
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&meta_ready[st]);
        }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int q = warp & 3;  // a warp may only touch TMEM lanes [32*(warp%4), +32)
    const int row = q * 32 + lane;
    const bool issuer = (threadIdx.x == 192);
    uint32_t lt = 0, chunk = 0;
    for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x, ++lt) {
      int t = tile;
      const int nt = t % p.tiles_n; t /= p.tiles_n;
      const int wt = t % p.tiles_w; t /= p.tiles_w;
      const int ht = t % p.tiles_h; t /= p.tiles_h;
      const int bt = t;
      const int acc = lt % NACC;
      const uint32_t aph = (lt / NACC) & 1u;
      ptx::mbar_wait(&acc_full[acc], aph, err, 0x600u + acc);
      ptx::tc_fence_after_sync();
      store_accumulator<BN, C::kOutBufs>(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN), sOut, &tmD,
                                         nt * BN, wt * p.TW, ht * p.TH, bt * p.TB, true, row, issuer, chunk);
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&acc_empty[acc]);
    }
    if (issuer) ptx::bulk_wait_group_all();  // dD is written before the CTA leaves
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  if (warp == 1) ptx::tmem_dealloc(tmem_base, kTmemCols);
}


// ------------------------------------------------------------------------------------------
// CTA-pair variant (cta_group::2). Two CTAs of a cluster own two neighbouring 128-pixel
// patches and one BN-wide column block: each stages its own A patch (+ metadata) and HALF of
// the W columns, and a single thread of the pair's first CTA issues 256-row MMAs that read
// both halves. Per CTA this halves the W bytes and TMA requests per FLOP and the shared-memory
// reads of B, and leaves room in TMEM for BN = 256.
//
// Barriers: full / meta_ready / acc_empty are waited on by the first CTA only and collect
// arrivals from both; empty / acc_full exist in both CTAs and are signalled together by a
// multicast tcgen05.commit; meta_full is local (each CTA's own metadata box).

template <bool SPARSE, int BN>
struct PairCfg {
  static constexpr int kKB = SPARSE ? 128 : 64;
  static constexpr int kBCols = BN / 2;                    // W columns staged by one CTA
  static constexpr int kBBytes = kKB * kBCols * 2;
  static constexpr int kStageBytes = kABytes + kBBytes + (SPARSE ? 2 * kEBytes : 0);
  static constexpr int kSmemBudget = 232448 - 2048;
  static constexpr int kOutBufs = ((kSmemBudget - 2 * kOutBytes) / kStageBytes >= 4) ? 2 : 1;
  static constexpr int kStagesFit = (kSmemBudget - kOutBufs * kOutBytes) / kStageBytes;
  static constexpr int kStages = kStagesFit > 8 ? 8 : kStagesFit;
  static constexpr int kAcc = (2 * BN + (SPARSE ? 4 * kStages : 0) <= (int)kTmemCols) ? 2 : 1;
  static constexpr int kMetaCol = kAcc * BN;
  static constexpr int kSmemBytes = kStages * kStageBytes + kOutBufs * kOutBytes + 2048;
  static_assert(kBCols % 64 == 0, "each CTA stages whole 64-column swizzle blocks of W");
  static_assert(kStages >= 2, "pipeline needs at least two stages");
};

__host__ __device__ constexpr uint32_t make_idesc_pair(int n, bool sparse) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(256 >> 4) << 24) | (sparse ? (1u << 2) : 0u);
}

template <bool SPARSE, int BN>
__global__ void __launch_bounds__(kThreadsGemm, 1)
dgrad_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmE,
                  const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmD,
                  const DgradParams p) {
  using C = PairCfg<SPARSE, BN>;
  constexpr int STAGES = C::kStages;
  constexpr int NACC = C::kAcc;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = smem;
  uint8_t* sB = sA + STAGES * kABytes;
  uint8_t* sEraw = sB + STAGES * C::kBBytes;
  uint8_t* sEhw = sEraw + (SPARSE ? STAGES * kEBytes : 0);
  uint8_t* sOut = sEhw + (SPARSE ? STAGES * kEBytes : 0);
  uint64_t* bars = (uint64_t*)(sOut + C::kOutBufs * kOutBytes);
  uint64_t* full = bars;
  uint64_t* empty = full + STAGES;
  uint64_t* meta_full = empty + STAGES;
  uint64_t* meta_ready = meta_full + STAGES;
  uint64_t* acc_full = meta_ready + STAGES;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = (uint32_t*)(acc_empty + 2);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();  // 0: issues the MMAs
  unsigned int* err = &g_device_error;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(&full[s], 1);
      ptx::mbar_init(&empty[s], 1);
      ptx::mbar_init(&meta_full[s], 1);
      ptx::mbar_init(&meta_ready[s], 2);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&acc_full[a], 1);
      ptx::mbar_init(&acc_empty[a], 8);
    }
    ptx::fence_mbar_init();
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmB);
    ptx::prefetch_tensormap(&tmD);
    if (SPARSE) ptx::prefetch_tensormap(&tmE);
  }
  if (warp == 1) {
    ptx::tmem_alloc_pair(tmem_slot, kTmemCols);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before_sync();
  ptx::cluster_sync();  // barrier inits and TMEM of both CTAs are ready before any cross-CTA signal
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  const int rows_used = p.TW * p.TH * p.TB;
  const int taps = p.R * p.S;
  const int k_iters = taps * p.k_blocks_per_tap;
  const int pair_stride = gridDim.x >> 1;
  const int first_pair = blockIdx.x >> 1;

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    if (ptx::elect_one()) {
      const uint32_t pair_tx = 2u * (uint32_t)(rows_used * 128 + C::kBBytes);
      uint32_t it = 0;
      for (int pt = first_pair; pt < p.pair_tiles; pt += pair_stride) {
        const int nt = pt % p.tiles_n;
        int t = 2 * (pt / p.tiles_n) + (int)rank;  // this CTA's patch; may lie past the last one
        const int wt = t % p.tiles_w; t /= p.tiles_w;
        const int ht = t % p.tiles_h; t /= p.tiles_h;
        const int bt = t;
        const int n0 = nt * BN + (int)rank * C::kBCols;
        const int w0 = wt * p.TW, h0 = ht * p.TH, b0 = bt * p.TB;
        for (int tap = 0; tap < taps; ++tap) {
          const int r = tap / p.S, s = tap - r * p.S;
          const int q0 = w0 + p.pad - s, p0 = h0 + p.pad - r;
          for (int cb = 0; cb < p.k_blocks_per_tap; ++cb, ++it) {
            const int st = it % STAGES;
            const uint32_t ph = (it / STAGES) & 1u;
            ptx::mbar_wait(&empty[st], ph ^ 1u, err, 0x1100u + st);
            if (rank == 0) ptx::mbar_arrive_expect_tx(&full[st], pair_tx);
            if (SPARSE) {
              ptx::mbar_arrive_expect_tx(&meta_full[st], (uint32_t)(rows_used * 16));
              if (p.meta_merged) ptx::tma_load_4d(sEraw + st * kEBytes, &tmE, &meta_full[st], 8 * q0, p0, b0, 0);
              else ptx::tma_load_4d(sEraw + st * kEBytes, &tmE, &meta_full[st], cb * 8, q0, p0, b0);
            }
            ptx::tma_load_4d_pair(sA + st * kABytes, &tmA, &full[st], cb * 64, q0, p0, b0);
#pragma unroll
            for (int j = 0; j < C::kBCols / 64; ++j)
              ptx::tma_load_2d_pair(sB + st * C::kBBytes + j * (C::kKB * 128), &tmB, &full[st],
                                    tap * p.Cin + n0 + 64 * j, cb * C::kKB);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------- MMA issuer (first CTA only)
    if (rank == 0 && ptx::elect_one()) {
      constexpr uint32_t idesc = make_idesc_pair(BN, SPARSE);
      uint32_t it = 0, lt = 0;
      for (int pt = first_pair; pt < p.pair_tiles; pt += pair_stride, ++lt) {
        const int acc = lt % NACC;
        const uint32_t aph = (lt / NACC) & 1u;
        ptx::mbar_wait(&acc_empty[acc], aph ^ 1u, err, 0x1200u + acc);
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < k_iters; ++kb, ++it) {
          const int st = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          ptx::mbar_wait(&full[st], ph, err, 0x1300u + st);
          if (SPARSE) ptx::mbar_wait(&meta_ready[st], ph, err, 0x1400u + st);
          ptx::tc_fence_after_sync();
          const uint64_t adesc = ptx::make_smem_desc(ptx::smem_u32(sA + st * kABytes), 16, 1024, 2);
          const uint64_t bdesc =
              ptx::make_smem_desc(ptx::smem_u32(sB + st * C::kBBytes), C::kKB * 128, 1024, 2);
          if (SPARSE) {
            const uint64_t edesc = ptx::make_smem_desc(ptx::smem_u32(sEhw + st * kEBytes), 128, 128, 0);
            ptx::tc_cp_128x128b_pair(tmem_base + (uint32_t)(C::kMetaCol + 4 * st), edesc);
          }
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t accumulate = (kb > 0 || j > 0) ? 1u : 0u;
            const uint64_t a_j = adesc + (uint64_t)(j * 2);
            const uint64_t b_j = bdesc + (uint64_t)(j * (C::kKB / 4) * 128 / 16);
            if (SPARSE) {
              const uint32_t col = (uint32_t)(C::kMetaCol + 4 * st + j);
              ptx::mma_sp_f16_ss_pair(d_tmem, a_j, b_j, tmem_base + (col & ~1u), idesc | (col & 1u), accumulate);
            } else {
              ptx::mma_f16_ss_pair(d_tmem, a_j, b_j, idesc, accumulate);
            }
          }
          ptx::tc_commit_pair(&empty[st], 3);
        }
        ptx::tc_commit_pair(&acc_full[acc], 3);
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------- metadata rearranger
    if (SPARSE) {
      uint32_t it = 0;
      for (int pt = first_pair; pt < p.pair_tiles; pt += pair_stride) {
        for (int kb = 0; kb < k_iters; ++kb, ++it) {
          if ((int)(it & 3u) != warp - 2) continue;
          const int st = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          ptx::mbar_wait(&meta_full[st], ph, err, 0x1500u + st);
          rearrange_metadata_stage(sEraw + st * kEBytes, sEhw + st * kEBytes, lane, rows_used);
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive_cluster(&meta_ready[st], 0);
        }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const bool issuer = (threadIdx.x == 192);
    uint32_t lt = 0, chunk = 0;
    for (int pt = first_pair; pt < p.pair_tiles; pt += pair_stride, ++lt) {
      const int nt = pt % p.tiles_n;
      const int mt = 2 * (pt / p.tiles_n) + (int)rank;
      int t = mt;
      const int wt = t % p.tiles_w; t /= p.tiles_w;
      const int ht = t % p.tiles_h; t /= p.tiles_h;
      const int bt = t;
      const int acc = lt % NACC;
      const uint32_t aph = (lt / NACC) & 1u;
      ptx::mbar_wait(&acc_full[acc], aph, err, 0x1600u + acc);
      ptx::tc_fence_after_sync();
      store_accumulator<BN, C::kOutBufs>(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN), sOut, &tmD,
                                         nt * BN, wt * p.TW, ht * p.TH, bt * p.TB, mt < p.m_tiles, row, issuer,
                                         chunk);
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive_cluster(&acc_empty[acc], 0);
    }
    if (issuer) ptx::bulk_wait_group_all();
  }

  ptx::tc_fence_before_sync();
  __syncwarp();
  ptx::cluster_sync();  // neither CTA leaves (or frees TMEM) while the other may still touch it
  ptx::tc_fence_after_sync();
  if (warp == 1) ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
}

// ------------------------------------------------------------------- host

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)ptr;
  }
  return fn;
}

bool encode(CUtensorMap* tm, CUtensorMapDataType dt, int rank, const void* base, const uint64_t* dims,
            const uint64_t* strides_bytes, const uint32_t* box, CUtensorMapSwizzle swz) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint32_t ones[5] = {1, 1, 1, 1, 1};
  return fn(tm, dt, (cuuint32_t)rank, const_cast<void*>(base), (const cuuint64_t*)dims,
            (const cuuint64_t*)strides_bytes, (const cuuint32_t*)box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int largest_divisor_at_most(int x, int cap) {
  for (int d = cap < x ? cap : x; d >= 1; --d)
    if (x % d == 0) return d;
  return 1;
}

// Pixel patch of one 128-row tile: whole image rows when the image is narrow, so that a
// filter tap shifts the patch as a block and the image border falls outside the box.
void choose_patch(int B, int H, int W, int* TW, int* TH, int* TB) {
  if (W >= kBM) {
    *TW = kBM; *TH = 1; *TB = 1;
    return;
  }
  *TW = W;
  const int max_h = kBM / W;
  if (H <= max_h) {
    *TH = H;
    const int max_b = kBM / (W * H);
    *TB = max_b < B ? max_b : B;
    if (*TB < 1) *TB = 1;
  } else {
    const int d = largest_divisor_at_most(H, max_h);
    *TH = (2 * d >= max_h) ? d : max_h;
    *TB = 1;
  }
}

int sm_count() {
  static int n = 0;
  if (!n) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (n <= 0) n = 148;
  }
  return n;
}

template <bool SPARSE, int BN>
sdgp_status launch_cfg(const CUtensorMap& tmA, const CUtensorMap& tmE, const CUtensorMap& tmB,
                       const CUtensorMap& tmD, const DgradParams& p, cudaStream_t stream) {
  using C = Cfg<SPARSE, BN>;
  static bool configured = false;
  auto kernel = dgrad_kernel<SPARSE, BN>;
  if (!configured) {
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes) != cudaSuccess)
      return SDGP_ERR_CUDA;
    configured = true;
  }
  const int grid = p.total_tiles < sm_count() ? p.total_tiles : sm_count();
  kernel<<<grid, kThreadsGemm, C::kSmemBytes, stream>>>(tmA, tmE, tmB, tmD, p);
  return cudaGetLastError() == cudaSuccess ? SDGP_OK : SDGP_ERR_CUDA;
}

template <bool SPARSE, int BN>
sdgp_status launch_pair_cfg(const CUtensorMap& tmA, const CUtensorMap& tmE, const CUtensorMap& tmB,
                            const CUtensorMap& tmD, const DgradParams& p, cudaStream_t stream) {
  using C = PairCfg<SPARSE, BN>;
  static bool configured = false;
  auto kernel = dgrad_pair_kernel<SPARSE, BN>;
  if (!configured) {
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes) != cudaSuccess)
      return SDGP_ERR_CUDA;
    configured = true;
  }
  const int max_pairs = sm_count() / 2;
  const int pairs = p.pair_tiles < max_pairs ? p.pair_tiles : max_pairs;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * pairs));
  cfg.blockDim = dim3(kThreadsGemm);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, tmA, tmE, tmB, tmD, p) == cudaSuccess ? SDGP_OK : SDGP_ERR_CUDA;
}

}  // namespace

// A: dense dL/dO [B,P,Q,Cout] (sparse == false) or compressed values [B,P,Q,Cout/2] with
// meta [B,P,Q,Cout/16]; Wt: [Cout, R, S, Cin]; dD: [B,H,W,Cin]. Stride 1.
sdgp_status launch_dgrad(bool sparse, const void* A, const void* meta, const void* Wt, void* dD, int B,
                         int H, int W, int Cin, int Cout, int R, int S, int pad, cudaStream_t stream) {
  const int P = H + 2 * pad - R + 1, Q = W + 2 * pad - S + 1;
  if (P < 1 || Q < 1) return SDGP_ERR_INVALID_ARG;
  if ((int64_t)B * H * W == 0) return SDGP_OK;
  if (Cin % 64 != 0 || Cout % (sparse ? 128 : 64) != 0) return SDGP_ERR_UNSUPPORTED;
  if ((int64_t)R * S * Cin > 0x7FFFFFFF) return SDGP_ERR_UNSUPPORTED;

  // CTA pairs whenever the column count allows whole 64-column halves; the single-CTA kernel
  // serves Cin = 64 (mod 128).
  const bool pair = (Cin % 128 == 0);
  const int BN = pair ? ((Cin % 256 == 0) ? 256 : 128) : 64;
  const int kb_channels = sparse ? 128 : 64;

  DgradParams p;
  p.B = B; p.H = H; p.W = W; p.Cin = Cin; p.Cout = Cout; p.R = R; p.S = S; p.pad = pad;
  choose_patch(B, H, W, &p.TW, &p.TH, &p.TB);
  p.tiles_w = (W + p.TW - 1) / p.TW;
  p.tiles_h = (H + p.TH - 1) / p.TH;
  p.tiles_b = (B + p.TB - 1) / p.TB;
  p.tiles_n = Cin / BN;
  const int64_t m_tiles = (int64_t)p.tiles_w * p.tiles_h * p.tiles_b;
  const int64_t total = m_tiles * p.tiles_n;
  if (total > 0x3FFFFFFF) return SDGP_ERR_UNSUPPORTED;
  p.m_tiles = (int)m_tiles;
  p.total_tiles = (int)total;
  p.pair_tiles = (int)((m_tiles + 1) / 2) * p.tiles_n;
  p.k_blocks_per_tap = (Cout + kb_channels - 1) / kb_channels;
  p.dD = (uint16_t*)dD;

  CUtensorMap tmA, tmE, tmB;
  const uint64_t CA = sparse ? (uint64_t)Cout / 2 : (uint64_t)Cout;  // stored elements per pixel
  {
    const uint64_t dims[4] = {CA, (uint64_t)Q, (uint64_t)P, (uint64_t)B};
    const uint64_t strides[3] = {CA * 2, CA * 2 * Q, CA * 2 * Q * P};
    const uint32_t box[4] = {64, (uint32_t)p.TW, (uint32_t)p.TH, (uint32_t)p.TB};
    if (!encode(&tmA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, A, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B))
      return SDGP_ERR_CUDA;
  }
  p.meta_merged = 0;
  if (sparse && Cout == 128 && p.TW <= 32) {
    // One pixel's metadata is a single 16-byte run and pixels of an image row are contiguous:
    // fetch whole rows of the patch per TMA request instead of one request per pixel.
    p.meta_merged = 1;
    const uint64_t dims[4] = {8ull * Q, (uint64_t)P, (uint64_t)B, 1};
    const uint64_t strides[3] = {16ull * Q, 16ull * Q * P, 16ull * Q * P * B};
    const uint32_t box[4] = {8u * (uint32_t)p.TW, (uint32_t)p.TH, (uint32_t)p.TB, 1};
    if (!encode(&tmE, CU_TENSOR_MAP_DATA_TYPE_UINT16, 4, meta, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE))
      return SDGP_ERR_CUDA;
  } else if (sparse) {
    const uint64_t CE = (uint64_t)Cout / 16;
    const uint64_t dims[4] = {CE, (uint64_t)Q, (uint64_t)P, (uint64_t)B};
    const uint64_t strides[3] = {CE * 2, CE * 2 * Q, CE * 2 * Q * P};
    const uint32_t box[4] = {8, (uint32_t)p.TW, (uint32_t)p.TH, (uint32_t)p.TB};
    if (!encode(&tmE, CU_TENSOR_MAP_DATA_TYPE_UINT16, 4, meta, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE))
      return SDGP_ERR_CUDA;
  } else {
    tmE = tmA;
  }
  {
    const uint64_t dims[2] = {(uint64_t)R * S * Cin, (uint64_t)Cout};
    const uint64_t strides[1] = {(uint64_t)R * S * Cin * 2};
    const uint32_t box[2] = {64, (uint32_t)kb_channels};
    if (!encode(&tmB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Wt, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B))
      return SDGP_ERR_CUDA;
  }

  CUtensorMap tmD;
  {
    const uint64_t dims[4] = {(uint64_t)Cin, (uint64_t)W, (uint64_t)H, (uint64_t)B};
    const uint64_t strides[3] = {(uint64_t)Cin * 2, (uint64_t)Cin * 2 * W, (uint64_t)Cin * 2 * W * H};
    const uint32_t box[4] = {64, (uint32_t)p.TW, (uint32_t)p.TH, (uint32_t)p.TB};
    if (!encode(&tmD, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, dD, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B))
      return SDGP_ERR_CUDA;
  }

  if (pair) {
    if (sparse)
      return BN == 256 ? launch_pair_cfg<true, 256>(tmA, tmE, tmB, tmD, p, stream)
                       : launch_pair_cfg<true, 128>(tmA, tmE, tmB, tmD, p, stream);
    return BN == 256 ? launch_pair_cfg<false, 256>(tmA, tmE, tmB, tmD, p, stream)
                     : launch_pair_cfg<false, 128>(tmA, tmE, tmB, tmD, p, stream);
  }
  return sparse ? launch_cfg<true, 64>(tmA, tmE, tmB, tmD, p, stream)
                : launch_cfg<false, 64>(tmA, tmE, tmB, tmD, p, stream);
}

sdgp_status read_device_error() {
  unsigned int word = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return SDGP_ERR_CUDA;
  if (cudaMemcpyFromSymbol(&word, g_device_error, sizeof(word)) != cudaSuccess) return SDGP_ERR_CUDA;
  if (word != 0) {
    const unsigned int zero = 0;
    cudaMemcpyToSymbol(g_device_error, &zero, sizeof(zero));
    return SDGP_ERR_TIMEOUT;
  }
  return SDGP_OK;
}

}  // namespace sdgp
