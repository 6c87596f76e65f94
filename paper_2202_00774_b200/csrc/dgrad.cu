// Data-gradient contraction dD = dOp . W on the sm_100a tensor cores (Section 2.1, Fig. 2/3).
//
// One persistent, warp-specialised kernel serves the fully connected layer and the stride-1
// convolution (an implicit GEMM whose K axis covers filter taps x output channels; a 4-element
// pruning chunk never straddles two taps), with A either dense dL/dO (tcgen05.mma) or
// 2:4-compressed dL/dO plus position metadata (tcgen05.mma.sp).
//
// CTA pairs (cta_group::2): the two CTAs of a cluster own two neighbouring 128-pixel patches
// and one BN-wide block of input channels. Each CTA stages its own A patch (+ metadata) and
// HALF of the W columns; one thread of the pair's first CTA issues 256-row MMAs that read
// both halves. What limits this kernel is the bytes an SM can pull in from L2 (about 64 B per
// clock), so everything is arranged to reuse what is already in shared memory:
//   * W column halves: half the W bytes per CTA and half the shared-memory reads of B;
//   * filter-row reuse: for an R x S filter one A "image" of TH + R - 1 pixel rows serves all R
//     vertical taps - a tap is just a row offset (a multiple of 8 rows, i.e. of the 1024-byte
//     swizzle period) in the A descriptor - so A is fetched S times instead of R*S times;
//   * resident W: when the layer's whole W slice fits next to two A stages it is loaded once
//     per CTA and never streamed again.
//
// Warp roles
//   warp 0      TMA producer (both CTAs): per stage one 4-D box of A (pixels outside the image
//               arrive as zeros), the matching box of metadata, and the W boxes of its half.
//   warp 1      MMA issuer (first CTA only): tcgen05.cp of the stage's metadata into TMEM,
//               four MMAs per (tap, channel block), tcgen05.commit to the stage's "empty" barrier.
//   warps 2-5   (sparse only) build the stage's metadata images: from the row-major order TMA
//               delivers to the lane/column order the tensor core reads from TMEM. Each warp
//               owns every fourth stage; with fused pruning these four warps and eight helper
//               warps (10-17) first prune the stage's pixel rows together.
//   warps 6-9   epilogue: TMEM -> registers -> bf16 -> swizzled staging tile -> TMA store,
//               overlapped with the next tile's main loop through a second accumulator.
//
// Barriers: full / acc_empty / w_full are waited on by the first CTA only and collect arrivals
// from both (full: the producer's byte count plus the metadata warps' arrivals, so the MMA
// thread waits once per stage); empty / acc_full exist in both CTAs and are signalled together
// by a multicast tcgen05.commit; meta_full is local (each CTA's own metadata box).
// Every wait is bounded: a wait that runs out records a code in g_device_error, the role
// stops issuing work, every other wait then gives up at once, and the kernel frees its TMEM
// and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include <string.h>

#include <type_traits>

#include "prune_core.cuh"
#include "ptx.cuh"
#include "sdgp_internal.cuh"

namespace sdgp {

__device__ unsigned int g_device_error = 0;

namespace {

constexpr int kBM = 128;             // output pixels (rows) per CTA tile = TMEM lanes
constexpr int kThreadsGemm = 320;    // 10 warps
// Fused pruning in the general kernel: eight more warps (10..17) prune beside warps 2..5. A lone warp
// runs the pruning code at a quarter of an instruction per clock; twelve of them keep up with the
// rate at which a memory-bound layer's dense dL/dO arrives.
constexpr int kFusedHelperWarps = 8;
constexpr int kThreadsGemmFused = kThreadsGemm + 32 * kFusedHelperWarps;
constexpr int kFusedPruners = 128 + 32 * kFusedHelperWarps;
constexpr int kEHwBytes = kBM * 16;  // rearranged metadata of one (tap, channel block): 128 lanes x 16 B
constexpr int kOutBytes = kBM * 128; // epilogue staging slab: 128 rows x 64 bf16 columns
constexpr uint32_t kTmemCols = 512;
constexpr int kMaxImgRows = 192;     // pixel rows of one A stage (filter-row reuse: TW * (TH + R - 1))
constexpr int kSmemLimit = 232448;   // opt-in dynamic shared memory per CTA
constexpr int kSmemSlack = 1536;     // 1024-byte alignment of the carve + barrier block
constexpr int kMaxStages = 8;

struct DgradParams {
  int B, H, W;            // dD pixel grid (fully connected: B = H = 1, W = rows)
  int Cin, Cout;
  int R, S;               // filter taps of this launch (stride 2: the taps of one output-parity class)
  int pad_h, pad_w;       // dO pixel of output pixel (h,w) under tap (r,s): (h + pad_h - r, w + pad_w - s)
  int r_first, r_step, s_first, s_step, S_full;  // tap (r,s) of the launch is filter tap (r_first + r_step*r, s_first + s_step*s)
  int TW, TH, TB;         // pixel patch of one CTA tile, TW * TH * TB <= 128
  int tiles_w, tiles_h, tiles_b, tiles_n;
  int m_tiles;            // tiles_w * tiles_h * tiles_b
  int pair_tiles;         // ceil(m_tiles / 2) * tiles_n
  int k_blocks;           // channel blocks per tap: ceil(Cout / channels per stage)
  int rr;                 // vertical taps served by one A stage: 1, or R (filter-row reuse)
  int img_rows;           // pixel rows of one A stage: TW * (TH + rr - 1) * TB
  int stages;             // shared-memory pipeline depth
  int nacc;               // TMEM accumulators (2 = epilogue overlaps the next tile)
  int meta_col;           // first TMEM column of the metadata slots
  int meta_shared;        // metadata slots live in the first columns of the accumulator NOT being written
  int w_resident;         // whole W half-slice kept in shared memory
  int out_bufs;           // epilogue staging slabs (1 or 2)
  // fused pruning (the kernel reads dense dL/dO and prunes it while staging A)
  int fused_n, fused_m, fused_scheme;
  uint32_t seed_lo, seed_hi;
  int P, Q;               // dO pixel grid (for the linear element index of the random scheme)
  int f16;                // element type of A, W and dD: 0 = bf16, 1 = IEEE binary16
  // grouped convolution (block-diagonal W): a tile of input channels sees only k_blocks channel blocks of dL/dO,
  // starting at first_k_block(); diag_cin_g == 0: every tile sees all of them
  int diag_cin_g, diag_cout_g, diag_last;
  int off_raw;            // dense dL/dO stages: 2 * a_bytes each (two boxes of 64 channels)
  // shared-memory carve (byte offsets from the 1024-aligned base) and per-stage sizes
  int a_bytes, b_bytes, eraw_bytes, ehw_bytes;
  int off_b, off_eraw, off_ehw, off_w, off_out, off_bar;
  int smem_bytes;
};

template <bool SPARSE, int BN>
struct Cfg {
  static constexpr int kKB = SPARSE ? 128 : 64;               // W rows (output channels) per MMA group
  static constexpr int kBCols = BN / 2;                       // W columns staged by one CTA
  static constexpr int kBoxCols = kBCols < 64 ? kBCols : 64;  // columns of one W box
  static constexpr int kBoxes = kBCols / kBoxCols;
  static constexpr int kRowB = kBoxCols * 2;                  // bytes of one W row in shared memory
  static constexpr uint32_t kBSwizzle = (kRowB == 128) ? 2u : 4u;  // descriptor code: 128-/64-byte swizzle
  static constexpr int kBoxBytes = kKB * kRowB;
  static constexpr int kTapBBytes = kBoxBytes * kBoxes;       // one CTA's W bytes of one (tap, channel block)
  static_assert(kBCols == 32 || kBCols % 64 == 0, "W half must be 32 columns or whole 64-column blocks");
};

// Grouped convolution: input channels n0 .. n0 + BN - 1 belong to groups n0 / cin_g and up, whose output channels
// start at (n0 / cin_g) * cout_g; the tile's window of channel blocks (kbc channels each) starts at that channel's
// block, or at `diag_last` where the window would otherwise run past the last block (W is zero outside the groups'
// own blocks, so a window that covers more than it must changes nothing).
template <class P>
__device__ __forceinline__ int first_k_block(const P& p, int n0, int kbc) {
  if (p.diag_cin_g == 0) return 0;
  const int kb = ((n0 / p.diag_cin_g) * p.diag_cout_g) / kbc;
  return kb < p.diag_last ? kb : p.diag_last;
}

// Instruction descriptor: fp32 accumulate, bf16 A and B, A K-major, B MN-major, M = 256 (pair).
__host__ __device__ constexpr uint32_t make_idesc(int n, bool sparse) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(256 >> 4) << 24) | (sparse ? (1u << 2) : 0u);
}
// The A-format (bits 7-9) and B-format (bits 10-12) fields: 1 = bf16, 0 = binary16. Both operands
// always have the same type.
constexpr uint32_t kIdescBf16Operands = (1u << 7) | (1u << 10);

// Metadata of an A tile: from the row-major order TMA delivers (16 bytes per pixel row: one uint16
// per 16 channels of a 128-channel block) to the order tcgen05.cp moves into TMEM. For the MMA
// covering channels [32*k2, 32*k2+32) of the block the tensor core reads one 32-bit TMEM column:
// lane (row%8) + 8*half + 16*(row/16) holds in its low 16 bits the four position nibbles of
// channels 32*k2 + 16*half + [0,16) of the row with bit 3 clear, in its high 16 bits those of
// row + 8. One call builds the 16 bytes of TMEM lane `tl` from its two rows. Rows that carry no
// data (past the patch, or outside the image where TMA filled zeros) get the well-formed
// position pair (0,1) in every chunk.
// Every position nibble of real metadata is at least 4 (p0 | p1 << 2 with p0 < p1), so a 16-bit
// group of four nibbles is at least 0x4444; pixels outside the image arrive as zeros. The
// per-half maximum with 0x4444 therefore leaves real metadata alone and turns a missing group
// into the well-formed position pair (0,1) in every chunk.
__device__ __forceinline__ uint32_t well_formed(uint32_t x) { return __vmaxu2(x, 0x44444444u); }

__device__ __forceinline__ void build_metadata_lane(const uint8_t* raw_rows, uint8_t* hw_tile, int tl, int rows_used) {
  const int row_a = ((tl >> 4) << 4) + (tl & 7), row_b = row_a + 8;
  const uint32_t sel = (tl & 8) ? 0x7632u : 0x5410u;
  const uint4 k01 = make_uint4(0x44444444u, 0x44444444u, 0x44444444u, 0x44444444u);
  uint4 lo = k01, hi = k01;
  if (row_a < rows_used) lo = *(const uint4*)(raw_rows + row_a * 16);
  if (row_b < rows_used) hi = *(const uint4*)(raw_rows + row_b * 16);
  *(uint4*)(hw_tile + tl * 16) =
      make_uint4(well_formed(prmt(lo.x, hi.x, sel)), well_formed(prmt(lo.y, hi.y, sel)),
                 well_formed(prmt(lo.z, hi.z, sel)), well_formed(prmt(lo.w, hi.w, sel)));
}

// The whole 128-lane image by one warp: four passes of 32 lanes, all loads before all stores
// (the compiler cannot tell the two shared-memory regions apart and would serialise them).
__device__ __forceinline__ void build_metadata_image(const uint8_t* raw_rows, uint8_t* hw_tile, int lane, int rows_used) {
  const uint32_t sel = (lane & 8) ? 0x7632u : 0x5410u;
  const uint4 k01 = make_uint4(0x44444444u, 0x44444444u, 0x44444444u, 0x44444444u);
  uint4 lo[4], hi[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int tl = 32 * i + lane;
    const int row_a = ((tl >> 4) << 4) + (tl & 7), row_b = row_a + 8;
    lo[i] = k01;
    hi[i] = k01;
    if (row_a < rows_used) lo[i] = *(const uint4*)(raw_rows + row_a * 16);
    if (row_b < rows_used) hi[i] = *(const uint4*)(raw_rows + row_b * 16);
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint4 a = lo[i], b = hi[i];
    *(uint4*)(hw_tile + (32 * i + lane) * 16) =
        make_uint4(well_formed(prmt(a.x, b.x, sel)), well_formed(prmt(a.y, b.y, sel)),
                   well_formed(prmt(a.z, b.z, sel)), well_formed(prmt(a.w, b.w, sel)));
  }
}

// Fused pruning of one eighth of a pixel row of a stage (the unit of work the pruning threads share
// out): the row's 128 dense channels lie in two 128-byte-swizzled boxes of 64; 16 of them = two
// vectors become one 16-byte chunk of the compressed row, written straight into the A tile's swizzled
// row, and two of the row's sixteen bytes of position metadata (row-major form, as the rearrangement
// step expects). vbase = number of the row's first 8-element vector in the whole dL/dO tensor (random keys).
template <int M, int N, int SCHEME>
__device__ __forceinline__ void fused_prune_eighth(const uint8_t* raw, int a_bytes, uint8_t* a_tile, uint8_t* meta_rows,
                                                   int i, int e, int64_t vbase, uint32_t seed_lo, uint32_t seed_hi) {
  const int sw = i & 7;
  uint32_t nibs = 0u;
  uint2 out[2];
  uint4 w[2];
#pragma unroll
  for (int jj = 0; jj < 2; ++jj) {
    const int j = 2 * e + jj;
    w[jj] = *(const uint4*)(raw + (j >> 3) * a_bytes + i * 128 + (((j & 7) ^ sw) << 4));
  }
  uint32_t y[2][4], km[2][4];
  if (M == 16) {  // the thread's two vectors are one group
    top2_prune_group16<SCHEME>(w[0], w[1], vbase + 2 * e, seed_lo, seed_hi, N, y[0], km[0], y[1], km[1]);
  } else {
#pragma unroll
    for (int jj = 0; jj < 2; ++jj) {
      if (M == 4)
        m4_prune_vector<N, SCHEME>(w[jj], vbase + 2 * e + jj, seed_lo, seed_hi, y[jj][0], y[jj][1], y[jj][2], y[jj][3], km[jj][0],
                                   km[jj][1], km[jj][2], km[jj][3]);
      else
        top2_prune_vector<8, SCHEME>(w[jj], vbase + 2 * e + jj, seed_lo, seed_hi, N, 0, 0u, y[jj][0], y[jj][1], y[jj][2], y[jj][3],
                                     km[jj][0], km[jj][1], km[jj][2], km[jj][3]);
    }
  }
#pragma unroll
  for (int jj = 0; jj < 2; ++jj) {
    uint32_t slot0, slot1, nib2;
    if (M == 4 && SCHEME == SDGP_RESCALED_MAGNITUDE)  // (the lanes above are dead code then: the slots are rescaled, not the lanes)
      m4_rescaled_compressed<N, false>(w[jj], slot0, slot1, nib2, km[jj][0], km[jj][1], km[jj][2], km[jj][3]);
    else
      compressed_slots(y[jj][0], y[jj][1], y[jj][2], y[jj][3], km[jj][0], km[jj][1], km[jj][2], km[jj][3], slot0, slot1, nib2);
    out[jj] = make_uint2(prmt(slot0, slot1, 0x5410), prmt(slot0, slot1, 0x7632));
    nibs |= nib2 << (8 * jj);
  }
  *(uint4*)(a_tile + i * 128 + ((e ^ sw) << 4)) = make_uint4(out[0].x, out[0].y, out[1].x, out[1].y);
  *(uint16_t*)(meta_rows + i * 16 + 2 * e) = (uint16_t)nibs;
}

// The four epilogue warps move one 128-row x BN accumulator to global memory in 64-column
// slabs: TMEM -> registers -> bf16 -> a 128-byte-swizzled staging tile -> one TMA store of the
// whole pixel patch (full-line writes; pixels outside the tensor are clipped by the TMA unit).
// With two staging slabs the store of one overlaps the packing of the next. `chunk` counts
// slabs over the kernel's lifetime and picks the slab.
// FIVE: dD's tensor map has five dimensions and (w0, h0, b0, e0) are coordinates 1..4.
template <int BN, bool FIVE = false>
__device__ __forceinline__ void store_accumulator(uint32_t taddr, uint8_t* staging, int out_bufs,
                                                  const CUtensorMap* tmD, int n0, int w0, int h0, int b0,
                                                  bool tile_in_range, int row, bool issuer, uint32_t& chunk,
                                                  uint64_t* first_slab_read, bool f16, int e0 = 0) {
#pragma unroll 1
  for (int c0 = 0; c0 < BN; c0 += 64, ++chunk) {
    uint32_t packed[32];
    uint32_t v0[32], v1[32];
    ptx::tmem_ld_32x32(taddr + (uint32_t)c0, v0);
    ptx::tmem_ld_32x32(taddr + (uint32_t)(c0 + 32), v1);
    ptx::tmem_ld_wait();
    if (c0 == 0 && first_slab_read != nullptr) {
      // the accumulator's first 64 columns are in registers: they may now hold the next
      // tile's metadata (signalled before the conversion work, the MMA thread is waiting)
      ptx::tc_fence_before_sync();
      __syncwarp();
      if ((threadIdx.x & 31) == 0) ptx::mbar_arrive_cluster(first_slab_read, 0);
    }
    if (f16) {
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const __half2 a2 = __floats2half2_rn(__uint_as_float(v0[2 * e]), __uint_as_float(v0[2 * e + 1]));
        const __half2 b2 = __floats2half2_rn(__uint_as_float(v1[2 * e]), __uint_as_float(v1[2 * e + 1]));
        packed[e] = *(const uint32_t*)&a2;
        packed[16 + e] = *(const uint32_t*)&b2;
      }
    } else {
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const __nv_bfloat162 a2 = __floats2bfloat162_rn(__uint_as_float(v0[2 * e]), __uint_as_float(v0[2 * e + 1]));
        const __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(v1[2 * e]), __uint_as_float(v1[2 * e + 1]));
        packed[e] = *(const uint32_t*)&a2;
        packed[16 + e] = *(const uint32_t*)&b2;
      }
    }
    uint8_t* buf = staging + (out_bufs == 2 ? (chunk & 1u) : 0u) * kOutBytes;
    if (issuer) {  // the store that last used this slab has finished reading it
      if (out_bufs == 2) ptx::bulk_wait_group_read<1>();
      else ptx::bulk_wait_group_read<0>();
    }
    ptx::named_bar_sync(1, 128);
#pragma unroll
    for (int c = 0; c < 8; ++c)
      *(uint4*)(buf + row * 128 + ((c ^ (row & 7)) << 4)) =
          make_uint4(packed[4 * c], packed[4 * c + 1], packed[4 * c + 2], packed[4 * c + 3]);
    ptx::fence_proxy_async_smem();
    ptx::named_bar_sync(1, 128);
    if (issuer && tile_in_range) {
      if (FIVE) ptx::tma_store_5d(tmD, buf, n0 + c0, w0, h0, b0, e0);
      else ptx::tma_store_4d(tmD, buf, n0 + c0, w0, h0, b0);
      ptx::bulk_commit_group();
    }
  }
}

template <bool SPARSE, int BN, bool FUSED>
__global__ void __launch_bounds__(FUSED ? kThreadsGemmFused : kThreadsGemm, 1)
dgrad_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmE,
             const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmD,
             const DgradParams p) {
  using C = Cfg<SPARSE, BN>;
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment: required by the 128-byte swizzle of the A, B and staging tiles
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = smem;
  uint8_t* sB = smem + p.off_b;
  uint8_t* sEraw = smem + p.off_eraw;
  uint8_t* sEhw = smem + p.off_ehw;
  uint8_t* sW = smem + p.off_w;
  uint8_t* sOut = smem + p.off_out;
  uint8_t* sRaw = smem + p.off_raw;
  uint64_t* full = (uint64_t*)(smem + p.off_bar);
  uint64_t* empty = full + kMaxStages;
  uint64_t* meta_full = empty + kMaxStages;
  uint64_t* acc_full = meta_full + kMaxStages;
  uint64_t* acc_empty = acc_full + 2;
  uint64_t* w_full = acc_empty + 2;
  uint64_t* meta_free = w_full + 1;
  uint64_t* raw_full = meta_free + 2;
  uint32_t* tmem_slot = (uint32_t*)(raw_full + kMaxStages);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();  // 0: issues the MMAs
  unsigned int* err = &g_device_error;
  const int STAGES = p.stages;
  const int NACC = p.nacc;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kMaxStages; ++s) {
      // full: the producer's arrival (with the stage's byte count) plus, for sparse A, the
      // arrivals of the warps that built the stage's metadata images in both CTAs (one warp per
      // CTA; all four when they also prune) - the MMA thread waits once per stage
      ptx::mbar_init(&full[s], SPARSE ? (FUSED ? 9 : 3) : 1);
      ptx::mbar_init(&empty[s], 1);
      ptx::mbar_init(&meta_full[s], 1);
      ptx::mbar_init(&raw_full[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&acc_full[a], 1);
      ptx::mbar_init(&acc_empty[a], 8);
      ptx::mbar_init(&meta_free[a], 8);
    }
    ptx::mbar_init(w_full, 1);
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
  // everything above touched no global memory; the previous kernel's results are needed from here on
  ptx::wait_for_previous_grid();
  // Only now may the next kernel of the stream be scheduled: every CTA of this grid owns its TMEM
  // and has passed its cluster barrier and its wait for the previous grid, so a younger grid can
  // never sit between this grid and a resource it still needs, and at most one grid is resident
  // behind a running one. The younger grid's own TMEM allocation then simply waits for this grid
  // to free its columns, which it does without anyone's help.
  ptx::launch_dependents();

  const int rows_used = p.TW * p.TH * p.TB;
  const int taps = p.R * p.S;
  const bool reuse = (p.rr == p.R) && p.R > 1;
  auto filter_tap = [&p](int r, int s) { return (p.r_first + p.r_step * r) * p.S_full + p.s_first + p.s_step * s; };
  const int groups = reuse ? p.S : taps;  // stage uses per channel block and tile
  const int uses_per_tile = groups * p.k_blocks;
  const int pair_stride = gridDim.x >> 1;
  const int first_pair = blockIdx.x >> 1;
  const int my_tiles = first_pair < p.pair_tiles ? (p.pair_tiles - first_pair + pair_stride - 1) / pair_stride : 0;
  const int n_half = (int)rank * C::kBCols;  // this CTA's column offset inside the BN block

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    if (ptx::elect_one()) {
      bool alive = true;
      if (p.w_resident) {
        // the layer's whole W half-slice, once: [tap][channel block][box] tiles of kKB rows
        if (rank == 0) ptx::mbar_arrive_expect_tx(w_full, 2u * (uint32_t)(taps * p.k_blocks * C::kTapBBytes));
        for (int t = 0; t < taps; ++t) {
          const int ft = filter_tap(t / p.S, t % p.S);
          for (int cb = 0; cb < p.k_blocks; ++cb)
#pragma unroll
            for (int j = 0; j < C::kBoxes; ++j)
              ptx::tma_load_2d_pair(sW + ((t * p.k_blocks + cb) * C::kBoxes + j) * C::kBoxBytes, &tmB, w_full,
                                    ft * p.Cin + n_half + C::kBoxCols * j, cb * C::kKB);
        }
      }
      const uint32_t pair_tx =
          2u * (uint32_t)((FUSED ? 0 : p.img_rows * 128) + (p.w_resident ? 0 : p.rr * C::kTapBBytes));
      const uint32_t meta_tx = (uint32_t)(p.img_rows * 16);
      int st = 0;
      uint32_t ph = 0;
      for (int pt = first_pair; alive && pt < p.pair_tiles; pt += pair_stride) {
        const int nt = pt % p.tiles_n;
        int t = 2 * (pt / p.tiles_n) + (int)rank;  // this CTA's patch; may lie past the last one
        const int wt = t % p.tiles_w; t /= p.tiles_w;
        const int ht = t % p.tiles_h; t /= p.tiles_h;
        const int bt = t;
        const int n0 = nt * BN + n_half;
        const int cb0 = first_k_block(p, nt * BN, C::kKB);
        const int w0 = wt * p.TW, h0 = ht * p.TH, b0 = bt * p.TB;
        // reuse: a group is the horizontal tap s and the image starts R-1 rows above the row
        // the last vertical tap needs; otherwise a group is the single tap (r, s).
        int r = reuse ? (p.R - 1) : 0, s = 0;
        for (int g = 0; alive && g < groups; ++g) {
          const int q0 = w0 + p.pad_w - s, p0 = h0 + p.pad_h - r;
          for (int cb = 0; cb < p.k_blocks; ++cb) {
            if (!ptx::mbar_wait(&empty[st], ph ^ 1u, err, 0x100u + st)) { alive = false; break; }
            if (rank == 0) ptx::mbar_arrive_expect_tx(&full[st], pair_tx);
            if (FUSED) {
              // dense dL/dO of this CTA's patch: 128 channels as two boxes of 64
              ptx::mbar_arrive_expect_tx(&raw_full[st], 2u * (uint32_t)(p.img_rows * 128));
              ptx::tma_load_4d(sRaw + st * 2 * p.a_bytes, &tmA, &raw_full[st], (cb0 + cb) * 128, q0, p0, b0);
              ptx::tma_load_4d(sRaw + st * 2 * p.a_bytes + p.a_bytes, &tmA, &raw_full[st], (cb0 + cb) * 128 + 64, q0, p0, b0);
            } else {
              if (SPARSE) {
                ptx::mbar_arrive_expect_tx(&meta_full[st], meta_tx);
                ptx::tma_load_4d(sEraw + st * p.eraw_bytes, &tmE, &meta_full[st], (cb0 + cb) * 8, q0, p0, b0);
              }
              ptx::tma_load_4d_pair(sA + st * p.a_bytes, &tmA, &full[st], (cb0 + cb) * 64, q0, p0, b0);
            }
            if (!p.w_resident) {
              for (int u = 0; u < p.rr; ++u) {
                const int tap = filter_tap(reuse ? u : r, s);
#pragma unroll
                for (int j = 0; j < C::kBoxes; ++j)
                  ptx::tma_load_2d_pair(sB + st * p.b_bytes + (u * C::kBoxes + j) * C::kBoxBytes, &tmB, &full[st],
                                        tap * p.Cin + n0 + C::kBoxCols * j, (cb0 + cb) * C::kKB);
              }
            }
            if (++st == STAGES) { st = 0; ph ^= 1u; }
          }
          if (++s == p.S) { s = 0; if (!reuse) ++r; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------- MMA issuer (first CTA only)
    // A single thread executes roughly one dependent instruction per ten clocks, so its path
    // per stage is short: one barrier wait, descriptor words kept as running sums.
    if (rank == 0 && ptx::elect_one()) {
      const uint32_t idesc = make_idesc(BN, SPARSE) & ~(p.f16 ? kIdescBf16Operands : 0u);
      bool alive = true;
      if (p.w_resident) alive = ptx::mbar_wait(w_full, 0u, err, 0x700u);
      // descriptors as two 32-bit halves: the start address only ever changes the low word
      const uint64_t adesc0 = ptx::make_smem_desc(0, 16, 1024, 2);
      const uint64_t bdesc0 = ptx::make_smem_desc(0, C::kBoxBytes, 8 * C::kRowB, C::kBSwizzle);
      const uint64_t edesc0 = ptx::make_smem_desc(0, 128, 128, 0);
      const uint32_t a_hi = (uint32_t)(adesc0 >> 32), b_hi = (uint32_t)(bdesc0 >> 32), e_hi = (uint32_t)(edesc0 >> 32);
      const uint32_t a_lo0 = (uint32_t)adesc0 + (ptx::smem_u32(sA) >> 4);
      const uint32_t b_lo0 = (uint32_t)bdesc0 + (ptx::smem_u32(sB) >> 4);
      const uint32_t w_lo0 = (uint32_t)bdesc0 + (ptx::smem_u32(sW) >> 4);
      const uint32_t e_lo0 = (uint32_t)edesc0 + (ptx::smem_u32(sEhw) >> 4);
      const uint32_t a_stage16 = (uint32_t)p.a_bytes >> 4, b_stage16 = (uint32_t)p.b_bytes >> 4,
                     e_stage16 = (uint32_t)p.ehw_bytes >> 4;
      constexpr uint32_t kTapB16 = (uint32_t)C::kTapBBytes >> 4;
      constexpr uint32_t kBStep = (uint32_t)((C::kKB / 4) * C::kRowB / 16);  // W rows of one MMA
      const uint32_t slot_cols = 4u * (uint32_t)p.rr;                         // metadata columns of one stage
      int st = 0, acc = 0;
      uint32_t ph = 0, aph = 0;
      uint32_t a_lo = a_lo0, b_lo = b_lo0, e_lo = e_lo0, mcol = 0;  // running words of the stage ring
      for (int lt = 0; alive && lt < my_tiles; ++lt) {
        if (!ptx::mbar_wait(&acc_empty[acc], aph ^ 1u, err, 0x200u + acc)) break;
        // Shared metadata region: this tile's slots are the first columns of the other
        // accumulator, which the epilogue of the previous tile must have read out first.
        if (p.meta_shared && lt > 0 &&
            !ptx::mbar_wait(&meta_free[acc ^ 1], (((uint32_t)lt - 1u) >> 1) & 1u, err, 0x800u + acc))
          break;
        const uint32_t meta_base = tmem_base + (uint32_t)(p.meta_shared ? (acc ^ 1) * BN : p.meta_col);
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        uint32_t accumulate = 0u;
        int r_single = 0, s = 0;
        for (int g = 0; alive && g < groups; ++g) {
          for (int cb = 0; cb < p.k_blocks; ++cb) {
            if (!ptx::mbar_wait(&full[st], ph, err, 0x300u + st)) { alive = false; break; }
            ptx::tc_fence_after_sync();
            const uint32_t e_col = meta_base + mcol;  // even: slots are multiples of 4 columns apart
            if (SPARSE) {
              for (int u = 0; u < p.rr; ++u)
                ptx::tc_cp_128x128b_pair(e_col + 4u * u, ((uint64_t)e_hi << 32) | (e_lo + (uint32_t)(u * (kEHwBytes / 16))));
            }
            for (int u = 0; u < p.rr; ++u) {
              // vertical tap r: the tile's rows start (R-1-r) image rows into the stage
              const int r = reuse ? u : r_single;
              const uint32_t a_u = a_lo + (reuse ? (uint32_t)((p.R - 1 - r) * p.TW * 8) : 0u);
              const uint32_t b_u = p.w_resident ? w_lo0 + (uint32_t)((r * p.S + s) * p.k_blocks + cb) * kTapB16
                                                : b_lo + (uint32_t)u * kTapB16;
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                // A: 32 bytes of a 128-byte swizzled row per MMA; B: 16 (dense) or 32 (sparse) rows
                const uint64_t a_q = ((uint64_t)a_hi << 32) | (a_u + (uint32_t)(q * 2));
                const uint64_t b_q = ((uint64_t)b_hi << 32) | (b_u + (uint32_t)q * kBStep);
                if (SPARSE)
                  ptx::mma_sp_f16_ss_pair(d_tmem, a_q, b_q, e_col + 4u * u + (uint32_t)(q & 2), idesc | (uint32_t)(q & 1),
                                          q == 0 ? accumulate : 1u);
                else
                  ptx::mma_f16_ss_pair(d_tmem, a_q, b_q, idesc, q == 0 ? accumulate : 1u);
              }
              accumulate = 1u;
            }
            ptx::tc_commit_pair(&empty[st], 3);
            if (++st == STAGES) { st = 0; ph ^= 1u; a_lo = a_lo0; b_lo = b_lo0; e_lo = e_lo0; mcol = 0; }
            else { a_lo += a_stage16; b_lo += b_stage16; e_lo += e_stage16; mcol += slot_cols; }
          }
          if (++s == p.S) { s = 0; ++r_single; }
        }
        if (alive) ptx::tc_commit_pair(&acc_full[acc], 3);
        if (++acc == NACC) { acc = 0; aph ^= 1u; }
      }
    }
  } else if (warp < 6 || warp >= 10) {  // warps 10.. exist only in the fused instantiation
    // ------------------------------------------------- metadata rearranger
    if (SPARSE && !FUSED) {
      // A lone warp runs a dependent chain slowly, so the four warps do not share a stage: warp k
      // owns stages k, k+G, ... of the ring and builds the TMEM metadata images of every use of
      // those stages (four passes of 32 lanes per image); consecutive uses fall to different warps,
      // so up to G are in flight.
      // Ownership goes by STAGE, not by use: a parity wait tells "the phase I expect has completed"
      // from "the phase two before it has" only if the waiter saw the phase in between complete.
      // The warp that owns a stage waits for each of its uses in turn, so it always has. (A warp
      // that took uses k, k+G, ... regardless of stage would wait for use u of a stage without
      // having waited for use u - STAGES; that box was requested earlier than the boxes the warp
      // did see land, but TMA boxes may land out of request order, and a box that is late lets
      // the wait pass one phase early.)
      const int G = STAGES < 4 ? STAGES : 4;
      const int total_uses = (warp - 2 < G) ? my_tiles * uses_per_tile : 0;
      uint32_t ph = 0;
      for (int first = 0; first < total_uses; first += STAGES, ph ^= 1u) {  // one pass over the ring
        bool alive = true;
        for (int st = warp - 2; st < STAGES && first + st < total_uses; st += G) {
          // the metadata box was requested after the stage's previous use had been consumed
          if (!ptx::mbar_wait(&meta_full[st], ph, err, 0x500u + st)) { alive = false; break; }
          for (int v = 0; v < p.rr; ++v) {
            const int row_off = reuse ? (p.R - 1 - v) * p.TW : 0;
            build_metadata_image(sEraw + st * p.eraw_bytes + row_off * 16, sEhw + st * p.ehw_bytes + v * kEHwBytes, lane,
                                 rows_used);
          }
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive_cluster(&full[st], 0);
        }
        if (!alive) break;
      }
    } else if (SPARSE) {
      // Fused pruning: warps 2..5 and the helper warps 10.. share out the stage's pixel rows in eighths
      // (item = row, eighth); then each thread of warps 2..5 builds one TMEM lane of every metadata image.
      const int pruner = warp < 6 ? (int)threadIdx.x - 64 : 128 + (int)threadIdx.x - kThreadsGemm;  // 0 .. kFusedPruners - 1
      const int row = threadIdx.x - 64;  // warps 2..5 only
      bool alive = true;
      int st = 0;
      uint32_t ph = 0;
      const int img_h = p.TH + p.rr - 1;
      for (int pt = first_pair; alive && pt < p.pair_tiles; pt += pair_stride) {
        int t = 2 * (pt / p.tiles_n) + (int)rank;
        const int wt = t % p.tiles_w; t /= p.tiles_w;
        const int ht = t % p.tiles_h; t /= p.tiles_h;
        const int w0 = wt * p.TW, h0 = ht * p.TH, b0 = t * p.TB;
        const int cb0 = first_k_block(p, (pt % p.tiles_n) * BN, C::kKB);
        int r = reuse ? (p.R - 1) : 0, s = 0, cb = 0;
        for (int k = 0; k < uses_per_tile; ++k) {
          // the pruning warps stay or leave together: they meet at a named barrier below
          if (!ptx::named_bar_all(2, kFusedPruners, ptx::mbar_wait(&raw_full[st], ph, err, 0x900u + st))) { alive = false; break; }
          const int q0 = w0 + p.pad_w - s, p0 = h0 + p.pad_h - r;
          const uint8_t* raw = sRaw + st * 2 * p.a_bytes;
          uint8_t* a_tile = sA + st * p.a_bytes;
          uint8_t* meta_rows = sEraw + st * p.eraw_bytes;
          for (int item = pruner; item < 8 * p.img_rows; item += kFusedPruners) {
            const int i = item >> 3, e = item & 7;
            const int iw = i % p.TW, ih = (i / p.TW) % img_h, ib = i / (p.TW * img_h);
            const int64_t pixel = ((int64_t)(b0 + ib) * p.P + (p0 + ih)) * p.Q + (q0 + iw);  // any value when outside
            const int64_t vbase = pixel * (p.Cout >> 3) + (cb0 + cb) * 16;
#define SDGP_FUSED_ITEM(MM, NN, SS) fused_prune_eighth<MM, NN, SS>(raw, p.a_bytes, a_tile, meta_rows, i, e, vbase, p.seed_lo, p.seed_hi)
#define SDGP_FUSED_M(MM)                                                                                                   \
  if (p.fused_scheme == SDGP_MAGNITUDE) { if (p.fused_n == 1) SDGP_FUSED_ITEM(MM, 1, SDGP_MAGNITUDE); else SDGP_FUSED_ITEM(MM, 2, SDGP_MAGNITUDE); } \
  else if (p.fused_scheme == SDGP_RANDOM) { if (p.fused_n == 1) SDGP_FUSED_ITEM(MM, 1, SDGP_RANDOM); else SDGP_FUSED_ITEM(MM, 2, SDGP_RANDOM); }    \
  else { if (p.fused_n == 1) SDGP_FUSED_ITEM(MM, 1, SDGP_RESCALED_MAGNITUDE); else SDGP_FUSED_ITEM(MM, 2, SDGP_RESCALED_MAGNITUDE); }
            if (p.fused_m == 4) { SDGP_FUSED_M(4) } else if (p.fused_m == 8) { SDGP_FUSED_M(8) } else { SDGP_FUSED_M(16) }
#undef SDGP_FUSED_M
#undef SDGP_FUSED_ITEM
          }
          ptx::fence_proxy_async_smem();                // the compressed tile is read by the tensor core
          ptx::named_bar_sync(2, kFusedPruners);        // every row's metadata is in place before it is rearranged
          if (warp < 6) {
            for (int u = 0; u < p.rr; ++u) {
              const int row_off = reuse ? (p.R - 1 - u) * p.TW : 0;
              build_metadata_lane(sEraw + st * p.eraw_bytes + row_off * 16, sEhw + st * p.ehw_bytes + u * kEHwBytes, row,
                                  rows_used);
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(&full[st], 0);
          }
          if (++st == STAGES) { st = 0; ph ^= 1u; }
          if (++cb == p.k_blocks) {
            cb = 0;
            if (++s == p.S) { s = 0; if (!reuse) ++r; }
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int q = warp & 3;  // a warp may only touch TMEM lanes [32*(warp%4), +32)
    const int row = q * 32 + lane;
    const bool issuer = (threadIdx.x == 192);
    uint32_t chunk = 0, aph = 0;
    int acc = 0;
    for (int pt = first_pair; pt < p.pair_tiles; pt += pair_stride) {
      const int nt = pt % p.tiles_n;
      const int mt = 2 * (pt / p.tiles_n) + (int)rank;
      int t = mt;
      const int wt = t % p.tiles_w; t /= p.tiles_w;
      const int ht = t % p.tiles_h; t /= p.tiles_h;
      const int bt = t;
      if (!ptx::mbar_wait(&acc_full[acc], aph, err, 0x600u + acc)) break;
      ptx::tc_fence_after_sync();
      store_accumulator<BN>(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN), sOut, p.out_bufs, &tmD,
                            nt * BN, wt * p.TW, ht * p.TH, bt * p.TB, mt < p.m_tiles, row, issuer, chunk,
                            p.meta_shared ? &meta_free[acc] : nullptr, p.f16 != 0);
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive_cluster(&acc_empty[acc], 0);
      if (++acc == NACC) { acc = 0; aph ^= 1u; }
    }
    // the staging slabs have been read; the writes themselves complete with the grid (whoever depends on dD waits for that)
    if (issuer) ptx::bulk_wait_group_read<0>();
  }

  __syncwarp();
  if (*(volatile unsigned int*)err != 0u) {
    // A wait gave up somewhere: loads may still be in flight towards this CTA's shared
    // memory. Give them a bounded while to land before the CTA goes away.
    const uint64_t t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 200000ull) {
    }
  }
  ptx::tc_fence_before_sync();
  __syncwarp();
  ptx::cluster_sync();  // neither CTA leaves (or frees TMEM) while the other may still touch it
  ptx::tc_fence_after_sync();
  if (warp == 1) ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
}

// ---------------------------------------------------------------- whole-filter reuse
//
// Convolutions with more than one filter tap.
// The shared-memory matrix descriptor swizzles by absolute address bits, so an A operand may
// start at ANY 128-byte row of a swizzled tile and its 8-row groups may lie any number of rows
// apart. A tile is therefore a strip of 16 rows of 8 pixels, and one TMA box holding the strip plus
// its (R-1, S-1) halo serves EVERY filter tap: tap (r, s) is the row offset
// (R-1-r) * tb * pitch + (S-1-s) in the A descriptor, group stride = pitch rows. dL/dO is
// read from L2 once per strip (plus halo) instead of once per horizontal tap, and with two
// neighbouring strips per CTA (two accumulators) each W stage feeds twice the MMAs.
// Strip geometries (th pixel rows x tb images, th * tb = 16): 16 rows of one image; 8 rows of two images
// (images at most 8 pixels tall; the box's rows are ordered (pixel row, image)); and, for images 4 pixels
// wide, 4 rows of eight images with two images side by side in a strip row and one box per filter column
// (column-split mode: no column halo, five-dimensional tensor maps).
//
// Rings: A boxes (2 or 4 stages; one stage = one tile set and one block of output channels, with the raw
// metadata box TMA delivers and the two metadata masters built from it), W taps (w_stages; one stage = the W
// rows of one tap and channel block, and a slot of TMEM columns for that tap's metadata).
// Metadata masters: the position metadata of a box is stored once, in the order the tensor core wants, and every
// tap copies a window of it into TMEM (see HaloParams). Two-pass: warps 2..5 build the masters of each box;
// fused: the pruning warps write them directly.

constexpr int kHaloRows = 16;  // 8-pixel rows of a strip: the 128 rows of an accumulator
constexpr int kHaloAStages = 4;  // at most: A stages in use are p.a_stages = 2, or 4 when the boxes are small (a power of two)
// Warp roles of the fused whole-filter-reuse kernel (24 warps: registers are granted to warps in fours, and
// 24 x 80 registers is what fits): warp 0 streams W, warp 1 issues the MMAs, warps 4..7 are the epilogue (one per
// TMEM lane quarter) and the other eighteen prune. Warp w runs on scheduler w % 4, so four pruning warps (9, 13, 17,
// 21) share the scheduler of the MMA-issuing warp; measured, their integer-pipe time is worth more than the issue
// slots they take from it (14 -> 16 -> 18 pruning warps: 1062 -> 1107 -> 1111 TFLOP/s on the ResNet-9 chain).
constexpr int kPruneWarps = 18;
constexpr unsigned kIdleWaitNs = 200;  // sleep between polls of the waits that are off the critical path
constexpr int kThreadsHaloFused = 24 * 32;

// Division by a divisor fixed for the launch: m = floor(2^32 / d) (0xFFFFFFFF for d = 1) gives a quotient
// that is at most one too small for any 32-bit x; one correction step makes it exact.
__host__ __device__ inline uint32_t div_magic(uint32_t d) { return d <= 1 ? 0xFFFFFFFFu : (uint32_t)(0x100000000ull / d); }
__device__ __forceinline__ void divmod(uint32_t x, uint32_t d, uint32_t m, uint32_t& q, uint32_t& r) {
  q = __umulhi(x, m);
  r = x - q * d;
  if (r >= d) { ++q; r -= d; }
}

struct HaloParams {
  int B, H, W, Cin, Cout;
  int R, S, pad_h, pad_w;
  int r_first, r_step, s_first, s_step, S_full;  // as in DgradParams
  int nt;                  // strips per CTA tile set (1 or 2), side by side, sharing every W stage
  int sets_w, tiles_h, tiles_n;
  int m_sets;              // sets_w * tiles_h * B
  uint32_t mg_tiles_n, mg_sets_w, mg_tiles_h;  // div_magic of the three counts above
  int pair_tiles;          // ceil(m_sets / 2) * tiles_n
  int units;               // work units: pair tiles, the last `units - split_from` of them split by strip
  int split_from;          // units >= split_from cover one strip of a pair tile each (quantisation of the last round)
  int k_blocks;
  int pitch;               // pixel columns of the A box: 8 * nt + S - 1
  int th, tb;              // a strip is 8 pixels wide and covers th pixel rows of tb images, th * tb = 16: 16 x 1, or 8 x 2
                           // for images at most 8 pixels tall. Its 16 rows are ordered (pixel row, image), so a vertical
                           // tap is still one uniform row offset (tb rows).
  int img_h;               // rows of the A box: (th + R - 1) * tb, ordered (pixel row, image)
  // Images 4 pixels wide: the 8 pixels of a strip row are the same pixel row of TWO images, a box row holds
  // img_per_row = 2 * nt images side by side with no column halo (an image's neighbour is another image), and
  // the horizontal taps are served by separate boxes: ss = S boxes per channel block, each fetched with its
  // own column offset (the tensor map zero-fills beyond an image's edge), sb = 1 filter column per box.
  // Otherwise img_per_row = 1, ss = 1, sb = S.
  int split, img_per_row, ss, sb;
  int k_uses;              // A boxes per tile set: k_blocks * ss
  int a_stages, a_shift;   // A ring depth (2 or 4) and its log2
  int img_rows;            // pitch * img_h
  // Fused mode, work units of the pruning warps (8 box pixels each). static_pad == 0: unit u = box pixels 8u .. 8u + 7
  // in row-major order, units_per_box = ceil(img_rows / 8). static_pad == 1 (a tile set spans its images from edge to
  // edge, so the halo rows and columns of EVERY box are padding): the stages are cleared once when the kernel starts and
  // only the units inside the images are ever pruned and written - unit u = 8 pixels from column unit_col0 + 8 * (u % nt)
  // of box row unit_row0 + u / nt, units_per_box = H * tb * nt. Fewer units per box also means fewer rounds of units
  // per pruning warp, which is what sets the time a box takes.
  int static_pad, units_per_box, unit_row0, unit_col0;
  int w_stages;
  int meta_col, meta_shared, out_bufs;
  int a_bytes, eraw_bytes, w_bytes;  // per stage
  // Position metadata of an A box in the order the tensor core wants, stored ONCE per box and shared by every
  // tap: "master" pi (pi = 0, 1) pairs box rows (pi + 2m, pi + 2m + 1); its 16-byte line ((2m + e) * pitch + x)
  // holds, for the four MMAs of a channel block, the metadata of channels 16e .. 16e+15 of the MMA's 32 at
  // box pixel (pi + 2m, x) in the low half-words and of the pixel below it in the high half-words. The
  // TMEM image of tap (r, s) and strip j is then the window of 16 groups of 8 lines that starts at line
  // ((R-1-r - pi) * pitch + 8j + S-1-s) of master pi = (R-1-r) % 2, groups pitch lines apart: one
  // tcgen05.cp whose descriptor carries that start address and stride.
  int pairs0, pairs1;      // row pairs of the two masters
  int m0_bytes, meta_bytes;  // bytes of master 0; of both (one A stage)
  int off_eraw, off_meta, off_w, off_out, off_bar;
  int smem_bytes;
  // fused pruning (A is the dense dL/dO; m = 4): the pruning warps read it straight from global memory
  const uint8_t* a_dense;  // dL/dO [B, P, Q, Cout], 16-bit elements
  int diag_cin_g, diag_cout_g, diag_last;  // grouped convolution: see first_k_block()
  uint32_t pitch_magic;    // ceil(2^20 / pitch): i / pitch == (i * pitch_magic) >> 20 for every box pixel row i
  int fused_n, fused_m, fused_scheme;
  uint32_t seed_lo, seed_hi;
  int P, Q;                // dO pixel grid (linear element index of the random scheme)
  int f16;                 // element type of A, W and dD: 0 = bf16, 1 = IEEE binary16
};

// Fused pruning of four vectors (8 channels each, already in registers) of one pixel row: out[v] = the 8
// compressed bytes of vector v, metaw = their four bytes of position metadata (byte v = the two nibbles of
// vector v). Number of vector v in the whole dL/dO tensor (random keys): vbase + vstep * v. Groups of M = 8, 16
// or 32 channels span 1, 2 or 4 vectors held by neighbouring lanes (lane bits 0 and up; `part` = which of
// them this lane's vectors are); all 32 lanes must call together.
template <int M, int N, int SCHEME>
__device__ __forceinline__ void fused_prune_vectors(const uint4 (&w)[4], int64_t vbase, int vstep, uint32_t seed_lo,
                                                    uint32_t seed_hi, int part, uint2 (&out)[4], uint32_t& metaw) {
  metaw = 0u;
#pragma unroll
  for (int v = 0; v < 4; ++v) {
    uint32_t y0, y1, y2, y3, km0, km1, km2, km3, slot0, slot1, nib2;
    if (M == 4 && SCHEME == SDGP_RESCALED_MAGNITUDE) {
      m4_rescaled_compressed<N, false>(w[v], slot0, slot1, nib2, km0, km1, km2, km3);  // the slots are rescaled, not the lanes
    } else if (SCHEME == SDGP_RESCALED_MAGNITUDE) {
      top2_rescaled_compressed<(M == 4 ? 8 : M), false>(w[v], N, part, 0xFFFFFFFFu, slot0, slot1, nib2, km0, km1, km2, km3);
    } else {
      if (M == 4)
        m4_prune_vector<N, SCHEME>(w[v], vbase + vstep * v, seed_lo, seed_hi, y0, y1, y2, y3, km0, km1, km2, km3);
      else
        top2_prune_vector<(M == 4 ? 8 : M), SCHEME>(w[v], vbase + vstep * v, seed_lo, seed_hi, N, part, 0xFFFFFFFFu, y0, y1, y2,
                                                    y3, km0, km1, km2, km3);
      compressed_slots(y0, y1, y2, y3, km0, km1, km2, km3, slot0, slot1, nib2);
    }
    out[v] = make_uint2(prmt(slot0, slot1, 0x5410), prmt(slot0, slot1, 0x7632));
    metaw |= nib2 << (8 * v);
  }
}

// 16 bytes from global memory, read-only path, kept out of L1 (each byte is used once by this SM).
__device__ __forceinline__ uint4 ldg_stream(const uint8_t* ptr) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(ptr));
  return v;
}

template <bool SPARSE, int BN, int NT, bool FUSED>
__global__ void __launch_bounds__(FUSED ? kThreadsHaloFused : kThreadsGemm, 1)
dgrad_halo_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmE,
                  const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmD,
                  const HaloParams p) {
  using C = Cfg<SPARSE, BN>;
  constexpr int kEpilogueWarp0 = FUSED ? 4 : 6;  // first of the four epilogue warps
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = smem;
  uint8_t* sEraw = smem + p.off_eraw;    // two-pass: the row-major metadata box as TMA delivers it
  uint8_t* sMeta = smem + p.off_meta;    // the two metadata masters of each A stage
  uint8_t* sW = smem + p.off_w;
  uint8_t* sOut = smem + p.off_out;
  uint64_t* a_full = (uint64_t*)(smem + p.off_bar);
  uint64_t* a_empty = a_full + kHaloAStages;
  uint64_t* meta_full = a_empty + kHaloAStages;
  uint64_t* meta_ready = meta_full + kHaloAStages;  // two-pass: the masters of the A stage are built (both CTAs)
  uint64_t* w_ready = meta_ready + kHaloAStages;    // W bytes landed
  uint64_t* w_empty = w_ready + kMaxStages;
  uint64_t* acc_full = w_empty + kMaxStages;
  uint64_t* acc_empty = acc_full + 2;
  uint64_t* meta_free = acc_empty + 2;
  uint32_t* tmem_slot = (uint32_t*)(meta_free + 2);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();
  unsigned int* err = &g_device_error;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kHaloAStages; ++s) {
      // fused: A and its metadata rows are complete when every pruning warp has arrived
      // (a_full: the warps of both CTAs; meta_full: this CTA's)
      // (one arrival per work unit of the box: 8 pixel rows)
      ptx::mbar_init(&a_full[s], FUSED ? 2 * p.units_per_box : 1);
      ptx::mbar_init(&a_empty[s], 1);
      ptx::mbar_init(&meta_full[s], 1);
      ptx::mbar_init(&meta_ready[s], 8);  // four metadata warps in each CTA
    }
    for (int s = 0; s < kMaxStages; ++s) {
      ptx::mbar_init(&w_ready[s], 1);  // the producer's arrival with the byte count
      ptx::mbar_init(&w_empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&acc_full[a], 1);
      ptx::mbar_init(&acc_empty[a], 8);
      ptx::mbar_init(&meta_free[a], 8);
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
  ptx::cluster_sync();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base_any = *tmem_slot;
  const uint32_t tmem_base = tmem_base_any;
  // everything above touched no global memory; the previous kernel's results are needed from here on
  ptx::wait_for_previous_grid();
  // Only now may the next kernel of the stream be scheduled: every CTA of this grid owns its TMEM
  // and has passed its cluster barrier and its wait for the previous grid, so a younger grid can
  // never sit between this grid and a resource it still needs, and at most one grid is resident
  // behind a running one. The younger grid's own TMEM allocation then simply waits for this grid
  // to free its columns, which it does without anyone's help.
  ptx::launch_dependents();

  const int taps = p.R * p.sb;  // filter taps served by one A box
  const int pair_stride = gridDim.x >> 1;
  const int first_pair = blockIdx.x >> 1;
  const int my_tiles = first_pair < p.units ? (p.units - first_pair + pair_stride - 1) / pair_stride : 0;
  const int n_half = (int)rank * C::kBCols;
  constexpr int set_cols = NT * BN;  // TMEM columns of one tile set's accumulators
  const int WS = p.w_stages;
  // Work unit u: a pair tile, or - for the units of the last, partly filled round - one strip of
  // a pair tile, so that the round costs half. strip_mask: the strips unit number lt of this CTA covers.
  auto strip_mask = [&p, first_pair, pair_stride](int lt) -> uint32_t {
    const int u = first_pair + lt * pair_stride;
    return u < p.split_from ? ((1u << NT) - 1u) : (1u << ((u - p.split_from) & 1));
  };
  // tile set of unit `u` for this CTA: first input channel, first pixel column / row, image
  auto locate = [&p, rank](int u, int& n0, int& w0, int& h0, int& b0) -> bool {
    const int pt = u < p.split_from ? u : p.split_from + ((u - p.split_from) >> 1);
    uint32_t q, r;
    divmod((uint32_t)pt, (uint32_t)p.tiles_n, p.mg_tiles_n, q, r);
    n0 = (int)r * BN;
    const uint32_t t = 2u * q + rank;
    const bool in_range = (int)t < p.m_sets;  // a set past the last one loads zeros and stores nothing
    divmod(t, (uint32_t)p.sets_w, p.mg_sets_w, q, r);
    w0 = (int)r * 8 * NT;
    divmod(q, (uint32_t)p.tiles_h, p.mg_tiles_h, q, r);
    h0 = (int)r * p.th;
    b0 = (int)q * p.tb * p.img_per_row;
    return in_range;
  };

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    if (ptx::elect_one()) {
      const uint32_t a_tx = 2u * (uint32_t)(p.img_rows * 128);
      const uint32_t meta_tx = (uint32_t)(p.img_rows * 16);
      const uint32_t w_tx = 2u * (uint32_t)C::kTapBBytes;
      const int a_uses = my_tiles * p.k_uses;
      int ia = 0, ast = 0;
      uint32_t aph = 0;
      // Loads the A box (and raw metadata) of stage use `ia`. blocking == false: only if the
      // stage is free right now. Returns 1 issued, 0 not free, -1 wait gave up.
      auto issue_a = [&](bool blocking) -> int {
        if (blocking) {
          if (!ptx::mbar_wait(&a_empty[ast], aph ^ 1u, err, 0x100u + ast)) return -1;
        } else if (!ptx::mbar_test(&a_empty[ast], aph ^ 1u)) {
          return 0;
        }
        const int lt = ia / p.k_uses, ku = ia - lt * p.k_uses;
        const int kl = ku / p.ss, si = ku - kl * p.ss;  // channel block of the tile's window, filter column of the box (column-split mode)
        int n0, w0, h0, b0;
        locate(first_pair + lt * pair_stride, n0, w0, h0, b0);
        const int kb = first_k_block(p, n0, C::kKB) + kl;
        const int q0 = w0 + p.pad_w - (p.sb - 1) - si, p0 = h0 + p.pad_h - (p.R - 1);
        // coordinates: channel, pixel column, image within a box row, image group, pixel row
        const int bg = b0 / p.img_per_row;
        if (rank == 0) ptx::mbar_arrive_expect_tx(&a_full[ast], a_tx);
        // (the tensor maps have the image-within-row dimension only in column-split mode)
        if (SPARSE) {
          ptx::mbar_arrive_expect_tx(&meta_full[ast], meta_tx);
          if (p.split) ptx::tma_load_5d(sEraw + ast * p.eraw_bytes, &tmE, &meta_full[ast], kb * 8, q0, 0, bg, p0);
          else ptx::tma_load_4d(sEraw + ast * p.eraw_bytes, &tmE, &meta_full[ast], kb * 8, q0, b0, p0);
        }
        if (p.split) ptx::tma_load_5d_pair(sA + ast * p.a_bytes, &tmA, &a_full[ast], kb * 64, q0, 0, bg, p0);
        else ptx::tma_load_4d_pair(sA + ast * p.a_bytes, &tmA, &a_full[ast], kb * 64, q0, b0, p0);
        ++ia;
        if (++ast == p.a_stages) { ast = 0; aph ^= 1u; }
        return 1;
      };
      bool alive = true;
      int wst = 0, use = 0;
      uint32_t wph = 0;
      for (int lt = 0; alive && lt < my_tiles; ++lt) {
        int n0, w0_unused, h0_unused, b0_unused;
        locate(first_pair + lt * pair_stride, n0, w0_unused, h0_unused, b0_unused);
        const int kb0 = first_k_block(p, n0, C::kKB);
        n0 += n_half;
        for (int ku = 0; alive && ku < p.k_uses; ++ku, ++use) {
          const int kl = ku / p.ss, si = ku - kl * p.ss, kb = kb0 + kl;
          // (fused: the pruning warps fetch dL/dO themselves; this thread streams W only)
          while (!FUSED && alive && ia <= use)
            if (issue_a(true) < 0) alive = false;
          for (int t = 0; alive && t < taps; ++t) {
            // the next A box goes out as soon as its stage is released, between W taps
            if (!FUSED && ia < a_uses && ia < use + p.a_stages && issue_a(false) < 0) { alive = false; break; }
            if (!ptx::mbar_wait<kIdleWaitNs>(&w_empty[wst], wph ^ 1u, err, 0x180u + wst)) { alive = false; break; }
            if (rank == 0) ptx::mbar_arrive_expect_tx(&w_ready[wst], w_tx);
            const int r = t / p.sb, s = t - r * p.sb + si;
            const int ft = (p.r_first + p.r_step * r) * p.S_full + p.s_first + p.s_step * s;
#pragma unroll
            for (int j = 0; j < C::kBoxes; ++j)
              ptx::tma_load_2d_pair(sW + wst * p.w_bytes + j * C::kBoxBytes, &tmB, &w_ready[wst],
                                    ft * p.Cin + n0 + C::kBoxCols * j, kb * C::kKB);
            if (++wst == WS) { wst = 0; wph ^= 1u; }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------- MMA issuer (first CTA only)
    // The whole warp walks the loops together and one elected lane issues the tensor-core instructions: every
    // address and descriptor word is then the same in all lanes, which lets the compiler keep them in the warp's
    // uniform registers, where those instructions take their operands from. The path per tap is kept short: one
    // barrier wait, running descriptor words updated by additions, compile-time offsets for the strips and the four
    // MMAs of a channel block.
    if (rank == 0) {
      const bool leader = ptx::elect_one();
      const uint32_t tmem_base = __shfl_sync(0xFFFFFFFFu, tmem_base_any, 0);  // one value for the warp, and known to be
      const uint32_t idesc = make_idesc(BN, SPARSE) & ~(p.f16 ? kIdescBf16Operands : 0u);
      // descriptors as two 32-bit halves: the start address only ever changes the low word
      const uint64_t adesc0 = ptx::make_smem_desc(0, 16, (uint32_t)p.pitch * 128u, 2);
      const uint64_t bdesc0 = ptx::make_smem_desc(0, C::kBoxBytes, 8 * C::kRowB, C::kBSwizzle);
      // metadata window: 16 groups of 8 consecutive 16-byte lines, one pitch of lines apart
      const uint64_t edesc0 = ptx::make_smem_desc(0, 128, (uint32_t)p.pitch * 16u, 0);
      const uint32_t a_hi = (uint32_t)(adesc0 >> 32), b_hi = (uint32_t)(bdesc0 >> 32), e_hi = (uint32_t)(edesc0 >> 32);
      const uint32_t a_lo0 = (uint32_t)adesc0 + (ptx::smem_u32(sA) >> 4);
      const uint32_t b_lo0 = (uint32_t)bdesc0 + (ptx::smem_u32(sW) >> 4);
      const uint32_t e_lo0 = (uint32_t)edesc0 + (ptx::smem_u32(sMeta) >> 4);
      const uint32_t a_stage16 = (uint32_t)p.a_bytes >> 4, w_stage16 = (uint32_t)p.w_bytes >> 4,
                     e_stage16 = (uint32_t)p.meta_bytes >> 4, m1_off16 = (uint32_t)p.m0_bytes >> 4;
      // first line (16-byte units) of the window of vertical tap offset dr = R-1-r: master dr % 2, pair dr / 2
      auto meta_row16 = [&p, m1_off16](int dr) -> uint32_t {
        const int off = dr * p.tb;  // box rows
        return ((off & 1) ? m1_off16 : 0u) + (uint32_t)((off >> 1) * 2 * p.pitch);
      };
      const uint32_t a_first16 = (uint32_t)(((p.R - 1) * p.tb * p.pitch + (p.sb - 1)) * 8);  // tap (0,0), in 16-byte units
      const uint32_t a_rowstep16 = (uint32_t)((p.tb * p.pitch - (p.sb - 1)) * 8);            // last tap of a filter row -> first of the next
      constexpr uint32_t kBStep = (uint32_t)((C::kKB / 4) * C::kRowB / 16);  // W rows of one MMA
      constexpr uint32_t kSlotCols = 4u * NT;                                // metadata columns of one W stage
      bool alive = true;
      int ast = 0, acc = 0, wst = 0;
      uint32_t aph = 0, wph = 0, cph = 0;
      // running words of the W ring: W descriptor, metadata column (relative)
      uint32_t b_lo = b_lo0, mcol = 0;
      // (a wait that gives up in one lane ends the role for the whole warp)
      auto wait_all = [&](uint64_t* bar, uint32_t parity, unsigned int code) -> bool {
        return __all_sync(0xFFFFFFFFu, ptx::mbar_wait(bar, parity, err, code));
      };
      for (int lt = 0; alive && lt < my_tiles; ++lt) {
        if (!wait_all(&acc_empty[acc], cph ^ 1u, 0x200u + acc)) break;
        // shared metadata region: the first columns of the other tile set's accumulators,
        // which the epilogue of the previous tile set reads out first
        if (p.meta_shared && lt > 0 && !wait_all(&meta_free[acc ^ 1], (((uint32_t)lt - 1u) >> 1) & 1u, 0x800u + acc)) break;
        const uint32_t meta_base = tmem_base + (uint32_t)(p.meta_shared ? (acc ^ 1) * set_cols : p.meta_col);
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * set_cols);
        const uint32_t strips = strip_mask(lt);
        const bool all_strips = strips == ((1u << NT) - 1u);
        uint32_t accumulate = 0u;
        for (int ku = 0; alive && ku < p.k_uses; ++ku) {
          if (!wait_all(&a_full[ast], aph, 0x300u + ast)) { alive = false; break; }
          if (SPARSE && !FUSED && !wait_all(&meta_ready[ast], aph, 0x340u + ast)) { alive = false; break; }
          uint32_t a_lo = a_lo0 + (uint32_t)ast * a_stage16 + a_first16;
          int s = p.sb, dr = p.R - 1;
          const uint32_t e_stage = e_lo0 + (uint32_t)ast * e_stage16;
          uint32_t e_lo = e_stage + meta_row16(dr) + (uint32_t)(p.sb - 1);
          for (int t = 0; t < taps; ++t) {
            if (!wait_all(&w_ready[wst], wph, 0x380u + wst)) { alive = false; break; }
            ptx::tc_fence_after_sync();
            const uint32_t e_col = meta_base + mcol;  // even: slots are 4 columns apart
            // ALL: every strip takes part (no per-strip test in the issue path)
            auto issue_tap = [&](auto all) {
              constexpr bool ALL = decltype(all)::value;
              if (SPARSE) {
#pragma unroll
                for (int j = 0; j < NT; ++j)
                  if (ALL || (strips & (1u << j)))
                    ptx::tc_cp_128x128b_pair(e_col + 4u * j, ((uint64_t)e_hi << 32) | (e_lo + (uint32_t)(8 * j)));
              }
#pragma unroll
              for (int j = 0; j < NT; ++j) {
                if (!ALL && !(strips & (1u << j))) continue;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                  // strip j: 8 pixels = 1024 bytes to the right; MMA q: 32 bytes along the row
                  const uint64_t a_q = ((uint64_t)a_hi << 32) | (a_lo + (uint32_t)(j * 64 + q * 2));
                  const uint64_t b_q = ((uint64_t)b_hi << 32) | (b_lo + (uint32_t)q * kBStep);
                  if (SPARSE)
                    ptx::mma_sp_f16_ss_pair(d_tmem + (uint32_t)(j * BN), a_q, b_q, e_col + (uint32_t)(4 * j + (q & 2)),
                                            idesc | (uint32_t)(q & 1), q == 0 ? accumulate : 1u);
                  else
                    ptx::mma_f16_ss_pair(d_tmem + (uint32_t)(j * BN), a_q, b_q, idesc, q == 0 ? accumulate : 1u);
                }
              }
            };
            if (leader) {
              if (all_strips) issue_tap(std::true_type{});
              else issue_tap(std::false_type{});
              ptx::tc_commit_pair(&w_empty[wst], 3);
            }
            accumulate = 1u;
            // next tap: one pixel to the left, or the end of the filter row above
            if (--s == 0) { s = p.sb; a_lo -= a_rowstep16; --dr; e_lo = e_stage + meta_row16(dr) + (uint32_t)(p.sb - 1); }
            else { a_lo -= 8u; e_lo -= 1u; }
            if (++wst == WS) { wst = 0; wph ^= 1u; b_lo = b_lo0; mcol = 0; }
            else { b_lo += w_stage16; mcol += kSlotCols; }
          }
          if (alive && leader) ptx::tc_commit_pair(&a_empty[ast], 3);
          if (++ast == p.a_stages) { ast = 0; aph ^= 1u; }
        }
        if (alive && leader) ptx::tc_commit_pair(&acc_full[acc], 3);
        if (++acc == 2) { acc = 0; cph ^= 1u; }
      }
    }
  } else if (!FUSED && warp < 6) {
    // ------------------------------------------------- metadata rearranger (two-pass)
    // Once per A box the four warps turn the row-major metadata box TMA delivered into the two masters
    // (one 16-byte line per lane and pass: two 16-byte loads, four prmt, one 16-byte store), then arrive
    // on meta_ready. Every warp waits for every box in turn (a parity wait must see each phase).
    if (SPARSE) {
      const int mw = warp - 2;
      const int lines0 = p.pairs0 * 2 * p.pitch, lines = (p.pairs0 + p.pairs1) * 2 * p.pitch;
      const int a_uses = my_tiles * p.k_uses;
      constexpr int kBatch = 3;  // lines per lane whose loads are issued before any store
      for (int ause = 0; ause < a_uses; ++ause) {
        const int ast = ause & (p.a_stages - 1);
        if (!ptx::mbar_wait(&meta_full[ast], (uint32_t)(ause >> p.a_shift) & 1u, err, 0x500u + ast)) break;
        const uint8_t* raw = sEraw + ast * p.eraw_bytes;
        uint8_t* master = sMeta + ast * p.meta_bytes;
        for (int first = mw * 32 + lane; first < lines; first += 128 * kBatch) {
          uint4 lo[kBatch], hi[kBatch];
          uint32_t sel[kBatch];
#pragma unroll
          for (int k = 0; k < kBatch; ++k) {
            const int L = first + 128 * k;
            if (L < lines) {
              const int pi = L >= lines0 ? 1 : 0;
              const int l = L - pi * lines0;
              const int m2e = (int)(((uint32_t)l * p.pitch_magic) >> 20), x = l - m2e * p.pitch;  // 2m + e, pixel column
              const int row_a = (pi + (m2e & ~1)) * p.pitch + x;  // box pixel (pi + 2m, x); its partner is one box row down
              lo[k] = *(const uint4*)(raw + row_a * 16);
              hi[k] = *(const uint4*)(raw + (row_a + p.pitch) * 16);
              sel[k] = (m2e & 1) ? 0x7632u : 0x5410u;
            }
          }
#pragma unroll
          for (int k = 0; k < kBatch; ++k) {
            const int L = first + 128 * k;
            if (L < lines)
              *(uint4*)(master + L * 16) =
                  make_uint4(well_formed(prmt(lo[k].x, hi[k].x, sel[k])), well_formed(prmt(lo[k].y, hi[k].y, sel[k])),
                             well_formed(prmt(lo[k].z, hi[k].z, sel[k])), well_formed(prmt(lo[k].w, hi[k].w, sel[k])));
          }
        }
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive_cluster(&meta_ready[ast], 0);
      }
    }
  } else if (FUSED && (((warp & 3) != 1 && (warp < 4 || warp >= 8)) || warp == 9 || warp == 13 || warp == 17 || warp == 21)) {
    // ------------------------------------------------------------ pruner
    // Work unit = 8 pixel rows of a box = one pass of a warp: lane = (row, c), and the thread owns vectors
    // c, c + 4, c + 8 and c + 12 (8 channels each) of the row's 16, so that every load instruction of the
    // warp reads 64 contiguous bytes per pixel. Units are numbered through all boxes of this CTA and dealt
    // round-robin to the pruning warps. A thread reads its 64 bytes of dense dL/dO straight from global
    // memory into registers (the loads of the next unit go out as soon as this one is pruned, and the lines
    // of the next box are asked into L2 a box ahead), prunes them and writes the compressed vectors and their
    // metadata into the A stage. These stores replace the TMA write of the compressed box, so the fused mode adds no
    // shared-memory traffic to the two-pass kernel's - which matters because with 64 or 128 input
    // channels the MMAs themselves are bound by shared-memory reads.
    {
      // number of this pruning warp, 0 .. kPruneWarps - 1: warps 2, 3, 8, then 10.. without those on scheduler 1 (0..13),
      // then the four on scheduler 1
      const int pw = warp == 9 ? 14 : warp == 13 ? 15 : warp == 17 ? 16 : warp == 21 ? 17 : warp < 4 ? warp - 2 : warp == 8 ? 2 : 3 + (warp - 10) - ((warp - 9) >> 2);
      const int upb = p.units_per_box;
      if (p.static_pad) {
        // every stage starts out as padding: zero values, metadata naming the position pair (0, 1)
        const int words = p.a_stages * p.a_bytes >> 4;
        for (int k = pw * 32 + lane; k < words; k += 32 * kPruneWarps) ((uint4*)sA)[k] = make_uint4(0u, 0u, 0u, 0u);
        const int mwords = p.a_stages * p.meta_bytes >> 4;
        for (int k = pw * 32 + lane; k < mwords; k += 32 * kPruneWarps)
          ((uint4*)sMeta)[k] = make_uint4(0x44444444u, 0x44444444u, 0x44444444u, 0x44444444u);
        ptx::fence_proxy_async_smem();
        ptx::named_bar_sync(3, 32 * kPruneWarps);  // no unit is announced before every stage is cleared
      }
      const int a_uses = my_tiles * p.k_uses;
      const int row8 = lane >> 2, c = lane & 3;
      const uint32_t px_bytes = (uint32_t)p.Cout * 2u;
      const int tb_shift = p.tb == 4 ? 2 : p.tb >> 1;  // tb is 1, 2 or 4
      auto prune_units = [&](auto m_tag, auto n_tag, auto scheme_tag) {
        constexpr int M = decltype(m_tag)::value;
        constexpr int N = decltype(n_tag)::value;
        constexpr int SCHEME = decltype(scheme_tag)::value;
        // ---- load cursor: the unit whose loads go out next, and the box it lies in
        int ia = 0, o = pw, lt = 0, ku = 0;  // ku: box of the tile set (channel block ku / ss, filter column ku % ss)
        auto normalise = [&]() { while (o >= upb) { o -= upb; ++ia; if (++ku == p.k_uses) { ku = 0; ++lt; } } };
        normalise();
        int org_box = -1;             // box the origin below belongs to
        const uint8_t* org_ptr = p.a_dense;  // address of box pixel (0, 0), channel block kb, quarter c (may lie outside the tensor)
        int org_p = 0, org_q = 0;     // dO pixel of box pixel (0, 0)
        int org_b = 0;                // its image
        int64_t org_pix = 0;          // its linear pixel number (random keys)
        bool org_ok = false;
        int org_kb0 = 0;              // first channel block of its tile's window
        auto set_origin = [&](int box_lt, int box_ku, const uint8_t*& ptr, int& p0, int& q0, int& b0, int64_t& pix, bool& ok, int& kb0) {
          int n0, w0, h0;
          ok = locate(first_pair + box_lt * pair_stride, n0, w0, h0, b0);
          const int box_kl = box_ku / p.ss, si = box_ku - box_kl * p.ss;
          kb0 = first_k_block(p, n0, 128);
          const int box_kb = kb0 + box_kl;
          q0 = w0 + p.pad_w - (p.sb - 1) - si;
          p0 = h0 + p.pad_h - (p.R - 1);
          pix = ((int64_t)b0 * p.P + p0) * p.Q + q0;
          ptr = p.a_dense + pix * (int64_t)px_bytes + box_kb * 256 + c * 16;
        };
        // box pixel (box row br, column col) -> image offset, pixel row and pixel column relative to the origin
        auto box_pixel = [&](int br, int col, int& ib, int& ih, int& iw) {
          ih = br >> tb_shift;
          ib = (br & (p.tb - 1)) * p.img_per_row;
          iw = col;
          if (p.split) { ib += col >> 2; iw = col & 3; }
        };
        // The unit whose loads are in flight: its 64 bytes, its pixel row in the box, its box
        uint4 w[4];
        int u_i = 0, u_ia = 0, u_kb = 0;  // (u_kb: channel block)
        int64_t u_pix = 0;
        bool u_live = false;  // some pixel of the unit lies inside the tensor (halo rows above / below an image: none does)
        auto fetch = [&]() {
          if (org_box != ia) {
            set_origin(lt, ku, org_ptr, org_p, org_q, org_b, org_pix, org_ok, org_kb0);
            org_box = ia;
            // ask the lines of the NEXT box into L2 now, a whole box ahead of their loads: 2 lines of 128
            // bytes per box pixel, dealt to the pruning threads
            int nlt = lt, nkb = ku + 1;
            if (nkb == p.k_uses) { nkb = 0; ++nlt; }
            if (ia + 1 < a_uses) {
              const uint8_t* nptr;
              int np0, nq0, nb0, nkb0;
              int64_t npix;
              bool nok;
              set_origin(nlt, nkb, nptr, np0, nq0, nb0, npix, nok, nkb0);
              for (int line = pw * 32 + lane; line < 2 * p.img_rows; line += 32 * kPruneWarps) {
                const int px = line >> 1;
                const int br = (int)(((uint32_t)px * p.pitch_magic) >> 20);  // box row
                int ib, ih, iw;
                box_pixel(br, px - br * p.pitch, ib, ih, iw);
                if (nok && nb0 + ib < p.B && (unsigned)(np0 + ih) < (unsigned)p.P && (unsigned)(nq0 + iw) < (unsigned)p.Q)
                  asm volatile("prefetch.global.L2 [%0];" ::"l"(nptr - c * 16 + (uint32_t)((ib * p.P + ih) * p.Q + iw) * px_bytes + (line & 1) * 128));
              }
            }
          }
          if (p.static_pad) {
            const int ur = NT == 2 ? (o >> 1) : o, uc = NT == 2 ? (o & 1) : 0;
            u_i = (p.unit_row0 + ur) * p.pitch + p.unit_col0 + 8 * uc + row8;
          } else {
            u_i = 8 * o + row8;
          }
          u_ia = ia;
          const int kb = org_kb0 + ku / p.ss;
          u_kb = kb;
          const int br = (int)(((uint32_t)u_i * p.pitch_magic) >> 20);  // box row
          int ib, ih, iw;
          box_pixel(br, u_i - br * p.pitch, ib, ih, iw);
          const uint32_t off = (uint32_t)((ib * p.P + ih) * p.Q + iw);
          u_pix = org_pix + off;
          const bool valid = org_ok && u_i < p.img_rows && org_b + ib < p.B && (unsigned)(org_p + ih) < (unsigned)p.P &&
                             (unsigned)(org_q + iw) < (unsigned)p.Q;
          u_live = __any_sync(0xFFFFFFFFu, valid);
#pragma unroll
          for (int v = 0; v < 4; ++v) w[v] = make_uint4(0u, 0u, 0u, 0u);
          if (valid) {
            const uint8_t* src = org_ptr + off * px_bytes;
            // vector c + 4v: channels beyond Cout (a last channel block that is half empty) read as zero
            const int chan0 = kb * 128 + c * 8;
#pragma unroll
            for (int v = 0; v < 4; ++v)
              if (chan0 + 32 * v < p.Cout) w[v] = ldg_stream(src + 64 * v);
          }
          o += kPruneWarps;
          normalise();
        };
        int boxes_seen = 0;  // stage hand-backs (a_empty phases) this warp has observed, one per box, in order
        int pending_ast = -1;  // stage of the unit whose stores are out but not yet announced
        // Makes the stores of the previous unit visible to the tensor core and announces them. Called a whole
        // unit later than the stores were issued, so the fence finds them done.
        auto announce = [&]() {
          if (pending_ast >= 0) {
            ptx::fence_proxy_async_smem();  // the tensor core reads A and the masters through the async proxy
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(&a_full[pending_ast], 0);
          }
        };
        bool more = ia < a_uses;  // a unit is in flight
        if (more) fetch();
        while (more) {
          const int i = u_i, cia = u_ia;
          const bool live = u_live;
          const int ast = cia & (p.a_stages - 1);
          uint2 out[4];
          uint32_t metaw;
          // (a group of M channels = vectors c + 4v of M / 8 neighbouring lanes c, same v)
          if (live) {
            fused_prune_vectors<M, N, SCHEME>(w, u_pix * (p.Cout >> 3) + u_kb * 16 + c, 4, p.seed_lo, p.seed_hi, c & (M / 8 - 1), out, metaw);
          } else {
            // a unit of padding only: zeros, whatever positions the metadata names (it names the pair (0, 1))
#pragma unroll
            for (int v = 0; v < 4; ++v) out[v] = make_uint2(0u, 0u);
            metaw = 0x44444444u;
          }
          // the registers of this unit are free: the loads of the next one go out before this one's stores
          more = ia < a_uses;
          if (more) fetch();
          // only now, with the unit pruned and the next one's loads in flight, does the warp need the stage
          if (boxes_seen <= cia) {  // the MMAs that read this stage's previous contents (box cia - 2) have completed
            // (whatever this warp still owes an earlier box goes out first: with fewer units per box than pruning warps
            // the stage waited for here can be the very one that unit belongs to)
            announce();
            pending_ast = -1;
            bool ok = true;
            while (boxes_seen <= cia) {
              const int bs = boxes_seen & (p.a_stages - 1);
              if (!ptx::mbar_wait<kIdleWaitNs>(&a_empty[bs], (((uint32_t)boxes_seen >> p.a_shift) & 1u) ^ 1u, err, 0x900u + bs)) { ok = false; break; }
              ++boxes_seen;
            }
            if (!__all_sync(0xFFFFFFFFu, ok)) break;
          }
          announce();
          const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, metaw, 1);  // (all lanes: before the rows part ways)
          if (i < p.img_rows) {
            const int sw = i & 7;
            // vector j = c + 4v -> 8 bytes at 16-byte chunk j / 2 = 2v + c / 2 (swizzled), half j % 2 = c % 2
            uint8_t* a_row = sA + ast * p.a_bytes + i * 128 + 8 * (c & 1);
            const int ch0 = (c >> 1) ^ sw;
#pragma unroll
            for (int v = 0; v < 4; ++v) *(uint2*)(a_row + ((ch0 ^ (2 * v)) << 4)) = out[v];
            // Metadata: byte v of metaw belongs to the 16-channel group 2v + c / 2, i.e. to 32-bit word v of the
            // master line e = c / 2, byte c % 2 of its low or high half-word. Lanes c and c ^ 1 hold the two bytes
            // of each half-word: they trade words, the even lane writes the half-words of v = 0, 1, the odd one
            // those of v = 2, 3.
            const uint32_t lo = (c & 1) ? other : metaw, hi = (c & 1) ? metaw : other;  // bytes of c even / c odd
            const uint32_t pair = (c & 1) ? prmt(lo, hi, 0x7362) : prmt(lo, hi, 0x5140);  // two half-words
            const int ih = (int)(((uint32_t)i * p.pitch_magic) >> 20), iw = i - ih * p.pitch;  // ih: box row
            uint8_t* master = sMeta + ast * p.meta_bytes + (iw << 4) + 8 * (c & 1) + (c >> 1) * (p.pitch << 4);
            if (ih < 2 * p.pairs0) {
              uint8_t* dst = master + (((ih & ~1) * p.pitch) << 4) + 2 * (ih & 1);
              *(uint16_t*)dst = (uint16_t)pair;
              *(uint16_t*)(dst + 4) = (uint16_t)(pair >> 16);
            }
            if (ih >= 1 && ih <= 2 * p.pairs1) {
              uint8_t* dst = master + p.m0_bytes + ((((ih - 1) & ~1) * p.pitch) << 4) + 2 * ((ih - 1) & 1);
              *(uint16_t*)dst = (uint16_t)pair;
              *(uint16_t*)(dst + 4) = (uint16_t)(pair >> 16);
            }
          }
          pending_ast = ast;
        }
        announce();
      };
      using std::integral_constant;
      auto with_m = [&](auto m_tag) {
        if (p.fused_scheme == SDGP_MAGNITUDE) {
          if (p.fused_n == 1) prune_units(m_tag, integral_constant<int, 1>{}, integral_constant<int, SDGP_MAGNITUDE>{});
          else prune_units(m_tag, integral_constant<int, 2>{}, integral_constant<int, SDGP_MAGNITUDE>{});
        } else if (p.fused_scheme == SDGP_RANDOM) {
          if (p.fused_n == 1) prune_units(m_tag, integral_constant<int, 1>{}, integral_constant<int, SDGP_RANDOM>{});
          else prune_units(m_tag, integral_constant<int, 2>{}, integral_constant<int, SDGP_RANDOM>{});
        } else {
          if (p.fused_n == 1) prune_units(m_tag, integral_constant<int, 1>{}, integral_constant<int, SDGP_RESCALED_MAGNITUDE>{});
          else prune_units(m_tag, integral_constant<int, 2>{}, integral_constant<int, SDGP_RESCALED_MAGNITUDE>{});
        }
      };
      if (p.fused_m == 4) with_m(integral_constant<int, 4>{});
      else if (p.fused_m == 8) with_m(integral_constant<int, 8>{});
      else if (p.fused_m == 16) with_m(integral_constant<int, 16>{});
      else with_m(integral_constant<int, 32>{});
    }
  } else if (warp >= kEpilogueWarp0 && warp < kEpilogueWarp0 + 4) {
    // ------------------------------------------------------------ epilogue
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const bool issuer = (threadIdx.x == kEpilogueWarp0 * 32);
    uint32_t chunk = 0, cph = 0;
    int acc = 0;
    for (int lt = 0; lt < my_tiles; ++lt) {
      int n0, w0, h0, b0;
      const bool in_range = locate(first_pair + lt * pair_stride, n0, w0, h0, b0);
      const uint32_t strips = strip_mask(lt);
      if (!ptx::mbar_wait<kIdleWaitNs>(&acc_full[acc], cph, err, 0x600u + acc)) break;
      ptx::tc_fence_after_sync();
#pragma unroll
      for (int j = 0; j < NT; ++j)
        if (p.split)  // coordinates of strip j: pixel column, image within the box row, image group, pixel row
          store_accumulator<BN, true>(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * set_cols + j * BN), sOut, p.out_bufs,
                                      &tmD, n0, 0, 2 * j, b0 / p.img_per_row, in_range && (strips & (1u << j)), row, issuer, chunk,
                                      (p.meta_shared && j == 0) ? &meta_free[acc] : nullptr, p.f16 != 0, h0);
        else          // pixel column, image, pixel row
          store_accumulator<BN>(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * set_cols + j * BN), sOut, p.out_bufs, &tmD,
                                n0, w0 + 8 * j, b0, h0, in_range && (w0 + 8 * j < p.W) && (strips & (1u << j)), row, issuer, chunk,
                                (p.meta_shared && j == 0) ? &meta_free[acc] : nullptr, p.f16 != 0);
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive_cluster(&acc_empty[acc], 0);
      if (++acc == 2) { acc = 0; cph ^= 1u; }
    }
    // the staging slabs have been read; the writes themselves complete with the grid (whoever depends on dD waits for that)
    if (issuer) ptx::bulk_wait_group_read<0>();
  }

  __syncwarp();
  if (*(volatile unsigned int*)err != 0u) {
    const uint64_t t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 200000ull) {
    }
  }
  ptx::tc_fence_before_sync();
  __syncwarp();
  ptx::cluster_sync();
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

// A tensor map is a pure function of these arguments (it holds the address, not the memory), and a training
// loop asks for the same few maps every step: each host thread keeps the last kMapCache it encoded. Outside a CUDA
// graph the four encodes of a launch otherwise cost about as much as a small layer's kernel.
struct MapKey {
  const void* base;
  uint64_t dims[5], strides[4];
  uint32_t box[5];
  int dt, rank, swz;
};
constexpr int kMapCache = 64;

bool encode(CUtensorMap* tm, CUtensorMapDataType dt, int rank, const void* base, const uint64_t* dims,
            const uint64_t* strides_bytes, const uint32_t* box, CUtensorMapSwizzle swz) {
  static thread_local MapKey keys[kMapCache];
  static thread_local CUtensorMap maps[kMapCache];
  static thread_local int used = 0, next = 0;
  MapKey key;
  memset(&key, 0, sizeof(key));
  key.base = base; key.dt = (int)dt; key.rank = rank; key.swz = (int)swz;
  for (int i = 0; i < rank; ++i) { key.dims[i] = dims[i]; key.box[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) key.strides[i] = strides_bytes[i];
  for (int i = 0; i < used; ++i)
    if (memcmp(&keys[i], &key, sizeof(key)) == 0) {
      *tm = maps[i];
      return true;
    }
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint32_t ones[5] = {1, 1, 1, 1, 1};
  if (fn(tm, dt, (cuuint32_t)rank, const_cast<void*>(base), (const cuuint64_t*)dims, (const cuuint64_t*)strides_bytes,
         (const cuuint32_t*)box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  const int slot = used < kMapCache ? used++ : (next = (next + 1) % kMapCache);
  keys[slot] = key;
  maps[slot] = *tm;
  return true;
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

// Per-device caches, indexed by the ordinal of the CURRENT device (the library follows the caller's
// current device, and a process may drive several). Filled on first use; concurrent first uses store the
// same values.
constexpr int kMaxDevices = 64;

int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
  return dev;
}

int sm_count() {
  static int n[kMaxDevices] = {};
  const int dev = current_device();
  if (dev < 0) return 148;
  if (!n[dev]) {
    int v = 0;
    cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
    n[dev] = v > 0 ? v : 148;
  }
  return n[dev];
}

// Opts `kernel` in to the large dynamic shared-memory carve, once per device and instantiation.
template <typename K>
bool configure_once(K kernel, bool (&done)[kMaxDevices]) {
  const int dev = current_device();
  if (dev < 0) return false;
  if (!done[dev]) {
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) != cudaSuccess) return false;
    done[dev] = true;
  }
  return true;
}

int round_up(int x, int a) { return (x + a - 1) / a * a; }

// Shared-memory plan for one launch: decides filter-row reuse, resident W, pipeline depth,
// accumulator count and the carve. Returns false if no variant fits.
template <bool SPARSE, int BN, bool FUSED>
bool plan(DgradParams* p) {
  using C = Cfg<SPARSE, BN>;
  const int taps = p->R * p->S;
  const int budget = kSmemLimit - kSmemSlack;
  // Filter-row reuse needs a single-image patch whose rows are whole groups of 8 pixels, so
  // that every vertical tap is an offset of whole 1024-byte swizzle periods.
  const bool can_reuse = p->R > 1 && p->TB == 1 && p->TW % 8 == 0 && p->TW * (p->TH + p->R - 1) <= kMaxImgRows;
  const bool can_reside = p->tiles_n == 1 && p->diag_cin_g == 0 && p->pair_tiles > sm_count() / 2;  // pays only if tiles repeat
  for (int attempt = 0; attempt < 4; ++attempt) {
    // attempt 0: reuse with streamed W (measured best where it fits: more stages in flight),
    // 1: reuse + resident W, 2: resident W, 3: neither
    const bool reuse = attempt < 2;
    const bool resident = (attempt == 1 || attempt == 2);
    if ((reuse && !can_reuse) || (resident && !can_reside)) continue;
    p->rr = reuse ? p->R : 1;
    p->img_rows = p->TW * (p->TH + p->rr - 1) * p->TB;
    p->w_resident = resident ? 1 : 0;
    p->a_bytes = round_up(p->img_rows * 128, 1024);
    p->b_bytes = resident ? 0 : p->rr * C::kTapBBytes;
    p->eraw_bytes = SPARSE ? round_up(p->img_rows * 16, 128) : 0;
    p->ehw_bytes = SPARSE ? p->rr * kEHwBytes : 0;
    const int w_bytes = resident ? taps * p->k_blocks * C::kTapBBytes : 0;
    const int raw_bytes = FUSED ? 2 * p->a_bytes : 0;
    const int stage_bytes = p->a_bytes + p->b_bytes + p->eraw_bytes + p->ehw_bytes + raw_bytes;
    int out_bufs = 2;
    int stages = (budget - w_bytes - out_bufs * kOutBytes) / stage_bytes;
    if (stages < 4) {
      out_bufs = 1;
      stages = (budget - w_bytes - out_bufs * kOutBytes) / stage_bytes;
    }
    if (stages > kMaxStages) stages = kMaxStages;
    // TMEM: accumulators first, metadata slots (4 columns per tap and stage) behind them
    const int meta_cols_per_stage = SPARSE ? 4 * p->rr : 0;
    const int meta_div = SPARSE ? meta_cols_per_stage : 1;  // divisor that is never zero
    int nacc = (2 * BN + 2 * meta_cols_per_stage <= (int)kTmemCols) ? 2 : 1;
    p->meta_shared = 0;
    if (meta_cols_per_stage > 0 && nacc == 1 && 2 * BN <= (int)kTmemCols) {
      // Two accumulators fill TMEM: the metadata slots share the first 64 columns of whichever
      // accumulator is being read out, released early by the epilogue.
      nacc = 2;
      p->meta_shared = 1;
      if (stages > 64 / meta_div) stages = 64 / meta_div;
    } else if (meta_cols_per_stage > 0) {
      const int max_meta_stages = ((int)kTmemCols - nacc * BN) / meta_div;
      if (stages > max_meta_stages) stages = max_meta_stages;
    }
    if (stages < ((resident || reuse || FUSED) ? 2 : 3)) continue;  // a reuse stage is R taps long
    p->stages = stages;
    p->nacc = nacc;
    p->meta_col = p->meta_shared ? 0 : nacc * BN;
    p->out_bufs = out_bufs;
    p->off_b = stages * p->a_bytes;
    p->off_eraw = p->off_b + stages * p->b_bytes;
    p->off_ehw = round_up(p->off_eraw + stages * p->eraw_bytes, 1024);
    p->off_w = round_up(p->off_ehw + stages * p->ehw_bytes, 1024);
    p->off_out = round_up(p->off_w + w_bytes, 1024);
    p->off_raw = p->off_out + out_bufs * kOutBytes;
    p->off_bar = p->off_raw + stages * raw_bytes;
    p->smem_bytes = p->off_bar + 512 + 1024;
    if (p->smem_bytes > kSmemLimit) continue;
    return true;
  }
  return false;
}

// Where one launch reads and writes: dO as stored (P x Q pixels of `a_channels` channels per image,
// a multiple of the channel block; W holds only the first `Cout` of them), the full filter
// width in W columns, and the (possibly strided) view of dD the launch fills.
struct DgradView {
  int P, Q, batch;
  int a_channels;
  int d_channels;                 // channels per pixel of dD as stored (<= Cin: a store is clipped there)
  int64_t w_cols;                 // R_full * S_full * Cin
  void* d_base;
  uint64_t d_stride_w, d_stride_h, d_stride_b;  // bytes
};

template <bool SPARSE, int BN, bool FUSED = false>
sdgp_status launch_cfg(const void* A, const void* meta, const void* Wt, const DgradView& view, DgradParams p,
                       cudaStream_t stream) {
  const int P = view.P, Q = view.Q;
  using C = Cfg<SPARSE, BN>;
  if (!plan<SPARSE, BN, FUSED>(&p)) return SDGP_ERR_UNSUPPORTED;

  CUtensorMap tmA, tmE, tmB, tmD;
  const uint32_t img_h = (uint32_t)(p.TH + p.rr - 1);
  const uint64_t CA = (SPARSE && !FUSED) ? (uint64_t)view.a_channels / 2 : (uint64_t)view.a_channels;  // stored elements per pixel
  {
    const uint64_t dims[4] = {CA, (uint64_t)Q, (uint64_t)P, (uint64_t)view.batch};
    const uint64_t strides[3] = {CA * 2, CA * 2 * Q, CA * 2 * Q * P};
    const uint32_t box[4] = {64, (uint32_t)p.TW, img_h, (uint32_t)p.TB};
    if (!encode(&tmA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, A, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B))
      return SDGP_ERR_CUDA;
  }
  if (SPARSE && !FUSED) {
    const uint64_t CE = (uint64_t)view.a_channels / 16;
    const uint64_t dims[4] = {CE, (uint64_t)Q, (uint64_t)P, (uint64_t)view.batch};
    const uint64_t strides[3] = {CE * 2, CE * 2 * Q, CE * 2 * Q * P};
    const uint32_t box[4] = {8, (uint32_t)p.TW, img_h, (uint32_t)p.TB};
    if (!encode(&tmE, CU_TENSOR_MAP_DATA_TYPE_UINT16, 4, meta, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE))
      return SDGP_ERR_CUDA;
  } else {
    tmE = tmA;
  }
  {
    const uint64_t dims[2] = {(uint64_t)view.w_cols, (uint64_t)p.Cout};
    const uint64_t strides[1] = {(uint64_t)view.w_cols * 2};
    const uint32_t box[2] = {(uint32_t)C::kBoxCols, (uint32_t)C::kKB};
    if (!encode(&tmB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Wt, dims, strides, box,
                C::kRowB == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B))
      return SDGP_ERR_CUDA;
  }
  {
    const uint64_t dims[4] = {(uint64_t)view.d_channels, (uint64_t)p.W, (uint64_t)p.H, (uint64_t)p.B};
    const uint64_t strides[3] = {view.d_stride_w, view.d_stride_h, view.d_stride_b};
    const uint32_t box[4] = {64, (uint32_t)p.TW, (uint32_t)p.TH, (uint32_t)p.TB};
    if (!encode(&tmD, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, view.d_base, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B))
      return SDGP_ERR_CUDA;
  }

  static bool configured[kMaxDevices] = {};
  auto kernel = dgrad_kernel<SPARSE, BN, FUSED>;
  if (!configure_once(kernel, configured)) return SDGP_ERR_CUDA;
  const int max_pairs = sm_count() / 2;
  const int pairs = p.pair_tiles < max_pairs ? p.pair_tiles : max_pairs;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * pairs));
  cfg.blockDim = dim3(FUSED ? kThreadsGemmFused : kThreadsGemm);
  cfg.dynamicSmemBytes = (size_t)p.smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // may be scheduled while the previous kernel of the stream drains (the kernel waits for it
  // after its set-up)
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kernel, tmA, tmE, tmB, tmD, p) == cudaSuccess ? SDGP_OK : SDGP_ERR_CUDA;
}

// Shared-memory and TMEM plan of the whole-filter-reuse kernel. Returns false if it does not fit.
template <bool SPARSE, int BN, bool FUSED>
bool plan_halo(HaloParams* p, int nt) {
  using C = Cfg<SPARSE, BN>;
  const int budget = kSmemLimit - kSmemSlack;
  {
    if (nt * BN > 256) return false;         // two tile sets of accumulators must fit the 512 TMEM columns
    p->split = (p->W == 4) ? 1 : 0;  // images 4 pixels wide: two per strip row, horizontal taps by separate boxes
    if (!p->split && nt == 2 && p->W <= 8) return false;  // a second strip would be empty
    p->nt = nt;
    p->img_per_row = p->split ? 2 * nt : 1;
    if (p->B % p->img_per_row != 0) return false;  // a box row of images must not reach past the batch
    p->ss = p->split ? p->S : 1;
    p->sb = p->split ? 1 : p->S;
    p->k_uses = p->k_blocks * p->ss;
    p->pitch = 8 * nt + p->sb - 1;
    p->th = p->H <= 4 ? 4 : p->H <= 8 ? 8 : kHaloRows;
    p->tb = kHaloRows / p->th;
    p->img_h = (p->th + p->R - 1) * p->tb;
    p->img_rows = p->pitch * p->img_h;
    p->static_pad = 0;
    p->units_per_box = (p->img_rows + 7) / 8;
    if (p->pitch > 256 || p->img_h > 256) return false;
    p->a_bytes = round_up(p->img_rows * 128, 1024);
    p->eraw_bytes = (SPARSE && !FUSED) ? round_up(p->img_rows * 16, 128) : 0;
    p->w_bytes = C::kTapBBytes;
    // vertical tap offset dr = 0 .. R-1 starts tb * dr box rows down: master (tb * dr) % 2, pair (tb * dr) / 2
    p->pairs0 = 8 + (p->tb == 1 ? (p->R - 1) >> 1 : (p->tb >> 1) * (p->R - 1));
    p->pairs1 = (p->tb == 1 && p->R > 1) ? 8 + ((p->R - 2) >> 1) : 0;
    p->m0_bytes = SPARSE ? p->pairs0 * 2 * p->pitch * 16 : 0;
    p->meta_bytes = SPARSE ? round_up((p->pairs0 + p->pairs1) * 2 * p->pitch * 16, 128) : 0;
    // A ring: two stages; four where a box feeds few taps (column-split mode: R taps per box), so that the loads
    // run further ahead of the MMAs, if that still leaves three W stages
    p->a_stages = 2;
    const int per_a = p->a_bytes + p->eraw_bytes + p->meta_bytes;
    if (p->split && (budget - 4 * per_a - 1024 - kOutBytes) / p->w_bytes >= 3) p->a_stages = 4;
    p->a_shift = p->a_stages == 4 ? 2 : 1;
    const int fixed = p->a_stages * per_a + 1024;
    int out_bufs = 2;
    int w_stages = (budget - fixed - out_bufs * kOutBytes) / p->w_bytes;
    if (w_stages < 4) {
      out_bufs = 1;
      w_stages = (budget - fixed - out_bufs * kOutBytes) / p->w_bytes;
    }
    if (w_stages > kMaxStages) w_stages = kMaxStages;
    p->meta_shared = 0;
    p->meta_col = 2 * nt * BN;
    if (SPARSE) {
      const int slot_cols = 4 * nt;  // TMEM columns of one W stage's metadata
      const int free_cols = (int)kTmemCols - 2 * nt * BN;
      if (free_cols >= 3 * slot_cols) {
        if (w_stages > free_cols / slot_cols) w_stages = free_cols / slot_cols;
      } else {
        p->meta_shared = 1;  // slots live in the first 64 columns of the tile set being read out
        p->meta_col = 0;
        if (w_stages > 64 / slot_cols) w_stages = 64 / slot_cols;
      }
    }
    if (w_stages < 3) return false;
    p->w_stages = w_stages;
    p->out_bufs = out_bufs;
    p->off_eraw = p->a_stages * p->a_bytes;
    p->off_meta = p->off_eraw + p->a_stages * p->eraw_bytes;
    p->off_w = round_up(p->off_meta + p->a_stages * p->meta_bytes, 1024);
    p->pitch_magic = ((1u << 20) + (uint32_t)p->pitch - 1u) / (uint32_t)p->pitch;
    p->off_out = round_up(p->off_w + w_stages * p->w_bytes, 1024);
    p->off_bar = p->off_out + out_bufs * kOutBytes;
    p->smem_bytes = p->off_bar + 512 + 1024;
    if (p->smem_bytes > kSmemLimit) return false;
    p->sets_w = p->split ? 1 : (p->W + 8 * nt - 1) / (8 * nt);
    p->tiles_h = (p->H + p->th - 1) / p->th;
    if (FUSED && p->sets_w == 1 && p->tiles_h == 1 && p->a_bytes % 16 == 0 && p->meta_bytes % 16 == 0) {
      // Box pixel row 0 is dL/dO row p0 and box column 0 is dL/dO column q0 (every tile set starts at h0 = w0 = 0); the
      // rows and columns of the box that lie inside dL/dO's P x Q pixels are the same for every box.
      const int p0 = p->pad_h - (p->R - 1), q0 = p->pad_w - (p->sb - 1);
      const int row_lo = p0 < 0 ? -p0 : 0;
      const int row_hi = (p->th + p->R - 1) < (p->P - p0) ? (p->th + p->R - 1) : (p->P - p0);
      const int col_lo = p->split ? 0 : (q0 < 0 ? -q0 : 0);
      const bool cols_fit = p->split ? p->Q <= 4 : (p->Q - q0 <= col_lo + 8 * nt);
      if (row_hi > row_lo && cols_fit) {
        p->static_pad = 1;
        p->unit_row0 = row_lo * p->tb;
        p->unit_col0 = col_lo;
        p->units_per_box = (row_hi - row_lo) * p->tb * nt;
      }
    }
    const int tile_imgs = p->tb * p->img_per_row;  // images of one tile set
    const int64_t m_sets = (int64_t)p->sets_w * p->tiles_h * ((p->B + tile_imgs - 1) / tile_imgs);
    if (m_sets * p->tiles_n > 0x3FFFFFFF) return false;
    p->m_sets = (int)m_sets;
    p->pair_tiles = (int)((m_sets + 1) / 2) * p->tiles_n;
    p->mg_tiles_n = div_magic((uint32_t)p->tiles_n);
    p->mg_sets_w = div_magic((uint32_t)p->sets_w);
    p->mg_tiles_h = div_magic((uint32_t)p->tiles_h);
    // The pair tiles of a last round that fills at most half the CTA pairs are dealt out strip by
    // strip: that round then costs about half.
    p->units = p->pair_tiles;
    p->split_from = p->pair_tiles;
    const int max_pairs = sm_count() / 2;
    const int rem = p->pair_tiles % max_pairs;
    if (nt == 2 && p->pair_tiles > max_pairs && rem > 0 && 2 * rem <= max_pairs) {
      p->split_from = p->pair_tiles - rem;
      p->units = p->pair_tiles + rem;
    }
    return true;
  }
  return false;
}

// Whole-filter reuse pays when there is more than one tap and strips of 8 x 16 pixels cover the
// image without much padding.
bool halo_applies(int H, int W, int taps) {
  if (taps < 2) return false;
  if (W == 4 && H >= 3 && H <= 4) return true;  // two images per strip row, four pixel rows of eight images per strip
  if (W < 8 || (H < 12 && H > 8) || H < 6) return false;
  const int th = H <= 8 ? 8 : kHaloRows;  // images at most 8 pixels tall: strips of 8 rows of two images
  const int64_t covered = (int64_t)((W + 7) / 8 * 8) * ((H + th - 1) / th * th);
  return covered * 100 <= (int64_t)H * W * 135;
}

template <bool SPARSE, int BN, int NT, bool FUSED>
sdgp_status launch_halo_nt(const void* A, const void* meta, const void* Wt, const DgradView& view, HaloParams p,
                           cudaStream_t stream) {
  using C = Cfg<SPARSE, BN>;
  if (!plan_halo<SPARSE, BN, FUSED>(&p, NT)) return SDGP_ERR_UNSUPPORTED;

  CUtensorMap tmA, tmE, tmB, tmD;
  const int P = view.P, Q = view.Q;
  const uint64_t CA = (SPARSE && !FUSED) ? (uint64_t)view.a_channels / 2 : (uint64_t)view.a_channels;
  // Dimensions: channel, pixel column, [column-split mode only: image within a box row (img_per_row images lie side by
  // side),] image (group), pixel row. A box then holds its rows in (pixel row, image group) order and, inside a row,
  // image after image.
  const uint64_t ipr = (uint64_t)p.img_per_row, groups = (uint64_t)view.batch / ipr;
  const uint32_t box_w = (uint32_t)(p.split ? 4 : p.pitch), box_h = (uint32_t)(p.img_h / p.tb);
  // builds the map of a [B, rows, cols, chan] tensor of 2-byte elements with the given strides and box extents
  auto encode_nhwc = [&](CUtensorMap* tm, CUtensorMapDataType dt, const void* base, uint64_t chan, uint64_t cols, uint64_t rows,
                         uint64_t images, uint64_t s_col, uint64_t s_row, uint64_t s_img, uint32_t b_chan, uint32_t b_col,
                         uint32_t b_ipr, uint32_t b_grp, uint32_t b_row, CUtensorMapSwizzle swz) -> bool {
    if (p.split) {
      const uint64_t dims[5] = {chan, cols, ipr, images / ipr, rows};
      const uint64_t strides[4] = {s_col, s_img, s_img * ipr, s_row};
      const uint32_t box[5] = {b_chan, b_col, b_ipr, b_grp, b_row};
      return encode(tm, dt, 5, base, dims, strides, box, swz);
    }
    const uint64_t dims[4] = {chan, cols, images, rows};
    const uint64_t strides[3] = {s_col, s_img, s_row};
    const uint32_t box[4] = {b_chan, b_col, b_grp, b_row};
    return encode(tm, dt, 4, base, dims, strides, box, swz);
  };
  // (fused: the pruning warps read dL/dO with plain loads and the A map goes unused)
  if (!encode_nhwc(&tmA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, A, CA, (uint64_t)Q, (uint64_t)P, (uint64_t)view.batch, CA * 2, CA * 2 * Q,
                   CA * 2 * Q * P, 64, box_w, (uint32_t)ipr, (uint32_t)p.tb, box_h, CU_TENSOR_MAP_SWIZZLE_128B))
    return SDGP_ERR_CUDA;
  tmE = tmA;
  p.a_dense = (const uint8_t*)A;
  if (SPARSE && !FUSED) {
    const uint64_t CE = (uint64_t)view.a_channels / 16;
    if (!encode_nhwc(&tmE, CU_TENSOR_MAP_DATA_TYPE_UINT16, meta, CE, (uint64_t)Q, (uint64_t)P, (uint64_t)view.batch, CE * 2, CE * 2 * Q,
                     CE * 2 * Q * P, 8, box_w, (uint32_t)ipr, (uint32_t)p.tb, box_h, CU_TENSOR_MAP_SWIZZLE_NONE))
      return SDGP_ERR_CUDA;
  }
  {
    const uint64_t dims[2] = {(uint64_t)view.w_cols, (uint64_t)p.Cout};
    const uint64_t strides[1] = {(uint64_t)view.w_cols * 2};
    const uint32_t box[2] = {(uint32_t)C::kBoxCols, (uint32_t)C::kKB};
    if (!encode(&tmB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Wt, dims, strides, box,
                C::kRowB == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B))
      return SDGP_ERR_CUDA;
  }
  // dD, one strip per store: 8 pixel columns of one image, or (column-split mode) the 4 columns of two neighbouring images
  if (!encode_nhwc(&tmD, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, view.d_base, (uint64_t)view.d_channels, (uint64_t)p.W, (uint64_t)p.H, (uint64_t)p.B,
                   view.d_stride_w, view.d_stride_h, view.d_stride_b, 64, (uint32_t)(p.split ? 4 : 8), 2, (uint32_t)p.tb,
                   (uint32_t)p.th, CU_TENSOR_MAP_SWIZZLE_128B))
    return SDGP_ERR_CUDA;

  static bool configured[kMaxDevices] = {};
  auto kernel = dgrad_halo_kernel<SPARSE, BN, NT, FUSED>;
  if (!configure_once(kernel, configured)) return SDGP_ERR_CUDA;
  const int max_pairs = sm_count() / 2;
  const int pairs = p.units < max_pairs ? p.units : max_pairs;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * pairs));
  cfg.blockDim = dim3(FUSED ? kThreadsHaloFused : kThreadsGemm);
  cfg.dynamicSmemBytes = (size_t)p.smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // may be scheduled while the previous kernel of the stream drains (the kernel waits for it
  // after its set-up)
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kernel, tmA, tmE, tmB, tmD, p) == cudaSuccess ? SDGP_OK : SDGP_ERR_CUDA;
}

// Two strips per CTA where the accumulators of two tile sets fit TMEM, else one.
template <bool SPARSE, int BN, bool FUSED = false>
sdgp_status launch_halo(const void* A, const void* meta, const void* Wt, const DgradView& view, const HaloParams& p,
                        cudaStream_t stream) {
  if (BN <= 128) {
    const sdgp_status st = launch_halo_nt<SPARSE, (BN <= 128 ? BN : 64), 2, FUSED>(A, meta, Wt, view, p, stream);
    if (st != SDGP_ERR_UNSUPPORTED) return st;
  }
  return launch_halo_nt<SPARSE, BN, 1, FUSED>(A, meta, Wt, view, p, stream);
}

}  // namespace

// A: dense dL/dO [B,P,Q,Cout] (sparse == false) or compressed values [B,P,Q,a_channels/2] with
// meta [B,P,Q,a_channels/16], a_channels = Cout rounded up to 128 (pad channels hold zero values
// and the position pair (0,1)); Wt: [Cout, R, S, Cin]; dD: [B,H,W,Cin].
// Stride 2 is split by the parity of the output pixel: pixel (2h'+ph, 2w'+pw) only meets the taps
// r = ph + pad (mod 2), s = pw + pad (mod 2), and on those it is a stride-1 problem from dO to
// the strided view dD[:, ph::2, pw::2, :].
// fused != nullptr (with sparse == true): A is the DENSE dL/dO and the kernel prunes it itself
// (m = 4, n = fused->n in {1, 2}); no compressed tensor exists in global memory.
sdgp_status launch_dgrad(bool sparse, const void* A, const void* meta, const void* Wt, void* dD, int B,
                         int H, int W, int Cin, int Cout, int R, int S, int stride, int pad, cudaStream_t stream,
                         const FusedPrune* fused, int dtype, const StoredChannels* stored, const ConvGroups* conv_groups) {
  if (fused && stored) return SDGP_ERR_UNSUPPORTED;  // the pruning warps address dL/dO by the channel count they tile by
  if (stored && (stored->a < 0 || stored->a > Cout || stored->a % 8 != 0 || stored->d < 0 || stored->d > Cin || stored->d % 8 != 0))
    return SDGP_ERR_INVALID_ARG;
  if (fused && (!sparse || fused->n < 1 || fused->n > 2)) return SDGP_ERR_UNSUPPORTED;
  if (fused && fused->m != 4 && fused->m != 8 && fused->m != 16 && fused->m != 32) return SDGP_ERR_UNSUPPORTED;
  if (dtype != SDGP_BF16 && dtype != SDGP_FP16) return SDGP_ERR_INVALID_ARG;
  if (fused && dtype == SDGP_FP16 && fused->scheme == SDGP_RESCALED_MAGNITUDE) return SDGP_ERR_UNSUPPORTED;
  if (stride != 1 && stride != 2) return SDGP_ERR_UNSUPPORTED;
  const int P = (H + 2 * pad - R) / stride + 1, Q = (W + 2 * pad - S) / stride + 1;
  if (P < 1 || Q < 1) return SDGP_ERR_INVALID_ARG;
  if ((int64_t)B * H * W == 0) return SDGP_OK;
  if (Cin % 64 != 0 || Cout % 64 != 0) return SDGP_ERR_UNSUPPORTED;
  if ((int64_t)R * S * Cin > 0x7FFFFFFF) return SDGP_ERR_UNSUPPORTED;

  const int BN = (Cin % 256 == 0) ? 256 : (Cin % 128 == 0) ? 128 : 64;
  const int kb_channels = sparse ? 128 : 64;

  DgradView view;
  view.P = P; view.Q = Q; view.batch = B;
  view.a_channels = (sparse && !fused) ? (Cout + 127) / 128 * 128 : (stored && stored->a) ? stored->a : Cout;
  view.d_channels = (stored && stored->d) ? stored->d : Cin;
  view.w_cols = (int64_t)R * S * Cin;
  const size_t Cd = (size_t)view.d_channels;

  // Output parities that no tap reaches are zero: clear dD first if there is any such class.
  bool any_empty = false;
  for (int ph = 0; ph < stride; ++ph)
    for (int pw = 0; pw < stride; ++pw)
      if ((ph + pad) % stride >= R || (pw + pad) % stride >= S) any_empty = true;
  if (any_empty && cudaMemsetAsync(dD, 0, (size_t)B * H * W * Cd * 2, stream) != cudaSuccess) return SDGP_ERR_CUDA;
  for (int ph = 0; ph < stride; ++ph) {
    for (int pw = 0; pw < stride; ++pw) {
      const int Hs = (H - ph + stride - 1) / stride, Ws = (W - pw + stride - 1) / stride;  // pixels of this class
      if (Hs <= 0 || Ws <= 0) continue;
      DgradParams p = {};
      p.r_first = (ph + pad) % stride; p.r_step = stride;
      p.s_first = (pw + pad) % stride; p.s_step = stride;
      p.S_full = S;
      p.R = p.r_first < R ? (R - p.r_first + stride - 1) / stride : 0;
      p.S = p.s_first < S ? (S - p.s_first + stride - 1) / stride : 0;
      if (p.R == 0 || p.S == 0) continue;  // cleared above
      p.pad_h = (ph + pad - p.r_first) / stride;
      p.pad_w = (pw + pad - p.s_first) / stride;
      p.B = B; p.H = Hs; p.W = Ws; p.Cin = Cin; p.Cout = Cout;
      choose_patch(B, Hs, Ws, &p.TW, &p.TH, &p.TB);
      p.tiles_w = (Ws + p.TW - 1) / p.TW;
      p.tiles_h = (Hs + p.TH - 1) / p.TH;
      p.tiles_b = (B + p.TB - 1) / p.TB;
      p.tiles_n = Cin / BN;
      const int64_t m_tiles = (int64_t)p.tiles_w * p.tiles_h * p.tiles_b;
      if (m_tiles * p.tiles_n > 0x3FFFFFFF) return SDGP_ERR_UNSUPPORTED;
      p.m_tiles = (int)m_tiles;
      p.pair_tiles = (int)((m_tiles + 1) / 2) * p.tiles_n;
      p.k_blocks = (Cout + kb_channels - 1) / kb_channels;
      if (conv_groups && conv_groups->cin_g > 0 && conv_groups->cout_g > 0) {
        // block-diagonal W: the widest window of channel blocks any tile of input channels needs
        int widest = 0;
        for (int nt = 0; nt < p.tiles_n; ++nt) {
          const int lo = ((nt * BN) / conv_groups->cin_g) * conv_groups->cout_g / kb_channels;
          int co_end = ((nt * BN + BN + conv_groups->cin_g - 1) / conv_groups->cin_g) * conv_groups->cout_g;
          if (co_end > Cout) co_end = Cout;
          const int hi = (co_end + kb_channels - 1) / kb_channels;
          if (hi - lo > widest) widest = hi - lo;
        }
        if (widest > 0 && widest < p.k_blocks) {
          p.diag_cin_g = conv_groups->cin_g; p.diag_cout_g = conv_groups->cout_g;
          p.diag_last = p.k_blocks - widest;
          p.k_blocks = widest;
        }
      }
      p.P = P; p.Q = Q;
      p.f16 = dtype == SDGP_FP16 ? 1 : 0;
      if (fused) {
        p.fused_n = fused->n; p.fused_m = fused->m; p.fused_scheme = fused->scheme;
        p.seed_lo = (uint32_t)fused->seed; p.seed_hi = (uint32_t)(fused->seed >> 32);
      }
      view.d_base = (uint8_t*)dD + ((size_t)ph * W + pw) * Cd * 2;
      view.d_stride_w = (uint64_t)stride * Cd * 2;
      view.d_stride_h = (uint64_t)stride * W * Cd * 2;
      view.d_stride_b = (uint64_t)H * W * Cd * 2;
      sdgp_status st = SDGP_ERR_UNSUPPORTED;
      // Images 4 pixels wide take the whole-filter-reuse kernel (column-split mode) with a sparse A: fused, it prunes
      // each box S times instead of R * S times; two-pass it measured the same as the general kernel; the dense twin
      // measured slower there (one tile per CTA pair: set-up and the single epilogue dominate either way) and stays
      // on the general kernel.
      if (halo_applies(Hs, Ws, p.R * p.S) && (Ws != 4 || sparse)) {
        HaloParams hp = {};
        hp.B = B; hp.H = Hs; hp.W = Ws; hp.Cin = Cin; hp.Cout = Cout;
        hp.R = p.R; hp.S = p.S; hp.pad_h = p.pad_h; hp.pad_w = p.pad_w;
        hp.r_first = p.r_first; hp.r_step = p.r_step; hp.s_first = p.s_first; hp.s_step = p.s_step;
        hp.S_full = S;
        hp.tiles_n = p.tiles_n; hp.k_blocks = p.k_blocks;
        hp.diag_cin_g = p.diag_cin_g; hp.diag_cout_g = p.diag_cout_g; hp.diag_last = p.diag_last;
        hp.P = P; hp.Q = Q;
        hp.f16 = p.f16;
        if (fused) {
          hp.fused_n = p.fused_n; hp.fused_m = p.fused_m; hp.fused_scheme = p.fused_scheme; hp.seed_lo = p.seed_lo; hp.seed_hi = p.seed_hi;
          st = BN == 256 ? launch_halo<true, 256, true>(A, meta, Wt, view, hp, stream)
             : BN == 128 ? launch_halo<true, 128, true>(A, meta, Wt, view, hp, stream)
                         : launch_halo<true, 64, true>(A, meta, Wt, view, hp, stream);
        } else if (sparse) {
          st = BN == 256 ? launch_halo<true, 256>(A, meta, Wt, view, hp, stream)
             : BN == 128 ? launch_halo<true, 128>(A, meta, Wt, view, hp, stream)
                         : launch_halo<true, 64>(A, meta, Wt, view, hp, stream);
        } else {
          st = BN == 256 ? launch_halo<false, 256>(A, meta, Wt, view, hp, stream)
             : BN == 128 ? launch_halo<false, 128>(A, meta, Wt, view, hp, stream)
                         : launch_halo<false, 64>(A, meta, Wt, view, hp, stream);
        }
        if (st == SDGP_OK) continue;
        if (st != SDGP_ERR_UNSUPPORTED) return st;  // otherwise: does not fit, use the general kernel
      }
      if (fused) {
        if (fused->m == 32) return SDGP_ERR_UNSUPPORTED;  // this kernel's threads hold 16 channels each: groups of up to 16
        st = BN == 256 ? launch_cfg<true, 256, true>(A, meta, Wt, view, p, stream)
           : BN == 128 ? launch_cfg<true, 128, true>(A, meta, Wt, view, p, stream)
                       : launch_cfg<true, 64, true>(A, meta, Wt, view, p, stream);
      } else if (sparse) {
        st = BN == 256 ? launch_cfg<true, 256>(A, meta, Wt, view, p, stream)
           : BN == 128 ? launch_cfg<true, 128>(A, meta, Wt, view, p, stream)
                       : launch_cfg<true, 64>(A, meta, Wt, view, p, stream);
      } else {
        st = BN == 256 ? launch_cfg<false, 256>(A, meta, Wt, view, p, stream)
           : BN == 128 ? launch_cfg<false, 128>(A, meta, Wt, view, p, stream)
                       : launch_cfg<false, 64>(A, meta, Wt, view, p, stream);
      }
      if (st != SDGP_OK) return st;
    }
  }
  return SDGP_OK;
}

// One CTA waits, with a 50 ms limit, on a barrier that nothing ever signals: the wait must give
// up, record its code and let the kernel end normally.
__global__ void bounded_wait_selftest_kernel() {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    ptx::fence_mbar_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) ptx::mbar_wait(&bar, 0u, &g_device_error, 0xE00u, 50000000ull);
  __syncthreads();
}

sdgp_status launch_bounded_wait_selftest(cudaStream_t stream) {
  bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>();
  return cudaGetLastError() == cudaSuccess ? SDGP_OK : SDGP_ERR_CUDA;
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
