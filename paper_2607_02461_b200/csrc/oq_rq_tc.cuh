// Fused rotate+quantize kernel for Hadamard blocks of 64 to 4096 with the block transform on the tensor cores.
//
// The rotation of Eq. 7 / Eq. 4 is  z = blkdiag(H_128 D_j) P x : a gather, a sign flip and, per block of 128
// rotated coordinates, a product with the 128 x 128 matrix of +-1.  Butterflies in registers cost ~6
// instructions per coordinate and 64 registers per lane; here the signed, permuted coordinates are written
// as bf16 into a shared-memory operand tile instead and one tcgen05.mma per 16 coordinates multiplies 128
// (token, block) pairs by H_128 (entries +-1 are exact in bf16, the inputs are bf16 already, the sums are
// accumulated in fp32 in tensor memory).  The rest of the path reads tensor memory twice: once for the row
// norms (||H x'||^2 = 128 ||x||^2), once for the level search and packing.  Blocks of 64 use a block-diagonal
// operand (two blocks per 128 coordinates); a block of 128 * 2^S coordinates (S = 1 .. 5) is H_{2^S} (x) H_128 in
// natural order, so after the tensor-core product its 2^S sub-blocks, which sit in adjacent tile rows of one
// warp, go through S butterfly stages of one shuffle and one FMA per coordinate.
//
// Work units.  A group is 2 th consecutive rows (th = 1, 2, 4 or 8 tokens per HALF group, chosen so that the
// P = th * dim / 128 (token, block) pairs of a half number at most 192).  Each half has its own row buffer and
// its own "rows landed" barrier.  The pairs of a group fill two or three operand tiles of 128 rows:
//     P <= 128:  tile 0 = half 0,  tile 1 = half 1;
//     P >  128:  tile 0 = first 128 pairs of half 0,  tile 2 = first 128 pairs of half 1,
//                tile 1 = the remaining pairs of half 0 (rows 0..63) and of half 1 (rows 64..127).
// Tiles are gathered in the order 0, 1, 2, so half 0's buffer is free one tile before half 1's and the copy of
// each half of the next group overlaps the gather of the other half.
//
// Warp roles (25 warps, every wait bounded, reporting to a status word):
//   gather  (8 warps)  a thread owns one row of a tile (a pair) and 64 of its rotated coordinates: offset table,
//                      16-bit shared-memory load (the th tokens of a warp sit in different banks), pair-wise sign
//                      mask, 16-byte stores into the K-major 128-byte-swizzled operand tile (two tile buffers).
//                      The warp that is the last to finish a half's loads requests the bulk copies (one per row,
//                      16-byte aligned pitch) of that half of the CTA's next group.  These warps run ahead of
//                      the others by up to two operand tiles / four accumulators;
//   mma     (1 thread) per tile: 8 x tcgen05.mma (M = 128 pairs, N = 128 coordinates, K = 16) into one of four
//                      128-column accumulators in tensor memory, committed to "accumulator ready" and
//                      "tile buffer free";
//   compute (16 warps) pass 1: every thread reads its 32 columns of every tile of a group and sums squares;
//                      partial sums meet in shared memory in a fixed order (deterministic norms);
//                      pass 2: reads the same columns again, finds the levels with the polynomial of QuantPoly,
//                      packs, stores, and frees the accumulator.
// Gather warps wait on shared memory, compute warps on the FMA and ALU pipes: the warp schedulers overlap them.
#pragma once
#include <cuda_bf16.h>

#include <type_traits>

#include "oq_internal.h"
#include "oq_rq_fast.cuh"
#include "oq_sm100.cuh"

namespace oq {

struct RqTcParams {
  const unsigned char* X;   // rows x ldx bf16
  int rows, dim, ldx;
  const uint32_t* offset;   // [dim] byte offset of the source element of rotated position k
  const uint32_t* posmask;  // [dim/2] bf16x2 sign-bit masks indexed by ROTATED position pair
  uint32_t* out_idx;
  int pitch_words;          // words per packed row
  void* out_norm;
  float* dbg;
  QuantPoly poly;
  int groups;               // number of groups of 2 th rows
  int ths;                  // log2(th), th = tokens per half group
  int pairs;                // P = th * dim / 128 pairs per half (<= 192)
  int ntiles;               // 2 (P <= 128) or 3
  int bf16_norm;            // 1: norms stored as bf16 (weights), 0: fp32 (activations)
  int stages;               // BLK = 512 only: the Hadamard block is 128 << stages (2 .. 5), th << stages <= 64
  // BITS = 6 (64 levels): the output is the matrix of bf16 levels C[idx] (the operand form of oq_qlinear_levels),
  // found with the grid tables of WideTables; out_idx is not written
  const WideTables* wide;   // device
  __nv_bfloat16* out_levels;
  int ld_levels;
  uint8_t* out_idx8;        // optional [rows][dim] level indices 0..63 (tests), or NULL
  float grid_scale;
  int* status;
};

namespace rqtc {
constexpr int H = 128;
constexpr int COMPUTE_WARPS = 16;                 // 4 lane quarters x 4 column quarters of a tile
constexpr int GATHER_WARPS = 8;                   // 4 lane quarters x 2 halves of the 128 coordinates
constexpr int COMPUTE_THREADS = COMPUTE_WARPS * 32;
constexpr int THREADS = (COMPUTE_WARPS + GATHER_WARPS + 1) * 32;
constexpr int MMA_WARP = COMPUTE_WARPS + GATHER_WARPS;
constexpr int SLOTS = 3;                          // accumulators of 128 columns in tensor memory
constexpr int ABUFS = 2;                          // operand tiles in tensor memory: 128 lanes x 64 columns of bf16 pairs
constexpr uint32_t A_COL0 = SLOTS * 128;          // first column of the operand tiles
constexpr int TMEM_COLS = 512;
constexpr int ROWBUFS = 3;                        // row buffers, one half group each
constexpr uint32_t ATOM = 128 * 128;              // 128 rows x 64 bf16: one swizzle atom column of a tile
constexpr uint32_t TILE = 2 * ATOM;               // 128 rows x 128 bf16
constexpr uint32_t OFF_H = 0, OFF_ROWS = TILE;
constexpr int TAB_PITCH = 132, MSK_PITCH = 68;    // words per block of the shared-memory table copies
constexpr int MAX_PAIRS = 192;
constexpr unsigned GATHER_SLEEP_NS = 256;         // between polls of a gather warp that waits for an operand tile
enum { WAIT_ROWS = 11, WAIT_AFULL = 12, WAIT_ACC = 13, WAIT_DRAIN = 14, WAIT_AFREE = 15, WAIT_ACCFREE = 16 };
__host__ __device__ constexpr uint32_t row_pitch_bytes(int dim) { return 2u * (uint32_t)dim + 16u; }
}  // namespace rqtc

// BITS: 2, 3, 4 (packed indices out, polynomial level search) or 6 (bf16 levels out, grid level search).
// TAB: where the gather tables live.  0: global memory (read-only path); 1: both copied to shared memory (32-bit
// offsets, masks); 2: offsets copied to shared memory as 16-bit values, masks stay in global memory.
// BLK: the Hadamard block, 64, 128 or 256 (256: one butterfly stage across two tile rows after the tensor-core product);
// 512 stands for every larger block, 128 << p.stages, with p.stages butterfly stages.
template <int BITS, int TAB, int BLK>
__global__ void __launch_bounds__(rqtc::THREADS, 1) rq_tc_kernel(const RqTcParams p) {
  using namespace rqtc;
  extern __shared__ unsigned char smem_dyn[];
  // 1024-byte alignment for the swizzled tiles, computed on the shared-window address so that the compiler keeps
  // treating everything below as shared memory (32-bit addresses, no generic-pointer arithmetic)
  unsigned char* smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  const int th = 1 << p.ths, T = 2 * th;
  const uint32_t pitch = row_pitch_bytes(p.dim);
  unsigned char* rows_s = smem + OFF_ROWS;          // [3 buffers][th rows][pitch]
  unsigned char* after_rows = rows_s + (size_t)ROWBUFS * th * pitch;
  // copies of the offset and sign-mask tables: the words of a block are followed by 4 words of padding, so that
  // the blocks a warp reads at once sit in different banks
  uint32_t* s_table = reinterpret_cast<uint32_t*>(after_rows);    // [dim/128][TAB_PITCH] (TAB 1) or [dim/128][MSK_PITCH] (TAB 2)
  uint32_t* s_mask = s_table + (TAB == 1 ? (p.dim / H) * TAB_PITCH : TAB == 2 ? (p.dim / H) * MSK_PITCH : 0);   // [dim/128][MSK_PITCH] (TAB 1)
  float* s_part = reinterpret_cast<float*>(s_mask + (TAB == 1 ? (p.dim / H) * MSK_PITCH : 0));                  // [2][16 warps][2 halves][8]
  uint64_t* bars = reinterpret_cast<uint64_t*>(s_part + 2 * COMPUTE_WARPS * 16);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 13);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  // [0..2]: gather warps that no longer need row buffer b (never reset; the warp that brings one to a multiple of
  // 8 requests the next copy into it); [3..5]: copies requested per buffer
  unsigned int* s_cnt = reinterpret_cast<unsigned int*>(tmem_slot + 2);
  // BITS = 6: copy of the grid tables (16-byte aligned: every region above is a multiple of 16 bytes, 144 up to here)
  const WideTables* s_wide = reinterpret_cast<const WideTables*>(s_cnt + 8);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rows_full0 = smem_u32(bars);          // [3] bulk copies of a half group have landed in buffer b
  const uint32_t a_full0 = smem_u32(bars + 3);         // [2] operand tile written by the 8 gather warps
  const uint32_t a_free0 = smem_u32(bars + 5);         // [2] operand tile read by its MMAs
  const uint32_t acc_ready0 = smem_u32(bars + 7);      // [3] accumulator written by its MMAs
  const uint32_t acc_free0 = smem_u32(bars + 10);      // [3] accumulator read twice by the 16 compute warps
  const uint32_t row_bytes = 2u * (uint32_t)p.dim;
  const int stride = (int)gridDim.x;
  const bool nt3 = p.ntiles == 3;
  const int rem = p.pairs - 128;     // pairs of a half that go to the shared middle tile (nt3)

  // Half groups are numbered hs = 2 * (index of the group within this CTA) + half and live in row buffer hs % 3.
  // Bulk copies of half group hs into its buffer; one that lies past the last row (or past the last group) still
  // completes its barrier phase (0 bytes).
  auto request_half = [&](uint32_t hs) {
    const uint32_t b = hs % 3u;
    const uint32_t bar = rows_full0 + 8 * b;
    const long long grp = (long long)blockIdx.x + (long long)(hs >> 1) * stride;
    const long long row0 = grp * T + (long long)(hs & 1u) * th;
    const int nvalid = grp < p.groups ? (int)max(0ll, min((long long)th, (long long)p.rows - row0)) : 0;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(row_bytes * (uint32_t)nvalid) : "memory");
    for (int r = 0; r < nvalid; ++r) {
      const unsigned char* src = p.X + (size_t)(row0 + r) * p.ldx * 2;
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(smem_u32(rows_s + ((size_t)b * th + r) * pitch)), "l"(src), "r"(row_bytes), "r"(bar) : "memory");
    }
    s_cnt[3 + b] += 1u;
  };

  if (tid == 0) {
    for (int b = 0; b < ROWBUFS; ++b) mbar_init(rows_full0 + 8 * b, 1);
    for (int b = 0; b < ABUFS; ++b) {
      mbar_init(a_full0 + 8 * b, GATHER_WARPS);
      mbar_init(a_free0 + 8 * b, 1);
    }
    for (int s = 0; s < SLOTS; ++s) {
      mbar_init(acc_ready0 + 8 * s, 1);
      mbar_init(acc_free0 + 8 * s, COMPUTE_WARPS);
    }
    *abort_flag = 0;
    for (int i = 0; i < 6; ++i) s_cnt[i] = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    // With programmatic dependent launch this CTA may have started while the previous kernel of the stream was still
    // running: its results (the rows read here, buffers this kernel overwrites) are safe to touch only after this wait.
    // Every other access to them in this CTA is ordered after it through barriers.  (A no-op in an ordinary launch.)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // the first rows travel while the CTA builds its tables
    if ((int)blockIdx.x < p.groups)
      for (uint32_t hs = 0; hs < (uint32_t)ROWBUFS; ++hs) request_half(hs);
  }
  if (warp == MMA_WARP) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "n"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // The B operand, K-major, 128-byte swizzle: H_128 with B[n][k] = (-1)^popcount(n & k) (symmetric) for blocks of 128
  // and 256, blkdiag(H_64, H_64) for blocks of 64.
  for (int c = tid; c < 128 * 16; c += THREADS) {
    const int n = c >> 4, k0 = (c & 15) * 8;
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int ka = k0 + 2 * e, kb2 = ka + 1;
      constexpr int hm = BLK == 64 ? 63 : 127;       // index bits inside one Hadamard block of the tile row
      uint32_t lo = (__popc(n & ka & hm) & 1) ? 0xBF80u : 0x3F80u;
      uint32_t hi = (__popc(n & kb2 & hm) & 1) ? 0xBF80u : 0x3F80u;
      if (BLK == 64) {           // two independent blocks of 64 per tile row: blkdiag(H_64, H_64)
        if ((n ^ ka) & 64) lo = 0u;
        if ((n ^ kb2) & 64) hi = 0u;
      }
      w[e] = lo | (hi << 16);
    }
    const uint32_t chunk = (uint32_t)((k0 & 63) >> 3);
    *reinterpret_cast<uint4*>(smem + OFF_H + (k0 >> 6) * ATOM + n * 128 + ((chunk ^ (n & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
  }
  for (int i = tid; i < 2 * COMPUTE_WARPS * 16; i += THREADS) s_part[i] = 0.f;
  if constexpr (BITS == 6) {
    uint32_t* dst = reinterpret_cast<uint32_t*>(s_cnt + 8);
    const uint32_t* src = reinterpret_cast<const uint32_t*>(p.wide);
    for (int i = tid; i < (int)(sizeof(WideTables) / 4); i += THREADS) dst[i] = __ldg(src + i);
  }
  if (TAB == 1) {
    // 16 bytes per thread and load: one or two loads per thread, all in flight together
    const uint4* src = reinterpret_cast<const uint4*>(p.offset);
    for (int i = tid; i < p.dim / 4; i += THREADS)
      reinterpret_cast<uint4*>(s_table)[(i >> 5) * (TAB_PITCH / 4) + (i & 31)] = __ldg(src + i);
    const uint4* msrc = reinterpret_cast<const uint4*>(p.posmask);
    for (int i = tid; i < p.dim / 8; i += THREADS)
      reinterpret_cast<uint4*>(s_mask)[(i >> 4) * (MSK_PITCH / 4) + (i & 15)] = __ldg(msrc + i);
  } else if (TAB == 2) {
    const uint4* src = reinterpret_cast<const uint4*>(p.offset);
    for (int i = tid; i < p.dim / 4; i += THREADS) {      // 4 offsets -> 2 words of the 16-bit table
      const uint4 o = __ldg(src + i);
      reinterpret_cast<uint2*>(s_table)[(i >> 5) * (MSK_PITCH / 2) + (i & 31)] = make_uint2(o.x | (o.y << 16), o.z | (o.w << 16));
    }
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *tmem_slot;
  // the next kernel of the stream may be scheduled on SMs as they become free (it waits for this grid to finish
  // before it touches anything this grid reads or writes)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  auto warp_wait = [&](uint32_t bar, uint32_t parity, int code) {
    if (lane == 0) mbar_wait(bar, parity, abort_flag, p.status, code);
    __syncwarp();
  };
  // Which pair row r of tile i holds: its half, its block of 128 coordinates, and whether the row is in use.
  // (q = r / 32.)  Pair number = block * th + token; for blocks above 256 the S low bits of the block number move
  // below the token bits, (block_hi * th + token) * 2^S + block_lo, so that the sub-blocks of one Hadamard block are
  // adjacent rows.  The token of a row is the same in every tile (th * 2^S divides 64).
  const int lg_lo = BLK == 512 ? p.stages : 0;
  auto tile_half = [&](int i, int q) { return nt3 ? (i == 0 ? 0 : (i == 2 ? 1 : (q >> 1))) : i; };
  auto tile_block = [&](int i, int r) {
    const int pr = (nt3 && i == 1) ? 128 + (r & 63) : r;
    if constexpr (BLK == 512) return ((pr >> (lg_lo + p.ths)) << lg_lo) | (pr & ((1 << lg_lo) - 1));
    else return pr >> p.ths;
  };
  auto tile_valid = [&](int i, int r) { return nt3 ? (i != 1 || (r & 63) < rem) : r < p.pairs; };
  auto row_token = [&](int r) { return ((r & 63) >> lg_lo) & (th - 1); };

  if (warp == MMA_WARP) {
    // ------------------------------- MMA issuer -------------------------------
    if (lane == 0) {
      constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      const uint64_t desc_h = smem_desc(smem_u32(smem + OFF_H));
      uint32_t n = 0;                               // tiles issued so far (operand buffer n & 1, accumulator n % 3)
      for (int grp = blockIdx.x; grp < p.groups; grp += stride) {
        for (int i = 0; i < p.ntiles; ++i, ++n) {
          const uint32_t buf = n & 1u, slot = n % 3u, use = n / 3u;
          mbar_wait(a_full0 + 8 * buf, (n >> 1) & 1u, abort_flag, p.status, WAIT_AFULL);
          if (use > 0u) mbar_wait(acc_free0 + 8 * slot, (use - 1u) & 1u, abort_flag, p.status, WAIT_ACCFREE);
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_tmem = tmem + A_COL0 + buf * 64u;     // 8 columns (16 bf16) per K step
#pragma unroll
          for (int k4 = 0; k4 < 8; ++k4) {
            const uint64_t db = desc_h + (uint64_t)((k4 >> 2) * (ATOM >> 4)) + 2 * (k4 & 3);
            const uint32_t acc = k4 > 0 ? 1u : 0u;
            asm volatile(
                "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                " tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
                ::"r"(tmem + slot * 128u), "r"(a_tmem + 8u * k4), "l"(db), "r"(IDESC), "r"(acc) : "memory");
          }
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(acc_ready0 + 8 * slot) : "memory");
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(a_free0 + 8 * buf) : "memory");
        }
      }
    }
  } else if (warp >= COMPUTE_WARPS) {
    // ------------------------------- gather warps -------------------------------
    const int gw = warp - COMPUTE_WARPS;
    const int gq = gw & 3, kh = gw >> 2;              // lane quarter of the tile, half of the 128 coordinates
    const int r = gq * 32 + lane;                     // row of the operand tile
    const int tl = row_token(r);                      // token within its half (the same in every tile)
    const uint32_t a_thr = tmem + ((uint32_t)(gq * 32) << 16) + A_COL0 + (uint32_t)kh * 32u;   // + 64 * buffer
    uint32_t n = 0;
    int it = 0;
    for (int grp = blockIdx.x; grp < p.groups; grp += stride, ++it) {
      for (int i = 0; i < p.ntiles; ++i, ++n) {
        const uint32_t buf = n & 1u;
        const int half = tile_half(i, gq), j = tile_block(i, r);
        const uint32_t hs = 2u * (uint32_t)it + (uint32_t)half, rb = hs % 3u;
        warp_wait(rows_full0 + 8 * rb, (hs / 3u) & 1u, WAIT_ROWS);
        if (n >= 2u) {     // the gather runs ahead of the other warps: a long sleep between polls leaves them the issue slots
          if (lane == 0) mbar_wait(a_free0 + 8 * buf, ((n >> 1) - 1u) & 1u, abort_flag, p.status, WAIT_AFREE, WAIT_CYCLES, GATHER_SLEEP_NS);
          __syncwarp();
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        uint32_t w[32];
        if (tile_valid(i, r)) {
          const unsigned char* rowbytes = rows_s + ((size_t)rb * th + tl) * pitch;
          // offsets of the thread's 64 coordinates, then the 64 loads (all in flight together), then masks and
          // pairing: 32 words of two bf16, the thread's half row of the operand tile
          if constexpr (TAB == 2) {
            // two rounds of 32 coordinates: 16-bit offsets from shared memory, masks from global memory (requested
            // before the gather loads so that their latency overlaps)
#pragma unroll
            for (int rd = 0; rd < 2; ++rd) {
              uint32_t h[32];
              const uint4* tab = reinterpret_cast<const uint4*>(s_table + j * MSK_PITCH + kh * 32 + rd * 16);
#pragma unroll
              for (int e8 = 0; e8 < 4; ++e8) {
                const uint4 o = tab[e8];
                h[8 * e8] = o.x & 0xFFFFu; h[8 * e8 + 1] = o.x >> 16; h[8 * e8 + 2] = o.y & 0xFFFFu; h[8 * e8 + 3] = o.y >> 16;
                h[8 * e8 + 4] = o.z & 0xFFFFu; h[8 * e8 + 5] = o.z >> 16; h[8 * e8 + 6] = o.w & 0xFFFFu; h[8 * e8 + 7] = o.w >> 16;
              }
              const uint4* msk = reinterpret_cast<const uint4*>(p.posmask + j * (H / 2) + kh * 32 + rd * 16);
              uint4 m[4];
#pragma unroll
              for (int c = 0; c < 4; ++c) m[c] = __ldg(msk + c);
#pragma unroll
              for (int e = 0; e < 32; ++e) h[e] = *reinterpret_cast<const unsigned short*>(rowbytes + h[e]);
#pragma unroll
              for (int c = 0; c < 4; ++c) {
                w[16 * rd + 4 * c] = prmt(h[8 * c], h[8 * c + 1], 0x5410u) ^ m[c].x;
                w[16 * rd + 4 * c + 1] = prmt(h[8 * c + 2], h[8 * c + 3], 0x5410u) ^ m[c].y;
                w[16 * rd + 4 * c + 2] = prmt(h[8 * c + 4], h[8 * c + 5], 0x5410u) ^ m[c].z;
                w[16 * rd + 4 * c + 3] = prmt(h[8 * c + 6], h[8 * c + 7], 0x5410u) ^ m[c].w;
              }
            }
          } else {
            uint32_t h[64];
            const uint4* tab = reinterpret_cast<const uint4*>(TAB == 1 ? s_table + j * TAB_PITCH + kh * 64 : p.offset + j * H + kh * 64);
#pragma unroll
            for (int e4 = 0; e4 < 16; ++e4) {
              const uint4 o = TAB == 1 ? tab[e4] : __ldg(tab + e4);
              h[4 * e4] = o.x; h[4 * e4 + 1] = o.y; h[4 * e4 + 2] = o.z; h[4 * e4 + 3] = o.w;
            }
#pragma unroll
            for (int e = 0; e < 64; ++e) h[e] = *reinterpret_cast<const unsigned short*>(rowbytes + h[e]);
            const uint4* msk = reinterpret_cast<const uint4*>(TAB == 1 ? s_mask + j * MSK_PITCH + kh * 32 : p.posmask + j * (H / 2) + kh * 32);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              const uint4 m = TAB == 1 ? msk[c] : __ldg(msk + c);
              w[4 * c] = prmt(h[8 * c], h[8 * c + 1], 0x5410u) ^ m.x;
              w[4 * c + 1] = prmt(h[8 * c + 2], h[8 * c + 3], 0x5410u) ^ m.y;
              w[4 * c + 2] = prmt(h[8 * c + 4], h[8 * c + 5], 0x5410u) ^ m.z;
              w[4 * c + 3] = prmt(h[8 * c + 6], h[8 * c + 7], 0x5410u) ^ m.w;
            }
          }
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) w[c] = 0u;
        }
        // the operand tile lives in tensor memory: 32 columns of this thread's lane
        tmem_store32(a_thr + buf * 64u, w);
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        // the last gather warp to finish with a row buffer requests the half group that reuses it
        const bool last0 = nt3 ? i == 1 : i == 0, last1 = i == p.ntiles - 1;
        __syncwarp();
        if (lane == 0) {
          if (last0 || last1) {
            __threadfence_block();
            const uint32_t hsr = 2u * (uint32_t)it + (last1 ? 1u : 0u), b = hsr % 3u;
            const unsigned int old = atomicAdd(&s_cnt[b], 1u);
            if ((old & (GATHER_WARPS - 1)) == GATHER_WARPS - 1 && !*abort_flag) {
              __threadfence_block();     // the other warps' reads of the buffer are ordered before the copies below
              const long long g3 = (long long)blockIdx.x + (long long)((hsr + 3u) >> 1) * stride;
              if (g3 < p.groups) request_half(hsr + 3u);
            }
          }
          asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(a_full0 + 8 * buf) : "memory");
        }
      }
    }
  } else {
    // ------------------------------- compute warps -------------------------------
    const int q = warp & 3, kq = warp >> 2;          // tensor-memory lane quarter, column quarter
    const int r = q * 32 + lane;                     // row of the tile = tensor-memory lane
    const int tl = row_token(r);
    // lane bits that number the token (the other bits run over the blocks of that token)
    const int tok_bits = BLK == 512 ? (((th - 1) << lg_lo) & 31) : th - 1;
    const Poly2<BITS == 6 ? 1 : (1 << (BITS - 1)) - 1> poly(p.poly);     // (unused with 6 bits)
    const float blk_f = BLK == 512 ? (float)(H << p.stages) : (float)BLK;      // coordinates per Hadamard block
    const float inv_sqrt_h = rsqrtf(blk_f);
    constexpr float mma_h = BLK < H ? (float)BLK : (float)H;   // the tensor-core product multiplies squared norms by this
    const uint32_t tmem_thr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(kq * 32);
    // Pass 1 of one tile (sequence number n, tile i of its group): the sum of squares of the thread's 32 columns,
    // zero for an unused row.
    auto tile_sumsq = [&](uint32_t n, int i) {
      const uint32_t slot = n % 3u;
      warp_wait(acc_ready0 + 8 * slot, (n / 3u) & 1u, WAIT_ACC);
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      uint32_t v[32];
      tmem_load32(tmem_thr + slot * 128u, v);
      unsigned long long qa = 0ull, qb = 0ull;      // two chains, fixed order
#pragma unroll
      for (int e = 0; e < 16; e += 2) {
        const unsigned long long xa = pack2(__uint_as_float(v[2 * e]), __uint_as_float(v[2 * e + 1]));
        const unsigned long long xb = pack2(__uint_as_float(v[2 * e + 2]), __uint_as_float(v[2 * e + 3]));
        qa = fma2(xa, xa, qa);
        qb = fma2(xb, xb, qb);
      }
      float a0, a1, b0, b1;
      unpack2(qa, a0, a1);
      unpack2(qb, b0, b1);
      return tile_valid(i, r) ? (a0 + a1) + (b0 + b1) : 0.f;
    };
    uint32_t n0 = 0;                                  // sequence number of the group's first tile
    int it = 0;
    // pass 1 of the CTA's first group; pass 1 of every later group is spread over the pass 2 of the group before it
    float ssq0 = 0.f, ssq1 = 0.f;
    if ((int)blockIdx.x < p.groups) {
      for (int i = 0; i < p.ntiles; ++i) {
        const float a = tile_sumsq((uint32_t)i, i);
        if (tile_half(i, q)) ssq1 += a; else ssq0 += a;
      }
    }
    for (int grp = blockIdx.x; grp < p.groups; grp += stride, ++it, n0 += (uint32_t)p.ntiles) {
      const int row0 = grp * T;
      const bool has_next = grp + stride < p.groups;
      // lanes of the warp that hold the same token add up (they differ in the lane bits that are not token bits) ...
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1)
        if (BLK == 512 ? !(o & tok_bits) : o >= th) {
          ssq0 += __shfl_xor_sync(0xffffffffu, ssq0, o);
          ssq1 += __shfl_xor_sync(0xffffffffu, ssq1, o);
        }
      // (with large blocks a warp may hold only some of the tokens; the slots of the others stay zero)
      float* part = s_part + (it & 1) * (COMPUTE_WARPS * 16);
      if ((lane & ~tok_bits) == 0) {
        part[warp * 16 + tl] = ssq0;
        part[warp * 16 + 8 + tl] = ssq1;
      }
      asm volatile("bar.sync 1, %0;" ::"n"(COMPUTE_THREADS) : "memory");
      // ... and the 16 warps' partial sums in a fixed order: lane L adds 8 warps for slot L & 15
      float tot = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) tot += part[((lane >> 4) * 8 + w) * 16 + (lane & 15)];
      tot += __shfl_xor_sync(0xffffffffu, tot, 16);
      const float nrm = sqrtf(tot * (1.0f / mma_h));               // of slot lane & 15 = (half, token)
      if (warp == 0 && lane < 16 && (lane & 7) < th) {
        const int row = row0 + (lane >> 3) * th + (lane & 7);
        if (row < p.rows) {
          if (p.bf16_norm) reinterpret_cast<__nv_bfloat16*>(p.out_norm)[row] = __float2bfloat16_rn(nrm);
          else reinterpret_cast<float*>(p.out_norm)[row] = nrm;
        }
      }
      const float s0 = __shfl_sync(0xffffffffu, nrm, tl), s1 = __shfl_sync(0xffffffffu, nrm, 8 + tl);
      // |z| / (sqrt(h) (s + eps) clamp) with z the unnormalised block transform
      // (6 bits: |z| * grid_scale / (sqrt(h) (s + eps)), the position on the level-search grid)
      const float kappa0 = BITS == 6 ? p.grid_scale / (sqrtf(blk_f) * (s0 + 1e-10f)) : 1.0f / (sqrtf(blk_f) * (s0 + 1e-10f) * p.poly.clamp);
      const float kappa1 = BITS == 6 ? p.grid_scale / (sqrtf(blk_f) * (s1 + 1e-10f)) : 1.0f / (sqrtf(blk_f) * (s1 + 1e-10f) * p.poly.clamp);
      // ---------------- pass 2: level search and packing; pass 1 of the next group, one tile at a time ----------------
      ssq0 = 0.f;
      ssq1 = 0.f;
      for (int i = 0; i < p.ntiles; ++i) {
        const uint32_t n = n0 + (uint32_t)i, slot = n % 3u;
        const int half = tile_half(i, q), j = tile_block(i, r);
        uint32_t vb[32];
        tmem_load32(tmem_thr + slot * 128u, vb);
        // the accumulator may be overwritten as soon as every compute warp has read it
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(acc_free0 + 8 * slot) : "memory");
        if constexpr (BLK == 256) {
          // H_256 = [[H_128, H_128], [H_128, -H_128]]: the two halves of a block sit th rows apart, in the same warp
          const float sg = (lane & th) ? -1.f : 1.f;
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const float mine = __uint_as_float(vb[e]);
            const float other = __shfl_xor_sync(0xffffffffu, mine, th);
            vb[e] = __float_as_uint(fmaf(mine, sg, other));      // low half: mine + other; high half: other - mine
          }
        } else if constexpr (BLK == 512) {
          // H_{2^S} (x) H_128: sub-block u of a block is the low S bits of the lane; stage s combines the rows that
          // differ in bit s of u (sum in the row with the bit clear, difference in the other)
          for (int s = 0; s < p.stages; ++s) {
            const int bit = 1 << s;
            const float sg = (lane & bit) ? -1.f : 1.f;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              const float mine = __uint_as_float(vb[e]);
              const float other = __shfl_xor_sync(0xffffffffu, mine, bit);
              vb[e] = __float_as_uint(fmaf(mine, sg, other));
            }
          }
        }
        const int row = row0 + half * th + tl;
        if (tile_valid(i, r) && row < p.rows) {
          float v[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(vb[e]);
          if (p.dbg != nullptr) {
            float* d = p.dbg + (size_t)row * p.dim + j * H + kq * 32;
#pragma unroll
            for (int e = 0; e < 32; ++e) d[e] = v[e] * inv_sqrt_h;
          }
          if constexpr (BITS == 6) {
            // grid level search (see WideTables): magnitude rank, then the bf16 level with the sign of z (z <= 0
            // counts as negative: the number of boundaries strictly below the value, as in the packed formats)
            const float kg = half ? kappa1 : kappa0;
            uint4* dl = reinterpret_cast<uint4*>(p.out_levels + (size_t)row * p.ld_levels + j * H + kq * 32);
            // (the index bytes are a test output: the loop that does not build them is the one that is timed)
            auto search32 = [&](auto want_idx) {
              uint32_t lv[16];
              [[maybe_unused]] uint32_t ib[8];
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                const float u = fabsf(v[e]) * kg;
                const int g = min(__float2int_rz(u), 255);
                const int cand = s_wide->cell[g];
                const int mag = cand + (u > s_wide->bound_scaled[cand] ? 1 : 0);
                const uint32_t neg = v[e] > 0.f ? 0u : 1u;
                const uint32_t bits = (uint32_t)s_wide->level_bf16[mag] | (neg << 15);
                if (e & 1) lv[e >> 1] |= bits << 16; else lv[e >> 1] = bits;
                if constexpr (decltype(want_idx)::value) {
                  const uint32_t idx = neg ? (uint32_t)(31 - mag) : (uint32_t)(32 + mag);
                  if (e & 3) ib[e >> 2] |= idx << (8 * (e & 3)); else ib[e >> 2] = idx;
                }
              }
#pragma unroll
              for (int c = 0; c < 4; ++c) dl[c] = make_uint4(lv[4 * c], lv[4 * c + 1], lv[4 * c + 2], lv[4 * c + 3]);
              if constexpr (decltype(want_idx)::value) {
                uint4* di = reinterpret_cast<uint4*>(p.out_idx8 + (size_t)row * p.dim + j * H + kq * 32);
                di[0] = make_uint4(ib[0], ib[1], ib[2], ib[3]);
                di[1] = make_uint4(ib[4], ib[5], ib[6], ib[7]);
              }
            };
            if (p.out_idx8 != nullptr) search32(std::true_type{});
            else search32(std::false_type{});
          } else {
          uint32_t words[BITS];
          pack32<BITS>(v, half ? kappa1 : kappa0, poly, words);
          uint32_t* dst = p.out_idx + (size_t)row * p.pitch_words + (j * (H / 32) + kq) * BITS;
          if constexpr (BITS == 4) *reinterpret_cast<uint4*>(dst) = make_uint4(words[0], words[1], words[2], words[3]);
          else if constexpr (BITS == 2) *reinterpret_cast<uint2*>(dst) = make_uint2(words[0], words[1]);
          else {
#pragma unroll
            for (int c = 0; c < BITS; ++c) dst[c] = words[c];
          }
          }
        }
        // the next group's tile i went into the accumulator that this tile's pass 2 freed (3-tile groups) or one
        // freed earlier: its MMAs ran while this warp packed
        if (has_next) {
          const float a = tile_sumsq(n + (uint32_t)p.ntiles, i);
          if (tile_half(i, q)) ssq1 += a; else ssq0 += a;
        }
      }
    }
  }
  __syncwarp();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  // after a wait gave up somewhere, a requested copy may still be in flight: let it land before the CTA ends
  if (tid == 0 && *abort_flag) {
    int keep_waiting = 0;      // (the CTA's abort flag is already up: it must not cut this wait short)
    for (int b = 0; b < ROWBUFS; ++b)
      if (s_cnt[3 + b] > 0u)
        mbar_wait(rows_full0 + 8 * b, (s_cnt[3 + b] - 1u) & 1u, &keep_waiting, p.status, WAIT_DRAIN, 200000000ll);
  }
  if (warp == MMA_WARP) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(TMEM_COLS) : "memory");
  }
}

}  // namespace oq
