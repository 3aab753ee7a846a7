// Fused rotate+quantize kernel, token-slab form (Hadamard blocks of 64, 128 and 256).
//
// The rotation of Eq. 7 / Eq. 4 is  z = blkdiag(H_128 D_j) P x.  The expensive part on a GPU is the gather P x: one
// 2-byte shared-memory access per coordinate when every thread walks its own row.  Here the rows of a SLAB of TOK
// consecutive tokens (8, 4 or 2, by row length) are first transposed into a buffer in which the TOK tokens of one
// source coordinate are adjacent (a "chunk" of 2 TOK bytes), so that ONE shared-memory load moves a coordinate of
// all TOK tokens.  The permuted, signed chunks are written into an operand tile that the tensor cores read with the
// row index (token, block) contiguous ("MN-major"), and one tcgen05.mma per 16 coordinates multiplies the tile by
// H_128 (entries +-1 are exact in bf16, inputs are bf16, sums are fp32 in tensor memory).
//
// Row norms (Eq. 7: s = ||x'|| = ||x||, the rotation is orthogonal) also come from the tensor cores: the transposed
// slab, read as both operands of one more product, gives the Gram matrix of its 16-byte rows; the diagonal entries
// that belong to a token add up to its squared norm (bf16 products are exact in fp32).  The norm of a token is
// therefore known before the first of its tiles is quantized, and every accumulator is read exactly once.
//
// Pipeline of one CTA (one per SM, persistent over its slabs; every wait is bounded and reports to a status word):
//   front end (16 w)  per slab: the rows of the NEXT slab are already in registers (16-byte global loads issued a slab
//                 ahead); sign flips by SOURCE position -> stmatrix.trans -> slab buffer; named barrier; then the tiles
//                 that the slab completes: table look-up of the chunk address, one load + one store per chunk into
//                 the operand tile (two halves of 64 coordinates, refilled as soon as their MMAs have completed)
//   MMA (1 thr)   Gram product of a slab; per tile 8 x tcgen05.mma (M = 128 pairs, N = 128, K = 16) into one of
//                 three accumulators
//   compute (8 w) per slab: the diagonal of the Gram matrix -> norms; per tile: 2 x 32 accumulator columns per thread,
//                 level search with the polynomial of QuantPoly, packing, stores.
#pragma once
#include <cuda_bf16.h>

#include "oq_internal.h"
#include "oq_rq_fast.cuh"
#include "oq_rq_mm_params.h"
#include "oq_sm100.cuh"

namespace oq {

namespace rqmm {
constexpr int COMPUTE_WARPS = 8, FE_WARPS = 16;
constexpr int PIECES = 2;                         // pieces of 32 accumulator columns one compute thread handles per tile
constexpr int FE_WARP0 = COMPUTE_WARPS, MMA_WARP = FE_WARP0 + FE_WARPS;
constexpr int THREADS = (MMA_WARP + 1) * 32;
constexpr int SLOTS = 3;                          // accumulators of 128 columns
constexpr uint32_t GRAM_COL = SLOTS * 128;        // Gram accumulator
constexpr int TMEM_COLS = 512;
constexpr uint32_t ATOM = 128 * 128;              // one 64-coordinate half of the K-major, 128-byte-swizzled H tile
constexpr uint32_t OFF_H = 0, OFF_A = 32768, OFF_T = 65536;   // H tile, operand tile, two slab buffers
constexpr int WIN_SLOTS = 8;                      // 16-byte global loads one front-end thread keeps in flight
constexpr int NORM_RING = 4;
enum { B_TFULL = 0, B_TDONE = 2, B_AFULL = 4, B_AFREE = 6, B_ACCRDY = 8, B_ACCFREE = 11, B_GRAMRDY = 14, B_GRAMFREE = 15, NBARS = 16 };
enum { WAIT_TFULL = 22, WAIT_TDONE = 23, WAIT_AFULL = 24, WAIT_AFREE = 25, WAIT_ACC = 26, WAIT_ACCFREE = 27, WAIT_GRAM = 28,
       WAIT_GRAMFREE = 29 };
__host__ __device__ constexpr int window_row(int cb) { return rq_mm_window_row(cb); }
}  // namespace rqmm

// Shared-memory matrix descriptor of an MN-major operand with the 128-byte swizzle: atoms of 64 elements along M/N
// (128 contiguous bytes, 16-byte pieces XOR-ed with the row number) x 8 rows along K; `mn_stride` bytes between atoms
// that are neighbours along M/N, `k_stride` bytes between neighbours along K.
__device__ __forceinline__ uint64_t mn_major_desc(uint32_t addr, uint32_t mn_stride, uint32_t k_stride) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((mn_stride >> 4) & 0x3FFFu) << 16) | ((uint64_t)((k_stride >> 4) & 0x3FFFu) << 32) |
         (1ull << 46) | (2ull << 61);
}

template <int BITS, int TOK, int BLK>
__global__ void __launch_bounds__(rqmm::THREADS, 1) rq_mm_kernel(const RqMmParams p) {
  using namespace rqmm;
  constexpr int CB = 2 * TOK;            // chunk bytes
  constexpr int SUBS = 8 / TOK;          // chunks per 16-byte row
  constexpr int BC = 128 / TOK;          // (slab, block) chunks of 128 rotated coordinates per tile
  constexpr int GPW = TOK / 2;           // groups of 8 * SUBS lanes per front-end warp
  constexpr int PASSES = 4 / GPW;        // passes over the 16 piece columns of the operand tile
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t slab_bytes = 256u * (uint32_t)p.seg_rows;
  const uint32_t a_base = sbase + OFF_A, t_base = sbase + OFF_T;
  const uint32_t tab_base = t_base + 2 * slab_bytes;
  const uint32_t msk_base = tab_base + (p.tab_smem ? 4u * (uint32_t)p.dim : 0u);
  unsigned char* small = smem + (msk_base - sbase) + (p.mask_smem ? 2u * (uint32_t)p.dim : 0u);
  float* s_part = reinterpret_cast<float*>(small);                       // [NORM_RING][4 lane quarters][8 row elements]
  uint64_t* bars = reinterpret_cast<uint64_t*>(s_part + NORM_RING * 32);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NBARS + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar0 = smem_u32(bars);
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int stride = (int)gridDim.x;
  const int nsl = ((int)blockIdx.x < p.nslabs) ? (p.nslabs - (int)blockIdx.x + stride - 1) / stride : 0;   // slabs of this CTA
  const int ntiles = (nsl * p.nb + BC - 1) / BC;
  const int raw_rows = p.nb * TOK;

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(B_TFULL + i), 1);
      mbar_init(bar(B_TDONE + i), 1);
      mbar_init(bar(B_AFULL + i), FE_WARPS / 2);
      mbar_init(bar(B_AFREE + i), 1);
    }
    for (int i = 0; i < SLOTS; ++i) {
      mbar_init(bar(B_ACCRDY + i), 1);
      mbar_init(bar(B_ACCFREE + i), COMPUTE_WARPS);
    }
    mbar_init(bar(B_GRAMRDY), 1);
    mbar_init(bar(B_GRAMFREE), 4);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    // With programmatic dependent launch this CTA may have started while the previous kernel of the stream was still
    // running: its results (the rows read here, buffers this kernel overwrites) are safe to touch only after this wait.
    // Every access to them in this CTA comes after the __syncthreads below.
    asm volatile("griddepcontrol.wait;" ::: "memory");
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
      constexpr int hm = BLK == 64 ? 63 : 127;
      uint32_t lo = (__popc(n & ka & hm) & 1) ? 0xBF80u : 0x3F80u;
      uint32_t hi = (__popc(n & kb2 & hm) & 1) ? 0xBF80u : 0x3F80u;
      if (BLK == 64) {
        if ((n ^ ka) & 64) lo = 0u;
        if ((n ^ kb2) & 64) hi = 0u;
      }
      w[e] = lo | (hi << 16);
    }
    const uint32_t chunk = (uint32_t)((k0 & 63) >> 3);
    *reinterpret_cast<uint4*>(smem + OFF_H + (k0 >> 6) * ATOM + n * 128 + ((chunk ^ (n & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
  }
  // the unused rows at the end of both halves of the two slab buffers take part in the Gram product: zero them once
  if (p.pad_rows > 0) {
    const int per_half = 8 * p.pad_rows;
    for (int i = tid; i < 4 * per_half; i += THREADS) {
      const int hb = i / per_half, r = i % per_half;      // hb: buffer * 2 + half
      *reinterpret_cast<uint4*>(smem + OFF_T + (size_t)(hb >> 1) * slab_bytes + 16u * (uint32_t)((hb & 1) * 8 * p.seg_rows + 8 * raw_rows + r)) =
          make_uint4(0u, 0u, 0u, 0u);
    }
  }
  if (p.tab_smem) {
    const uint4* src = reinterpret_cast<const uint4*>(p.table);
    uint4* dst = reinterpret_cast<uint4*>(smem + (tab_base - sbase));
    for (int i = tid; i < p.dim / 4; i += THREADS) dst[i] = __ldg(src + i);
  }
  if (p.mask_smem) {
    const uint4* src = reinterpret_cast<const uint4*>(p.srcmask);
    uint4* dst = reinterpret_cast<uint4*>(smem + (msk_base - sbase));
    for (int i = tid; i < p.dim / 8; i += THREADS) dst[i] = __ldg(src + i);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *tmem_slot;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

#ifdef OQ_RQMM_TRACE
  // trace build: CTA 0 records clock64 at pipeline events, p.dbg receives [16 kinds][64 events] 64-bit stamps
#define OQ_EV(kind, idx) if (blockIdx.x == 0 && lane == 0 && (idx) < 64 && p.dbg != nullptr) reinterpret_cast<long long*>(p.dbg)[(kind) * 64 + (idx)] = clock64();
#else
#define OQ_EV(kind, idx)
#endif
  auto wait1 = [&](uint32_t b, uint32_t parity, int code) { mbar_wait(b, parity, abort_flag, p.status, code); };
  auto warp_wait = [&](uint32_t b, uint32_t parity, int code) {
    if (lane == 0) wait1(b, parity, code);
    __syncwarp();
  };
  // Position of a chunk of this CTA's chunk stream: (local slab, block of 128 coordinates inside the row).  The roles
  // walk the stream tile by tile and keep the position of the tile's first chunk; divisions by the runtime row
  // length are replaced by a few subtractions (a tile spans at most three slabs).
  const int nb = p.nb;
  auto advance = [&](int& sl, int& j, int chunks) {
    j += chunks;
    while (j >= nb) { j -= nb; ++sl; }
  };
  // local slab of the last chunk of the tile that starts at (sl0, j0) that exists
  auto tile_last_slab = [&](int sl0, int j0) {
    int sl = sl0, j = j0;
    advance(sl, j, BC - 1);
    return min(sl, nsl - 1);
  };

  if (warp == MMA_WARP) {
    // ------------------------------- MMA issuer -------------------------------
    if (lane == 0) {
      constexpr uint32_t IDESC_H = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      constexpr uint32_t IDESC_G = IDESC_H | (1u << 16);
      const uint64_t desc_h = smem_desc(sbase + OFF_H);
      const int ngram = p.seg_rows / 16;
      int next_gram = 0;
      int sl0 = 0, j0 = 0;                           // first chunk of tile i
      for (int i = 0; i < ntiles; ++i, advance(sl0, j0, BC)) {
        const int sl_last = tile_last_slab(sl0, j0);
        for (; next_gram <= sl_last; ++next_gram) {
          const int s = next_gram;
          wait1(bar(B_TFULL + (s & 1)), (uint32_t)(s >> 1) & 1u, WAIT_TFULL);
          if (s > 0) wait1(bar(B_GRAMFREE), (uint32_t)(s - 1) & 1u, WAIT_GRAMFREE);
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          OQ_EV(3, s)
          const uint32_t tb = t_base + (uint32_t)(s & 1) * slab_bytes;
          for (int g = 0; g < ngram; ++g) {
            const uint64_t dsc = mn_major_desc(tb + 2048u * (uint32_t)g, 128u * (uint32_t)p.seg_rows, 1024u);
            const uint32_t acc = g > 0 ? 1u : 0u;
            asm volatile(
                "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                ::"r"(tmem + GRAM_COL), "l"(dsc), "l"(dsc), "r"(IDESC_G), "r"(acc) : "memory");
          }
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar(B_GRAMRDY)) : "memory");
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar(B_TDONE + (s & 1))) : "memory");
        }
        const uint32_t slot = (uint32_t)i % 3u, use = (uint32_t)i / 3u;
        if (use > 0u) wait1(bar(B_ACCFREE + slot), (use - 1u) & 1u, WAIT_ACCFREE);
        OQ_EV(4, i)
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          wait1(bar(B_AFULL + half), (uint32_t)i & 1u, WAIT_AFULL);
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
          for (int k4 = 4 * half; k4 < 4 * half + 4; ++k4) {
            const uint64_t da = mn_major_desc(a_base + 4096u * (uint32_t)k4, 1024u, 2048u);
            const uint64_t db = desc_h + (uint64_t)((k4 >> 2) * (ATOM >> 4)) + 2 * (k4 & 3);
            const uint32_t acc = k4 > 0 ? 1u : 0u;
            asm volatile(
                "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                ::"r"(tmem + slot * 128u), "l"(da), "l"(db), "r"(IDESC_H), "r"(acc) : "memory");
          }
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar(B_AFREE + half)) : "memory");
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar(B_ACCRDY + slot)) : "memory");
        OQ_EV(5, i)
      }
    }
  } else if (warp >= FE_WARP0) {
    // ------------------------------- front end: global rows -> transposed slab -> operand tiles -------------------------------
    const int fw = warp - FE_WARP0;
    // as loader: lane = (fragment row, 8 coordinates); as provider of a row address: matrix lane / 8, transposed row lane % 8
    const int frow = lane >> 2;
    const int tok = frow % TOK, h = frow / TOK;               // its token, its 32-coordinate sub-window
    const int c8 = (lane & 3) * 8;
    const int cb_addr = ((lane & 7) >> 1) * 8 + 2 * (lane >> 3) + (lane & 1);
    const int wrow = window_row(cb_addr);
    const int nwin = p.dim / (32 * SUBS);                     // windows of 32 * SUBS coordinates per row
    const int coord_thr = fw * 32 * SUBS + h * 32 + c8;       // this lane's coordinates in the warp's first window
    // as gatherer: piece column mm of the tile (per pass), coordinates k = 8 kg + kr with kg in [4 kq, 4 kq + 4)
    const int gw = fw & 3, kq = fw >> 2, half = kq >> 1;
    const int sub = lane % SUBS, kr = (lane / SUBS) & 7, grp = lane / (8 * SUBS);
    const uint32_t tab_thr = (uint32_t)kr * 16u + 4u * (uint32_t)kq;     // + j * 128: 4 consecutive entries
    uint32_t r[WIN_SLOTS][4];
    auto load_slab = [&](int sl) {        // the warp's windows fw, fw + FE_WARPS, ... of slab sl -> registers
      const int row = ((int)blockIdx.x + sl * stride) * TOK + tok;
      const bool row_ok = sl < nsl && row < p.rows;
      const unsigned char* src = p.X + ((size_t)(row_ok ? row : 0) * p.ldx + coord_thr) * 2;
#pragma unroll
      for (int u = 0; u < WIN_SLOTS; ++u) {
        r[u][0] = r[u][1] = r[u][2] = r[u][3] = 0u;
        if (row_ok && fw + u * FE_WARPS < nwin)
          asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r[u][0]), "=r"(r[u][1]), "=r"(r[u][2]), "=r"(r[u][3])
                       : "l"(src + (size_t)u * (FE_WARPS * 64 * SUBS)));
      }
    };
    // Rows reach the registers through L2: one thread asks for the rows of a slab two slabs before they are loaded, so
    // that the loads (issued right after a slab has been stored, used one slab later) are short when the next fence of
    // this thread has to wait for them.
    auto prefetch_slab = [&](int sl) {
      if (sl >= nsl) return;
      const int row0 = ((int)blockIdx.x + sl * stride) * TOK;
      for (int rr = 0; rr < TOK && row0 + rr < p.rows; ++rr)
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p.X + (size_t)(row0 + rr) * p.ldx * 2), "r"(2u * (uint32_t)p.dim) : "memory");
    };
    if (fw == 1 && lane == 0) {
      prefetch_slab(1);
      prefetch_slab(2);
    }
    load_slab(0);
    int next_tile = 0;
    int sl0 = 0, j0 = 0;                             // first chunk of tile next_tile
    for (int sl = 0; sl < nsl; ++sl) {
      const uint32_t tb = t_base + (uint32_t)(sl & 1) * slab_bytes;
      // the buffer held slab sl - 2: its Gram product must have been read by the tensor cores, and every front-end warp
      // must have finished the tiles that gathered from it (they were gathered before this point of the program)
      if (sl >= 2) warp_wait(bar(B_TDONE + (sl & 1)), (uint32_t)((sl >> 1) - 1) & 1u, WAIT_TDONE);
      if (sl >= 1) asm volatile("bar.sync 2, %0;" ::"n"(FE_WARPS * 32) : "memory");
      if (fw == 0) { OQ_EV(0, sl) }
      // sign flips first (the mask loads of all windows are in flight together), then the transposing stores
#pragma unroll
      for (int u = 0; u < WIN_SLOTS; ++u) {
        if (fw + u * FE_WARPS < nwin) {
          const int coord = coord_thr + u * (FE_WARPS * 32 * SUBS);
          uint4 m;
          if (p.mask_smem)
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(m.x), "=r"(m.y), "=r"(m.z), "=r"(m.w) : "r"(msk_base + 2u * (uint32_t)coord));
          else
            m = __ldg(reinterpret_cast<const uint4*>(p.srcmask + (coord >> 1)));
          r[u][0] ^= m.x; r[u][1] ^= m.y; r[u][2] ^= m.z; r[u][3] ^= m.w;
        }
      }
#pragma unroll
      for (int u = 0; u < WIN_SLOTS; ++u) {
        if (fw + u * FE_WARPS < nwin) {
          int lin = (fw + u * FE_WARPS) * 32 + wrow;          // row of the slab buffer before padding
          if (lin >= 8 * raw_rows) lin += 8 * p.pad_rows;
          asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1,%2,%3,%4};"
                       ::"r"(tb + 16u * (uint32_t)lin), "r"(r[u][0]), "r"(r[u][1]), "r"(r[u][2]), "r"(r[u][3]) : "memory");
        }
      }
      // the tensor cores read the slab buffer (Gram product): make this thread's writes visible to the async proxy
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("bar.sync 3, %0;" ::"n"(FE_WARPS * 32) : "memory");
      if (fw == 0) {
        OQ_EV(2, sl)
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar(B_TFULL + (sl & 1))) : "memory");
      }
      if (fw == 1 && lane == 0) prefetch_slab(sl + 3);
      load_slab(sl + 1);                               // from L2; used when the next slab is stored
      // the tiles that this slab completes
      while (next_tile < ntiles && tile_last_slab(sl0, j0) == sl) {
        const int i = next_tile;
        if (fw == 0) { OQ_EV(8, i) }
        if (i > 0) warp_wait(bar(B_AFREE + half), (uint32_t)(i - 1) & 1u, WAIT_AFREE);
#pragma unroll
        for (int ps = 0; ps < PASSES; ++ps) {
          const int mm = ps * (4 * GPW) + gw * GPW + grp;
          int s2 = sl0, j = j0;
          advance(s2, j, mm * SUBS + sub);
          if (s2 < nsl) {
            uint32_t off[4];
            if (p.tab_smem) {
              asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(off[0]), "=r"(off[1]), "=r"(off[2]), "=r"(off[3])
                           : "r"(tab_base + 4u * ((uint32_t)j * 128u + tab_thr)));
            } else {
              const uint4 o = __ldg(reinterpret_cast<const uint4*>(p.table + (uint32_t)j * 128u + tab_thr));
              off[0] = o.x; off[1] = o.y; off[2] = o.z; off[3] = o.w;
            }
            const uint32_t srcb = t_base + (uint32_t)(s2 & 1) * slab_bytes;
            // operand tile: [coordinates k / 8][2 halves of the 128 rows][k % 8][8 pieces of 16 bytes, XOR-ed with k % 8]
            const uint32_t dst = a_base + (uint32_t)(4 * kq) * 2048u + (uint32_t)(mm >> 3) * 1024u + (uint32_t)kr * 128u +
                                 (uint32_t)(((mm & 7) ^ kr) << 4) + (uint32_t)sub * CB;
            if constexpr (TOK == 8) {
              uint4 c[4];
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(c[kk].x), "=r"(c[kk].y), "=r"(c[kk].z), "=r"(c[kk].w) : "r"(srcb + off[kk]));
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(dst + 2048u * kk), "r"(c[kk].x), "r"(c[kk].y), "r"(c[kk].z), "r"(c[kk].w) : "memory");
            } else if constexpr (TOK == 4) {
              uint2 c[4];
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(c[kk].x), "=r"(c[kk].y) : "r"(srcb + off[kk]));
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) asm volatile("st.shared.v2.u32 [%0], {%1,%2};" ::"r"(dst + 2048u * kk), "r"(c[kk].x), "r"(c[kk].y) : "memory");
            } else {
              uint32_t c[4];
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(c[kk]) : "r"(srcb + off[kk]));
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) asm volatile("st.shared.u32 [%0], %1;" ::"r"(dst + 2048u * kk), "r"(c[kk]) : "memory");
            }
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar(B_AFULL + half)) : "memory");
        if (fw == 0) { OQ_EV(9, i) }
        ++next_tile;
        advance(sl0, j0, BC);
      }
    }
  } else {
    // ------------------------------- compute warps -------------------------------
    const int q = warp & 3, colpart = warp >> 2;
    const int n = q * 32 + lane;                     // row of the tile = tensor-memory lane = pair
    const int t = n % TOK;
    const Poly2<(1 << (BITS - 1)) - 1> poly(p.poly);
    constexpr float blk_f = (float)BLK;
    const float inv_sqrt_h = rsqrtf(blk_f);
    const uint32_t tmem_thr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(colpart * (32 * PIECES));
    int next_norm = 0;
    int sl0 = 0, j0 = 0;                             // first chunk of tile i
    for (int i = 0; i < ntiles; ++i, advance(sl0, j0, BC)) {
      int sl = sl0, j = j0;
      advance(sl, j, n / TOK);
      const int row = ((int)blockIdx.x + sl * stride) * TOK + t;
      const bool valid = sl < nsl && row < p.rows;
      const int sl_last = tile_last_slab(sl0, j0);
      // norms of the slabs that this tile is the first to touch: the diagonal of the Gram matrix, added up over the
      // 16 row groups in a fixed order (4 per lane quarter by shuffles, the 4 quarters by every reader)
      for (; next_norm <= sl_last; ++next_norm) {
        const int s = next_norm;
        float* part = s_part + (s & (NORM_RING - 1)) * 32;
        if (colpart == 0) {
          warp_wait(bar(B_GRAMRDY), (uint32_t)s & 1u, WAIT_GRAM);
          if (warp == 0) { OQ_EV(6, s) }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          uint32_t v[32];
          tmem_load32(tmem + ((uint32_t)(q * 32) << 16) + GRAM_COL + (uint32_t)q * 32u, v);
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar(B_GRAMFREE)) : "memory");
          // entry (lane, lane) of the warp's 32 x 32 diagonal block
#pragma unroll
          for (int hb = 16; hb >= 1; hb >>= 1) {
            const bool up = (lane & hb) != 0;
#pragma unroll
            for (int e = 0; e < hb; ++e) v[e] = up ? v[e + hb] : v[e];
          }
          float dsum = __uint_as_float(v[0]);
          dsum += __shfl_xor_sync(0xffffffffu, dsum, 8);
          dsum += __shfl_xor_sync(0xffffffffu, dsum, 16);
          if (lane < 8) part[q * 8 + lane] = dsum;
        }
        asm volatile("bar.sync 1, %0;" ::"n"(COMPUTE_WARPS * 32) : "memory");
        if (warp == 0 && lane < TOK) {
          float tot = 0.f;
#pragma unroll
          for (int qq = 0; qq < 4; ++qq)
#pragma unroll
            for (int hh = 0; hh < SUBS; ++hh) tot += part[qq * 8 + hh * TOK + lane];
          const float nrm = sqrtf(tot);
          const int orow = ((int)blockIdx.x + s * stride) * TOK + lane;
          if (orow < p.rows) {
            if (p.bf16_norm) reinterpret_cast<__nv_bfloat16*>(p.out_norm)[orow] = __float2bfloat16_rn(nrm);
            else reinterpret_cast<float*>(p.out_norm)[orow] = nrm;
          }
          OQ_EV(7, s)
        }
      }
      float tot = 0.f;
      {
        const float* part = s_part + (min(sl, nsl - 1) & (NORM_RING - 1)) * 32;
#pragma unroll
        for (int qq = 0; qq < 4; ++qq)
#pragma unroll
          for (int hh = 0; hh < SUBS; ++hh) tot += part[qq * 8 + hh * TOK + t];
      }
      const float s = sqrtf(tot);
      // |z| / (sqrt(h) (s + eps) clamp) with z the unnormalised block transform
      const float kappa = 1.0f / (sqrtf(blk_f) * (s + 1e-10f) * p.poly.clamp);
      const uint32_t slot = (uint32_t)i % 3u;
      warp_wait(bar(B_ACCRDY + slot), ((uint32_t)i / 3u) & 1u, WAIT_ACC);
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (warp == 0) { OQ_EV(10, i) }
#pragma unroll 1
      for (int piece = 0; piece < PIECES; ++piece) {
        uint32_t vb[32];
        tmem_load32(tmem_thr + slot * 128u + 32u * piece, vb);
        if (piece == PIECES - 1) {
          // the accumulator may be overwritten as soon as the compute warps have read it
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar(B_ACCFREE + slot)) : "memory");
        }
        if constexpr (BLK == 256) {
          // H_256 = [[H_128, H_128], [H_128, -H_128]]: the two halves of a block sit TOK rows apart, in the same warp
          const float sg = (lane & TOK) ? -1.f : 1.f;
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const float mine = __uint_as_float(vb[e]);
            const float other = __shfl_xor_sync(0xffffffffu, mine, TOK);
            vb[e] = __float_as_uint(fmaf(mine, sg, other));      // low half: mine + other; high half: other - mine
          }
        }
        if (valid) {
          float v[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(vb[e]);
          const int cq = colpart * PIECES + piece;
#ifndef OQ_RQMM_TRACE
          if (p.dbg != nullptr) {
            float* d = p.dbg + (size_t)row * p.dim + j * 128 + cq * 32;
#pragma unroll
            for (int e = 0; e < 32; ++e) d[e] = v[e] * inv_sqrt_h;
          }
#endif
          uint32_t words[BITS];
          pack32<BITS>(v, kappa, poly, words);
          uint32_t* dst = p.out_idx + (size_t)row * p.pitch_words + (j * 4 + cq) * BITS;
          if constexpr (BITS == 4) *reinterpret_cast<uint4*>(dst) = make_uint4(words[0], words[1], words[2], words[3]);
          else if constexpr (BITS == 2) *reinterpret_cast<uint2*>(dst) = make_uint2(words[0], words[1]);
          else {
#pragma unroll
            for (int c = 0; c < BITS; ++c) dst[c] = words[c];
          }
        }
      }
      if (warp == 0) { OQ_EV(11, i) }
    }
  }
  __syncwarp();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == MMA_WARP) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(TMEM_COLS) : "memory");
  }
}

}  // namespace oq
