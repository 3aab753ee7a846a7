// Fused rotate+quantize kernel for Hadamard blocks of 128 with the block transform on the tensor cores.
//
// The rotation of Eq. 7 / Eq. 4 is  z = blkdiag(H_128 D_j) P x : a gather, a sign flip and, per block of 128
// rotated coordinates, a product with the 128 x 128 matrix of +-1.  Butterflies in registers cost ~6
// instructions per coordinate and 64 registers per lane; here the signed, permuted coordinates are written
// as bf16 into a shared-memory operand tile instead and one tcgen05.mma per 16 coordinates multiplies 128
// (token, block) pairs by H_128 (entries +-1 are exact in bf16, the inputs are bf16 already, the sums are
// accumulated in fp32 in tensor memory).  The rest of the path reads tensor memory twice: once for the row
// norms (||H x'||^2 = 128 ||x||^2), once for the level search and packing.
//
// Data flow per CTA (persistent over groups of T consecutive rows, T a power of two <= 16):
//   copy      a bulk copy per row (global -> shared, 16-byte aligned row pitch); the rows of the next group are
//             requested by whichever warp is the last to finish the
//             shared-memory loads of this group's last tile;
//   gather    512 threads; a thread owns one of the 128 (token, block) pairs of a tile and 32 of its rotated
//             coordinates: table look-up, 16-bit shared-memory load, pair-wise sign mask, 16-byte store into
//             the K-major 128-byte-swizzled operand tile (two tile buffers);
//   mma       the warp that finishes a tile last issues 8 x tcgen05.mma (M = 128 pairs, N = 128 coordinates,
//             K = 16) into the tile's own 128-column accumulator (a group's whole rotated output stays in
//             tensor memory) and commits to a barrier;
//   pass 1    every thread reads its 32 columns of every tile, sums squares; partial sums meet in shared
//             memory in a fixed order (deterministic norms);
//   pass 2    reads the same columns again, finds the levels with the polynomial of QuantPoly, packs, stores.
//             It is fused with the gather of the NEXT group, 8 coordinates at a time: the level search keeps
//             the FMA and ALU pipes busy while the gather waits for shared memory.
// Every wait is bounded and reports to a status word.
#pragma once
#include <cuda_bf16.h>

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
  int groups;               // number of T-row groups
  int tshift;               // log2(T)
  int ntiles;               // tiles of 128 (token, block) pairs per group (1..4)
  int tmem_cols;            // 128 * ntiles rounded up to a power of two
  int bf16_norm;            // 1: norms stored as bf16 (weights), 0: fp32 (activations)
  int* status;
};

namespace rqtc {
constexpr int H = 128;
constexpr int THREADS = 512;                      // 16 warps: 4 lane quarters x 4 column quarters of a tile
constexpr int WARPS = THREADS / 32;
constexpr uint32_t ATOM = 128 * 128;              // 128 rows x 64 bf16: one swizzle atom column of a tile
constexpr uint32_t TILE = 2 * ATOM;               // 128 rows x 128 bf16
constexpr uint32_t OFF_H = 0, OFF_A = TILE, OFF_ROWS = 3 * TILE;
constexpr int TAB_PITCH = 132, MSK_PITCH = 68;    // words per block of the shared-memory table copies
enum { WAIT_ROWS = 11, WAIT_ACC = 13, WAIT_DRAIN = 14 };
__host__ __device__ constexpr uint32_t row_pitch_bytes(int dim) { return 2u * (uint32_t)dim + 16u; }
}  // namespace rqtc


template <int BITS, bool TAB_SMEM>
__global__ void __launch_bounds__(rqtc::THREADS, 1) rq_tc_kernel(const RqTcParams p) {
  using namespace rqtc;
  extern __shared__ unsigned char smem_dyn[];
  // 1024-byte alignment for the swizzled tiles, computed on the shared-window address so that the compiler keeps
  // treating everything below as shared memory (32-bit addresses, no generic-pointer arithmetic)
  unsigned char* smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  const int T = 1 << p.tshift;
  const uint32_t pitch = row_pitch_bytes(p.dim);
  unsigned char* rows_s = smem + OFF_ROWS;
  unsigned char* after_rows = rows_s + (size_t)T * pitch;
  // copies of the offset and sign-mask tables (TAB_SMEM): the 128 / 64 words of a block are followed by 4 words
  // of padding, so that the four blocks a warp reads at once sit in different banks
  uint32_t* s_table = reinterpret_cast<uint32_t*>(after_rows);                                 // [dim/128][TAB_PITCH]
  uint32_t* s_mask = s_table + (TAB_SMEM ? (p.dim / H) * TAB_PITCH : 0);                       // [dim/128][MSK_PITCH]
  float* s_part = reinterpret_cast<float*>(s_mask + (TAB_SMEM ? (p.dim / H) * MSK_PITCH : 0)); // [16 warps][16]
  uint64_t* bars = reinterpret_cast<uint64_t*>(s_part + WARPS * 16);                           // rows_full, acc_ready[4]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 5);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  // arrival counters (never reset; the warp that brings one to a multiple of 16 acts): [0], [1] operand tile
  // buffers finished, [2] row buffer no longer needed, [3] row groups requested so far
  unsigned int* s_cnt = reinterpret_cast<unsigned int*>(tmem_slot + 2);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rows_full = smem_u32(bars), acc_ready0 = smem_u32(bars + 1);

  const int kblocks = p.dim / H;
  const uint32_t row_bytes = 2u * (uint32_t)p.dim;
  const int stride = (int)gridDim.x;
  // Bulk copies of the rows of group `grp` into the row buffer.
  auto request_rows = [&](int grp) {
    const int row0 = grp * T;
    const int nvalid = min(T, p.rows - row0);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(rows_full), "r"(row_bytes * (uint32_t)nvalid) : "memory");
    for (int r = 0; r < nvalid; ++r) {
      const unsigned char* src = p.X + (size_t)(row0 + r) * p.ldx * 2;
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(smem_u32(rows_s + (size_t)r * pitch)), "l"(src), "r"(row_bytes), "r"(rows_full) : "memory");
    }
    s_cnt[3] += 1u;
  };
  if (tid == 0) {
    mbar_init(rows_full, 1);
    for (int i = 0; i < 4; ++i) mbar_init(acc_ready0 + 8 * i, 1);                   // tcgen05.commit
    *abort_flag = 0;
    for (int i = 0; i < 4; ++i) s_cnt[i] = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    // the first rows travel while the CTA builds its tables
    if ((int)blockIdx.x < p.groups) request_rows(blockIdx.x);
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // H_128 as the B operand: B[n][k] = (-1)^popcount(n & k), K-major, 128-byte swizzle (the matrix is symmetric)
  for (int c = tid; c < 128 * 16; c += THREADS) {
    const int n = c >> 4, k0 = (c & 15) * 8;
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const uint32_t lo = (__popc(n & (k0 + 2 * e)) & 1) ? 0xBF80u : 0x3F80u;
      const uint32_t hi = (__popc(n & (k0 + 2 * e + 1)) & 1) ? 0xBF80u : 0x3F80u;
      w[e] = lo | (hi << 16);
    }
    const uint32_t chunk = (uint32_t)((k0 & 63) >> 3);
    *reinterpret_cast<uint4*>(smem + OFF_H + (k0 >> 6) * ATOM + n * 128 + ((chunk ^ (n & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
  }
  for (int i = tid; i < WARPS * 16; i += THREADS) s_part[i] = 0.f;
  if (TAB_SMEM) {
    for (int i = tid; i < p.dim; i += THREADS) s_table[(i >> 7) * TAB_PITCH + (i & 127)] = __ldg(p.offset + i);
    for (int i = tid; i < p.dim / 2; i += THREADS) s_mask[(i >> 6) * MSK_PITCH + (i & 63)] = __ldg(p.posmask + i);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *tmem_slot;


  const int q = warp & 3, kq = warp >> 2;          // tensor-memory lane quarter, column quarter
  const int r = q * 32 + lane;                     // row of the operand tile = tensor-memory lane
  // (token, block) pair of that row.  For T = 16 bits 3 and 5 of the row number trade places, so that a warp
  // holds 8 tokens x 4 blocks: rows are 16-byte aligned in shared memory, tokens t and t + 8 share banks.
  const int rp = (p.tshift == 4) ? ((r & ~0x28) | ((r & 8) << 2) | ((r & 32) >> 2)) : r;
  const int t = rp & (T - 1);
  const int j0 = rp >> p.tshift, jstep = H >> p.tshift;
  const unsigned char* rowbytes = rows_s + (size_t)t * pitch;
  const uint32_t a_row = (uint32_t)r * 128u;
  const uint32_t sw = (uint32_t)(r & 7);
  const Poly2<(1 << (BITS - 1)) - 1> poly(p.poly);
  const float inv_sqrt_h = rsqrtf((float)H);
  const uint32_t tmem_thr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(kq * 32);
  const uint64_t desc_h = smem_desc(smem_u32(smem + OFF_H));

  // ---- pieces of the gather of tile i: offsets of the thread's 32 coordinates ...
  auto gather_offsets = [&](int i, uint32_t (&h)[32]) {
    const int j = j0 + i * jstep;
    const uint4* tab = reinterpret_cast<const uint4*>(TAB_SMEM ? s_table + j * TAB_PITCH + kq * 32 : p.offset + j * H + kq * 32);
#pragma unroll
    for (int e4 = 0; e4 < 8; ++e4) {
      const uint4 o = TAB_SMEM ? tab[e4] : __ldg(tab + e4);
      h[4 * e4] = o.x; h[4 * e4 + 1] = o.y; h[4 * e4 + 2] = o.z; h[4 * e4 + 3] = o.w;
    }
  };
  // ... the 16-bit loads of chunk c (8 coordinates), in place of their offsets ...
  auto gather_chunk_loads = [&](int c, uint32_t (&h)[32]) {
#pragma unroll
    for (int e = 0; e < 8; ++e) h[8 * c + e] = *reinterpret_cast<const unsigned short*>(rowbytes + h[8 * c + e]);
  };
  // ... and the sign masks, the pairing and the 16-byte store of chunk c into the swizzled tile.
  auto gather_chunk_store = [&](int i, int c, const uint32_t (&h)[32]) {
    const int j = j0 + i * jstep;
    const uint4* msk = reinterpret_cast<const uint4*>(TAB_SMEM ? s_mask + j * MSK_PITCH + kq * 16 : p.posmask + j * (H / 2) + kq * 16);
    const uint4 m = TAB_SMEM ? msk[c] : __ldg(msk + c);
    uint4 o;
    o.x = prmt(h[8 * c], h[8 * c + 1], 0x5410u) ^ m.x;
    o.y = prmt(h[8 * c + 2], h[8 * c + 3], 0x5410u) ^ m.y;
    o.z = prmt(h[8 * c + 4], h[8 * c + 5], 0x5410u) ^ m.z;
    o.w = prmt(h[8 * c + 6], h[8 * c + 7], 0x5410u) ^ m.w;
    unsigned char* abuf = smem + OFF_A + (i & 1) * TILE + (kq >> 1) * ATOM + a_row;
    const uint32_t chunk = (uint32_t)((kq & 1) * 4 + c);
    *reinterpret_cast<uint4*>(abuf + ((chunk ^ sw) << 4)) = o;
  };
  auto warp_wait = [&](uint32_t bar, uint32_t parity, int code) {
    if (lane == 0) mbar_wait(bar, parity, abort_flag, p.status, code);
    __syncwarp();
  };
  // This warp has taken everything it needs from the row buffer for group `grp`; the last warp to say so
  // requests the rows of the CTA's next group.
  auto rows_done = [&](int grp) {
    __syncwarp();
    if (lane == 0) {
      __threadfence_block();
      const unsigned int old = atomicAdd(&s_cnt[2], 1u);
      if ((old & (WARPS - 1)) == WARPS - 1) {
        const int nxt = grp + stride;
        if (nxt < p.groups && !*abort_flag) request_rows(nxt);
      }
    }
  };
  // This warp has written its part of operand tile i and has read what it needed from accumulator i; the last
  // warp to say so multiplies the tile by H_128 into accumulator i and commits to acc_ready[i].
  auto tile_done = [&](int i) {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (lane == 0) {
      __threadfence_block();
      const unsigned int old = atomicAdd(&s_cnt[i & 1], 1u);
      if ((old & (WARPS - 1)) == WARPS - 1) {
        __threadfence_block();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        const uint32_t a_addr = smem_u32(smem + OFF_A + (i & 1) * TILE);
#pragma unroll
        for (int k4 = 0; k4 < 8; ++k4) {
          const uint64_t da = smem_desc(a_addr + (k4 >> 2) * ATOM) + 2 * (k4 & 3);
          const uint64_t db = desc_h + (uint64_t)((k4 >> 2) * (ATOM >> 4)) + 2 * (k4 & 3);
          const uint32_t acc = k4 > 0 ? 1u : 0u;
          asm volatile(
              "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
              " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
              ::"r"(tmem + (uint32_t)i * 128u), "l"(da), "l"(db), "r"(IDESC), "r"(acc) : "memory");
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(acc_ready0 + 8 * i) : "memory");
      }
    }
  };

  // prologue: the tiles of the CTA's first group
  if ((int)blockIdx.x < p.groups) {
    warp_wait(rows_full, 0u, WAIT_ROWS);
    for (int i = 0; i < p.ntiles; ++i) {
      if (i >= 2) warp_wait(acc_ready0 + 8 * (i - 2), 0u, WAIT_ACC);   // the tile buffer was read by the MMAs of tile i - 2
      if (j0 + i * jstep < kblocks) {
        uint32_t h[32];
        gather_offsets(i, h);
#pragma unroll
        for (int c = 0; c < 4; ++c) gather_chunk_loads(c, h);
#pragma unroll
        for (int c = 0; c < 4; ++c) gather_chunk_store(i, c, h);
      }
      if (i == p.ntiles - 1) rows_done(blockIdx.x);
      tile_done(i);
    }
  }
  int it = 0;
  for (int grp = blockIdx.x; grp < p.groups; grp += stride, ++it) {
    const int row0 = grp * T;
    const uint32_t par = (uint32_t)it & 1u;
    // ---------------- pass 1: squared norms from the rotated values ----------------
    float ssq = 0.f;
    for (int i = 0; i < p.ntiles; ++i) {
      warp_wait(acc_ready0 + 8 * i, par, WAIT_ACC);
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      uint32_t v[32];
      tmem_load32(tmem_thr + (uint32_t)i * 128u, v);
      if (j0 + i * jstep < kblocks) {
        unsigned long long acc2 = 0ull;
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const unsigned long long x2 = pack2(__uint_as_float(v[2 * e]), __uint_as_float(v[2 * e + 1]));
          acc2 = fma2(x2, x2, acc2);
        }
        float a0, a1;
        unpack2(acc2, a0, a1);
        ssq += a0 + a1;
      }
    }
    // lanes of the warp that hold the same token add up; the lowest of them publishes the warp's partial sum
    bool leader = true;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
      const float other = __shfl_xor_sync(0xffffffffu, ssq, o);
      const int ot = __shfl_xor_sync(0xffffffffu, t, o);
      if (ot == t) {
        ssq += other;
        if (lane & o) leader = false;
      }
    }
    if (leader) s_part[warp * 16 + t] = ssq;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < WARPS; ++w) tot += s_part[w * 16 + t];
    const float s = sqrtf(tot * (1.0f / (float)H));
    const bool row_ok = row0 + t < p.rows;
    // warps 0 and 1 (lane quarters 0 and 1, column quarter 0) hold every token between them
    if (warp == ((p.tshift == 4) ? (t >> 3) : 0) && leader && row_ok) {
      if (p.bf16_norm) reinterpret_cast<__nv_bfloat16*>(p.out_norm)[row0 + t] = __float2bfloat16_rn(s);
      else reinterpret_cast<float*>(p.out_norm)[row0 + t] = s;
    }
    // ---------------- pass 2 of this group, fused with the gather of the CTA's next group ----------------
    // |z| / (sqrt(h) (s + eps) clamp) with z the unnormalised block transform
    const float kappa = 1.0f / (sqrtf((float)H) * (s + 1e-10f) * p.poly.clamp);
    const int nxt = grp + stride;
    const bool has_next = nxt < p.groups;
    const uint32_t npar = par ^ 1u;
    if (has_next) warp_wait(rows_full, npar, WAIT_ROWS);
    for (int i = 0; i < p.ntiles; ++i) {
      const int j = j0 + i * jstep;
      const bool pair_ok = j < kblocks;
      const bool gat = has_next && pair_ok;
      if (has_next && i >= 2) warp_wait(acc_ready0 + 8 * (i - 2), npar, WAIT_ACC);
      uint32_t h[32];
      if (gat) {
        gather_offsets(i, h);
        gather_chunk_loads(0, h);
        gather_chunk_loads(1, h);
      }
      uint32_t vb[32];
      tmem_load32(tmem_thr + (uint32_t)i * 128u, vb);
      float v[32];
#pragma unroll
      for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(vb[e]);
      const bool out_ok = pair_ok && row_ok;
      if (p.dbg != nullptr && out_ok) {
        float* d = p.dbg + (size_t)(row0 + t) * p.dim + j * H + kq * 32;
#pragma unroll
        for (int e = 0; e < 32; ++e) d[e] = v[e] * inv_sqrt_h;
      }
      uint32_t words[BITS];
      if constexpr (BITS == 4) {
        // The gather sits in the first half of the tile: chunks 2 and 3 are loaded before word 0 is packed and
        // stored before word 1, so every shared-memory load has a level search between its issue and its use,
        // and the tile is handed over (and its MMAs start) while words 1 to 3 are still being packed.
        if (gat) {
          gather_chunk_loads(2, h);
          gather_chunk_loads(3, h);
          gather_chunk_store(i, 0, h);
          gather_chunk_store(i, 1, h);
        }
        words[0] = pack8_4bit(v, kappa, poly);
        if (gat) {
          gather_chunk_store(i, 2, h);
          gather_chunk_store(i, 3, h);
        }
        if (has_next) {
          if (i == p.ntiles - 1) rows_done(nxt);
          tile_done(i);
        }
#pragma unroll
        for (int c = 1; c < 4; ++c) words[c] = pack8_4bit(v + 8 * c, kappa, poly);
      } else {
        if (gat) {
          gather_chunk_loads(2, h);
          gather_chunk_loads(3, h);
        }
        pack32<BITS>(v, kappa, poly, words);
        if (gat) {
#pragma unroll
          for (int c = 0; c < 4; ++c) gather_chunk_store(i, c, h);
        }
        if (has_next) {
          if (i == p.ntiles - 1) rows_done(nxt);
          tile_done(i);
        }
      }
      if (out_ok) {
        uint32_t* dst = p.out_idx + (size_t)(row0 + t) * p.pitch_words + (j * (H / 32) + kq) * BITS;
        if constexpr (BITS == 4) *reinterpret_cast<uint4*>(dst) = make_uint4(words[0], words[1], words[2], words[3]);
        else if constexpr (BITS == 2) *reinterpret_cast<uint2*>(dst) = make_uint2(words[0], words[1]);
        else {
#pragma unroll
          for (int c = 0; c < BITS; ++c) dst[c] = words[c];
        }
      }
    }
  }
  __syncwarp();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  // after a wait gave up somewhere, a requested copy may still be in flight: let it land before the CTA ends
  if (tid == 0 && *abort_flag && s_cnt[3] > 0u) mbar_wait(rows_full, (s_cnt[3] - 1u) & 1u, abort_flag, p.status, WAIT_DRAIN);
  if (warp == 0) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(p.tmem_cols) : "memory");
  }
}

}  // namespace oq
