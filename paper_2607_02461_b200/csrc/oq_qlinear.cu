// Codebook-decode GEMM:  Y[n][i] = s_n * r'_i * sum_k C_a[idxA[n][k]] * C_w[idxW[i][k]]
// (the product W^' x^' of Sec. 4.3 with the magnitudes of Eq. 6 and Eq. 8 applied in the epilogue).
//
// Packed indices are fetched from global memory into registers (one stage ahead), decoded to bf16 levels
// with byte-permute table look-ups, written into shared memory in the tensor core's K-major
// 128-byte-swizzled layout, and contracted with tcgen05.mma.cta_group::2 (fp32 accumulators in tensor
// memory, two SMs per 256 x 256 tile).  Every device-side wait is bounded and reports to a status word.
#include <cuda_bf16.h>

#include "oq_internal.h"
#include "oq_sm100.cuh"

namespace oq {

namespace {

constexpr int BK = 64;                  // coordinates per swizzle atom: 64 bf16 = one 128-byte swizzled row
constexpr int DECODE_THREADS = 512;    // 16 decoding warps per CTA
constexpr int TMEM_COLS = 512;         // two 128 x 256 fp32 accumulators per CTA

// Byte tables of the positive levels: lo/hi bytes of bf16(c_j), j = magnitude rank.
struct Tables {
  uint32_t lo0, lo1, hi0, hi1;
};
__device__ __forceinline__ Tables make_tables(const CodebookParams& cb) {
  const int M = (1 << cb.bits) >> 1;
  Tables t = {0u, 0u, 0u, 0u};
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint32_t v = j < M ? cb.level_bf16[M + j] : 0u;
    if (j < 4) {
      t.lo0 |= (v & 0xFFu) << (8 * j);
      t.hi0 |= (v >> 8) << (8 * j);
    } else {
      t.lo1 |= (v & 0xFFu) << (8 * (j - 4));
      t.hi1 |= (v >> 8) << (8 * (j - 4));
    }
  }
  return t;
}

// Decodes 32 consecutive coordinates (BITS words of one packed row) into four 16-byte chunks of bf16.
// Raw packed words of 32 coordinates of one row (BITS words), fetched ahead of their use.
template <int BITS>
struct Raw {
  uint32_t w[BITS];
};
template <int BITS>
__device__ __forceinline__ Raw<BITS> load_raw(const uint32_t* __restrict__ src) {
  Raw<BITS> r;
  if (BITS == 4) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(src));
    r.w[0] = v.x; r.w[1] = v.y; r.w[2] = v.z; r.w[BITS - 1] = v.w;
  } else if (BITS == 3) {
    r.w[0] = __ldg(src); r.w[1] = __ldg(src + 1); r.w[2] = __ldg(src + 2);
  } else {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(src));
    r.w[0] = v.x; r.w[1] = v.y;
  }
  return r;
}

// The 2 * BITS contiguous words of 64 coordinates of one row, as two 32-coordinate pieces.
template <int BITS>
__device__ __forceinline__ void load_raw64(const uint32_t* __restrict__ src, Raw<BITS>& a, Raw<BITS>& b) {
  if (BITS == 4) {          // 32 bytes, 16-byte aligned
    a = load_raw<BITS>(src);
    b = load_raw<BITS>(src + 4);
  } else if (BITS == 3) {   // 24 bytes, 8-byte aligned
    const uint2 v0 = __ldg(reinterpret_cast<const uint2*>(src));
    const uint2 v1 = __ldg(reinterpret_cast<const uint2*>(src) + 1);
    const uint2 v2 = __ldg(reinterpret_cast<const uint2*>(src) + 2);
    a.w[0] = v0.x; a.w[1] = v0.y; a.w[BITS - 1] = v1.x;
    b.w[0] = v1.y; b.w[1] = v2.x; b.w[BITS - 1] = v2.y;
  } else {                  // 16 bytes, 16-byte aligned
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(src));
    a.w[0] = v.x; a.w[1] = v.y;
    b.w[0] = v.z; b.w[1] = v.w;
  }
}

template <int BITS>
__device__ __forceinline__ void decode32(const Raw<BITS>& raw, const Tables& t, uint4 out[4]) {
  if (BITS == 4) {
    const uint32_t* w = raw.w;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint32_t sel = w[q] & 0x77777777u;
      const uint32_t loA = prmt(t.lo0, t.lo1, sel), loB = prmt(t.lo0, t.lo1, sel >> 16);
      const uint32_t hiA = prmt(t.hi0, t.hi1, sel) ^ (w[q] & 0x80808080u);
      const uint32_t hiB = prmt(t.hi0, t.hi1, sel >> 16) ^ ((w[q] << 4) & 0x80808080u);
      out[q] = make_uint4(prmt(loA, hiA, 0x5140u), prmt(loA, hiA, 0x7362u), prmt(loB, hiB, 0x5140u),
                          prmt(loB, hiB, 0x7362u));
    }
  } else {
    const uint32_t mw[2] = {raw.w[0], raw.w[BITS == 3 ? 1 : 0]};
    const uint32_t s = raw.w[BITS - 1];
    // byte-permute selectors of the 8 groups of 4 coordinates: the permute reads only the low 16 bits of a
    // selector, so one mask serves two groups (the second after a shift by 16)
    uint32_t selv[8];
    if (BITS == 3) {
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const uint32_t e = mw[u] & 0x33333333u, o = (mw[u] >> 2) & 0x33333333u;
        selv[4 * u] = e; selv[4 * u + 1] = o; selv[4 * u + 2] = e >> 16; selv[4 * u + 3] = o >> 16;
      }
    } else {
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const uint32_t e = (mw[0] >> g) & 0x11111111u;
        selv[g] = e; selv[4 + g] = e >> 16;
      }
    }
    uint32_t r[16];
#pragma unroll
    for (int G = 0; G < 8; ++G) {
      const uint32_t sel = selv[G];
      const uint32_t lo = prmt(t.lo0, t.lo0, sel);
      const uint32_t hi = prmt(t.hi0, t.hi0, sel) ^ ((s << G) & 0x80808080u);
      r[2 * G] = prmt(lo, hi, 0x5140u);
      r[2 * G + 1] = prmt(lo, hi, 0x7362u);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) out[q] = make_uint4(r[4 * q], r[4 * q + 1], r[4 * q + 2], r[4 * q + 3]);
  }
}

// ---------------------------------------------------------------------------------------------------------
namespace pair {
constexpr int PSTAGES = 3;
constexpr int PBK = 2 * BK;                                            // 128 coordinates per stage: two swizzle atoms
constexpr uint32_t ATOM_BYTES = 128 * BK * 2;                          // 128 rows x 128 bytes = 16 KB
constexpr uint32_t PA_BYTES = 2 * ATOM_BYTES, PB_BYTES = 2 * ATOM_BYTES;
constexpr uint32_t PSTAGE_BYTES = PA_BYTES + PB_BYTES;                 // 64 KB
constexpr int EPI_THREADS = 128;
constexpr int PTHREADS = DECODE_THREADS + EPI_THREADS + 32;   // 16 decode warps, 4 epilogue warps, 1 MMA warp
constexpr size_t PSMEM_BYTES = PSTAGES * PSTAGE_BYTES + 1024 + 256;
}  // namespace pair

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive on the barrier at the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t local_bar, uint32_t rank) {
  asm volatile(
      "{\n .reg .b32 ra;\n mapa.shared::cluster.u32 ra, %0, %1;\n"
      " mbarrier.arrive.shared::cluster.b64 _, [ra];\n}"
      ::"r"(local_bar), "r"(rank) : "memory");
}
__device__ __forceinline__ bool mbar_try_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait with cluster-scope acquire (the arrivals may come from the other CTA of the pair).
__device__ __forceinline__ void mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                                  int code) {
  if (mbar_try_cluster(bar, parity)) return;
  const long long t0 = clock64();
  int polls = 0;
  while (!mbar_try_cluster(bar, parity)) {
    if (*abort_flag) return;
    if ((++polls & 1023) == 0) {
      if (*reinterpret_cast<volatile int*>(status) != 0 || clock64() - t0 > WAIT_CYCLES) {
        atomicCAS(status, 0, code);
        *abort_flag = 1;
        return;
      }
    }
  }
}
__device__ __forceinline__ void commit_multicast(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3) : "memory");
}

// Decode loop of one thread of the two-SM kernel: the thread owns one (row, 32-coordinate half) of this CTA's
// 128 rows of ONE operand (IS_A: activations, else weights) and, per 128-coordinate stage, decodes the two
// 32-coordinate pieces that fall into the stage's two swizzle atoms.
template <int BITS, bool IS_A>
__device__ __forceinline__ void pair_decode_loop(const uint32_t* __restrict__ packed, int nrows, int dim, const Tables& t,
                                                 unsigned char* smem, uint32_t full0, uint32_t empty0, int t2,
                                                 uint32_t rank, int pair_id, int npairs, int ntiles, int tiles_n,
                                                 int kblocks, volatile int* abort_flag, int* status) {
  using namespace pair;
  const int lane = threadIdx.x & 31;
  // Two ways to split a stage's 128 rows x 128 coordinates among 256 threads:
  //  * 4-bit operands: thread = (row t2/2, 32-coordinate half t2%2) of BOTH 64-coordinate swizzle atoms: one
  //    16-byte load per piece, adjacent lanes read adjacent 16 bytes;
  //  * 3- and 2-bit operands: thread = (row t2/2, atom t2%2), 64 contiguous coordinates: 24 / 16 bytes, 8- / 16-byte
  //    aligned, instead of 12- / 8-byte pieces; adjacent lanes read the two adjacent pieces of one row (whole
  //    sectors per warp).  The thread of atom 1 handles its two 32-coordinate pieces in the opposite order.
  // Inside an atom row r occupies 128 bytes and its 16-byte chunk c sits at position c ^ (r & 7); both
  // mappings give the 8 lanes of a quarter warp 8 different chunk positions, i.e. all 32 banks (4 rows x 2
  // lanes: the lanes of atom 0 store chunks q ^ r, those of atom 1 chunks (q + 4) ^ r at the same time).
  constexpr bool CONTIG = BITS != 4;
  const int row = t2 >> 1;
  const int sub = t2 & 1;                             // atom (CONTIG) or half of each atom
  const int pitch = dim / 32 * BITS;
  constexpr int WPA = 2 * BITS;                       // words per 64 coordinates of one row
  unsigned char* const tile0 = smem + (IS_A ? 0u : PA_BYTES) + (uint32_t)row * 128u + (CONTIG ? (uint32_t)sub * ATOM_BYTES : 0u);
  const uint32_t rx = (uint32_t)(row & 7) << 4;
  const uint32_t c0b = CONTIG ? (uint32_t)sub * 64u : (uint32_t)sub * 64u;   // first chunk (in bytes) of the piece stored first
  const uint32_t second = CONTIG ? (sub ? 0u : 64u) : ATOM_BYTES;    // where the other piece goes (CONTIG: chunk offset; else: atom)
  uint32_t st = 0, ph = 0;
  bool first_round = true;
  Raw<BITS> n0r, n1r;                                 // packed words of the NEXT stage
  int f_tile = pair_id, f_kb = 0;
  const uint32_t* fsrc = nullptr;
  auto set_fetch_tile = [&](int tile) {
    const int r0 = (IS_A ? (tile % tiles_n) : (tile / tiles_n)) * 256 + (int)rank * 128;
    fsrc = packed + (size_t)min(r0 + row, nrows - 1) * pitch + sub * (CONTIG ? WPA : BITS);   // rows past the end re-read the last
  };
  auto fetch_next = [&]() {
    if (f_tile >= ntiles) return;
    if (CONTIG) {
      load_raw64<BITS>(fsrc, n0r, n1r);
    } else {
      n0r = load_raw<BITS>(fsrc);
      n1r = load_raw<BITS>(fsrc + WPA);
    }
    fsrc += 2 * WPA;
    if (++f_kb == kblocks) {
      f_kb = 0;
      f_tile += npairs;
      if (f_tile < ntiles) set_fetch_tile(f_tile);
    }
  };
  if (f_tile < ntiles) set_fetch_tile(f_tile);
  fetch_next();
  for (int tile = pair_id; tile < ntiles; tile += npairs) {
    for (int kb = 0; kb < kblocks; ++kb) {
      const Raw<BITS> c0 = (CONTIG && sub) ? n1r : n0r, c1 = (CONTIG && sub) ? n0r : n1r;
      fetch_next();
      if (!first_round) {
        if (lane == 0) mbar_wait(empty0 + 8 * st, ph ^ 1, abort_flag, status, WAIT_EMPTY);
        __syncwarp();
      }
      unsigned char* Ss = tile0 + st * PSTAGE_BYTES;
      uint4 v[4];
      decode32<BITS>(c0, t, v);
#pragma unroll
      for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4*>(Ss + ((c0b + ((uint32_t)q << 4)) ^ rx)) = v[q];
      decode32<BITS>(c1, t, v);
      if (CONTIG) {
#pragma unroll
        for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4*>(Ss + ((second + ((uint32_t)q << 4)) ^ rx)) = v[q];
      } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4*>(Ss + second + ((c0b + ((uint32_t)q << 4)) ^ rx)) = v[q];
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy stores -> visible to the MMA
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(full0 + 8 * st, 0);          // to CTA 0, where the MMAs are issued
      if (++st == PSTAGES) { st = 0; ph ^= 1; first_round = false; }
    }
  }
}

template <int BITS_A, int BITS_W, bool F32_OUT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(pair::PTHREADS, 1)
qlinear_pair_kernel(const uint32_t* __restrict__ Aq, const float* __restrict__ a_norm, int n_tokens,
                    const uint32_t* __restrict__ Wq, const __nv_bfloat16* __restrict__ w_norm, int m, int dim,
                    CodebookParams cba, CodebookParams cbw, void* __restrict__ Y, int ldy, int* status) {
  using namespace pair;
  extern __shared__ unsigned char smem_dyn[];
  // 1024-byte alignment computed on the shared-window address: the compiler keeps treating the tiles as shared
  // memory (32-bit addresses) instead of falling back to generic-pointer arithmetic
  unsigned char* smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + PSTAGES * PSTAGE_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * PSTAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + PSTAGES);
  const uint32_t accfull0 = smem_u32(bars + 2 * PSTAGES), accempty0 = smem_u32(bars + 2 * PSTAGES + 2);
  constexpr int MMA_WARP = (DECODE_THREADS + EPI_THREADS) / 32;

  if (tid == 0) {
    for (int s = 0; s < PSTAGES; ++s) {
      mbar_init(full0 + 8 * s, 2 * (DECODE_THREADS / 32));   // one arrival per decoding warp of BOTH CTAs (used in CTA 0)
      mbar_init(empty0 + 8 * s, 1);                          // multicast commit
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(accfull0 + 8 * b, 1);                        // multicast commit
      mbar_init(accempty0 + 8 * b, 2 * (EPI_THREADS / 32));  // epilogue warps of both CTAs (used in CTA 0)
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == MMA_WARP) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();     // barriers of both CTAs are initialised before anyone arrives remotely
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *tmem_slot;
  // Programmatic dependent launch: the set-up above may have run while the previous kernel of the stream (normally
  // the rotate+quantize pass that produces Aq) was finishing; nothing below may start before that grid is complete.
  // The next kernel may in turn be scheduled on SMs as this grid frees them.  (Both are no-ops in an ordinary launch.)
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const int kblocks = dim / PBK;
  const int tiles_n = (n_tokens + 255) / 256;
  const int ntiles = tiles_n * ((m + 255) / 256);
  const int npairs = gridDim.x >> 1, pair_id = blockIdx.x >> 1;

  if (warp == MMA_WARP) {
    // ------------------------------- MMA issuer: one thread of CTA 0 -------------------------------
    if (rank == 0 && lane == 0) {
      uint32_t st = 0, ph = 0, lt = 0;
      constexpr uint32_t IDESC2 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
      for (int tile = pair_id; tile < ntiles; tile += npairs, ++lt) {
        const uint32_t buf = lt & 1;
        if (lt >= 2) mbar_wait_cluster(accempty0 + 8 * buf, ((lt >> 1) - 1) & 1, abort_flag, status, WAIT_ACC_EMPTY);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        for (int kb = 0; kb < kblocks; ++kb) {
          mbar_wait_cluster(full0 + 8 * st, ph, abort_flag, status, WAIT_FULL);
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = smem_u32(smem + st * PSTAGE_BYTES);
#pragma unroll
          for (int k4 = 0; k4 < PBK / 16; ++k4) {
            // K step k4: swizzle atom k4 / 4, 32 bytes per step inside the atom
            const uint64_t da = smem_desc(a_addr + (k4 >> 2) * ATOM_BYTES) + 2 * (k4 & 3);
            const uint64_t db = smem_desc(a_addr + PA_BYTES + (k4 >> 2) * ATOM_BYTES) + 2 * (k4 & 3);
            const uint32_t acc = (kb > 0 || k4 > 0) ? 1u : 0u;
            asm volatile(
                "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
                ::"r"(tmem + buf * 256), "l"(da), "l"(db), "r"(IDESC2), "r"(acc) : "memory");
          }
          commit_multicast(empty0 + 8 * st);       // both CTAs may refill the stage once these MMAs have read it
          if (++st == PSTAGES) { st = 0; ph ^= 1; }
        }
        commit_multicast(accfull0 + 8 * buf);      // both CTAs' epilogue warps may read accumulator `buf`
      }
    }
  } else if (warp >= DECODE_THREADS / 32) {
    // ------------------------------- epilogue warps (4 per CTA) -------------------------------
    const int q = warp & 3;                          // TMEM lane quarter of this warp
    uint32_t lt = 0;
    for (int tile = pair_id; tile < ntiles; tile += npairs, ++lt) {
      const uint32_t buf = lt & 1;
      const int n0 = (tile % tiles_n) * 256 + (int)rank * 128, i0 = (tile / tiles_n) * 256;
      if (lane == 0) mbar_wait(accfull0 + 8 * buf, (lt >> 1) & 1, abort_flag, status, WAIT_ACC_FULL);
      __syncwarp();
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int trow = n0 + q * 32 + lane;
      const float s = trow < n_tokens ? a_norm[trow] : 0.f;
#pragma unroll 1
      for (int c = 0; c < 8; ++c) {
        uint32_t r[32];
        tmem_load32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 256 + c * 32), r);
        if (trow < n_tokens) {
#pragma unroll
          for (int g8 = 0; g8 < 4; ++g8) {
            const int i = i0 + c * 32 + g8 * 8;
            if (i < m) {
              const uint4 rn = __ldg(reinterpret_cast<const uint4*>(w_norm + i));
              const uint32_t rw[4] = {rn.x, rn.y, rn.z, rn.w};
              float y[8];
#pragma unroll
              for (int jj = 0; jj < 4; ++jj) {
                y[2 * jj] = (__uint_as_float(r[g8 * 8 + 2 * jj]) * s) * __uint_as_float(rw[jj] << 16);
                y[2 * jj + 1] = (__uint_as_float(r[g8 * 8 + 2 * jj + 1]) * s) * __uint_as_float(rw[jj] & 0xFFFF0000u);
              }
              if (F32_OUT) {
                float* dst = reinterpret_cast<float*>(Y) + (size_t)trow * ldy + i;
                *reinterpret_cast<float4*>(dst) = make_float4(y[0], y[1], y[2], y[3]);
                *reinterpret_cast<float4*>(dst + 4) = make_float4(y[4], y[5], y[6], y[7]);
              } else {
                __nv_bfloat162 p0 = __floats2bfloat162_rn(y[0], y[1]), p1 = __floats2bfloat162_rn(y[2], y[3]);
                __nv_bfloat162 p2 = __floats2bfloat162_rn(y[4], y[5]), p3 = __floats2bfloat162_rn(y[6], y[7]);
                uint4 pk;
                pk.x = *reinterpret_cast<uint32_t*>(&p0); pk.y = *reinterpret_cast<uint32_t*>(&p1);
                pk.z = *reinterpret_cast<uint32_t*>(&p2); pk.w = *reinterpret_cast<uint32_t*>(&p3);
                *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(Y) + (size_t)trow * ldy + i) = pk;
              }
            }
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(accempty0 + 8 * buf, 0);   // CTA 0 may let the MMAs overwrite `buf`
    }
  } else {
    // ------------------------------- decoders (16 warps per CTA) -------------------------------
    // threads 0-255: this CTA's 128 rows of A; threads 256-511: its 128 rows of B
    if (tid < 256) {
      const Tables ta = make_tables(cba);
      pair_decode_loop<BITS_A, true>(Aq, n_tokens, dim, ta, smem, full0, empty0, tid, rank, pair_id, npairs, ntiles,
                                     tiles_n, kblocks, abort_flag, status);
    } else {
      const Tables tw = make_tables(cbw);
      pair_decode_loop<BITS_W, false>(Wq, m, dim, tw, smem, full0, empty0, tid - 256, rank, pair_id, npairs, ntiles,
                                      tiles_n, kblocks, abort_flag, status);
    }
  }
  __syncwarp();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();     // neither CTA leaves (or frees TMEM) while the other may still signal it or read its tiles
  if (warp == MMA_WARP) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
}

// One thread waits, with a short limit, on a barrier that nobody ever arrives at: the wait must give up by
// itself, record its code and let the kernel end normally.
__global__ void bounded_wait_probe_kernel(int* status, long long max_cycles) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_wait(smem_u32(&bar), 0, &abort_flag, status, WAIT_SELFTEST, max_cycles);
  }
}

template <int BA, int BW, bool F32>
cudaError_t launch_pair(int sms, cudaStream_t st, const uint32_t* Aq, const float* an, int n, const uint32_t* Wq,
                        const __nv_bfloat16* wn, int m, int dim, const CodebookParams& ca, const CodebookParams& cw,
                        void* Y, int ldy, int* status) {
  auto k = qlinear_pair_kernel<BA, BW, F32>;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pair::PSMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int ntiles = ((n + 255) / 256) * ((m + 255) / 256);
  // persistent grid: as many pairs as can be resident at once (SM pairs must sit in one cluster-capable group,
  // so this can be fewer than sms / 2)
  static int max_pairs[64] = {0};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && max_pairs[dev] == 0) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sms / 2 * 2);
    cfg.blockDim = dim3(pair::PTHREADS);
    cfg.dynamicSmemBytes = pair::PSMEM_BYTES;
    int nclusters = 0;
    e = cudaOccupancyMaxActiveClusters(&nclusters, k, &cfg);
    if (e != cudaSuccess) return e;
    max_pairs[dev] = nclusters > 0 ? nclusters : 1;
  }
  int pairs = (dev >= 0 && dev < 64) ? max_pairs[dev] : sms / 2;
  if (pairs > sms / 2) pairs = sms / 2;
  if (pairs > ntiles) pairs = ntiles;
  return launch_dependent(k, 2 * pairs, pair::PTHREADS, pair::PSMEM_BYTES, st, Aq, an, n, Wq, wn, m, dim, ca, cw, Y, ldy, status);
}

template <int BA, int BW>
int launch_bits(bool f32, int sms, cudaStream_t st, const uint32_t* Aq, const float* an, int n, const uint32_t* Wq,
                const __nv_bfloat16* wn, int m, int dim, const CodebookParams& ca, const CodebookParams& cw, void* Y,
                int ldy, int* status) {
  const cudaError_t e = f32 ? launch_pair<BA, BW, true>(sms, st, Aq, an, n, Wq, wn, m, dim, ca, cw, Y, ldy, status)
                            : launch_pair<BA, BW, false>(sms, st, Aq, an, n, Wq, wn, m, dim, ca, cw, Y, ldy, status);
  if (e != cudaSuccess) return cuda_fail(e, "oq_qlinear launch");
  return OQ_OK;
}

}  // namespace
}  // namespace oq

namespace oq {

// Validates and launches; `status` is the device word that bounded waits report to (NULL: the library's own
// word, allocated on first use).
int qlinear_launch(const void* Xq_idx, const float* Xq_norm, int n_tokens, const oq_codebook* cb_a,
                   const void* Wq_idx, const void* Wq_norm_bf16, int m, const oq_codebook* cb_w, int dim, void* Y,
                   int ldy, int y_dtype, int* status, void* stream) {
  if (!cb_a || !cb_w) return fail(OQ_ERR_INVALID_ARG, "oq_qlinear: NULL codebook");
  if (n_tokens < 0 || m < 0 || dim <= 0) return fail(OQ_ERR_INVALID_ARG, "oq_qlinear: bad sizes");
  if (cb_a->dim != dim || cb_w->dim != dim) return fail(OQ_ERR_INVALID_ARG, "oq_qlinear: codebook dim differs from dim");
  if (dim % 128) return fail(OQ_ERR_UNSUPPORTED, "oq_qlinear: dim must be a multiple of 128");
  if (m % 8) return fail(OQ_ERR_UNSUPPORTED, "oq_qlinear: m must be a multiple of 8");
  if (y_dtype != OQ_BF16 && y_dtype != OQ_F32) return fail(OQ_ERR_INVALID_ARG, "oq_qlinear: unknown y_dtype");
  const int ba = cb_a->bits, bw = cb_w->bits;
  if (ba < 2 || ba > 4 || bw < 2 || bw > 4) return fail(OQ_ERR_UNSUPPORTED, "oq_qlinear: bits must be 2, 3 or 4");
  if (n_tokens == 0 || m == 0) return OQ_OK;
  if (!Xq_idx || !Xq_norm || !Wq_idx || !Wq_norm_bf16 || !Y) return fail(OQ_ERR_INVALID_ARG, "oq_qlinear: NULL buffer");
  if (ldy < m) return fail(OQ_ERR_INVALID_ARG, "oq_qlinear: ldy smaller than m");
  if (ldy % 8 || !aligned16(Xq_idx) || !aligned16(Wq_idx) || !aligned16(Y) || !aligned16(Wq_norm_bf16))
    return fail(OQ_ERR_ALIGNMENT, "oq_qlinear: pointers must be 16-byte aligned and ldy a multiple of 8");
  if (!status) status = device_status_word();
  if (!status) return fail(OQ_ERR_CUDA, "oq_qlinear: cannot allocate the device status word");
  const CodebookParams ca = codebook_params(cb_a), cw = codebook_params(cb_w);
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaError_t ce = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (ce != cudaSuccess) return cuda_fail(ce, "cudaDeviceGetAttribute");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const uint32_t* A = reinterpret_cast<const uint32_t*>(Xq_idx);
  const uint32_t* W = reinterpret_cast<const uint32_t*>(Wq_idx);
  const __nv_bfloat16* wn = reinterpret_cast<const __nv_bfloat16*>(Wq_norm_bf16);
  const bool f32 = y_dtype == OQ_F32;
#define OQ_CASE(a, w) \
  if (ba == a && bw == w) return launch_bits<a, w>(f32, sms, st, A, Xq_norm, n_tokens, W, wn, m, dim, ca, cw, Y, ldy, status);
  OQ_CASE(4, 4) OQ_CASE(3, 3) OQ_CASE(4, 2) OQ_CASE(3, 2) OQ_CASE(4, 3) OQ_CASE(2, 2) OQ_CASE(3, 4) OQ_CASE(2, 4) OQ_CASE(2, 3)
#undef OQ_CASE
  return fail(OQ_ERR_UNSUPPORTED, "oq_qlinear: unsupported bit-width pair");
}

}  // namespace oq

extern "C" int oq_selftest_bounded_wait(void* stream) {
  int* status = oq::device_status_word();
  if (!status) return oq::fail(OQ_ERR_CUDA, "oq_selftest_bounded_wait: cannot allocate the device status word");
  oq::bounded_wait_probe_kernel<<<1, 32, 0, reinterpret_cast<cudaStream_t>(stream)>>>(status, 2000000ll);   // ~1 ms
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return oq::cuda_fail(e, "oq_selftest_bounded_wait");
  return OQ_OK;
}

extern "C" int oq_qlinear(const void* Xq_idx, const float* Xq_norm, int n_tokens, const oq_codebook* cb_a,
                          const void* Wq_idx, const void* Wq_norm_bf16, int m, const oq_codebook* cb_w, int dim,
                          void* Y, int ldy, int y_dtype, void* stream) {
  return oq::qlinear_launch(Xq_idx, Xq_norm, n_tokens, cb_a, Wq_idx, Wq_norm_bf16, m, cb_w, dim, Y, ldy, y_dtype,
                            nullptr, stream);
}
