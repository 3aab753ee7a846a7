// Codebook-decode GEMM:  Y[n][i] = s_n * r'_i * sum_k C_a[idxA[n][k]] * C_w[idxW[i][k]]
// (the product W^' x^' of Sec. 4.3 with the magnitudes of Eq. 6 and Eq. 8 applied in the epilogue).
//
// Packed indices are fetched from global memory into registers (one stage ahead), decoded to bf16 levels
// with byte-permute table look-ups, written into shared memory in the tensor core's K-major
// 128-byte-swizzled layout, and contracted with tcgen05.mma.cta_group::2 (fp32 accumulators in tensor
// memory, two SMs per 256 x 256 tile).  Every device-side wait is bounded and reports to a status word.
//
// The activation operand comes in one of two forms: packed indices, decoded here like the weights (BITS_A = 2, 3,
// 4), or the bf16 levels C_a[idx] written out once by the producer (BITS_A = 0).  An activation tile is used by
// every column tile of the output, so decoding it once per layer instead of once per tile takes half of the decode
// work out of this kernel: the tiles then arrive by TMA (cp.async.bulk.tensor, 128-byte swizzle, no SM
// instructions), and all 16 decoding warps work on the weights.  Both forms feed the same bf16 values to the same
// MMAs in the same order: the outputs are bit-identical.
#include <atomic>
#include <cuda.h>
#include <cuda_bf16.h>

#include "oq_decode.cuh"
#include "oq_internal.h"
#include "oq_sm100.cuh"

namespace oq {

namespace {

constexpr int BK = 64;                  // coordinates per swizzle atom: 64 bf16 = one 128-byte swizzled row
constexpr int DECODE_THREADS = 512;    // 16 decoding warps per CTA
constexpr int TMEM_COLS = 512;         // two 128 x 256 fp32 accumulators per CTA

// ---------------------------------------------------------------------------------------------------------
namespace pair {
constexpr int PSTAGES = 3;
constexpr int PBK = 2 * BK;                                            // 128 coordinates per stage: two swizzle atoms
constexpr uint32_t ATOM_BYTES = 128 * BK * 2;                          // 128 rows x 128 bytes = 16 KB
constexpr uint32_t PA_BYTES = 2 * ATOM_BYTES, PB_BYTES = 2 * ATOM_BYTES;
constexpr uint32_t PSTAGE_BYTES = PA_BYTES + PB_BYTES;                 // 64 KB
constexpr int EPI_THREADS = 128;
constexpr int PTHREADS = DECODE_THREADS + EPI_THREADS + 64;   // 16 decode warps, 4 epilogue warps, 1 MMA warp, 1 TMA warp
constexpr size_t PSMEM_BYTES = PSTAGES * PSTAGE_BYTES + 1024 + 256 + 2048;   // tiles, alignment slack, barriers, the epilogue warps' weight norms
// Activations as bf16 levels: the TMA-fed activation tiles have a ring of their own, one stage deeper than the
// weights' (their latency is the L2 round trip of a copy that can only be requested once its buffer is free; the
// decoders hide theirs by holding the next stage's packed words in registers).
constexpr int DA_STAGES = 4;
constexpr uint32_t DB_BASE = DA_STAGES * PA_BYTES;                     // weight ring behind the activation ring
constexpr uint32_t DBAR_OFF = DB_BASE + PSTAGES * PB_BYTES;            // 224 KB
constexpr size_t DSMEM_BYTES = DBAR_OFF + 1024 + 256;
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

// Address of the barrier at the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
  uint32_t ra;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
  return ra;
}
__device__ __forceinline__ void mbar_arrive_expect_tx_cluster(uint32_t cluster_bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.release.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_bar), "r"(bytes) : "memory");
}
// One box of the activation matrix (64 coordinates x 128 rows, 128-byte swizzle) into this CTA's shared memory; the
// bytes are counted on a barrier of the pair's leading CTA (each CTA fetches its own rows into its own memory).
__device__ __forceinline__ void tma_load_box(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t cluster_bar) {
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(cluster_bar), "r"(x), "r"(y) : "memory");
}

// Weight decode loop of the kernel whose activations arrive as bf16 levels: all 512 decoding threads work on this
// CTA's 128 weight rows.  Warps 0-7 fill swizzle atom 0 of a stage, warps 8-15 atom 1; inside an atom a thread owns
// (row t2/2, 32-coordinate half t2%2): one load of BITS words (adjacent lanes read adjacent pieces), four 16-byte
// stores; the 8 lanes of a quarter warp hit 8 different chunk positions, i.e. all 32 banks.
template <int BITS>
__device__ __forceinline__ void dense_b_decode_loop(const uint32_t* __restrict__ packed, int nrows, int dim, const Tables& t,
                                                    unsigned char* smem, uint32_t full0, uint32_t empty0, int tid512,
                                                    uint32_t rank, int pair_id, int npairs, int ntiles, int tiles_m,
                                                    int kblocks, volatile int* abort_flag, int* status) {
  using namespace pair;
  const int lane = threadIdx.x & 31;
  const int atom = tid512 >> 8, t2 = tid512 & 255, row = t2 >> 1, half = t2 & 1;
  const int pitch = dim / 32 * BITS;
  unsigned char* const tile0 = smem + DB_BASE + (uint32_t)atom * ATOM_BYTES + (uint32_t)row * 128u;
  const uint32_t rx = (uint32_t)(row & 7) << 4, c0b = (uint32_t)half * 64u;
  uint32_t st = 0, ph = 0;
  bool first_round = true;
  Raw<BITS> nxt;                                      // packed words of the NEXT stage
  int f_tile = pair_id, f_kb = 0;
  const uint32_t* fsrc = nullptr;
  auto set_fetch_tile = [&](int tile) {
    const int r0 = (tile % tiles_m) * 256 + (int)rank * 128;     // column tiles vary fastest (see the kernel)
    fsrc = packed + (size_t)min(r0 + row, nrows - 1) * pitch + (atom * 2 + half) * BITS;   // rows past the end re-read the last
  };
  auto fetch_next = [&]() {
    if (f_tile >= ntiles) return;
    nxt = load_raw<BITS>(fsrc);
    fsrc += 4 * BITS;                                 // 128 coordinates per stage
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
      const Raw<BITS> cur = nxt;
      fetch_next();
      uint4 v[4];
      decode32<BITS>(cur, t, v);                       // (registers only: before the stage is known to be free)
      if (!first_round) {
        if (lane == 0) mbar_wait(empty0 + 8 * st, ph ^ 1, abort_flag, status, WAIT_EMPTY);
        __syncwarp();
      }
      unsigned char* Ss = tile0 + st * PB_BYTES;
#pragma unroll
      for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4*>(Ss + ((c0b + ((uint32_t)q << 4)) ^ rx)) = v[q];
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy stores -> visible to the MMA
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(full0 + 8 * st, 0);          // to CTA 0, where the MMAs are issued
      if (++st == PSTAGES) { st = 0; ph ^= 1; first_round = false; }
    }
  }
}

// Tile order of the kernel with the activation operand in tensor memory: bands of `width` column tiles; inside a band the
// column tile varies fastest.  With width 1 the row tile varies fastest over the whole matrix (the pairs that run together
// share one weight tile and read npairs different activation tiles: fine while the packed activations stay in L2).  With
// width 8 they work on ~npairs / 8 row tiles x 8 column tiles, so both packed operands of a wave are a few MB: chosen by
// the launcher when the packed activations are too large to stay in L2 next to the output stream (Wan-sized layers: +4 %).
constexpr int TILE_BAND_WIDE = 8;
__device__ __forceinline__ void banded_tile(int tile, int tiles_n, int tiles_m, int width, int& rt, int& ct) {
  const int band = tile / (width * tiles_n);
  const int c0 = band * width;
  const int gc = min(width, tiles_m - c0);
  const int r = tile - band * width * tiles_n;
  rt = r / gc;
  ct = c0 + r - rt * gc;
}

// Decode loop of one thread of the two-SM kernel: the thread owns one (row, 32-coordinate half) of this CTA's
// 128 rows of ONE operand (IS_A: activations, else weights) and, per 128-coordinate stage, decodes the two
// 32-coordinate pieces that fall into the stage's two swizzle atoms.
template <int BITS, bool IS_A, uint32_t STAGE_STRIDE = pair::PSTAGE_BYTES, int NSTAGES = pair::PSTAGES, uint32_t B_OFF = pair::PA_BYTES, bool BANDED = false>
__device__ __forceinline__ void pair_decode_loop(const uint32_t* __restrict__ packed, int nrows, int dim, const Tables& t,
                                                 unsigned char* smem, uint32_t full0, uint32_t empty0, int t2,
                                                 uint32_t rank, int pair_id, int npairs, int ntiles, int tiles_n,
                                                 int kblocks, volatile int* abort_flag, int* status, int tiles_m = 0, int band = 1) {
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
  unsigned char* const tile0 = smem + (IS_A ? 0u : B_OFF) + (uint32_t)row * 128u + (CONTIG ? (uint32_t)sub * ATOM_BYTES : 0u);
  const uint32_t rx = (uint32_t)(row & 7) << 4;
  const uint32_t c0b = CONTIG ? (uint32_t)sub * 64u : (uint32_t)sub * 64u;   // first chunk (in bytes) of the piece stored first
  const uint32_t second = CONTIG ? (sub ? 0u : 64u) : ATOM_BYTES;    // where the other piece goes (CONTIG: chunk offset; else: atom)
  uint32_t st = 0, ph = 0;
  bool first_round = true;
  Raw<BITS> n0r, n1r;                                 // packed words of the NEXT stage
  int f_tile = pair_id, f_kb = 0;
  const uint32_t* fsrc = nullptr;
  auto set_fetch_tile = [&](int tile) {
    int rt = tile % tiles_n, ct = tile / tiles_n;
    if constexpr (BANDED) banded_tile(tile, tiles_n, tiles_m, band, rt, ct);
    const int r0 = (IS_A ? rt : ct) * 256 + (int)rank * 128;
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
      // the first piece is decoded (registers only) before the stage is known to be free: when the decoders are ahead
      // of the MMAs, half of the decode arithmetic is off the path from "stage free" to "stage full" (+3-4 %; decoding
      // both pieces first needs more registers than there are and was slower)
      uint4 v[4];
      decode32<BITS>(c0, t, v);
      if (!first_round) {
        if (lane == 0) mbar_wait(empty0 + 8 * st, ph ^ 1, abort_flag, status, WAIT_EMPTY);
        __syncwarp();
      }
      unsigned char* Ss = tile0 + st * STAGE_STRIDE;
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
      if (++st == NSTAGES) { st = 0; ph ^= 1; first_round = false; }
    }
  }
}

template <int BITS_A, int BITS_W, bool F32_OUT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(pair::PTHREADS, 1)
qlinear_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const uint32_t* __restrict__ Aq,
                    const float* __restrict__ a_norm, int n_tokens,
                    const uint32_t* __restrict__ Wq, const __nv_bfloat16* __restrict__ w_norm, int m, int dim,
                    CodebookParams cba, CodebookParams cbw, void* __restrict__ Y, int ldy, int* status) {
  using namespace pair;
  extern __shared__ unsigned char smem_dyn[];
  // 1024-byte alignment computed on the shared-window address: the compiler keeps treating the tiles as shared
  // memory (32-bit addresses) instead of falling back to generic-pointer arithmetic
  unsigned char* smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  constexpr bool DENSE_A = BITS_A == 0;               // activations as bf16 levels, fetched by TMA
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (DENSE_A ? DBAR_OFF : PSTAGES * PSTAGE_BYTES));
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * PSTAGES + 4 + 2 * DA_STAGES);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + PSTAGES);
  const uint32_t accfull0 = smem_u32(bars + 2 * PSTAGES), accempty0 = smem_u32(bars + 2 * PSTAGES + 2);
  // (levels form only) activation ring: bytes landed / stage read by its MMAs
  const uint32_t afull0 = smem_u32(bars + 2 * PSTAGES + 4), aempty0 = smem_u32(bars + 2 * PSTAGES + 4 + DA_STAGES);
  constexpr int MMA_WARP = (DECODE_THREADS + EPI_THREADS) / 32, TMA_WARP = MMA_WARP + 1;

  if (tid == 0) {
    for (int s = 0; s < PSTAGES; ++s) {
      mbar_init(full0 + 8 * s, 2 * (DECODE_THREADS / 32));   // one arrival per decoding warp of BOTH CTAs (used in CTA 0)
      mbar_init(empty0 + 8 * s, 1);                          // multicast commit
    }
    for (int s = 0; s < DA_STAGES; ++s) {
      mbar_init(afull0 + 8 * s, 2);                          // one arrival per CTA that announces its bytes (used in CTA 0)
      mbar_init(aempty0 + 8 * s, 1);                         // multicast commit
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
  const int tiles_m = (m + 255) / 256;
  const int ntiles = tiles_n * tiles_m;
  // Tile order.  Packed activations: row tiles vary fastest (the pairs running together share a weight tile).  bf16
  // levels: column tiles vary fastest, so that the pairs running together share activation tiles, which are four
  // times larger than packed ones and may not fit in L2 as a whole.
  const int npairs = gridDim.x >> 1, pair_id = blockIdx.x >> 1;

  if (warp == MMA_WARP) {
    // ------------------------------- MMA issuer: one thread of CTA 0 -------------------------------
    if (rank == 0 && lane == 0) {
      uint32_t st = 0, ph = 0, lt = 0;
      uint32_t sa = 0, pha = 0;                      // stage and phase of the activation ring (levels form)
      constexpr uint32_t IDESC2 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
      for (int tile = pair_id; tile < ntiles; tile += npairs, ++lt) {
        const uint32_t buf = lt & 1;
        if (lt >= 2) mbar_wait_cluster(accempty0 + 8 * buf, ((lt >> 1) - 1) & 1, abort_flag, status, WAIT_ACC_EMPTY);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        for (int kb = 0; kb < kblocks; ++kb) {
          if (DENSE_A) mbar_wait_cluster(afull0 + 8 * sa, pha, abort_flag, status, WAIT_FULL);
          mbar_wait_cluster(full0 + 8 * st, ph, abort_flag, status, WAIT_FULL);
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = smem_u32(smem + (DENSE_A ? sa * PA_BYTES : st * PSTAGE_BYTES));
          const uint32_t b_addr = smem_u32(smem + (DENSE_A ? DB_BASE + st * PB_BYTES : st * PSTAGE_BYTES + PA_BYTES));
#pragma unroll
          for (int k4 = 0; k4 < PBK / 16; ++k4) {
            // K step k4: swizzle atom k4 / 4, 32 bytes per step inside the atom
            const uint64_t da = smem_desc(a_addr + (k4 >> 2) * ATOM_BYTES) + 2 * (k4 & 3);
            const uint64_t db = smem_desc(b_addr + (k4 >> 2) * ATOM_BYTES) + 2 * (k4 & 3);
            const uint32_t acc = (kb > 0 || k4 > 0) ? 1u : 0u;
            asm volatile(
                "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
                ::"r"(tmem + buf * 256), "l"(da), "l"(db), "r"(IDESC2), "r"(acc) : "memory");
          }
          commit_multicast(empty0 + 8 * st);       // both CTAs may refill the stage once these MMAs have read it
          if (++st == PSTAGES) { st = 0; ph ^= 1; }
          if (DENSE_A) {
            commit_multicast(aempty0 + 8 * sa);
            if (++sa == DA_STAGES) { sa = 0; pha ^= 1; }
          }
        }
        commit_multicast(accfull0 + 8 * buf);      // both CTAs' epilogue warps may read accumulator `buf`
      }
    }
  } else if (warp == TMA_WARP) {
    // ------------------------------- activation tiles by TMA: one thread per CTA -------------------------------
    if (DENSE_A && lane == 0) {
      const uint32_t full_leader = map_to_cta(afull0, 0);
      uint32_t st = 0, ph = 0;
      bool first_round = true;
      for (int tile = pair_id; tile < ntiles && !*abort_flag; tile += npairs) {
        const int n0 = (tile / tiles_m) * 256 + (int)rank * 128;       // rows past the last token read as zeros
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!first_round) mbar_wait(aempty0 + 8 * st, ph ^ 1, abort_flag, status, WAIT_EMPTY);
          if (*abort_flag) break;
          mbar_arrive_expect_tx_cluster(full_leader + 8 * st, PA_BYTES);
          const uint32_t dst = smem_u32(smem + st * PA_BYTES);
          tma_load_box(dst, &tmap_a, kb * PBK, n0, full_leader + 8 * st);
          tma_load_box(dst + ATOM_BYTES, &tmap_a, kb * PBK + BK, n0, full_leader + 8 * st);
          if (++st == DA_STAGES) { st = 0; ph ^= 1; first_round = false; }
        }
      }
      // after a wait gave up somewhere, tiles requested above may still be on their way into this CTA's shared memory:
      // give them time to land before the CTA ends (they complete within microseconds)
      if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) {}
      }
    }
  } else if (warp >= DECODE_THREADS / 32) {
    // ------------------------------- epilogue warps (4 per CTA) -------------------------------
    const int q = warp & 3;                          // TMEM lane quarter of this warp
    // (packed form) the weight norms r' of the tile's 256 columns, one copy per warp, fetched before the warp waits for
    // the accumulator so that the epilogue of a pair's last tile does not wait for them chunk by chunk
    uint4* wn_s = reinterpret_cast<uint4*>(smem + PSTAGES * PSTAGE_BYTES + 256) + q * 32;
    uint32_t lt = 0;
    for (int tile = pair_id; tile < ntiles; tile += npairs, ++lt) {
      const uint32_t buf = lt & 1;
      const int n0 = (DENSE_A ? tile / tiles_m : tile % tiles_n) * 256 + (int)rank * 128;
      const int i0 = (DENSE_A ? tile % tiles_m : tile / tiles_n) * 256;
      if constexpr (!DENSE_A) {
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (i0 + lane * 8 < m) v = __ldg(reinterpret_cast<const uint4*>(w_norm + i0 + lane * 8));
        __syncwarp();                                  // the other lanes have read the previous tile's copy
        wn_s[lane] = v;
        __syncwarp();
      }
      if (lane == 0) mbar_wait(accfull0 + 8 * buf, (lt >> 1) & 1, abort_flag, status, WAIT_ACC_FULL);
      __syncwarp();
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int trow = n0 + q * 32 + lane;
      const float s = trow < n_tokens ? a_norm[trow] : 0.f;
#pragma unroll 1
      for (int c = 0; c < 8; ++c) {
        uint32_t r[32];
        tmem_load32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 256 + c * 32), r);
        if constexpr (F32_OUT) {
          if (trow < n_tokens) {
#pragma unroll
            for (int g8 = 0; g8 < 4; ++g8) {
              const int i = i0 + c * 32 + g8 * 8;
              if (i < m) {
                const uint4 rn = DENSE_A ? __ldg(reinterpret_cast<const uint4*>(w_norm + i)) : wn_s[c * 4 + g8];
                const uint32_t rw[4] = {rn.x, rn.y, rn.z, rn.w};
                float y[8];
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                  y[2 * jj] = (__uint_as_float(r[g8 * 8 + 2 * jj]) * s) * __uint_as_float(rw[jj] << 16);
                  y[2 * jj + 1] = (__uint_as_float(r[g8 * 8 + 2 * jj + 1]) * s) * __uint_as_float(rw[jj] & 0xFFFF0000u);
                }
                float* dst = reinterpret_cast<float*>(Y) + (size_t)trow * ldy + i;
                *reinterpret_cast<float4*>(dst) = make_float4(y[0], y[1], y[2], y[3]);
                *reinterpret_cast<float4*>(dst + 4) = make_float4(y[4], y[5], y[6], y[7]);
              }
            }
          }
        } else {
          // bf16: a thread holds 64 contiguous bytes of its row (four 16-byte chunks).  Neighbouring lanes (rows t, t + 1)
          // swap two chunks each, so that every store instruction writes whole 32-byte sectors: lane pair (2j, 2j + 1)
          // stores chunks (0, 1) and (2, 3) of row t, then of row t + 1.
          uint4 pk[4];
#pragma unroll
          for (int g8 = 0; g8 < 4; ++g8) {
            const int i = i0 + c * 32 + g8 * 8;
            pk[g8] = make_uint4(0u, 0u, 0u, 0u);
            if (i < m) {                               // (uniform over the warp)
              const uint4 rn = DENSE_A ? __ldg(reinterpret_cast<const uint4*>(w_norm + i)) : wn_s[c * 4 + g8];
              const uint32_t rw[4] = {rn.x, rn.y, rn.z, rn.w};
              float y[8];
#pragma unroll
              for (int jj = 0; jj < 4; ++jj) {
                y[2 * jj] = (__uint_as_float(r[g8 * 8 + 2 * jj]) * s) * __uint_as_float(rw[jj] << 16);
                y[2 * jj + 1] = (__uint_as_float(r[g8 * 8 + 2 * jj + 1]) * s) * __uint_as_float(rw[jj] & 0xFFFF0000u);
              }
              __nv_bfloat162 p0 = __floats2bfloat162_rn(y[0], y[1]), p1 = __floats2bfloat162_rn(y[2], y[3]);
              __nv_bfloat162 p2 = __floats2bfloat162_rn(y[4], y[5]), p3 = __floats2bfloat162_rn(y[6], y[7]);
              pk[g8].x = *reinterpret_cast<uint32_t*>(&p0); pk[g8].y = *reinterpret_cast<uint32_t*>(&p1);
              pk[g8].z = *reinterpret_cast<uint32_t*>(&p2); pk[g8].w = *reinterpret_cast<uint32_t*>(&p3);
            }
          }
          const bool odd = lane & 1;
          const uint4 s0 = odd ? pk[0] : pk[1], s1 = odd ? pk[2] : pk[3];
          uint4 r0, r1;
          r0.x = __shfl_xor_sync(0xffffffffu, s0.x, 1); r0.y = __shfl_xor_sync(0xffffffffu, s0.y, 1);
          r0.z = __shfl_xor_sync(0xffffffffu, s0.z, 1); r0.w = __shfl_xor_sync(0xffffffffu, s0.w, 1);
          r1.x = __shfl_xor_sync(0xffffffffu, s1.x, 1); r1.y = __shfl_xor_sync(0xffffffffu, s1.y, 1);
          r1.z = __shfl_xor_sync(0xffffffffu, s1.z, 1); r1.w = __shfl_xor_sync(0xffffffffu, s1.w, 1);
          const int row_a = odd ? trow - 1 : trow, row_b = row_a + 1;
          const uint4 a0 = odd ? r0 : pk[0], a1 = odd ? r1 : pk[2];
          const uint4 b0 = odd ? pk[1] : r0, b1 = odd ? pk[3] : r1;
          const int ca = i0 + c * 32 + (odd ? 8 : 0);
          __nv_bfloat16* Yb = reinterpret_cast<__nv_bfloat16*>(Y);
          if (row_a < n_tokens) {
            if (ca < m) *reinterpret_cast<uint4*>(Yb + (size_t)row_a * ldy + ca) = a0;
            if (ca + 16 < m) *reinterpret_cast<uint4*>(Yb + (size_t)row_a * ldy + ca + 16) = a1;
          }
          if (row_b < n_tokens) {
            if (ca < m) *reinterpret_cast<uint4*>(Yb + (size_t)row_b * ldy + ca) = b0;
            if (ca + 16 < m) *reinterpret_cast<uint4*>(Yb + (size_t)row_b * ldy + ca + 16) = b1;
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(accempty0 + 8 * buf, 0);   // CTA 0 may let the MMAs overwrite `buf`
    }
  } else {
    // ------------------------------- decoders (16 warps per CTA) -------------------------------
    // threads 0-255: this CTA's 128 rows of A; threads 256-511: its 128 rows of B (all 512 on B when A comes by TMA)
    if constexpr (DENSE_A) {
      const Tables tw = make_tables(cbw);
      dense_b_decode_loop<BITS_W>(Wq, m, dim, tw, smem, full0, empty0, tid, rank, pair_id, npairs, ntiles, tiles_m,
                                  kblocks, abort_flag, status);
    } else if (tid < 256) {
      const Tables ta = make_tables(cba);
      pair_decode_loop<(DENSE_A ? 4 : BITS_A), true>(Aq, n_tokens, dim, ta, smem, full0, empty0, tid, rank, pair_id, npairs, ntiles,
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


// ---------------------------------------------------------------------------------------------------------
// Variant with the ACTIVATION operand in tensor memory (packed activations, bf16 output).  The decoders of A write
// their bf16 levels with tcgen05.st into a ring of four 64-column stages (lane = token row, a column = two
// coordinates) and tcgen05.mma takes A from there, so shared memory carries only the weights (four 32 KB stages): per
// 128-coordinate stage and SM 96 KB of shared-memory traffic instead of 160 KB.  The ring takes the columns of the
// second accumulator, so the epilogue does not overlap the next tile's MMAs; it is made short instead: the four
// epilogue warps move the scaled, rounded tile into a shared-memory staging area (64 KB, 16-byte units XOR-ed with the
// row so that both sides are conflict-free), hand the accumulator back, and only then write the rows out (whole 512-byte
// row segments per instruction), which overlaps the next tile's main loop.
namespace pairt {
constexpr int TSTAGES = 4;
constexpr uint32_t TB_BYTES = pair::PB_BYTES;                      // 32 KB of weights per stage and CTA
constexpr uint32_t STAGING_OFF = TSTAGES * TB_BYTES;               // 128 KB
constexpr uint32_t STAGING_WARP = 32 * 512;                        // 32 rows x 256 bf16 per epilogue warp
constexpr uint32_t TBAR_OFF = STAGING_OFF + 4 * STAGING_WARP;      // 192 KB
constexpr size_t TSMEM_BYTES = TBAR_OFF + 1024 + 256 + 4096;       // + alignment slack, barriers, the epilogue warps' weight norms (fp32)
constexpr int TTHREADS = DECODE_THREADS + pair::EPI_THREADS + 32;  // 16 decode warps, 4 epilogue warps, 1 MMA warp
constexpr uint32_t A_COL0 = 256;                                   // columns 0..255: the accumulator
}  // namespace pairt

template <int BITS_A, int BITS_W>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(pairt::TTHREADS, 1)
qlinear_pair_tmem_a_kernel(const uint32_t* __restrict__ Aq, const float* __restrict__ a_norm, int n_tokens,
                           const uint32_t* __restrict__ Wq, const __nv_bfloat16* __restrict__ w_norm, int m, int dim,
                           CodebookParams cba, CodebookParams cbw, __nv_bfloat16* __restrict__ Y, int ldy, int band, int* status) {
  using namespace pair;
  using namespace pairt;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + TBAR_OFF);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * TSTAGES + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + TSTAGES);
  const uint32_t accfull = smem_u32(bars + 2 * TSTAGES), accempty = smem_u32(bars + 2 * TSTAGES + 1);
  constexpr int MMA_WARP = (DECODE_THREADS + EPI_THREADS) / 32;

  if (tid == 0) {
    for (int s = 0; s < TSTAGES; ++s) {
      mbar_init(full0 + 8 * s, 2 * (DECODE_THREADS / 32));   // one arrival per decoding warp of BOTH CTAs (used in CTA 0)
      mbar_init(empty0 + 8 * s, 1);                          // multicast commit
    }
    mbar_init(accfull, 1);                                   // multicast commit
    mbar_init(accempty, 2 * (EPI_THREADS / 32));             // epilogue warps of both CTAs (used in CTA 0)
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
  cluster_sync_all();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *tmem_slot;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const int kblocks = dim / PBK;
  const int tiles_n = (n_tokens + 255) / 256;
  const int tiles_m = (m + 255) / 256;
  const int ntiles = tiles_n * tiles_m;
  const int npairs = gridDim.x >> 1, pair_id = blockIdx.x >> 1;

  if (warp == MMA_WARP) {
    // ------------------------------- MMA issuer: one thread of CTA 0 -------------------------------
    if (rank == 0 && lane == 0) {
      uint32_t st = 0, ph = 0, lt = 0;
      constexpr uint32_t IDESC2 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
      for (int tile = pair_id; tile < ntiles; tile += npairs, ++lt) {
        if (lt >= 1) mbar_wait_cluster(accempty, (lt - 1) & 1, abort_flag, status, WAIT_ACC_EMPTY);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        for (int kb = 0; kb < kblocks; ++kb) {
          mbar_wait_cluster(full0 + 8 * st, ph, abort_flag, status, WAIT_FULL);
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_tmem = tmem + A_COL0 + st * 64u;                 // 8 columns (16 coordinates) per K step
          const uint32_t b_addr = smem_u32(smem + st * TB_BYTES);
#pragma unroll
          for (int k4 = 0; k4 < PBK / 16; ++k4) {
            const uint64_t db = smem_desc(b_addr + (k4 >> 2) * ATOM_BYTES) + 2 * (k4 & 3);
            const uint32_t acc = (kb > 0 || k4 > 0) ? 1u : 0u;
            asm volatile(
                "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                " tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n}"
                ::"r"(tmem), "r"(a_tmem + 8u * k4), "l"(db), "r"(IDESC2), "r"(acc) : "memory");
          }
          commit_multicast(empty0 + 8 * st);       // both CTAs may refill the stage once these MMAs have read it
          if (++st == TSTAGES) { st = 0; ph ^= 1; }
        }
        commit_multicast(accfull);                 // both CTAs' epilogue warps may read the accumulator
      }
    }
  } else if (warp >= DECODE_THREADS / 32) {
    // ------------------------------- epilogue warps (4 per CTA) -------------------------------
    const int q = warp & 3;                          // TMEM lane quarter of this warp
    float* wn_s = reinterpret_cast<float*>(smem + TBAR_OFF + 256) + q * 256;     // weight norms r' of the tile's 256 columns, fp32
    unsigned char* stage_w = smem + STAGING_OFF + (uint32_t)q * STAGING_WARP;   // this warp's 32 rows x 512 bytes
    const uint32_t acc_thr = tmem + ((uint32_t)(q * 32) << 16);
    uint32_t lt = 0;
    for (int tile = pair_id; tile < ntiles; tile += npairs, ++lt) {
      int rt, ct;
      banded_tile(tile, tiles_n, tiles_m, band, rt, ct);
      const int n0 = rt * 256 + (int)rank * 128;
      const int i0 = ct * 256;
      {
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (i0 + lane * 8 < m) v = __ldg(reinterpret_cast<const uint4*>(w_norm + i0 + lane * 8));
        __syncwarp();                                  // the other lanes have read the previous tile's copy
        reinterpret_cast<float4*>(wn_s)[2 * lane] = make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u),
                                                                  __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xFFFF0000u));
        reinterpret_cast<float4*>(wn_s)[2 * lane + 1] = make_float4(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xFFFF0000u),
                                                                      __uint_as_float(v.w << 16), __uint_as_float(v.w & 0xFFFF0000u));
        __syncwarp();
      }
      const int trow = n0 + q * 32 + lane;
      const float s = trow < n_tokens ? a_norm[trow] : 0.f;
      if (lane == 0) mbar_wait(accfull, lt & 1, abort_flag, status, WAIT_ACC_FULL);
      __syncwarp();
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      unsigned char* my_row = stage_w + (uint32_t)lane * 512u;
      // 16 pieces of 16 columns; the load of a piece is in flight while the one before it is scaled, rounded and staged
      auto stage16 = [&](const uint32_t (&r)[16], int pc) {
#pragma unroll
        for (int g8 = 0; g8 < 2; ++g8) {
          const float4 ra = reinterpret_cast<const float4*>(wn_s)[pc * 4 + g8 * 2], rb = reinterpret_cast<const float4*>(wn_s)[pc * 4 + g8 * 2 + 1];
          const float rw[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
          float y[8];
#pragma unroll
          for (int jj = 0; jj < 8; ++jj) y[jj] = (__uint_as_float(r[g8 * 8 + jj]) * s) * rw[jj];
          __nv_bfloat162 p0 = __floats2bfloat162_rn(y[0], y[1]), p1 = __floats2bfloat162_rn(y[2], y[3]);
          __nv_bfloat162 p2 = __floats2bfloat162_rn(y[4], y[5]), p3 = __floats2bfloat162_rn(y[6], y[7]);
          const uint4 pk = make_uint4(*reinterpret_cast<uint32_t*>(&p0), *reinterpret_cast<uint32_t*>(&p1),
                                      *reinterpret_cast<uint32_t*>(&p2), *reinterpret_cast<uint32_t*>(&p3));
          // 16-byte unit u = 2 pc + g8 of the row sits at position u ^ lane
          *reinterpret_cast<uint4*>(my_row + ((uint32_t)((pc * 2 + g8) ^ lane) << 4)) = pk;
        }
      };
      uint32_t ra[16], rb[16];
      tmem_load16_nowait(acc_thr, ra);
#pragma unroll 1
      for (int pc = 0; pc < 16; pc += 2) {
        tmem_wait_ld();
        tmem_load16_nowait(acc_thr + (uint32_t)(pc + 1) * 16u, rb);
        stage16(ra, pc);
        tmem_wait_ld();
        if (pc + 2 < 16) tmem_load16_nowait(acc_thr + (uint32_t)(pc + 2) * 16u, ra);
        stage16(rb, pc + 1);
      }
      // the accumulator has been read: the MMAs of the pair's next tile may overwrite it
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(accempty, 0);
      // rows out: lane L moves unit L of every row (512 contiguous bytes per instruction)
      const int col = i0 + lane * 8;
#pragma unroll 4
      for (int rr = 0; rr < 32; ++rr) {
        const int row = n0 + q * 32 + rr;
        const uint4 v = *reinterpret_cast<const uint4*>(stage_w + (uint32_t)rr * 512u + ((uint32_t)(lane ^ rr) << 4));
        if (row < n_tokens && col < m) *reinterpret_cast<uint4*>(Y + (size_t)row * ldy + col) = v;
      }
      __syncwarp();                                    // the staging rows are rewritten by the next tile
    }
  } else if (tid < 256) {
    // ------------------------------- decoders of A (8 warps): packed indices -> bf16 levels in tensor memory -------------------------------
    // warp = (lane quarter, 64-coordinate half of the stage); thread = one token row, 64 coordinates per stage
    const Tables ta = make_tables(cba);
    const int quarter = warp & 3, khalf = warp >> 2;
    const int row = quarter * 32 + lane;
    const int pitch = dim / 32 * BITS_A;
    const uint32_t a_thr = tmem + ((uint32_t)(quarter * 32) << 16) + A_COL0 + (uint32_t)khalf * 32u;   // + 64 * stage
    uint32_t st = 0, ph = 0;
    bool first_round = true;
    Raw<BITS_A> n0r, n1r;                              // packed words of the NEXT stage
    int f_tile = pair_id, f_kb = 0;
    const uint32_t* fsrc = nullptr;
    auto set_fetch_tile = [&](int tile) {
      int rt, ct;
      banded_tile(tile, tiles_n, tiles_m, band, rt, ct);
      const int r0 = rt * 256 + (int)rank * 128;
      fsrc = Aq + (size_t)min(r0 + row, n_tokens - 1) * pitch + khalf * 2 * BITS_A;   // rows past the end re-read the last
    };
    auto fetch_next = [&]() {
      if (f_tile >= ntiles) return;
      load_raw64<BITS_A>(fsrc, n0r, n1r);
      fsrc += 4 * BITS_A;
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
        const Raw<BITS_A> c0 = n0r, c1 = n1r;
        fetch_next();
        uint4 v0[4], v1[4];
        decode32<BITS_A>(c0, ta, v0);
        decode32<BITS_A>(c1, ta, v1);
        uint32_t w[32];
#pragma unroll
        for (int qq = 0; qq < 4; ++qq) {
          w[4 * qq] = v0[qq].x; w[4 * qq + 1] = v0[qq].y; w[4 * qq + 2] = v0[qq].z; w[4 * qq + 3] = v0[qq].w;
          w[16 + 4 * qq] = v1[qq].x; w[16 + 4 * qq + 1] = v1[qq].y; w[16 + 4 * qq + 2] = v1[qq].z; w[16 + 4 * qq + 3] = v1[qq].w;
        }
        if (!first_round) {
          if (lane == 0) mbar_wait(empty0 + 8 * st, ph ^ 1, abort_flag, status, WAIT_EMPTY);
          __syncwarp();
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        tmem_store32(a_thr + st * 64u, w);
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(full0 + 8 * st, 0);
        if (++st == TSTAGES) { st = 0; ph ^= 1; first_round = false; }
      }
    }
  } else {
    // ------------------------------- decoders of the weights (8 warps) -------------------------------
    const Tables tw = make_tables(cbw);
    pair_decode_loop<BITS_W, false, TB_BYTES, TSTAGES, 0u, true>(Wq, m, dim, tw, smem, full0, empty0, tid - 256, rank, pair_id, npairs,
                                                                  ntiles, tiles_n, kblocks, abort_flag, status, tiles_m, band);
  }
  __syncwarp();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();
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

// Writes an operand out as bf16 levels: thread = 32 consecutive coordinates of one row.
template <int BITS>
__global__ void decode_levels_kernel(const uint32_t* __restrict__ packed, int rows, int dim, CodebookParams cb,
                                     __nv_bfloat16* __restrict__ out, int ldo) {
  const Tables t = make_tables(cb);
  const int per_row = dim / 32, pitch = per_row * BITS;
  const long long total = (long long)rows * per_row;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int row = (int)(i / per_row), c = (int)(i - (long long)row * per_row);
    const Raw<BITS> raw = load_raw<BITS>(packed + (size_t)row * pitch + c * BITS);
    uint4 v[4];
    decode32<BITS>(raw, t, v);
    uint4* dst = reinterpret_cast<uint4*>(out + (size_t)row * ldo + c * 32);
#pragma unroll
    for (int q = 0; q < 4; ++q) dst[q] = v[q];
  }
}

// Tensor map of a row-major bf16 matrix [rows][ld] for boxes of 64 coordinates x 128 rows with the 128-byte swizzle
// (the driver entry point is looked up once; no link-time dependency on the driver library).
cudaError_t make_levels_map(const void* base, int rows, int dim, int ld, CUtensorMap* map) {
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                               const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static std::atomic<EncodeFn> encode_cached{nullptr};     // (threads racing here store the same pointer)
  EncodeFn encode = encode_cached.load(std::memory_order_acquire);
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    encode = reinterpret_cast<EncodeFn>(fn);
    encode_cached.store(encode, std::memory_order_release);
  }
  const cuuint64_t gdim[2] = {(cuuint64_t)dim, (cuuint64_t)rows};
  const cuuint64_t gstride[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {(cuuint32_t)BK, 128u};
  const cuuint32_t estride[2] = {1u, 1u};
  const CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estride,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int BA, int BW, bool F32>
cudaError_t launch_pair(const CUtensorMap& tmap, int sms, cudaStream_t st, const uint32_t* Aq, const float* an, int n, const uint32_t* Wq,
                        const __nv_bfloat16* wn, int m, int dim, const CodebookParams& ca, const CodebookParams& cw,
                        void* Y, int ldy, int* status) {
  auto k = qlinear_pair_kernel<BA, BW, F32>;
  constexpr size_t smem_bytes = BA == 0 ? pair::DSMEM_BYTES : pair::PSMEM_BYTES;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
  if (e != cudaSuccess) return e;
  const int ntiles = ((n + 255) / 256) * ((m + 255) / 256);
  // persistent grid: as many pairs as can be resident at once (SM pairs must sit in one cluster-capable group,
  // so this can be fewer than sms / 2)
  static std::atomic<int> max_pairs[64];                    // zero-initialised; threads racing here store the same value
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && max_pairs[dev].load(std::memory_order_relaxed) == 0) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sms / 2 * 2);
    cfg.blockDim = dim3(pair::PTHREADS);
    cfg.dynamicSmemBytes = smem_bytes;
    int nclusters = 0;
    e = cudaOccupancyMaxActiveClusters(&nclusters, k, &cfg);
    if (e != cudaSuccess) return e;
    max_pairs[dev].store(nclusters > 0 ? nclusters : 1, std::memory_order_relaxed);
  }
  int pairs = (dev >= 0 && dev < 64) ? max_pairs[dev].load(std::memory_order_relaxed) : sms / 2;
  if (pairs > sms / 2) pairs = sms / 2;
  if (pairs > ntiles) pairs = ntiles;
  return launch_dependent(k, 2 * pairs, pair::PTHREADS, smem_bytes, st, tmap, Aq, an, n, Wq, wn, m, dim, ca, cw, Y, ldy, status);
}

int g_gemm_kernel = 0;       // oq_debug_select_gemm_kernel: 0 by output type, 1 activation operand in shared memory, 2 in tensor memory,
                             // 3 in tensor memory with the wide tile bands at any size

template <int BA, int BW>
cudaError_t launch_pair_tmem_a(int sms, cudaStream_t st, const uint32_t* Aq, const float* an, int n, const uint32_t* Wq,
                               const __nv_bfloat16* wn, int m, int dim, const CodebookParams& ca, const CodebookParams& cw,
                               void* Y, int ldy, int* status) {
  auto k = qlinear_pair_tmem_a_kernel<BA, BW>;
  constexpr size_t smem_bytes = pairt::TSMEM_BYTES;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
  if (e != cudaSuccess) return e;
  const int ntiles = ((n + 255) / 256) * ((m + 255) / 256);
  static std::atomic<int> max_pairs[64];
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && max_pairs[dev].load(std::memory_order_relaxed) == 0) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sms / 2 * 2);
    cfg.blockDim = dim3(pairt::TTHREADS);
    cfg.dynamicSmemBytes = smem_bytes;
    int nclusters = 0;
    e = cudaOccupancyMaxActiveClusters(&nclusters, k, &cfg);
    if (e != cudaSuccess) return e;
    max_pairs[dev].store(nclusters > 0 ? nclusters : 1, std::memory_order_relaxed);
  }
  int pairs = (dev >= 0 && dev < 64) ? max_pairs[dev].load(std::memory_order_relaxed) : sms / 2;
  if (pairs > sms / 2) pairs = sms / 2;
  if (pairs > ntiles) pairs = ntiles;
  // (see banded_tile) packed activations above 32 MB: bands of 8 column tiles
  const int band = (g_gemm_kernel == 3 || (size_t)n * dim * BA / 8 > ((size_t)32 << 20)) ? TILE_BAND_WIDE : 1;
  return launch_dependent(k, 2 * pairs, pairt::TTHREADS, smem_bytes, st, Aq, an, n, Wq, wn, m, dim, ca, cw,
                          reinterpret_cast<__nv_bfloat16*>(Y), ldy, band, status);
}

template <int BA, int BW>
int launch_bits(bool f32, int sms, cudaStream_t st, const uint32_t* Aq, const float* an, int n, const uint32_t* Wq,
                const __nv_bfloat16* wn, int m, int dim, const CodebookParams& ca, const CodebookParams& cw, void* Y,
                int ldy, int* status) {
  static const CUtensorMap no_map = {};
  // bf16 output: the kernel with the activation operand in tensor memory (8-12 % faster on the benchmark shapes); fp32
  // output: the kernel with both operands in shared memory and two accumulators (an fp32 tile does not fit the staging area)
  if (!f32 && g_gemm_kernel != 1) {
    const cudaError_t e1 = launch_pair_tmem_a<BA, BW>(sms, st, Aq, an, n, Wq, wn, m, dim, ca, cw, Y, ldy, status);
    if (e1 != cudaSuccess) return cuda_fail(e1, "oq_qlinear launch (tensor-memory A)");
    return OQ_OK;
  }
  const cudaError_t e = f32 ? launch_pair<BA, BW, true>(no_map, sms, st, Aq, an, n, Wq, wn, m, dim, ca, cw, Y, ldy, status)
                            : launch_pair<BA, BW, false>(no_map, sms, st, Aq, an, n, Wq, wn, m, dim, ca, cw, Y, ldy, status);
  if (e != cudaSuccess) return cuda_fail(e, "oq_qlinear launch");
  return OQ_OK;
}

// Activations as bf16 levels (fetched by TMA through `tmap`).
template <int BW>
int launch_levels_bits(const CUtensorMap& tmap, bool f32, int sms, cudaStream_t st, const float* an, int n, const uint32_t* Wq,
                       const __nv_bfloat16* wn, int m, int dim, const CodebookParams& cw, void* Y, int ldy, int* status) {
  const cudaError_t e = f32 ? launch_pair<0, BW, true>(tmap, sms, st, nullptr, an, n, Wq, wn, m, dim, cw, cw, Y, ldy, status)
                            : launch_pair<0, BW, false>(tmap, sms, st, nullptr, an, n, Wq, wn, m, dim, cw, cw, Y, ldy, status);
  if (e != cudaSuccess) return cuda_fail(e, "oq_qlinear_levels launch");
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

namespace oq {

int qlinear_levels_launch(const void* Xd_bf16, int ldxd, const float* Xq_norm, int n_tokens, const void* Wq_idx,
                          const void* Wq_norm_bf16, int m, const oq_codebook* cb_w, int dim, void* Y, int ldy, int y_dtype,
                          int* status, void* stream) {
  if (!cb_w) return fail(OQ_ERR_INVALID_ARG, "oq_qlinear_levels: NULL codebook");
  if (n_tokens < 0 || m < 0 || dim <= 0) return fail(OQ_ERR_INVALID_ARG, "oq_qlinear_levels: bad sizes");
  if (cb_w->dim != dim) return fail(OQ_ERR_INVALID_ARG, "oq_qlinear_levels: codebook dim differs from dim");
  if (dim % 128) return fail(OQ_ERR_UNSUPPORTED, "oq_qlinear_levels: dim must be a multiple of 128");
  if (m % 8) return fail(OQ_ERR_UNSUPPORTED, "oq_qlinear_levels: m must be a multiple of 8");
  if (y_dtype != OQ_BF16 && y_dtype != OQ_F32) return fail(OQ_ERR_INVALID_ARG, "oq_qlinear_levels: unknown y_dtype");
  const int bw = cb_w->bits;
  if (bw < 2 || bw > 4) return fail(OQ_ERR_UNSUPPORTED, "oq_qlinear_levels: weight bits must be 2, 3 or 4");
  if (n_tokens == 0 || m == 0) return OQ_OK;
  if (!Xd_bf16 || !Xq_norm || !Wq_idx || !Wq_norm_bf16 || !Y) return fail(OQ_ERR_INVALID_ARG, "oq_qlinear_levels: NULL buffer");
  if (ldy < m || ldxd < dim) return fail(OQ_ERR_INVALID_ARG, "oq_qlinear_levels: leading dimension too small");
  if (ldy % 8 || ldxd % 8 || !aligned16(Xd_bf16) || !aligned16(Wq_idx) || !aligned16(Y) || !aligned16(Wq_norm_bf16))
    return fail(OQ_ERR_ALIGNMENT, "oq_qlinear_levels: pointers must be 16-byte aligned and leading dimensions multiples of 8");
  if (!status) status = device_status_word();
  if (!status) return fail(OQ_ERR_CUDA, "oq_qlinear_levels: cannot allocate the device status word");
  CUtensorMap tmap;
  cudaError_t ce = make_levels_map(Xd_bf16, n_tokens, dim, ldxd, &tmap);
  if (ce != cudaSuccess) return cuda_fail(ce, "oq_qlinear_levels: tensor map");
  const CodebookParams cw = codebook_params(cb_w);
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  ce = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (ce != cudaSuccess) return cuda_fail(ce, "cudaDeviceGetAttribute");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const uint32_t* W = reinterpret_cast<const uint32_t*>(Wq_idx);
  const __nv_bfloat16* wn = reinterpret_cast<const __nv_bfloat16*>(Wq_norm_bf16);
  const bool f32 = y_dtype == OQ_F32;
  if (bw == 4) return launch_levels_bits<4>(tmap, f32, sms, st, Xq_norm, n_tokens, W, wn, m, dim, cw, Y, ldy, status);
  if (bw == 3) return launch_levels_bits<3>(tmap, f32, sms, st, Xq_norm, n_tokens, W, wn, m, dim, cw, Y, ldy, status);
  return launch_levels_bits<2>(tmap, f32, sms, st, Xq_norm, n_tokens, W, wn, m, dim, cw, Y, ldy, status);
}

int decode_levels_launch(const void* idx, int rows, int dim, const oq_codebook* cb, void* out_bf16, int ldo, void* stream) {
  if (!cb) return fail(OQ_ERR_INVALID_ARG, "oq_decode_levels: NULL codebook");
  if (rows < 0 || dim <= 0 || cb->dim != dim) return fail(OQ_ERR_INVALID_ARG, "oq_decode_levels: bad sizes");
  if (dim % 128) return fail(OQ_ERR_UNSUPPORTED, "oq_decode_levels: dim must be a multiple of 128");
  if (cb->bits < 2 || cb->bits > 4) return fail(OQ_ERR_UNSUPPORTED, "oq_decode_levels: bits must be 2, 3 or 4");
  if (rows == 0) return OQ_OK;
  if (!idx || !out_bf16) return fail(OQ_ERR_INVALID_ARG, "oq_decode_levels: NULL buffer");
  if (ldo < dim) return fail(OQ_ERR_INVALID_ARG, "oq_decode_levels: ldo smaller than dim");
  if (ldo % 8 || !aligned16(idx) || !aligned16(out_bf16))
    return fail(OQ_ERR_ALIGNMENT, "oq_decode_levels: pointers must be 16-byte aligned and ldo a multiple of 8");
  const CodebookParams cp = codebook_params(cb);
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
  const long long total = (long long)rows * (dim / 32);
  long long blocks = (total + 255) / 256;
  if (blocks > (long long)sms * 8) blocks = (long long)sms * 8;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const uint32_t* p = reinterpret_cast<const uint32_t*>(idx);
  __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(out_bf16);
  if (cb->bits == 4) e = launch_dependent(decode_levels_kernel<4>, (int)blocks, 256, 0, st, p, rows, dim, cp, o, ldo);
  else if (cb->bits == 3) e = launch_dependent(decode_levels_kernel<3>, (int)blocks, 256, 0, st, p, rows, dim, cp, o, ldo);
  else e = launch_dependent(decode_levels_kernel<2>, (int)blocks, 256, 0, st, p, rows, dim, cp, o, ldo);
  if (e != cudaSuccess) return cuda_fail(e, "oq_decode_levels");
  return OQ_OK;
}

}  // namespace oq

extern "C" int oq_qlinear_levels(const void* Xd_bf16, int ldxd, const float* Xq_norm, int n_tokens, const void* Wq_idx,
                                 const void* Wq_norm_bf16, int m, const oq_codebook* cb_w, int dim, void* Y, int ldy,
                                 int y_dtype, void* stream) {
  return oq::qlinear_levels_launch(Xd_bf16, ldxd, Xq_norm, n_tokens, Wq_idx, Wq_norm_bf16, m, cb_w, dim, Y, ldy, y_dtype,
                                   nullptr, stream);
}

extern "C" int oq_decode_levels(const void* idx, int rows, int dim, const oq_codebook* cb, void* out_bf16, int ldo,
                                void* stream) {
  return oq::decode_levels_launch(idx, rows, dim, cb, out_bf16, ldo, stream);
}

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

extern "C" int oq_debug_select_gemm_kernel(int which) {
  if (which < 0 || which > 3) return oq::fail(OQ_ERR_INVALID_ARG, "oq_debug_select_gemm_kernel: unknown kernel");
  oq::g_gemm_kernel = which;
  return OQ_OK;
}
