// Codebook-decode GEMM:  Y[n][i] = s_n * r'_i * sum_k C_a[idxA[n][k]] * C_w[idxW[i][k]]
// (the product W^' x^' of Sec. 4.3 with the magnitudes of Eq. 6 and Eq. 8 applied in the epilogue).
//
// Packed indices are fetched from global memory, decoded to bf16 levels with byte-permute table
// look-ups, written into shared memory in the tensor core's K-major 128-byte-swizzled layout, and
// contracted with tcgen05.mma (fp32 accumulators in tensor memory).
#include <cuda_bf16.h>

#include "oq_internal.h"

namespace oq {

namespace {

constexpr int BM = 256;   // tokens per tile: two MMAs of M = 128, one accumulator each
constexpr int BN_MAX = 256;   // features per tile (MMA N): 256, or 192 when that fills the last wave better
constexpr int BK = 64;    // coordinates per stage: 64 bf16 = one 128-byte swizzled row
constexpr int STAGES = 3;
constexpr int DECODE_THREADS = 512;            // 16 warps decode and, after the last stage, run the epilogue
constexpr int THREADS = DECODE_THREADS + 32;   // + one warp whose lane 0 issues the MMAs
constexpr int TMEM_COLS = 512;                 // 2 accumulators x 256 fp32 columns
constexpr uint32_t A_BYTES = BM * BK * 2, B_BYTES = BN_MAX * BK * 2;
constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
constexpr size_t SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr long long WAIT_CYCLES = 4000000000ll;   // ~2 s: a wait that lasts longer reports and gives up

enum { WAIT_EMPTY = 1, WAIT_FULL = 2, WAIT_ACC_FULL = 3, WAIT_ACC_EMPTY = 4, WAIT_SELFTEST = 9 };

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  On expiry (or when another thread of the CTA / any CTA already gave up) it records
// `code` in the global status word, raises the CTA's abort flag and returns; callers carry on to the
// common tear-down so tensor memory is always released.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                          int code, long long max_cycles = WAIT_CYCLES) {
  if (mbar_try(bar, parity)) return;
  const long long t0 = clock64();
  int polls = 0;
  while (!mbar_try(bar, parity)) {
    if (*abort_flag) return;
    if ((++polls & 1023) == 0) {
      if (*reinterpret_cast<volatile int*>(status) != 0 || clock64() - t0 > max_cycles) {
        atomicCAS(status, 0, code);
        *abort_flag = 1;
        return;
      }
    }
  }
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

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
    uint32_t r[16];
#pragma unroll
    for (int G = 0; G < 8; ++G) {
      uint32_t sel;
      if (BITS == 3) sel = (mw[G >> 2] >> (2 * (G & 1) + 16 * ((G >> 1) & 1))) & 0x3333u;
      else sel = (mw[0] >> ((G & 3) + 16 * (G >> 2))) & 0x1111u;
      const uint32_t lo = prmt(t.lo0, t.lo0, sel);
      const uint32_t hi = prmt(t.hi0, t.hi0, sel) ^ ((s << G) & 0x80808080u);
      r[2 * G] = prmt(lo, hi, 0x5140u);
      r[2 * G + 1] = prmt(lo, hi, 0x7362u);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) out[q] = make_uint4(r[4 * q], r[4 * q + 1], r[4 * q + 2], r[4 * q + 3]);
  }
}

// Shared-memory matrix descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: D = f32, A = B = bf16, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t idesc_for(int n) { return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24); }

template <int BITS_A, int BITS_W, bool F32_OUT, int BN>
__global__ void __launch_bounds__(THREADS, 1)
qlinear_kernel(const uint32_t* __restrict__ Aq, const float* __restrict__ a_norm, int n_tokens,
               const uint32_t* __restrict__ Wq, const __nv_bfloat16* __restrict__ w_norm, int m, int dim,
               CodebookParams cba, CodebookParams cbw, void* __restrict__ Y, int ldy, int* status) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + STAGES);
  const uint32_t accfull = smem_u32(bars + 2 * STAGES), accempty = smem_u32(bars + 2 * STAGES + 1);

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full0 + 8 * s, DECODE_THREADS);   // every decoding thread arrives once per stage
      mbar_init(empty0 + 8 * s, 1);               // tcgen05.commit arrives once the MMAs have read the stage
    }
    mbar_init(accfull, 1);                        // tcgen05.commit after the last stage of a tile
    mbar_init(accempty, DECODE_THREADS);          // every epilogue thread arrives after reading its columns
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *tmem_slot;

  const int kblocks = dim / BK;
  const int tiles_n = (n_tokens + BM - 1) / BM, tiles_m = (m + BN - 1) / BN;
  const int ntiles = tiles_n * tiles_m;   // token tiles vary fastest: CTAs running together share weight rows

  if (warp == DECODE_THREADS / 32) {
    // ------------------------------- MMA issuer (one thread) -------------------------------
    if (lane == 0) {
      uint32_t st = 0, ph = 0, lt = 0;
      for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++lt) {
        if (lt > 0) mbar_wait(accempty, (lt - 1) & 1, abort_flag, status, WAIT_ACC_EMPTY);   // epilogue drained TMEM
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        for (int kb = 0; kb < kblocks; ++kb) {
          mbar_wait(full0 + 8 * st, ph, abort_flag, status, WAIT_FULL);
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = smem_u32(smem + st * STAGE_BYTES);
          const uint64_t da0 = smem_desc(a_addr), da1 = smem_desc(a_addr + 128 * 128), db = smem_desc(a_addr + A_BYTES);
#pragma unroll
          for (int k4 = 0; k4 < BK / 16; ++k4) {
            const uint32_t acc = (kb > 0 || k4 > 0) ? 1u : 0u;
            asm volatile(
                "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                ::"r"(tmem), "l"(da0 + 2 * k4), "l"(db + 2 * k4), "r"(idesc_for(BN)), "r"(acc) : "memory");
            asm volatile(
                "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                ::"r"(tmem + BN), "l"(da1 + 2 * k4), "l"(db + 2 * k4), "r"(idesc_for(BN)), "r"(acc) : "memory");
          }
          // arrives on empty[st] once every MMA issued so far has finished reading shared memory
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(empty0 + 8 * st) : "memory");
          if (++st == STAGES) { st = 0; ph ^= 1; }
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(accfull) : "memory");
      }
    }
  } else {
    // ------------------- decoders (all 16 warps), then the epilogue of the tile -------------------
    const Tables ta = make_tables(cba), tw = make_tables(cbw);
    const int pitch_a = dim / 32 * BITS_A, pitch_w = dim / 32 * BITS_W;   // words per packed row
    const int row = tid >> 1, half = tid & 1;          // one (row, 32-coordinate half) of A and one of B per stage
    uint32_t st = 0, ph = 0, lt = 0;   // ring slot, phase parity of its current round, local tile count
    bool first_round = true;           // nothing to wait for while the ring is filled for the first time
    // byte offsets of this thread's four 16-byte chunks inside a K-major 128-byte-swizzled tile:
    // row r occupies 128 bytes, its chunk c sits at chunk position c ^ (r & 7)
    uint32_t toff[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) toff[q] = (uint32_t)row * 128u + ((uint32_t)((half * 4 + q) ^ (row & 7)) << 4);
    // Packed words are fetched PF stages ahead of their decode (global/L2 latency under load is longer than
    // one stage): ring of PF register sets, slot (stage index % PF).  dim % 128 == 0 makes the number of
    // stages per tile even, so with PF = 2 the slot of a stage is the parity of its K block in every tile.
    constexpr int PF = 2;
    Raw<BITS_A> ra[PF];
    Raw<BITS_W> rb[PF];
    // position of the fetch stream: tile and K block of the next stage to fetch
    int f_tile = blockIdx.x, f_kb = 0;
    const uint32_t* fa = nullptr;
    const uint32_t* fb = nullptr;
    auto set_fetch_tile = [&](int tile) {
      const int n0 = (tile % tiles_n) * BM, i0 = (tile / tiles_n) * BN;
      fa = Aq + (size_t)min(n0 + row, n_tokens - 1) * pitch_a + half * BITS_A;   // rows past the end re-read the last
      fb = Wq + (size_t)min(i0 + row, m - 1) * pitch_w + half * BITS_W;          // row; their outputs are never stored
    };
    auto fetch_next = [&](Raw<BITS_A>& da, Raw<BITS_W>& db) {
      if (f_tile >= ntiles) return;
      da = load_raw<BITS_A>(fa);
      db = load_raw<BITS_W>(fb);
      fa += 2 * BITS_A;
      fb += 2 * BITS_W;
      if (++f_kb == kblocks) {
        f_kb = 0;
        f_tile += gridDim.x;
        if (f_tile < ntiles) set_fetch_tile(f_tile);
      }
    };
    if (f_tile < ntiles) set_fetch_tile(f_tile);
#pragma unroll
    for (int i = 0; i < PF; ++i) fetch_next(ra[i], rb[i]);
    auto epilogue = [&](int tile, uint32_t lt) {
      const int n0 = (tile % tiles_n) * BM, i0 = (tile / tiles_n) * BN;
      // ---- epilogue: warp w reads TMEM lanes 32 (w % 4) .., columns 128 (w / 4) ..; lane = one token row ----
      mbar_wait(accfull, lt & 1, abort_flag, status, WAIT_ACC_FULL);
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      __syncwarp();   // the per-thread wait loops may leave the warp diverged; tcgen05.ld is warp-collective
      {
        const int cg = warp >> 2;                        // column group: accumulator cg / 2, feature half cg % 2
        const int trow = n0 + (cg >> 1) * 128 + (warp & 3) * 32 + lane;
        const float s = trow < n_tokens ? a_norm[trow] : 0.f;
#pragma unroll 1
        for (int c = 0; c < BN / 64; ++c) {
          const int fcol = (cg & 1) * (BN / 2) + c * 32;   // feature offset inside the tile
          uint32_t r[32];
          const uint32_t taddr = tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((cg >> 1) * BN + fcol);
          asm volatile(
              "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
              "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
              : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
                "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
                "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
              : "r"(taddr)
              : "memory");
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          if (trow < n_tokens) {
#pragma unroll
            for (int g8 = 0; g8 < 4; ++g8) {   // 8 features per group
              const int i = i0 + fcol + g8 * 8;
              if (i < m) {
                const uint4 rn = __ldg(reinterpret_cast<const uint4*>(w_norm + i));   // 8 bf16 row norms
                const uint32_t rw[4] = {rn.x, rn.y, rn.z, rn.w};
                float y[8];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  y[2 * j] = (__uint_as_float(r[g8 * 8 + 2 * j]) * s) * __uint_as_float(rw[j] << 16);
                  y[2 * j + 1] = (__uint_as_float(r[g8 * 8 + 2 * j + 1]) * s) * __uint_as_float(rw[j] & 0xFFFF0000u);
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
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive(accempty);   // this thread's TMEM reads are done: the next tile may overwrite the accumulators
    };
    for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++lt) {
     for (int kb = 0; kb < kblocks; kb += PF) {
#pragma unroll
      for (int u = 0; u < PF; ++u) {      // u = register set of this stage
        const Raw<BITS_A> ca = ra[u];
        const Raw<BITS_W> cb = rb[u];
        fetch_next(ra[u], rb[u]);          // the stage PF ahead goes into the register set just freed
        if (!first_round) mbar_wait(empty0 + 8 * st, ph ^ 1, abort_flag, status, WAIT_EMPTY);
        unsigned char* As = smem + st * STAGE_BYTES;
        uint4 v[4];
        decode32<BITS_A>(ca, ta, v);
#pragma unroll
        for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4*>(As + toff[q]) = v[q];
        if (BN == BN_MAX || row < BN) {
          decode32<BITS_W>(cb, tw, v);
#pragma unroll
          for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4*>(As + A_BYTES + toff[q]) = v[q];
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy stores -> visible to the MMA
        mbar_arrive(full0 + 8 * st);
        if (++st == STAGES) { st = 0; ph ^= 1; first_round = false; }
      }
     }
     epilogue(tile, lt);
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
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

template <int BA, int BW, bool F32, int BN>
cudaError_t launch_one(dim3 grid, cudaStream_t st, const uint32_t* Aq, const float* an, int n, const uint32_t* Wq,
                       const __nv_bfloat16* wn, int m, int dim, const CodebookParams& ca, const CodebookParams& cw,
                       void* Y, int ldy, int* status) {
  auto k = qlinear_kernel<BA, BW, F32, BN>;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
  if (e != cudaSuccess) return e;
  k<<<grid, THREADS, SMEM_BYTES, st>>>(Aq, an, n, Wq, wn, m, dim, ca, cw, Y, ldy, status);
  return cudaGetLastError();
}

template <int BA, int BW>
int launch_bits(bool f32, int bn, dim3 grid, cudaStream_t st, const uint32_t* Aq, const float* an, int n,
                const uint32_t* Wq, const __nv_bfloat16* wn, int m, int dim, const CodebookParams& ca,
                const CodebookParams& cw, void* Y, int ldy, int* status) {
  cudaError_t e;
  if (f32) {
    e = bn == 256 ? launch_one<BA, BW, true, 256>(grid, st, Aq, an, n, Wq, wn, m, dim, ca, cw, Y, ldy, status)
                  : launch_one<BA, BW, true, 192>(grid, st, Aq, an, n, Wq, wn, m, dim, ca, cw, Y, ldy, status);
  } else {
    e = bn == 256 ? launch_one<BA, BW, false, 256>(grid, st, Aq, an, n, Wq, wn, m, dim, ca, cw, Y, ldy, status)
                  : launch_one<BA, BW, false, 192>(grid, st, Aq, an, n, Wq, wn, m, dim, ca, cw, Y, ldy, status);
  }
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
  // Tile width: 256 features, or 192 when the narrower tiles leave less of the last wave empty
  // (a 192-wide tile does 3/4 of the work at roughly 9/10 of the efficiency).
  const int tiles_tok = (n_tokens + BM - 1) / BM;
  const int t256 = tiles_tok * ((m + 255) / 256), t192 = tiles_tok * ((m + 191) / 192);
  const double cost256 = (double)((t256 + sms - 1) / sms), cost192 = 0.85 * (double)((t192 + sms - 1) / sms);
  const int bn = cost192 < cost256 ? 192 : 256;
  const int ntiles = bn == 256 ? t256 : t192;
  dim3 grid(ntiles < sms ? ntiles : sms);   // persistent: one CTA per SM walks the tiles
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const uint32_t* A = reinterpret_cast<const uint32_t*>(Xq_idx);
  const uint32_t* W = reinterpret_cast<const uint32_t*>(Wq_idx);
  const __nv_bfloat16* wn = reinterpret_cast<const __nv_bfloat16*>(Wq_norm_bf16);
  const bool f32 = y_dtype == OQ_F32;
#define OQ_CASE(a, w) \
  if (ba == a && bw == w) return launch_bits<a, w>(f32, bn, grid, st, A, Xq_norm, n_tokens, W, wn, m, dim, ca, cw, Y, ldy, status);
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
