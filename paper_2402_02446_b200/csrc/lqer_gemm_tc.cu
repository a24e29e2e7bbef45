// Main GEMM of the prefill path on the 5th-generation tensor cores (paper Section 3.1 /
// 3.2: the low-precision product X W_q and the correction (X A_k) B_k, with the "regular,
// blocked, no scatter/gather" pattern realised as ONE contraction over the concatenated
// K dimension):
//
//     Y[M,N] = [X_q | T_q] . [W_q ; B_q]
//
// Every operand element is m * 2^s with |m| <= 127, which bf16 holds exactly, so the
// per-block scaling 2^(e_x + e_w) happens exactly inside the multiply and only the fp32
// accumulation in tensor memory rounds.
//
// One persistent CTA per SM, 128 x 256 output tiles, K stepped 64 at a time:
//   warp 0      TMA producer: bf16 activations (128x64 box, 128-byte swizzle) and the packed
//               4-bit weight tiles (plain bulk copies) into a 4-stage ring
//   warps 6-13  converters: packed nibbles + block exponents -> exact bf16, written in the
//               128-byte-swizzled K-major layout the MMA reads (3-stage ring)
//   warp 1      issues tcgen05.mma (kind::f16, bf16 x bf16 -> fp32 in TMEM, M=128 N=256 K=16)
//   warps 2-5   epilogue: tcgen05.ld of a finished accumulator, fp32 stores to Y, while the
//               other accumulator (TMEM is double buffered: 2 x 256 columns) is being filled
// The rank tiles of B_q are appended as the last K stages of the same loop.
#include <cuda.h>

#include "lqer_common.cuh"

namespace lqer {
namespace tc {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int RAW_STAGES = 4, B_STAGES = 3;
constexpr int A_TILE_BYTES = BM * BK * 2;                    // 16384
constexpr int PK_HALF_BYTES = kWTileBytes;                   // 4608: one 128-column packed tile
constexpr int RAW_STAGE_BYTES = A_TILE_BYTES + 2 * PK_HALF_BYTES;  // 25600 (multiple of 1024)
constexpr int B_STAGE_BYTES = BN * BK * 2;                   // 32768
constexpr int RANK_PER_STAGE = 32;                           // rank columns per K stage (2 blocks)
constexpr int NUM_BARRIERS = 2 * RAW_STAGES + 2 * B_STAGES + 4;
constexpr int SMEM_BYTES = RAW_STAGES * RAW_STAGE_BYTES + B_STAGES * B_STAGE_BYTES + 256 + 1024;
constexpr int NUM_THREADS = 14 * 32;
constexpr int CONVERTER_WARPS = 8;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000LL;        // about two seconds
static_assert(RAW_STAGE_BYTES % 1024 == 0 && B_STAGE_BYTES % 1024 == 0, "swizzle atoms need 1024-byte bases");
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");

// ---------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: gives up after WAIT_LIMIT_CYCLES or as soon as another role has given up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  int spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255) == 0) {
      if (*abort_flag != 0) return false;
      if (clock64() - t0 > WAIT_LIMIT_CYCLES) { *abort_flag = 1; return false; }
    }
  }
  return true;
}
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);       // start address
  d |= (uint64_t)1 << 16;                         // leading byte offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                         // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                         // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t make_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

__device__ __forceinline__ uint32_t fma_bf16x2(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
// Eight offset-binary nibbles of one block word -> eight bf16 (n - 8) * 2^(e-2), exact:
// 0x4300 | n is the bf16 value 128 + n, and (128 + n) * s - 136 * s rounds nothing away.
__device__ __forceinline__ uint4 convert_word(uint32_t w, uint32_t s2, uint32_t c2) {
  uint4 o;
  o.x = fma_bf16x2((w & 0x000F000Fu) | 0x43004300u, s2, c2);
  o.y = fma_bf16x2(((w >> 4) & 0x000F000Fu) | 0x43004300u, s2, c2);
  o.z = fma_bf16x2(((w >> 8) & 0x000F000Fu) | 0x43004300u, s2, c2);
  o.w = fma_bf16x2(((w >> 12) & 0x000F000Fu) | 0x43004300u, s2, c2);
  return o;
}
__device__ __forceinline__ void w_scales(uint32_t eb, uint32_t& s2, uint32_t& c2) {
  const uint32_t s = (eb - 2u) << 7;                       // bf16 bits of 2^(e-2), eb = e + 127
  const uint32_t c = 0x8000u | ((eb + 5u) << 7) | 8u;      // bf16 bits of -136 * 2^(e-2)
  s2 = s | (s << 16);
  c2 = c | (c << 16);
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  return (__float_as_uint(lo) >> 16) | (__float_as_uint(hi) & 0xFFFF0000u);   // exact values: truncation loses nothing
}
__device__ __forceinline__ uint4 convert_i8x8(uint32_t w0, uint32_t w1, float scale) {
  uint4 o;
  o.x = pack_bf16x2((float)(int8_t)(w0) * scale, (float)(int8_t)(w0 >> 8) * scale);
  o.y = pack_bf16x2((float)(int8_t)(w0 >> 16) * scale, (float)(int8_t)(w0 >> 24) * scale);
  o.z = pack_bf16x2((float)(int8_t)(w1) * scale, (float)(int8_t)(w1 >> 8) * scale);
  o.w = pack_bf16x2((float)(int8_t)(w1 >> 16) * scale, (float)(int8_t)(w1 >> 24) * scale);
  return o;
}

struct Params {
  const uint8_t* wsec;
  const uint8_t* bsec;
  float* Y;
  DeviceStatus* status;
  int M, N, K64;
  int n_tiles;        // 128-column packed tiles
  int k_slabs;        // K stages from W
  int r_blocks;       // 16-row rank blocks of B
  int m_tiles, n256_tiles;
  int lr_shift;       // lr_bits - 2
};

__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* raw_base = smem;
  uint8_t* b_base = smem + RAW_STAGES * RAW_STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(b_base + B_STAGES * B_STAGE_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NUM_BARRIERS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const uint32_t bar0 = smem_u32(bars);
  auto raw_full = [&](int s) { return bar0 + 8u * s; };
  auto raw_empty = [&](int s) { return bar0 + 8u * (RAW_STAGES + s); };
  auto b_full = [&](int s) { return bar0 + 8u * (2 * RAW_STAGES + s); };
  auto b_empty = [&](int s) { return bar0 + 8u * (2 * RAW_STAGES + B_STAGES + s); };
  auto acc_full = [&](int a) { return bar0 + 8u * (2 * RAW_STAGES + 2 * B_STAGES + a); };
  auto acc_empty = [&](int a) { return bar0 + 8u * (2 * RAW_STAGES + 2 * B_STAGES + 2 + a); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < RAW_STAGES; ++s) { mbar_init(raw_full(s), 1); mbar_init(raw_empty(s), CONVERTER_WARPS + 1); }
    for (int s = 0; s < B_STAGES; ++s) { mbar_init(b_full(s), CONVERTER_WARPS); mbar_init(b_empty(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(acc_full(a), 1); mbar_init(acc_empty(a), 4); }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int rank_stages = (p.r_blocks + 1) / 2;
  const int stages_per_tile = p.k_slabs + rank_stages;
  const int num_tiles = p.m_tiles * p.n256_tiles;
  const int b_tile_stride = p.r_blocks * kTileN * 17;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
        const int mt = t % p.m_tiles, nt = t / p.m_tiles;
        const int halves = min(2, p.n_tiles - 2 * nt);
        for (int s = 0; s < stages_per_tile; ++s, ++it) {
          const int st = it % RAW_STAGES;
          if (!mbar_wait(raw_empty(st), ((it / RAW_STAGES) & 1) ^ 1, abort_flag)) { ok = false; break; }
          uint8_t* stage = raw_base + st * RAW_STAGE_BYTES;
          const uint32_t a_dst = smem_u32(stage);
          if (s < p.k_slabs) {
            mbar_expect_tx(raw_full(st), A_TILE_BYTES + halves * PK_HALF_BYTES);
            tma_load_2d(a_dst, &tmap_x, s * BK, mt * BM, raw_full(st));
            for (int h = 0; h < halves; ++h)
              bulk_load(a_dst + A_TILE_BYTES + h * PK_HALF_BYTES,
                        p.wsec + ((size_t)(2 * nt + h) * p.k_slabs + s) * kWTileBytes, kWTileBytes, raw_full(st));
          } else {
            const int rs = s - p.k_slabs;
            const int rb0 = rs * 2, nb = min(2, p.r_blocks - rb0);
            mbar_expect_tx(raw_full(st), A_TILE_BYTES + halves * nb * (kTileN * 17));
            tma_load_2d(a_dst, &tmap_x, p.K64 + rs * RANK_PER_STAGE, mt * BM, raw_full(st));
            for (int h = 0; h < halves; ++h) {
              const uint8_t* tile = p.bsec + (size_t)(2 * nt + h) * b_tile_stride;
              const uint32_t dst = a_dst + A_TILE_BYTES + h * PK_HALF_BYTES;
              bulk_load(dst, tile + (size_t)rb0 * kTileN * 16, nb * kTileN * 16, raw_full(st));
              bulk_load(dst + 4096, tile + (size_t)p.r_blocks * kTileN * 16 + rb0 * kTileN, nb * kTileN, raw_full(st));
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t it = 0, tile_it = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++tile_it) {
        const int nt = t / p.m_tiles;
        const int halves = min(2, p.n_tiles - 2 * nt);
        const uint32_t idesc = make_idesc(halves * kTileN);
        const int acc = tile_it & 1;
        if (!mbar_wait(acc_empty(acc), ((tile_it >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int s = 0; s < stages_per_tile; ++s, ++it) {
          const int st = it % RAW_STAGES, bst = it % B_STAGES;
          if (!mbar_wait(raw_full(st), (it / RAW_STAGES) & 1, abort_flag)) { ok = false; break; }
          if (!mbar_wait(b_full(bst), (it / B_STAGES) & 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t a_desc = make_desc(smem_u32(raw_base + st * RAW_STAGE_BYTES));
          const uint64_t b_desc = make_desc(smem_u32(b_base + bst * B_STAGE_BYTES));
          const int nk = (s < p.k_slabs) ? BK / 16 : min(2, p.r_blocks - (s - p.k_slabs) * 2);
          for (int j = 0; j < nk; ++j)     // 16 K = 32 bytes along the swizzled row: +2 in the address field
            umma_bf16(d_tmem, a_desc + 2 * j, b_desc + 2 * j, idesc, (s > 0 || j > 0) ? 1u : 0u);
          umma_commit(raw_empty(st));
          umma_commit(b_empty(bst));
        }
        if (ok) umma_commit(acc_full(acc));
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------------ epilogue
    const int q = warp & 3;              // TMEM lane quarter this warp may read
    uint32_t tile_it = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++tile_it) {
      const int mt = t % p.m_tiles, nt = t / p.m_tiles;
      const int acc = tile_it & 1;
      if (!mbar_wait(acc_full(acc), (tile_it >> 1) & 1, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int row = mt * BM + q * 32 + lane;
      const int ncols = min(BN, p.N - nt * BN);
      float* yrow = p.Y + (size_t)row * p.N + (size_t)nt * BN;
      for (int c = 0; c < BN; c += 32) {
        if (c >= ncols) break;           // uniform over the warp
        uint32_t r[32];
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN + c, r);
        tmem_ld_wait();
        if (row < p.M) {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (c + 4 * j < ncols)
              *reinterpret_cast<uint4*>(yrow + c + 4 * j) = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty(acc));
    }
  } else {
    // ------------------------------------------------------------------ converters
    const int c = threadIdx.x - 6 * 32;  // 0..255: output column within the 256-wide tile
    const int half = c >> 7, nl = c & 127;
    uint32_t it = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
      const int nt = t / p.m_tiles;
      const int halves = min(2, p.n_tiles - 2 * nt);
      for (int s = 0; s < stages_per_tile; ++s, ++it) {
        const int st = it % RAW_STAGES, bst = it % B_STAGES;
        if (!mbar_wait(raw_full(st), (it / RAW_STAGES) & 1, abort_flag)) { ok = false; break; }
        if (!mbar_wait(b_empty(bst), ((it / B_STAGES) & 1) ^ 1, abort_flag)) { ok = false; break; }
        const uint8_t* pk = raw_base + st * RAW_STAGE_BYTES + A_TILE_BYTES + half * PK_HALF_BYTES;
        uint8_t* brow = b_base + bst * B_STAGE_BYTES + c * 128;
        const int sw = c & 7;
        if (half < halves) {
          if (s < p.k_slabs) {
#pragma unroll
            for (int bp = 0; bp < 2; ++bp) {
              const uint4 w = *reinterpret_cast<const uint4*>(pk + (bp * kTileN + nl) * 16);
              const uint32_t eb = *reinterpret_cast<const uint16_t*>(pk + kWTileNibbleBytes + nl * 4 + bp * 2);
              uint32_t s2, c2;
              w_scales(eb & 0xFFu, s2, c2);
              *reinterpret_cast<uint4*>(brow + (((bp * 4 + 0) ^ sw) << 4)) = convert_word(w.x, s2, c2);
              *reinterpret_cast<uint4*>(brow + (((bp * 4 + 1) ^ sw) << 4)) = convert_word(w.y, s2, c2);
              w_scales(eb >> 8, s2, c2);
              *reinterpret_cast<uint4*>(brow + (((bp * 4 + 2) ^ sw) << 4)) = convert_word(w.z, s2, c2);
              *reinterpret_cast<uint4*>(brow + (((bp * 4 + 3) ^ sw) << 4)) = convert_word(w.w, s2, c2);
            }
          } else {
            const int nb = min(2, p.r_blocks - (s - p.k_slabs) * 2);
            for (int rb = 0; rb < nb; ++rb) {
              const uint4 w = *reinterpret_cast<const uint4*>(pk + (rb * kTileN + nl) * 16);
              const float scale = pow2f((int)pk[4096 + rb * kTileN + nl] - 127 - p.lr_shift);
              *reinterpret_cast<uint4*>(brow + (((rb * 2 + 0) ^ sw) << 4)) = convert_i8x8(w.x, w.y, scale);
              *reinterpret_cast<uint4*>(brow + (((rb * 2 + 1) ^ sw) << 4)) = convert_i8x8(w.z, w.w, scale);
            }
          }
        }
        fence_proxy_async_smem();        // generic-proxy writes -> visible to the MMA's async proxy
        __syncwarp();
        if (lane == 0) { mbar_arrive(b_full(bst)); mbar_arrive(raw_empty(st)); }
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  if (*abort_flag != 0) {
    // A wait ran out: let whatever is still in flight drain before shared and tensor memory go away.
    const long long t0 = clock64();
    while (clock64() - t0 < 400000) { }
    if (threadIdx.x == 0) report_error(p.status, LQER_ERR_TIMEOUT, 300, blockIdx.x);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &f, 12000, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

}  // namespace tc

cudaError_t launch_gemm_tc(const void* xcat, int M, const PackedMeta& m, const void* packed, float* Y,
                           DeviceStatus* st, cudaStream_t s) {
  using namespace tc;
  EncodeTiledFn enc = encode_fn();
  if (enc == nullptr) return cudaErrorNotSupported;
  CUtensorMap tmap;
  const cuuint64_t dims[2] = {(cuuint64_t)xcat_cols(m), (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)xcat_cols(m) * 2};
  const cuuint32_t box[2] = {BK, BM};
  const cuuint32_t estr[2] = {1, 1};
  if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(xcat), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;

  static int sm_count = 0;
  static bool attr_set = false;
  if (!attr_set) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  Params p;
  const uint8_t* base = static_cast<const uint8_t*>(packed);
  p.wsec = base + m.off_w;
  p.bsec = base + m.off_b;
  p.Y = Y;
  p.status = st;
  p.M = M; p.N = m.N; p.K64 = m.K64;
  p.n_tiles = m.n_tiles; p.k_slabs = m.k_slabs; p.r_blocks = m.r_blocks;
  p.m_tiles = (M + BM - 1) / BM;
  p.n256_tiles = (m.n_tiles + 1) / 2;
  p.lr_shift = m.lr_bits - 2;
  const int num_tiles = p.m_tiles * p.n256_tiles;
  const int grid = num_tiles < sm_count ? num_tiles : sm_count;
  gemm_tc_kernel<<<grid, NUM_THREADS, SMEM_BYTES, s>>>(tmap, p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace lqer
