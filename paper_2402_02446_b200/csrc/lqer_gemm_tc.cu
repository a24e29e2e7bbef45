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
//               4-bit weight tiles (plain bulk copies) into a 6-stage ring
//   warps 6-13  converters: packed nibbles + block exponents -> exact bf16, written in the
//               128-byte-swizzled K-major layout the MMA reads (2-stage ring)
//   warp 1      issues tcgen05.mma (kind::f16, bf16 x bf16 -> fp32 in TMEM, M=128 N=256 K=16)
//   warps 2-5   epilogue: tcgen05.ld of a finished accumulator, fp32 stores to Y, while the
//               other accumulator (TMEM is double buffered: 2 x 256 columns) is being filled
// The rank tiles of B_q are appended as the last K stages of the same loop.
#include "lqer_tc_ptx.cuh"

namespace lqer {
namespace tc {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int RAW_STAGES = 6, B_STAGES = 2;
constexpr int A_TILE_BYTES = BM * BK * 2;                    // 16384
constexpr int PK_HALF_BYTES = kWTileBytes;                   // 4608: one 128-column packed tile
constexpr int RAW_STAGE_BYTES = A_TILE_BYTES + 2 * PK_HALF_BYTES;  // 25600 (multiple of 1024)
constexpr int B_STAGE_BYTES = BN * BK * 2;                   // 32768
constexpr int RANK_PER_STAGE = 32;                           // rank columns per K stage (2 blocks)
constexpr int NUM_BARRIERS = 2 * RAW_STAGES + 2 * B_STAGES + 4;
constexpr int SMEM_BYTES = RAW_STAGES * RAW_STAGE_BYTES + B_STAGES * B_STAGE_BYTES + 256 + 1024;
constexpr int NUM_THREADS = 14 * 32;
constexpr int CONVERTER_WARPS = 8;
static_assert(RAW_STAGE_BYTES % 1024 == 0 && B_STAGE_BYTES % 1024 == 0, "swizzle atoms need 1024-byte bases");
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");

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
        const uint32_t idesc = make_idesc(BM, halves * kTileN);
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
    const int sw = c & 7;
    // byte offsets of the eight 16-byte chunks of this thread's row after the 128-byte swizzle
    uint32_t chunk[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) chunk[i] = (uint32_t)(c * 128 + ((i ^ sw) << 4));
    const uint32_t pk_off = A_TILE_BYTES + half * PK_HALF_BYTES;
    int st = 0, bst = 0;
    uint32_t ph = 0, bph = 0;            // phase parities of the two rings
    bool ok = true;
    for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
      const int nt = t / p.m_tiles;
      const bool mine = half < min(2, p.n_tiles - 2 * nt);
      for (int s = 0; s < stages_per_tile; ++s) {
        if (!mbar_wait(raw_full(st), ph, abort_flag)) { ok = false; break; }
        if (!mbar_wait(b_empty(bst), bph ^ 1, abort_flag)) { ok = false; break; }
        const uint8_t* pk = raw_base + st * RAW_STAGE_BYTES + pk_off;
        uint8_t* bt = b_base + bst * B_STAGE_BYTES;
        if (mine) {
          if (s < p.k_slabs) {
            const uint4 wa = *reinterpret_cast<const uint4*>(pk + nl * 16);
            const uint4 wb = *reinterpret_cast<const uint4*>(pk + (kTileN + nl) * 16);
            const uint32_t eb = *reinterpret_cast<const uint32_t*>(pk + kWTileNibbleBytes + nl * 4);
            uint32_t s2, c2;
            w_scales(eb & 0xFFu, s2, c2);
            *reinterpret_cast<uint4*>(bt + chunk[0]) = convert_word(wa.x, s2, c2);
            *reinterpret_cast<uint4*>(bt + chunk[1]) = convert_word(wa.y, s2, c2);
            w_scales((eb >> 8) & 0xFFu, s2, c2);
            *reinterpret_cast<uint4*>(bt + chunk[2]) = convert_word(wa.z, s2, c2);
            *reinterpret_cast<uint4*>(bt + chunk[3]) = convert_word(wa.w, s2, c2);
            w_scales((eb >> 16) & 0xFFu, s2, c2);
            *reinterpret_cast<uint4*>(bt + chunk[4]) = convert_word(wb.x, s2, c2);
            *reinterpret_cast<uint4*>(bt + chunk[5]) = convert_word(wb.y, s2, c2);
            w_scales(eb >> 24, s2, c2);
            *reinterpret_cast<uint4*>(bt + chunk[6]) = convert_word(wb.z, s2, c2);
            *reinterpret_cast<uint4*>(bt + chunk[7]) = convert_word(wb.w, s2, c2);
          } else {
            const int nb = min(2, p.r_blocks - (s - p.k_slabs) * 2);
            for (int rb = 0; rb < nb; ++rb) {
              const uint4 w = *reinterpret_cast<const uint4*>(pk + (rb * kTileN + nl) * 16);
              const float scale = pow2f((int)pk[4096 + rb * kTileN + nl] - 127 - p.lr_shift);
              *reinterpret_cast<uint4*>(bt + chunk[rb * 2]) = convert_i8x8(w.x, w.y, scale);
              *reinterpret_cast<uint4*>(bt + chunk[rb * 2 + 1]) = convert_i8x8(w.z, w.w, scale);
            }
          }
        }
        fence_proxy_async_smem();        // generic-proxy writes -> visible to the MMA's async proxy
        __syncwarp();
        if (lane == 0) { mbar_arrive(b_full(bst)); mbar_arrive(raw_empty(st)); }
        if (++st == RAW_STAGES) { st = 0; ph ^= 1; }
        if (++bst == B_STAGES) { bst = 0; bph ^= 1; }
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
  LaunchScope scope(kFamGemmTc, s);
  gemm_tc_kernel<<<grid, NUM_THREADS, SMEM_BYTES, s>>>(tmap, p);
  return cudaGetLastError();
}

}  // namespace lqer
