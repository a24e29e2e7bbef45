// CTA-pair form of the main GEMM (paper Section 3.1 / 3.2: Y = [X_q | T_q] . [W_q ; B_q]).
//
// Two CTAs on neighbouring SMs (a cluster of 2) share one 256 x 256 output tile.  CTA r holds
// token rows [128 r, 128 r + 128) of the tile (its own A operand and its own accumulator
// lanes) and output columns [128 r, 128 r + 128) of the weight tile (its half of the B
// operand).  Each CTA therefore fetches and converts only HALF of the 4-bit weights per
// tensor-core stage, and reads half of B from its shared memory; tcgen05.mma.cta_group::2,
// issued by CTA 0 alone, combines the halves.  Roles per CTA:
//   warp 0      TMA producer (own activation tile + own packed weight half)
//   warp 1      tensor memory allocation; in CTA 0 also the MMA issuer
//   warps 2-5   epilogue (tcgen05.ld of the finished accumulator, fp32 stores to Y)
//   warps 6-29  converters in six groups; a group converts every sixth stage (one weight
//               column = 64 weights per thread), so that its fixed per-stage latencies
//               (barrier wait, shared-memory round trip, proxy fence) overlap the other groups
// One ring of six stages; a stage holds the activation tile, the packed weight tile and the
// converted weight tile, so each role waits on one barrier and signals one per stage:
//   loaded[s]   (per CTA)  TMA bytes have landed          -> converters
//   ready[s]    (in CTA 0) both CTAs' converters are done -> MMA issuer; implies both
//                          activation tiles have landed, since a converter waits for loaded[s]
//   free[s]     (per CTA)  tcgen05.commit with a two-CTA mask: the MMAs that read the stage
//                          have finished                   -> TMA producer
// "accumulator full" is the same kind of commit; "accumulator free" lives in CTA 0 and
// collects the epilogue warps of both CTAs.
// A launch may serve several layers with one M: their tiles form one list (layers with more K
// stages per tile first) that the pairs walk round robin, so pairs idle only at the end of the
// list and set-up and the last epilogue are paid once per launch.
#include <algorithm>

#include "lqer_tc_ptx.cuh"

namespace lqer {
namespace tc2 {
using namespace tc;

constexpr int BM = 128;                    // token rows per CTA (256 per pair)
constexpr int BN = 256;                    // output columns per pair tile
constexpr int BNH = 128;                   // columns converted by one CTA
constexpr int BK = 64;
constexpr int STAGES = 6;
constexpr int A_TILE_BYTES = BM * BK * 2;                     // 16384: activations (TMA, swizzled)
constexpr int B_TILE_BYTES = BNH * BK * 2;                    // 16384: converted weights (swizzled)
constexpr int PK_OFFSET = A_TILE_BYTES + B_TILE_BYTES;        // packed weight tile (4608) behind them
constexpr int STAGE_BYTES = 37 * 1024;
constexpr int RANK_PER_STAGE = 32;
constexpr int NUM_BARRIERS = 3 * STAGES + 4;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 256 + 1024;
constexpr int CONVERTER_WARPS = 24;
constexpr int CONVERTER_GROUPS = 6;          // group g converts the stages with index = g (mod 6): with six ring
                                             // slots a group meets one slot only, exactly one pass apart, so
                                             // the parity of its wait can never alias an older pass
constexpr int WARPS_PER_GROUP = CONVERTER_WARPS / CONVERTER_GROUPS;
constexpr int NUM_THREADS = (6 + CONVERTER_WARPS) * 32;
static_assert(PK_OFFSET + kWTileBytes <= STAGE_BYTES && STAGE_BYTES % 1024 == 0, "stage layout");
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
static_assert(STAGES % CONVERTER_GROUPS == 0, "a converter group must revisit a ring slot exactly one pass later");

constexpr int MAX_GROUP = 8;               // independent layers with one M that may share a launch

struct TensorMaps {                        // one activation map per layer of the group
  CUtensorMap m[MAX_GROUP];
};

struct Layer {
  const uint8_t* wsec;
  const uint8_t* bsec;
  void* Y;                     // [M, N] fp32; bf16 or the MXINT8 sections by Params::y_type (never for the K ranges of a split layer)
  size_t y_extent;             // bytes of the buffer behind Y, for the checked build
  size_t w_extent, b_extent;   // bytes of the packed W and B sections
  int N, K64;
  int n_tiles, k_slabs, r_blocks;
  int slab0, slab_stride;      // a layer may be a K range of a real layer (split K): its first weight slab, and the
                               // real layer's slab count (the stride between column tiles of the packed weights)
  int spt;                     // K stages per tile: k_slabs + rank stages
  int tile_begin;              // first tile of this layer in the launch's list (256 x 256 tiles, row tile fastest)
};

struct Params {
  Layer L[MAX_GROUP];          // ordered by falling spt: the long tiles run first, the short ones fill the end
  int group;                   // layers in this launch
  int num_tiles;               // tiles of all layers
  DeviceStatus* status;
  int M, m_tiles;              // row tiles of 256 (the same M for every layer)
  int lr_shift;
  int y_type;                  // kYF32; kYBF16 (round to nearest even); kYMXINT8 (blocks of 16 along N, format below)
  int a_bits, exp_min, exp_max;// activation format, for an MXINT8 Y
  int w_bits;                  // mantissa bits of W_q: 4 or 2 (one value for all layers of a launch)
  long long wait_limit;        // bound of every wait, in clock cycles
  int stall;                   // test hook: the producers withhold the last stage of their last tile, so the waits run out
};

// Two fp32 bit patterns -> two bf16 (round to nearest even) in one word, the first in the low half.
__device__ __forceinline__ uint32_t bf16x2_rn(uint32_t lo, uint32_t hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(__uint_as_float(hi)), "f"(__uint_as_float(lo)));
  return d;
}

__device__ __forceinline__ int layer_of(const Params& p, int t) {
  int l = 0;
#pragma unroll
  for (int i = 1; i < MAX_GROUP; ++i)
    if (i < p.group && t >= p.L[i].tile_begin) l = i;
  return l;
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc2_kernel(const __grid_constant__ TensorMaps tmaps, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* stage_base = smem;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NUM_BARRIERS);
  volatile WaitState* abort_flag = reinterpret_cast<volatile WaitState*>(tmem_slot + 2);

  const uint32_t bar0 = smem_u32(bars);
  auto loaded = [&](int s) { return bar0 + 8u * s; };                        // local
  auto ready = [&](int s) { return bar0 + 8u * (STAGES + s); };              // used in CTA 0
  auto freed = [&](int s) { return bar0 + 8u * (2 * STAGES + s); };          // local, pair commit
  auto acc_full = [&](int a) { return bar0 + 8u * (3 * STAGES + a); };       // local, pair commit
  auto acc_empty = [&](int a) { return bar0 + 8u * (3 * STAGES + 2 + a); };  // used in CTA 0

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();          // 0 = leader (issues the MMAs)
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(loaded(s), 1);
      mbar_init(ready(s), 2 * WARPS_PER_GROUP);
      mbar_init(freed(s), 1);
    }
    for (int a = 0; a < 2; ++a) { mbar_init(acc_full(a), 1); mbar_init(acc_empty(a), 8); }
    abort_flag->abort = 0;
    abort_flag->limit = p.wait_limit;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), 512);
  tc_fence_before();
  __syncthreads();
  cluster_barrier();                             // both CTAs' barriers exist before any remote arrive
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // barriers and tensor memory are set up: let the next kernel start its own setup, then wait for the
  // prologue's Xcat (and for the previous user of Y and the workspace) before touching global memory
  pdl_launch_dependents();
  pdl_wait();

  const int num_tiles = p.num_tiles;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (own halves)
    if (lane == 0) {
      int st = 0;
      uint32_t ph = 0;
      bool ok = true;
      const uint32_t w_tile = (uint32_t)w_tile_bytes(p.w_bits);
      for (int t = pair; t < num_tiles && ok; t += num_pairs) {
        const int layer = layer_of(p, t), tl = t - p.L[layer].tile_begin;
        const int mt = tl % p.m_tiles, nt = tl / p.m_tiles;
        const CUtensorMap* tmap_x = &tmaps.m[layer];
        const uint8_t* wsec = p.L[layer].wsec;
        const uint8_t* bsec = p.L[layer].bsec;
        const int k_slabs = p.L[layer].k_slabs, r_blocks = p.L[layer].r_blocks, K64 = p.L[layer].K64;
        const int stages_per_tile = p.L[layer].spt, n_tiles = p.L[layer].n_tiles;
        const int slab0 = p.L[layer].slab0, slab_stride = p.L[layer].slab_stride;
        const int b_tile_stride = r_blocks * kTileN * 17;
        const int my_ntile = 2 * nt + (int)rank;
        const bool has_w = my_ntile < n_tiles;
        const int row0 = mt * 2 * BM + (int)rank * BM;
        for (int s = 0; s < stages_per_tile; ++s) {
          if (p.stall != 0 && s == stages_per_tile - 1 && t + num_pairs >= num_tiles) { ok = false; break; }
          if (!mbar_wait<true>(freed(st), ph ^ 1, abort_flag)) { ok = false; break; }
          const uint32_t a_dst = smem_u32(stage_base + st * STAGE_BYTES);
          if (s < k_slabs) {
            const size_t w_off = ((size_t)my_ntile * slab_stride + slab0 + s) * w_tile;
            if (has_w && !LQER_IN_BOUNDS(p.status, w_off, w_tile, p.L[layer].w_extent, 605)) { ok = false; break; }
            mbar_expect_tx(loaded(st), A_TILE_BYTES + (has_w ? w_tile : 0));
            tma_load_2d(a_dst, tmap_x, (slab0 + s) * BK, row0, loaded(st));
            if (has_w) bulk_load(a_dst + PK_OFFSET, wsec + w_off, w_tile, loaded(st));
          } else {
            const int rs = s - k_slabs;
            const int rb0 = rs * 2, nb = min(2, r_blocks - rb0);
            if (has_w && !LQER_IN_BOUNDS(p.status, (size_t)my_ntile * b_tile_stride + (size_t)r_blocks * kTileN * 16 + rb0 * kTileN,
                                         nb * kTileN, p.L[layer].b_extent, 606)) { ok = false; break; }
            mbar_expect_tx(loaded(st), A_TILE_BYTES + (has_w ? nb * (kTileN * 17) : 0));
            tma_load_2d(a_dst, tmap_x, K64 + rs * RANK_PER_STAGE, row0, loaded(st));
            if (has_w) {
              const uint8_t* tile = bsec + (size_t)my_ntile * b_tile_stride;
              bulk_load(a_dst + PK_OFFSET, tile + (size_t)rb0 * kTileN * 16, nb * kTileN * 16, loaded(st));
              bulk_load(a_dst + PK_OFFSET + 4096, tile + (size_t)r_blocks * kTileN * 16 + rb0 * kTileN,
                        nb * kTileN, loaded(st));
            }
          }
          if (++st == STAGES) { st = 0; ph ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    // The whole warp runs the loop, so that barrier addresses and descriptors are warp-uniform values, and one
    // elected lane issues: the tensor pipe takes an MMA of this shape every 128 cycles and queues very few, so every
    // cycle the issuing warp spends between two MMAs beyond that is a cycle the pipe idles.
    if (rank == 0) {
      int st = 0;
      uint32_t ph = 0, tile_it = 0;
      const uint32_t idesc = make_idesc(2 * BM, BN);
      const uint64_t a_desc0 = make_desc(smem_u32(stage_base));
      const uint64_t b_desc0 = make_desc(smem_u32(stage_base + A_TILE_BYTES));
      bool ok = true;
      for (int t = pair; t < num_tiles && ok; t += num_pairs, ++tile_it) {
        const int layer = layer_of(p, t);
        const int k_slabs = p.L[layer].k_slabs, r_blocks = p.L[layer].r_blocks, stages_per_tile = p.L[layer].spt;
        const int acc = tile_it & 1;
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(acc_empty(acc), ((tile_it >> 1) & 1) ^ 1, abort_flag)) != 0;
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int s = 0; s < stages_per_tile; ++s) {
          // everything that does not depend on the wait is computed before it
          const uint64_t a_desc = a_desc0 + (uint64_t)(st * (STAGE_BYTES >> 4));
          const uint64_t b_desc = b_desc0 + (uint64_t)(st * (STAGE_BYTES >> 4));
          const uint32_t first = s > 0 ? 1u : 0u;
          const uint32_t free_bar = freed(st);
          const int nk = s < k_slabs ? 4 : min(2, r_blocks - (s - k_slabs) * 2);
          ok = __all_sync(0xFFFFFFFFu, mbar_wait(ready(st), ph, abort_flag)) != 0;
          if (!ok) break;
          tc_fence_after();
          if (elect_one()) {
            umma_bf16_pair(d_tmem, a_desc, b_desc, idesc, first);           // +2 in the address field = 32 bytes = 16 K
            if (nk > 1) umma_bf16_pair(d_tmem, a_desc + 2, b_desc + 2, idesc, 1u);
            if (nk > 2) {
              umma_bf16_pair(d_tmem, a_desc + 4, b_desc + 4, idesc, 1u);
              umma_bf16_pair(d_tmem, a_desc + 6, b_desc + 6, idesc, 1u);
            }
            umma_commit_pair(free_bar);
          }
          __syncwarp();
          if (++st == STAGES) { st = 0; ph ^= 1; }
        }
        if (ok && elect_one()) umma_commit_pair(acc_full(acc));
        __syncwarp();
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------------ epilogue (own 128 rows)
    const int q = warp & 3;
    uint32_t tile_it = 0;
    bool ok = true;
    for (int t = pair; t < num_tiles && ok; t += num_pairs, ++tile_it) {
      const int layer = layer_of(p, t), tl = t - p.L[layer].tile_begin;
      const int mt = tl % p.m_tiles, nt = tl / p.m_tiles;
      const int Nl = p.L[layer].N;
      const int acc = tile_it & 1;
      if (!mbar_wait<true>(acc_full(acc), (tile_it >> 1) & 1, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int row = mt * 2 * BM + (int)rank * BM + q * 32 + lane;
      const int ncols = min(BN, Nl - nt * BN);
      const size_t yoff = (size_t)row * Nl + (size_t)nt * BN;
      float* yrow = static_cast<float*>(p.L[layer].Y) + yoff;
      uint16_t* yrow16 = static_cast<uint16_t*>(p.L[layer].Y) + yoff;
      // MXINT8 Y: mantissas [M, N], then exponent bytes [M, N / 16]; a thread holds whole 16-blocks of its row
      uint8_t* yq = static_cast<uint8_t*>(p.L[layer].Y) + yoff;
      uint8_t* yqe = static_cast<uint8_t*>(p.L[layer].Y) + (size_t)p.M * Nl + ((size_t)row * Nl + (size_t)nt * BN) / 16;
      const QuantConsts qc = quant_consts(p.a_bits, p.exp_min, p.exp_max);
      for (int c = 0; c < BN; c += 32) {
        if (c >= ncols) break;
        uint32_t r[32];
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN + c, r);
        tmem_ld_wait();
        if (row < p.M) {
          if (p.y_type == kYBF16) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (c + 8 * j < ncols && LQER_IN_BOUNDS(p.status, (yoff + c + 8 * j) * 2, 16, p.L[layer].y_extent, 601))   // N is a multiple of 8
                *reinterpret_cast<uint4*>(yrow16 + c + 8 * j) =
                    make_uint4(bf16x2_rn(r[8 * j], r[8 * j + 1]), bf16x2_rn(r[8 * j + 2], r[8 * j + 3]),
                               bf16x2_rn(r[8 * j + 4], r[8 * j + 5]), bf16x2_rn(r[8 * j + 6], r[8 * j + 7]));
          } else if (p.y_type == kYMXINT8) {
#pragma unroll
            for (int j = 0; j < 2; ++j)
              if (c + 16 * j < ncols && LQER_IN_BOUNDS(p.status, yoff + c + 16 * j, 16, p.L[layer].y_extent, 602) &&
                  LQER_IN_BOUNDS(p.status, (size_t)p.M * Nl + yoff / 16 + (c >> 4) + j, 1, p.L[layer].y_extent, 603)) {   // N is a multiple of 16 here
                float v[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[16 * j + i]);
                uint4 m8, b0, b1;
                int e;
                quantize_block16(v, qc, e, m8, b0, b1);
                *reinterpret_cast<uint4*>(yq + c + 16 * j) = m8;
                yqe[(c >> 4) + j] = (uint8_t)(e + 127);
              }
          } else {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if (c + 4 * j < ncols && LQER_IN_BOUNDS(p.status, (yoff + c + 4 * j) * 4, 16, p.L[layer].y_extent, 604))
                *reinterpret_cast<uint4*>(yrow + c + 4 * j) = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (rank == 0) mbar_arrive(acc_empty(acc)); else mbar_arrive_remote(acc_empty(acc), 0);
      }
    }
  } else {
    // ------------------------------------------------------------------ converters (own weight half)
    const int c = threadIdx.x - 6 * 32;          // 0..767
    const int group = c >> 7, nl = c & 127;      // stage group; weight column of the half tile
    const int sw = nl & 7;
    uint32_t chunk[8];                           // the row's eight 16-byte chunks after the 128-byte swizzle
#pragma unroll
    for (int i = 0; i < 8; ++i) chunk[i] = (uint32_t)(nl * 128 + ((i ^ sw) << 4));
    // the pair's tiles one after the other; their K stages form one sequence of which this group takes every sixth
    int tile = pair, s = group;                  // s may run past the tile; normalised below
    int stages_per_tile = 0, k_slabs = 0, r_blocks = 0;
    bool has_w = false;
    auto enter_tile = [&]() {
      if (tile < num_tiles) {
        const int layer = layer_of(p, tile);
        stages_per_tile = p.L[layer].spt; k_slabs = p.L[layer].k_slabs; r_blocks = p.L[layer].r_blocks;
        const int nt = (tile - p.L[layer].tile_begin) / p.m_tiles;
        has_w = 2 * nt + (int)rank < p.L[layer].n_tiles;
      }
    };
    enter_tile();
    bool ok = true;
    for (int it = group; tile < num_tiles && ok; it += CONVERTER_GROUPS, s += CONVERTER_GROUPS) {
      while (tile < num_tiles && s >= stages_per_tile) { s -= stages_per_tile; tile += num_pairs; enter_tile(); }
      if (tile >= num_tiles) break;
      const int st = it % STAGES;
      const uint32_t ph = (uint32_t)((it / STAGES) & 1);
      if (!mbar_wait(loaded(st), ph, abort_flag)) { ok = false; break; }
      const uint8_t* pk = stage_base + st * STAGE_BYTES + PK_OFFSET;
      uint8_t* bt = stage_base + st * STAGE_BYTES + A_TILE_BYTES;
      if (s < k_slabs) {
        if (has_w) {
          convert_column(pk, nl, p.w_bits, bt, chunk);
        } else {                                 // columns beyond N: a zero operand half
#pragma unroll
          for (int i = 0; i < 8; ++i) *reinterpret_cast<uint4*>(bt + chunk[i]) = make_uint4(0u, 0u, 0u, 0u);
        }
      } else {
        const int nb = min(2, r_blocks - (s - k_slabs) * 2);
        for (int rb = 0; rb < nb; ++rb) {
          uint4 o0 = make_uint4(0u, 0u, 0u, 0u), o1 = o0;
          if (has_w) {
            const uint4 w = *reinterpret_cast<const uint4*>(pk + (rb * kTileN + nl) * 16);
            const float scale = pow2f((int)pk[4096 + rb * kTileN + nl] - 127 - p.lr_shift);
            o0 = convert_i8x8(w.x, w.y, scale);
            o1 = convert_i8x8(w.z, w.w, scale);
          }
          *reinterpret_cast<uint4*>(bt + chunk[rb * 2]) = o0;
          *reinterpret_cast<uint4*>(bt + chunk[rb * 2 + 1]) = o1;
        }
      }
      fence_proxy_async_smem();        // generic-proxy writes -> visible to the MMA's async proxy
      __syncwarp();
      if (lane == 0) {
        if (rank == 0) mbar_arrive(ready(st)); else mbar_arrive_remote(ready(st), 0);
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  __syncthreads();                      // every role is done (or has given up): the flag below is final for this CTA
  if (abort_flag->abort != 0) {
    const long long t0 = clock64();
    while (clock64() - t0 < 400000) { }
    if (threadIdx.x == 0) report_error(p.status, LQER_ERR_TIMEOUT, 400, blockIdx.x);
  }
  tc_fence_before();
  __syncthreads();
  cluster_barrier();                    // the peer may still read this CTA's shared / tensor memory until here
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 512);
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

}  // namespace tc2

namespace tc2 {

static cudaError_t launch_params(const TensorMaps& tmaps, Params& p, cudaStream_t s) {
  static OncePerDevice once;
  cudaError_t e = once.run([] {
    return cudaFuncSetAttribute(gemm_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  });
  if (e != cudaSuccess) return e;
  const int max_pairs = sm_count() / 2;
  if (max_pairs < 1) return cudaErrorInvalidDevice;
  p.wait_limit = wait_limit_cycles();
  p.stall = take_stall(kFamGemmTcPair) ? 1 : 0;
  const int pairs = p.num_tiles < max_pairs ? p.num_tiles : max_pairs;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(NUM_THREADS);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may set up while the prologue drains
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  LaunchScope scope(kFamGemmTcPair, s);
  return cudaLaunchKernelEx(&cfg, gemm_tc2_kernel, tmaps, p);
}

// Y += P_0 + P_1 + ... in that order: the K ranges of a split layer other than the first.
__global__ void __launch_bounds__(256) splitk_sum_kernel(float4* __restrict__ Y, const float4* __restrict__ P, int parts,
                                                         size_t quads) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < quads; i += (size_t)gridDim.x * blockDim.x) {
    float4 y = Y[i];
    for (int c = 0; c < parts; ++c) {
      const float4 v = __ldcs(P + (size_t)c * quads + i);
      y.x += v.x; y.y += v.y; y.z += v.z; y.w += v.w;
    }
    Y[i] = y;
  }
}

}  // namespace tc2

// Small batches have few tiles; their K range is cut into ranges that run as layers of one launch, the first into Y,
// the others into scratch that a second kernel adds to Y in a fixed order.
cudaError_t launch_gemm_tc2_splitk(const void* xcat, int M, const PackedMeta& m, const void* packed, void* Yv, int y_type,
                                   float* partials, DeviceStatus* st, cudaStream_t s) {
  using namespace tc2;
  const int C = gemm_splitk_ranges(m, M);
  // only an fp32 Y can collect the ranges' sums: a layer with another output type runs whole
  if (C < 2 || y_type != kYF32) return launch_gemm_tc2(xcat, M, m, packed, Yv, y_type, st, s);
  float* Y = static_cast<float*>(Yv);
  if ((m.N & 3) != 0) return cudaErrorInvalidValue;
  EncodeTiledFn enc = encode_fn();
  if (enc == nullptr) return cudaErrorNotSupported;
  TensorMaps tmaps;
  const cuuint64_t dims[2] = {(cuuint64_t)xcat_cols(m), (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)xcat_cols(m) * 2};
  const cuuint32_t box[2] = {BK, BM};
  const cuuint32_t estr[2] = {1, 1};
  if (enc(&tmaps.m[0], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(xcat), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  for (int g = 1; g < MAX_GROUP; ++g) tmaps.m[g] = tmaps.m[0];
  Params p;
  p.m_tiles = (M + 2 * BM - 1) / (2 * BM);
  const uint8_t* base = static_cast<const uint8_t*>(packed);
  const int per_layer = p.m_tiles * ((m.n_tiles + 1) / 2);
  // the last range (it carries the rank stages and is the longest) first
  for (int slot = 0; slot < MAX_GROUP; ++slot) {
    const int c = slot < C ? C - 1 - slot : C - 1;
    const int lo = (int)((long long)c * m.k_slabs / C), hi = (int)((long long)(c + 1) * m.k_slabs / C);
    Layer& ly = p.L[slot];
    ly.wsec = base + m.off_w;
    ly.bsec = base + m.off_b;
    ly.Y = c == 0 ? Y : partials + (size_t)(c - 1) * M * m.N;
    ly.y_extent = (size_t)M * m.N * 4;
    ly.w_extent = m.off_b - m.off_w; ly.b_extent = m.off_a - m.off_b;
    ly.N = m.N; ly.K64 = m.K64;
    ly.n_tiles = m.n_tiles; ly.k_slabs = hi - lo;
    ly.r_blocks = c == C - 1 ? m.r_blocks : 0;
    ly.slab0 = lo; ly.slab_stride = m.k_slabs;
    ly.spt = ly.k_slabs + (ly.r_blocks + 1) / 2;
    ly.tile_begin = slot * per_layer;
  }
  p.group = C;
  p.num_tiles = C * per_layer;
  p.status = st;
  p.M = M;
  p.lr_shift = m.lr_bits - 2;
  p.y_type = kYF32;
  p.a_bits = m.a_bits; p.exp_min = m.exp_min; p.exp_max = m.exp_max;
  p.w_bits = m.w_bits;
  cudaError_t e = launch_params(tmaps, p, s);
  if (e != cudaSuccess) return e;
  const size_t quads = (size_t)M * m.N / 4;
  int blocks = (int)((quads + 255) / 256);
  if (blocks > sm_count() * 8) blocks = sm_count() * 8;
  LaunchScope scope(kFamGemmTcPair, s);
  splitk_sum_kernel<<<blocks, 256, 0, s>>>(reinterpret_cast<float4*>(Y), reinterpret_cast<const float4*>(partials), C - 1, quads);
  return cudaGetLastError();
}

cudaError_t launch_gemm_tc2(const void* xcat, int M, const PackedMeta& m, const void* packed, void* Y, int y_type,
                            DeviceStatus* st, cudaStream_t s) {
  return launch_gemm_tc2_group(&xcat, &packed, &Y, y_type, &m, 1, M, st, s);
}

int gemm_tc2_max_group() { return tc2::MAX_GROUP; }

// n layers with one M (shapes may differ, formats must not) as ONE launch: the tiles of all layers form one list that
// the CTA pairs walk, so the pairs idle only at the end of the whole list, and set-up and the last epilogue are paid
// once.  Layers with more K stages per tile come first in the list.
cudaError_t launch_gemm_tc2_group(const void* const* xcats, const void* const* packed, void* const* Ys, int y_type,
                                  const PackedMeta* metas, int n, int M, DeviceStatus* st, cudaStream_t s) {
  using namespace tc2;
  if (n < 1 || n > MAX_GROUP) return cudaErrorInvalidValue;
  EncodeTiledFn enc = encode_fn();
  if (enc == nullptr) return cudaErrorNotSupported;
  // order: falling number of K stages per tile (stable, so equal layers keep the caller's order)
  int order[MAX_GROUP];
  for (int g = 0; g < n; ++g) order[g] = g;
  auto spt_of = [&](int g) { return metas[g].k_slabs + (metas[g].r_blocks + 1) / 2; };
  for (int a = 1; a < n; ++a)
    for (int b = a; b > 0 && spt_of(order[b]) > spt_of(order[b - 1]); --b) { const int t = order[b]; order[b] = order[b - 1]; order[b - 1] = t; }

  TensorMaps tmaps;
  Params p;
  p.m_tiles = (M + 2 * BM - 1) / (2 * BM);
  int tile_begin = 0;
  for (int slot = 0; slot < MAX_GROUP; ++slot) {
    const int g = order[slot < n ? slot : 0];
    const PackedMeta& m = metas[g];
    if (m.lr_bits != metas[0].lr_bits || m.w_bits != metas[0].w_bits) return cudaErrorInvalidValue;
    const cuuint64_t dims[2] = {(cuuint64_t)xcat_cols(m), (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)xcat_cols(m) * 2};
    const cuuint32_t box[2] = {BK, BM};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&tmaps.m[slot], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(xcats[g]), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
    const uint8_t* base = static_cast<const uint8_t*>(packed[g]);
    Layer& ly = p.L[slot];
    ly.wsec = base + m.off_w;
    ly.bsec = base + m.off_b;
    ly.Y = Ys[g];
    ly.y_extent = y_bytes(y_type, (size_t)M, (size_t)m.N);
    if (kDebugBounds) ly.y_extent -= std::min(ly.y_extent, debug_y_shrink());
    ly.w_extent = m.off_b - m.off_w; ly.b_extent = m.off_a - m.off_b;
    ly.N = m.N; ly.K64 = m.K64;
    ly.n_tiles = m.n_tiles; ly.k_slabs = m.k_slabs; ly.r_blocks = m.r_blocks;
    ly.slab0 = 0; ly.slab_stride = m.k_slabs;
    ly.spt = m.k_slabs + (m.r_blocks + 1) / 2;
    ly.tile_begin = tile_begin;
    if (slot < n) tile_begin += p.m_tiles * ((m.n_tiles + 1) / 2);
  }
  p.group = n;
  p.num_tiles = tile_begin;
  p.status = st;
  p.M = M;
  p.lr_shift = metas[0].lr_bits - 2;
  p.y_type = y_type;
  p.a_bits = metas[0].a_bits; p.exp_min = metas[0].exp_min; p.exp_max = metas[0].exp_max;
  p.w_bits = metas[0].w_bits;
  return launch_params(tmaps, p, s);
}

}  // namespace lqer
