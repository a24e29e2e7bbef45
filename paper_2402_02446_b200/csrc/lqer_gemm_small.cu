// Small-batch form of the layer's contraction (paper Section 3.1 / 3.2: Y = [X_q | T_q] . [W_q ; B_q];
// Section 2.1: few tokens per step make the layer memory bound on its weights).
//
// The 5th-generation tensor core takes one row of the M-side operand per cycle against up to 256 columns of
// the N-side operand (measured: a tcgen05.mma of M = 128, K = 16 takes 134 cycles whether N is 16 or 256).  So
// with few tokens the tokens go on the M side, padded to the smallest tile (64 rows, or 128), and the weights
// take the full 256-wide N side:
//     D[MT tokens, 256 weight columns] += Xtile[MT, 16 K] . Wtile[256, 16 K]^T      (tcgen05.mma, bf16 -> fp32)
// A CTA streams packed weight tiles exactly once (two 128-column tiles = 256 columns x 64 K per stage, one bulk
// copy each), converts the 4-bit mantissas to their exact bf16 values in shared memory (as the large-batch
// GEMM does) and multiplies them with an [MT, 64] tile of the quantised activations that TMA brings from
// Xcat (rows beyond the batch arrive as zeros).
//
// Work items are (layer, 256-column tile, K chunk).  The chunks of a tile are fixed by the shape alone (so a
// result never depends on the number of SMs or on which layers share a launch); each chunk is summed from
// zero in tensor memory and, if a tile has more than one, leaves its fp32 partial in scratch; the CTA whose
// partial arrives last adds the chunks in chunk order and writes Y.  Nothing waits for another CTA.
// Roles per CTA:
//   warp 0      producer: bulk copies of packed weight tiles (issued before the dependency wait: weights
//               depend on no earlier kernel) and TMA loads of activation tiles (after it)
//   warp 1      tensor memory allocation, MMA issue (the whole warp runs the loop, one elected lane issues)
//   warps 2-5   epilogue (tcgen05.ld, Y or partial sums, the last-arriver reduction)
//   warps 6-29  converters in three groups of 256 threads (a weight column each); group g converts the stages
//               with index = g (mod 3), so it meets one CV slot only and its PK slots in phase order
// Two rings: PK slots hold {activation tile, two packed weight tiles}, with a barrier for the weights and one for
// the activations (the converters need only the former, so they work while the prologue still runs); CV slots
// hold converted weight tiles.
#include <algorithm>

#include "lqer_gemm_small.cuh"
#include "lqer_tc_ptx.cuh"

namespace lqer {
namespace sg {
using namespace tc;

constexpr int BK = 64;
constexpr int CV_TILE_BYTES = BN * BK * 2; // 32768
constexpr int CV_SLOTS = 3;
constexpr int CONVERTER_GROUPS = 3;
constexpr int WARPS_PER_GROUP = 8;
constexpr int NUM_THREADS = (6 + CONVERTER_GROUPS * WARPS_PER_GROUP) * 32;
constexpr int RANK_PER_STAGE = 32;

__device__ __forceinline__ void epilogue_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

template <int MT, int PK_SLOTS>
struct Cfg {
  static constexpr int X_TILE_BYTES = MT * 128;
  static constexpr int PK_SLOT_BYTES = (X_TILE_BYTES + 2 * kWTileBytes + 1023) / 1024 * 1024;
  static constexpr int OFF_PK = CV_SLOTS * CV_TILE_BYTES;
  static constexpr int OFF_BARS = OFF_PK + PK_SLOTS * PK_SLOT_BYTES;
  static constexpr int NUM_BARS = 3 * PK_SLOTS + 2 * CV_SLOTS + 4;
  static constexpr int SMEM_BYTES = OFF_BARS + NUM_BARS * 8 + 64 + 1024;
  static constexpr int TMEM_COLS = 512;    // two accumulators of 256 columns
  static_assert(MT == 64 || MT == 128, "MMA tile rows");
  static_assert(PK_SLOTS % CONVERTER_GROUPS == 0, "a converter group must meet a PK slot in phase order");
  static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
};

struct TensorMaps {
  CUtensorMap m[MAX_LAYERS];   // Xcat of each layer: bf16 [M, K64 + k_pad], box 64 x x_rows
};


template <int MT, int PK_SLOTS>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_small_kernel(const __grid_constant__ TensorMaps tmaps, const __grid_constant__ Params p) {
  using C = Cfg<MT, PK_SLOTS>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* cv_base = smem;
  uint8_t* pk_base = smem + C::OFF_PK;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BARS);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + C::NUM_BARS);
  int* last_flag = reinterpret_cast<int*>(tmem_slot + 1);
  int* deferred = reinterpret_cast<int*>(tmem_slot + 6);       // item whose chunks the whole CTA adds up at the end, or -1
  volatile WaitState* abort_flag = reinterpret_cast<volatile WaitState*>(tmem_slot + 2);

  const uint32_t bar0 = smem_u32(bars);
  auto w_full = [&](int s) { return bar0 + 8u * s; };                       // packed weights of a PK slot have landed
  auto x_full = [&](int s) { return bar0 + 8u * (PK_SLOTS + s); };          // its activation tile has landed
  auto pk_free = [&](int s) { return bar0 + 8u * (2 * PK_SLOTS + s); };
  auto cv_ready = [&](int s) { return bar0 + 8u * (3 * PK_SLOTS + s); };
  auto cv_free = [&](int s) { return bar0 + 8u * (3 * PK_SLOTS + CV_SLOTS + s); };
  auto acc_full = [&](int a) { return bar0 + 8u * (3 * PK_SLOTS + 2 * CV_SLOTS + a); };
  auto acc_empty = [&](int a) { return bar0 + 8u * (3 * PK_SLOTS + 2 * CV_SLOTS + 2 + a); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, num_ctas = gridDim.x;
  const int num_items = p.num_items;

  if (threadIdx.x == 0) {
    for (int s = 0; s < PK_SLOTS; ++s) { mbar_init(w_full(s), 1); mbar_init(x_full(s), 1); mbar_init(pk_free(s), 1); }
    for (int s = 0; s < CV_SLOTS; ++s) { mbar_init(cv_ready(s), WARPS_PER_GROUP); mbar_init(cv_free(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(acc_full(a), 1); mbar_init(acc_empty(a), 4); }
    abort_flag->abort = 0;
    abort_flag->limit = p.wait_limit;
    *deferred = -1;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), C::TMEM_COLS);
  // rows of the activation tiles beyond the batch are zero for the whole launch: TMA only ever writes the first x_rows
  for (int i = threadIdx.x; i < PK_SLOTS * (C::X_TILE_BYTES / 16); i += NUM_THREADS) {
    const int slot = i / (C::X_TILE_BYTES / 16), o = i % (C::X_TILE_BYTES / 16);
    if (o * 16 >= p.x_rows * 128) *reinterpret_cast<uint4*>(pk_base + slot * C::PK_SLOT_BYTES + o * 16) = make_uint4(0u, 0u, 0u, 0u);
  }
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_launch_dependents();               // the next kernel may set up (it waits for this one before it touches memory)

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      // Packed weights depend on no earlier kernel: the first PK_SLOTS stages are requested at once, and only
      // then does the producer wait for the kernel before (the prologue that writes Xcat) and request the
      // activation tiles of those stages.
      int pend_slot[PK_SLOTS], pend_x[PK_SLOTS], pend_layer[PK_SLOTS];
      int npend = 0;
      bool waited = false;
      // the activation tiles of the stages requested before the wait land on a barrier of their own (x_full, used
      // once per slot); later ones share the weights' barrier, so that the MMA warp has one barrier to watch
      auto load_x = [&](int slot, int layer, int xcol) {
        mbar_expect_tx(x_full(slot), p.x_rows * 128);        // rows of the box beyond the batch arrive as zeros
        tma_load_2d(smem_u32(pk_base + slot * C::PK_SLOT_BYTES), &tmaps.m[layer], xcol, 0, x_full(slot));
      };
      auto flush = [&]() {
        pdl_wait();
        for (int q = 0; q < npend; ++q) load_x(pend_slot[q], pend_layer[q], pend_x[q]);
        npend = 0;
        waited = true;
      };
      int pk = 0;
      uint32_t ph = 0;
      bool ok = true;
      const uint32_t w_tile = (uint32_t)w_tile_bytes(p.w_bits);
      for (int i = cta; i < num_items && ok; i += num_ctas) {
        const Item it = item_of(p, i);
        const Layer& ly = p.L[it.layer];
        const int b_tile_stride = ly.r_blocks * kTileN * 17;
        const int nt0 = 2 * it.tile;
        const int n_half = nt0 + 1 < ly.n_tiles ? 2 : 1;       // 128-column tiles of this 256-column tile that exist
        for (int s = it.s_lo; s < it.s_hi; ++s) {
          if (p.stall != 0 && s == it.s_hi - 1 && i + num_ctas >= num_items) { ok = false; break; }
          if (!waited && npend == PK_SLOTS) flush();
          if (!mbar_wait<true>(pk_free(pk), ph ^ 1, abort_flag)) { ok = false; break; }
          const uint32_t dst = smem_u32(pk_base + pk * C::PK_SLOT_BYTES) + C::X_TILE_BYTES;
          int xcol;
          const uint32_t x_bytes = waited ? (uint32_t)p.x_rows * 128u : 0u;
          if (s < ly.k_slabs) {
            if (!LQER_IN_BOUNDS(p.status, ((size_t)(nt0 + n_half - 1) * ly.k_slabs + s) * w_tile, w_tile, ly.w_extent, 705)) { ok = false; break; }
            mbar_expect_tx(w_full(pk), n_half * w_tile + x_bytes);
            for (int h = 0; h < n_half; ++h)
              bulk_load(dst + h * kWTileBytes, ly.wsec + ((size_t)(nt0 + h) * ly.k_slabs + s) * w_tile, w_tile, w_full(pk));
            xcol = s * BK;
          } else {
            const int rs = s - ly.k_slabs;
            const int rb0 = rs * 2, nb = min(2, ly.r_blocks - rb0);
            if (!LQER_IN_BOUNDS(p.status, (size_t)(nt0 + n_half - 1) * b_tile_stride + (size_t)ly.r_blocks * kTileN * 16 + rb0 * kTileN,
                                nb * kTileN, ly.b_extent, 706)) { ok = false; break; }
            mbar_expect_tx(w_full(pk), n_half * nb * (kTileN * 17) + x_bytes);
            for (int h = 0; h < n_half; ++h) {
              const uint8_t* tile = ly.bsec + (size_t)(nt0 + h) * b_tile_stride;
              bulk_load(dst + h * kWTileBytes, tile + (size_t)rb0 * kTileN * 16, nb * kTileN * 16, w_full(pk));
              bulk_load(dst + h * kWTileBytes + 4096, tile + (size_t)ly.r_blocks * kTileN * 16 + rb0 * kTileN, nb * kTileN, w_full(pk));
            }
            xcol = ly.K64 + rs * RANK_PER_STAGE;
          }
          if (waited) {
            tma_load_2d(smem_u32(pk_base + pk * C::PK_SLOT_BYTES), &tmaps.m[it.layer], xcol, 0, w_full(pk));
          } else {
            pend_slot[npend] = pk; pend_x[npend] = xcol; pend_layer[npend] = it.layer;
            ++npend;
          }
          if (++pk == PK_SLOTS) { pk = 0; ph ^= 1; }
        }
      }
      if (!waited) flush();
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issue
    // The tensor pipe queues very few MMAs, so what the issuing warp spends between two of them beyond the pipe's
    // own time is idle time of the pipe: the whole warp runs the loop (barrier addresses and descriptors are
    // warp-uniform values) and one elected lane issues.
    constexpr uint32_t idesc = make_idesc(MT, BN);
    const uint32_t cv0 = smem_u32(cv_base), pk0 = smem_u32(pk_base);
    uint32_t it_no = 0, tile_it = 0;
    bool ok = true;
    for (int i = cta; i < num_items && ok; i += num_ctas, ++tile_it) {
      const Item it = item_of(p, i);
      const Layer& ly = p.L[it.layer];
      const int acc = tile_it & 1;
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(acc_empty(acc), ((tile_it >> 1) & 1) ^ 1, abort_flag)) != 0;
      if (!ok) break;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + acc * BN;
      for (int s = it.s_lo; s < it.s_hi; ++s, ++it_no) {
        const int cv = it_no % CV_SLOTS, pk = it_no % PK_SLOTS;
        const uint64_t a_desc = make_desc(pk0 + pk * C::PK_SLOT_BYTES);
        const uint64_t b_desc = make_desc(cv0 + cv * CV_TILE_BYTES);
        const int nk = s < ly.k_slabs ? 4 : min(2, ly.r_blocks - (s - ly.k_slabs) * 2);
        // a converted tile implies its packed tile had landed, and with it (from the second pass over the ring on) the
        // activation tile; on the first pass the activation tiles have their own barrier
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(cv_ready(cv), (it_no / CV_SLOTS) & 1, abort_flag) &&
                                         (it_no >= (uint32_t)PK_SLOTS || mbar_wait(x_full(pk), 0, abort_flag))) != 0;
        if (!ok) break;
        tc_fence_after();
        if (elect_one()) {
          for (int j = 0; j < nk; ++j)              // +2 in the address field = 32 bytes = 16 K
            umma_bf16(d_tmem, a_desc + 2 * j, b_desc + 2 * j, idesc, (s > it.s_lo || j > 0) ? 1u : 0u);
          umma_commit(cv_free(cv));
          umma_commit(pk_free(pk));
        }
        __syncwarp();
      }
      if (ok && elect_one()) umma_commit(acc_full(acc));
      __syncwarp();
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------------ epilogue
    // A lane of tensor memory holds a token: the 128-row MMA puts row r in lane r, the 64-row MMA puts rows
    // 16 q .. 16 q + 15 in the first 16 lanes of lane quarter q.
    const int q = warp & 3;
    const int token = MT == 128 ? q * 32 + lane : (lane < 16 ? q * 16 + lane : p.M);
    const bool warp_has_rows = (MT == 128 ? q * 32 : q * 16) < p.M;
    const int et = threadIdx.x - 64;               // 0..127: index among the epilogue threads
    uint32_t tile_it = 0;
    bool ok = true;
    pdl_wait();                                    // Y, the scratch and the counters may be in use by the kernel before
    for (int i = cta; i < num_items && ok; i += num_ctas, ++tile_it) {
      const Item it = item_of(p, i);
      const Layer& ly = p.L[it.layer];
      const int acc = tile_it & 1;
      if (!mbar_wait<true>(acc_full(acc), (tile_it >> 1) & 1, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int col0 = it.tile * BN;
      const bool direct = ly.chunks == 1;
      if (warp_has_rows) {
        float* prow = direct ? nullptr : ly.partials + ((size_t)(it.tile * ly.chunks + it.chunk) * p.M + token) * BN;
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 32) {
          if (col0 + c0 >= ly.N) break;
          uint32_t r[32];
          tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN + c0, r);
          tmem_ld_wait();
          if (token < p.M) {
            if (direct && p.y_type == kYMXINT8) {
              // a token's 32 columns are two whole 16-blocks of its row
              const QuantConsts qc = quant_consts(p.a_bits, p.exp_min, p.exp_max);
              uint8_t* yq = static_cast<uint8_t*>(ly.Y);
#pragma unroll
              for (int j = 0; j < 2; ++j)
                if (col0 + c0 + 16 * j < ly.N) {          // N is a multiple of 16 here
                  float v[16];
#pragma unroll
                  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[16 * j + i]);
                  uint4 m8, b0, b1;
                  int e;
                  quantize_block16(v, qc, e, m8, b0, b1);
                  const size_t idx = (size_t)token * ly.N + col0 + c0 + 16 * j;
                  if (LQER_IN_BOUNDS(p.status, (size_t)p.M * ly.N + idx / 16, 1, ly.y_extent, 703)) {
                    *reinterpret_cast<uint4*>(yq + idx) = m8;
                    yq[(size_t)p.M * ly.N + idx / 16] = (uint8_t)(e + 127);
                  }
                }
            } else {
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const float4 v = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]),
                                             __uint_as_float(r[4 * j + 3]));
                if (!direct) {
                  if (LQER_IN_BOUNDS(p.status, (size_t)(prow + c0 + 4 * j - ly.partials) * 4, 16, ly.partial_extent, 704))
                    *reinterpret_cast<float4*>(prow + c0 + 4 * j) = v;
                }
                else if (col0 + c0 + 4 * j < ly.N) store_y4(ly.Y, (size_t)token * ly.N + col0 + c0 + 4 * j, v, p.y_type, p.status, ly.y_extent);   // N is a multiple of 8
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty(acc));
      if (!direct) {
        // count this chunk in; whoever brings the last partial of the tile adds them all up, in chunk order
        __threadfence();
        epilogue_barrier();
        if (et == 0) *last_flag = (atomicAdd(ly.counters + it.tile, 1) == ly.chunks - 1) ? 1 : 0;
        epilogue_barrier();
        if (*last_flag != 0) {
          if (i + num_ctas >= num_items) {
            // the CTA's last item: every other role is about to fall idle, so the whole CTA adds the chunks up at the end
            if (et == 0) *deferred = i;
          } else {
            __threadfence();
            reduce_tile(p, ly, it.tile, et, 128);
            if (et == 0) ly.counters[it.tile] = 0;    // zero again for the next call
          }
        }
        epilogue_barrier();                         // last_flag may be rewritten only after everyone has read it
      }
    }
  } else {
    // ------------------------------------------------------------------ converters
    const int c = threadIdx.x - 6 * 32;          // 0..767
    const int group = c >> 8, col = c & 255;     // stage group; weight column of the 256-column stage
    const int half = col >> 7, nl = col & 127;   // its 128-column packed tile, and the column within it
    const int sw = col & 7;
    uint32_t chunk[8];                           // the row's eight 16-byte chunks after the 128-byte swizzle
#pragma unroll
    for (int i = 0; i < 8; ++i) chunk[i] = (uint32_t)(col * 128 + ((i ^ sw) << 4));
    // the CTA's items one after the other; their K stages form one sequence of which this group takes every third
    int item = cta, s = group;                   // s: offset into the current item's stages; normalised below
    Item cur;
    cur.layer = 0; cur.tile = 0; cur.chunk = 0; cur.s_lo = 0; cur.s_hi = 0;
    if (item < num_items) cur = item_of(p, item);
    bool ok = true;
    for (uint32_t it_no = group; item < num_items && ok; it_no += CONVERTER_GROUPS, s += CONVERTER_GROUPS) {
      while (item < num_items && s >= cur.s_hi - cur.s_lo) {
        s -= cur.s_hi - cur.s_lo;
        item += num_ctas;
        if (item < num_items) cur = item_of(p, item);
      }
      if (item >= num_items) break;
      const Layer& ly = p.L[cur.layer];
      const int stage = cur.s_lo + s;
      const int pk = it_no % PK_SLOTS;
      const bool has_w = 2 * cur.tile + half < ly.n_tiles;
      if (!mbar_wait(w_full(pk), (it_no / PK_SLOTS) & 1, abort_flag)) { ok = false; break; }
      if (!mbar_wait(cv_free(group), ((it_no / CV_SLOTS) & 1) ^ 1, abort_flag)) { ok = false; break; }
      const uint8_t* pkt = pk_base + pk * C::PK_SLOT_BYTES + C::X_TILE_BYTES + half * kWTileBytes;
      uint8_t* bt = cv_base + group * CV_TILE_BYTES;
      if (!has_w) {                                // columns beyond N: a zero operand row
        const int nchunks = stage < ly.k_slabs ? 8 : 4;
        for (int i = 0; i < nchunks; ++i) *reinterpret_cast<uint4*>(bt + chunk[i]) = make_uint4(0u, 0u, 0u, 0u);
      } else if (stage < ly.k_slabs) {
        convert_column(pkt, nl, p.w_bits, bt, chunk);
      } else {
        const int nb = min(2, ly.r_blocks - (stage - ly.k_slabs) * 2);
        for (int rb = 0; rb < nb; ++rb) {
          const uint4 w = *reinterpret_cast<const uint4*>(pkt + (rb * kTileN + nl) * 16);
          const float scale = pow2f((int)pkt[4096 + rb * kTileN + nl] - 127 - p.lr_shift);
          *reinterpret_cast<uint4*>(bt + chunk[rb * 2]) = convert_i8x8(w.x, w.y, scale);
          *reinterpret_cast<uint4*>(bt + chunk[rb * 2 + 1]) = convert_i8x8(w.z, w.w, scale);
        }
      }
      fence_proxy_async_smem();        // generic-proxy writes -> visible to the MMA's async proxy
      __syncwarp();
      if (lane == 0) mbar_arrive(cv_ready(group));
    }
  }

  // ------------------------------------------------------------------ teardown
  __syncthreads();                      // every role is done (or has given up): the flags below are final for this CTA
  if (*deferred >= 0 && abort_flag->abort == 0) {
    const Item it = item_of(p, *deferred);
    __threadfence();
    reduce_tile(p, p.L[it.layer], it.tile, threadIdx.x, NUM_THREADS);
    if (threadIdx.x == 0) p.L[it.layer].counters[it.tile] = 0;     // zero again for the next call
  }
  if (abort_flag->abort != 0) {
    const long long t0 = clock64();
    while (clock64() - t0 < 400000) { }
    if (threadIdx.x == 0) report_error(p.status, LQER_ERR_TIMEOUT, 600, blockIdx.x);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
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

template <int MT, int PK_SLOTS>
static cudaError_t launch_mt(const TensorMaps& tmaps, const Params& p, int ctas, cudaStream_t s) {
  using C = Cfg<MT, PK_SLOTS>;
  static OncePerDevice once;
  cudaError_t e = once.run([] {
    return cudaFuncSetAttribute(gemm_small_kernel<MT, PK_SLOTS>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
  });
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(ctas);
  cfg.blockDim = dim3(NUM_THREADS);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may set up and prefetch weights while the prologue runs
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  LaunchScope scope(kFamDecode, s);
  return cudaLaunchKernelEx(&cfg, gemm_small_kernel<MT, PK_SLOTS>, tmaps, p);
}

}  // namespace sg

int gemm_small_max_layers() { return sg::MAX_LAYERS; }

cudaError_t launch_gemm_small(const SmallGemmLayer* layers, int n, int M, int y_type, bool tensor_memory_form, int epoch,
                              DeviceStatus* st, cudaStream_t s) {
  using namespace sg;
  if (n < 1 || n > MAX_LAYERS || M < 1 || M > kSmallMaxM) return cudaErrorInvalidValue;
  // up to 16 tokens: the register-operand kernel, unless the caller asks for this file's
  const bool use_mma = !tensor_memory_form && small_takes_mma(*layers[0].meta, M);
  EncodeTiledFn enc = use_mma ? nullptr : encode_fn();
  if (enc == nullptr && !use_mma) return cudaErrorNotSupported;
  const int MT = M <= 64 ? 64 : 128;
  const int x_rows = (M + 7) / 8 * 8;
  TensorMaps tmaps;
  Params p;
  int item_begin = 0;
  // K chunks per tile.  A layer alone is cut as its shape says (small_gemm_chunks: enough work items for every SM).
  // Layers that share a launch bring many tiles between them, and every chunk costs a pass of partial sums through
  // L2, so they are cut less: just enough for about two work items per SM in all, never more than alone (the scratch
  // is sized for that; finer cuts that would even out the last round of items were measured and lose more in
  // epilogues than they gain).  The sums of a tile are then grouped differently, so a layer's result in a shared launch
  // may differ from its result alone in the last bits; it is the same whenever the same layers share a launch.
  const int sms = sm_count();
  if (sms < 1) return cudaErrorInvalidDevice;
  int total_tiles = 0;
  for (int i = 0; i < n; ++i) total_tiles += small_gemm_col_tiles(*layers[i].meta);
  int group_chunks = (2 * 148 + total_tiles - 1) / total_tiles;            // about two work items per SM in all
  if (use_mma && n > 1) {
    // The register-operand kernel runs two CTAs per SM, an item each at a time, and an item costs about ten slabs' worth
    // of time beside its own slabs (activation copy, rank term, partial sums): the cut that makes (rounds of items over
    // 2 x 148 CTAs) x (slabs per item + 10) smallest, a function of the shapes alone like the rule above.
    long best = -1;
    for (int c = 1; c <= 16; ++c) {
      long items = 0, len = 0;
      for (int i = 0; i < n; ++i) {
        const PackedMeta& m = *layers[i].meta;
        const int ci = std::min(c, small_gemm_chunks(m));
        items += (long)small_gemm_col_tiles(m) * ci;
        len = std::max(len, (long)(m.k_slabs + ci - 1) / ci);
      }
      const long cost = ((items + 2 * 148 - 1) / (2 * 148)) * (len + 10);
      if (best < 0 || cost < best) { best = cost; group_chunks = c; }
    }
  }
  for (int i = 0; i < MAX_LAYERS; ++i) {
    const SmallGemmLayer& src = layers[i < n ? i : 0];
    const PackedMeta& m = *src.meta;
    if (m.lr_bits != layers[0].meta->lr_bits || m.w_bits != layers[0].meta->w_bits) return cudaErrorInvalidValue;
    const cuuint64_t dims[2] = {(cuuint64_t)xcat_cols(m), (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)xcat_cols(m) * 2};
    const cuuint32_t box[2] = {BK, (cuuint32_t)x_rows};
    const cuuint32_t estr[2] = {1, 1};
    if (!use_mma &&
        enc(&tmaps.m[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(src.xcat), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
    const uint8_t* base = static_cast<const uint8_t*>(src.packed);
    Layer& ly = p.L[i];
    ly.wsec = base + m.off_w;
    ly.bsec = base + m.off_b;
    ly.xfrag = static_cast<const uint8_t*>(src.xcat);
    ly.flags = src.flags;
    ly.plane = (m.k_slabs + frag_rank_slabs(m)) * 256;
    ly.Y = src.Y;
    ly.y_extent = y_bytes(y_type, (size_t)M, (size_t)m.N);
    if (kDebugBounds) ly.y_extent -= std::min(ly.y_extent, debug_y_shrink());
    ly.w_extent = m.off_b - m.off_w; ly.b_extent = m.off_a - m.off_b;
    ly.partials = src.partials;
    ly.counters = src.counters;
    ly.N = m.N; ly.K64 = m.K64;
    ly.n_tiles = m.n_tiles; ly.k_slabs = m.k_slabs; ly.r_blocks = m.r_blocks;
    ly.spt = m.k_slabs + (m.r_blocks + 1) / 2;
    int want = small_gemm_chunks(m);
    if (n > 1 && group_chunks < want) want = group_chunks;
    ly.chunk_stages = (m.k_slabs + want - 1) / want;
    ly.chunks = (m.k_slabs + ly.chunk_stages - 1) / ly.chunk_stages;
    ly.partial_extent = ly.chunks > 1 ? (size_t)small_gemm_col_tiles(m) * ly.chunks * M * 256 * 4 : 0;
    ly.item_begin = item_begin;
    if (i < n) item_begin += small_gemm_col_tiles(m) * ly.chunks;
  }
  p.n = n;
  p.num_items = item_begin;
  p.status = st;
  p.M = M;
  p.lr_shift = layers[0].meta->lr_bits - 2;
  p.y_type = y_type;
  p.a_bits = layers[0].meta->a_bits; p.exp_min = layers[0].meta->exp_min; p.exp_max = layers[0].meta->exp_max;
  p.x_rows = x_rows;
  p.w_bits = layers[0].meta->w_bits;
  p.wait_limit = wait_limit_cycles();
  p.epoch = epoch;
  p.exit_count = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(st) + kFlagAreaOffset + 2 * MAX_LAYERS * 4);
  p.stall = take_stall(kFamDecode) ? 1 : 0;
  if (use_mma) return launch_gemm_mma(p, s);
  const int ctas = p.num_items < sms ? p.num_items : sms;
  return MT == 64 ? launch_mt<64, 6>(tmaps, p, ctas, s) : launch_mt<128, 3>(tmaps, p, ctas, s);
}

}  // namespace lqer
