// Small-batch form of the layer's contraction (paper Section 3.1 / 3.2: Y = [X_q | T_q] . [W_q ; B_q];
// Section 2.1: few tokens per step make the layer memory bound on its weights).
//
// With up to 128 tokens the weights are the large operand, so here they take the M side of the
// 5th-generation tensor-core MMA and the tokens the N side:
//     D[128 weight columns, NT tokens] += Wtile[128, 16 K] . Xtile[NT, 16 K]^T      (tcgen05.mma, bf16 -> fp32)
// A CTA streams packed weight tiles (128 columns x 64 K, one bulk copy each) exactly once, converts the
// 4-bit mantissas to their exact bf16 values in shared memory (as the large-batch GEMM does) and multiplies
// them with a [NT, 64] tile of the quantised activations that TMA brings from Xcat.  The accumulator
// lives in tensor memory with a weight column per lane, so the epilogue writes rows of Y that are
// contiguous across the lanes of a warp.
//
// Work items are (layer, column tile, K chunk).  The chunks of a tile are fixed by the shape alone (so a
// result never depends on the number of SMs or on which layers share a launch); each chunk is summed from
// zero in tensor memory and, if a tile has more than one, leaves its fp32 partial in scratch; the CTA whose
// partial arrives last adds the chunks in chunk order and writes Y.  Nothing waits for another CTA.
// Roles per CTA:
//   warp 0      producer: bulk copies of packed weight tiles (issued before the dependency wait: weights
//               depend on no earlier kernel) and TMA loads of activation tiles
//   warp 1, 30  MMA issuers (even / odd stages of an item, an accumulator each); warp 1 also allocates tensor memory
//   warps 2-5   epilogue (tcgen05.ld, Y or partial sums, the last-arriver reduction)
//   warps 6-29  converters in six groups; group g converts the stages with index = g (mod 6)
// Two rings: PK slots hold {activation tile, packed weight tile} and are deep, because the bytes in flight
// bound the bandwidth; CV slots hold converted weight tiles.
#include "lqer_tc_ptx.cuh"

namespace lqer {
namespace tn {
using namespace tc;

constexpr int BMW = 128;                   // weight columns per tile = rows of the MMA
constexpr int BK = 64;
constexpr int CV_TILE_BYTES = BMW * BK * 2;   // 16384
constexpr int CV_SLOTS = 6;
constexpr int CONVERTER_GROUPS = 6;        // = CV_SLOTS: a group meets one CV slot only, and PK slots in phase order
constexpr int WARPS_PER_GROUP = 4;
constexpr int ISSUER_B_WARP = 6 + CONVERTER_GROUPS * WARPS_PER_GROUP;   // the second MMA-issuing warp
constexpr int NUM_THREADS = (ISSUER_B_WARP + 1) * 32;
constexpr int RANK_PER_STAGE = 32;
constexpr int MAX_LAYERS = 16;

template <int NT, int PK_SLOTS>
struct Cfg {
  static constexpr int X_TILE_BYTES = NT * 128;
  static constexpr int PK_SLOT_BYTES = (X_TILE_BYTES + kWTileBytes + 1023) / 1024 * 1024;
  static constexpr int OFF_PK = CV_SLOTS * CV_TILE_BYTES;
  static constexpr int OFF_BARS = OFF_PK + PK_SLOTS * PK_SLOT_BYTES;
  static constexpr int NUM_BARS = 2 * PK_SLOTS + 2 * CV_SLOTS + 4;
  static constexpr int SMEM_BYTES = OFF_BARS + NUM_BARS * 8 + 64 + 1024;
  static constexpr int TMEM_COLS = 4 * NT < 32 ? 32 : 4 * NT;   // two accumulators per item (one per issuing warp), two items
  static_assert(PK_SLOTS % CONVERTER_GROUPS == 0, "a converter group must meet a PK slot in phase order");
  static_assert((TMEM_COLS & (TMEM_COLS - 1)) == 0 && TMEM_COLS <= 512, "tensor memory columns");
  static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
};

struct Layer {
  const uint8_t* wsec;
  const uint8_t* bsec;
  void* Y;                     // [M, N] fp32 or bf16
  float* partials;             // [tile][chunk][M][128] fp32 (tiles with more than one chunk)
  int* counters;               // [tile] arrivals, zero between calls
  int N, K64, n_tiles, k_slabs, r_blocks;
  int spt;                     // K stages per tile: k_slabs + rank stages
  int chunks, chunk_stages;    // K chunks per tile; weight stages per chunk (the last chunk also takes the rank stages)
  int item_begin;              // first item of this layer in the launch's list
};

struct Params {
  Layer L[MAX_LAYERS];
  int n;                       // layers in this launch
  int num_items;
  DeviceStatus* status;
  int M;
  int lr_shift;
  int y_bf16;                  // Y is bf16 (round to nearest even), else fp32
  long long wait_limit;
  int stall;                   // test hook: the producer withholds the last stage of its last item
};

struct TensorMaps {
  CUtensorMap m[MAX_LAYERS];   // Xcat of each layer: bf16 [M, K64 + k_pad], box 64 x NT
};

struct Item {
  int layer, tile, chunk, s_lo, s_hi;
};
__device__ __forceinline__ Item item_of(const Params& p, int i) {
  int l = 0;
#pragma unroll
  for (int q = 1; q < MAX_LAYERS; ++q)
    if (q < p.n && i >= p.L[q].item_begin) l = q;
  const Layer& ly = p.L[l];
  const int local = i - ly.item_begin;
  Item it;
  it.layer = l;
  it.tile = local / ly.chunks;
  it.chunk = local - it.tile * ly.chunks;
  it.s_lo = it.chunk * ly.chunk_stages;
  it.s_hi = it.chunk == ly.chunks - 1 ? ly.spt : it.s_lo + ly.chunk_stages;
  return it;
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void epilogue_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ uint16_t bf16_rn(float v) {
  uint32_t u = __float_as_uint(v);
  if ((u & 0x7F800000u) == 0x7F800000u) return (uint16_t)((u >> 16) | ((u & 0xFFFFu) ? 0x40u : 0u));   // inf / NaN
  u += 0x7FFFu + ((u >> 16) & 1u);                                                                  // round to nearest even
  return (uint16_t)(u >> 16);
}

template <int NT, int PK_SLOTS>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tn_kernel(const __grid_constant__ TensorMaps tmaps, const __grid_constant__ Params p) {
  using C = Cfg<NT, PK_SLOTS>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* cv_base = smem;
  uint8_t* pk_base = smem + C::OFF_PK;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BARS);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + C::NUM_BARS);
  int* last_flag = reinterpret_cast<int*>(tmem_slot + 1);
  volatile WaitState* abort_flag = reinterpret_cast<volatile WaitState*>(tmem_slot + 2);

  const uint32_t bar0 = smem_u32(bars);
  auto pk_full = [&](int s) { return bar0 + 8u * s; };
  auto pk_free = [&](int s) { return bar0 + 8u * (PK_SLOTS + s); };
  auto cv_ready = [&](int s) { return bar0 + 8u * (2 * PK_SLOTS + s); };
  auto cv_free = [&](int s) { return bar0 + 8u * (2 * PK_SLOTS + CV_SLOTS + s); };
  auto acc_full = [&](int a) { return bar0 + 8u * (2 * PK_SLOTS + 2 * CV_SLOTS + a); };
  auto acc_empty = [&](int a) { return bar0 + 8u * (2 * PK_SLOTS + 2 * CV_SLOTS + 2 + a); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, num_ctas = gridDim.x;
  const int num_items = p.num_items;

  if (threadIdx.x == 0) {
    for (int s = 0; s < PK_SLOTS; ++s) { mbar_init(pk_full(s), 1); mbar_init(pk_free(s), 1); }
    for (int s = 0; s < CV_SLOTS; ++s) { mbar_init(cv_ready(s), WARPS_PER_GROUP); mbar_init(cv_free(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(acc_full(a), 2); mbar_init(acc_empty(a), 4); }
    abort_flag->abort = 0;
    abort_flag->limit = p.wait_limit;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), C::TMEM_COLS);
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
      auto flush = [&]() {
        pdl_wait();
        for (int q = 0; q < npend; ++q)
          tma_load_2d(smem_u32(pk_base + pend_slot[q] * C::PK_SLOT_BYTES), &tmaps.m[pend_layer[q]], pend_x[q], 0, pk_full(pend_slot[q]));
        npend = 0;
        waited = true;
      };
      int pk = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int i = cta; i < num_items && ok; i += num_ctas) {
        const Item it = item_of(p, i);
        const Layer& ly = p.L[it.layer];
        const int b_tile_stride = ly.r_blocks * kTileN * 17;
        for (int s = it.s_lo; s < it.s_hi; ++s) {
          if (p.stall != 0 && s == it.s_hi - 1 && i + num_ctas >= num_items) { ok = false; break; }
          if (!waited && npend == PK_SLOTS) flush();
          if (!mbar_wait<true>(pk_free(pk), ph ^ 1, abort_flag)) { ok = false; break; }
          const uint32_t dst = smem_u32(pk_base + pk * C::PK_SLOT_BYTES);
          int xcol;
          if (s < ly.k_slabs) {
            mbar_expect_tx(pk_full(pk), C::X_TILE_BYTES + kWTileBytes);
            bulk_load(dst + C::X_TILE_BYTES, ly.wsec + ((size_t)it.tile * ly.k_slabs + s) * kWTileBytes, kWTileBytes, pk_full(pk));
            xcol = s * BK;
          } else {
            const int rs = s - ly.k_slabs;
            const int rb0 = rs * 2, nb = min(2, ly.r_blocks - rb0);
            mbar_expect_tx(pk_full(pk), C::X_TILE_BYTES + nb * (kTileN * 17));
            const uint8_t* tile = ly.bsec + (size_t)it.tile * b_tile_stride;
            bulk_load(dst + C::X_TILE_BYTES, tile + (size_t)rb0 * kTileN * 16, nb * kTileN * 16, pk_full(pk));
            bulk_load(dst + C::X_TILE_BYTES + 4096, tile + (size_t)ly.r_blocks * kTileN * 16 + rb0 * kTileN, nb * kTileN, pk_full(pk));
            xcol = ly.K64 + rs * RANK_PER_STAGE;
          }
          if (waited) {
            tma_load_2d(dst, &tmaps.m[it.layer], xcol, 0, pk_full(pk));
          } else {
            pend_slot[npend] = pk; pend_x[npend] = xcol; pend_layer[npend] = it.layer;
            ++npend;
          }
          if (++pk == PK_SLOTS) { pk = 0; ph ^= 1; }
        }
      }
      if (!waited) flush();
    }
  } else if (warp == 1 || warp == ISSUER_B_WARP) {
    // ------------------------------------------------------------------ MMA issuers
    // An MMA with so few tokens costs the tensor core far more than its arithmetic, and what bounds the kernel is
    // the rate at which MMAs can be handed over.  So two warps issue: one takes the even stages of an item, the
    // other the odd ones, each into an accumulator of its own (the epilogue adds the two).  The whole warp runs the
    // loop, so that descriptors and addresses are warp-uniform values; one elected lane issues.
    const int which = warp == 1 ? 0 : 1;
    constexpr uint32_t idesc = make_idesc(BMW, NT);
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
      const uint32_t d_tmem = tmem_base + acc * 2 * NT + which * NT;
      for (int s = it.s_lo; s < it.s_hi; ++s, ++it_no) {
        if (((s - it.s_lo) & 1) != which) continue;
        const int cv = it_no % CV_SLOTS, pk = it_no % PK_SLOTS;
        const uint64_t a_desc = make_desc(cv0 + cv * CV_TILE_BYTES);
        const uint64_t b_desc = make_desc(pk0 + pk * C::PK_SLOT_BYTES);
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(cv_ready(cv), (it_no / CV_SLOTS) & 1, abort_flag)) != 0;
        if (!ok) break;
        tc_fence_after();
        const int nk = s < ly.k_slabs ? 4 : min(2, ly.r_blocks - (s - ly.k_slabs) * 2);
        if (elect_one()) {
          for (int j = 0; j < nk; ++j)              // +2 in the address field = 32 bytes = 16 K
            umma_bf16(d_tmem, a_desc + 2 * j, b_desc + 2 * j, idesc, (s > it.s_lo + which || j > 0) ? 1u : 0u);
          umma_commit(cv_free(cv));
          umma_commit(pk_free(pk));
        }
        __syncwarp();
      }
      if (ok && elect_one()) umma_commit(acc_full(acc));   // with no stage of its own (a one-stage item) it arrives at once
      __syncwarp();
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------------ epilogue
    const int q = warp & 3;                        // lane quarter of tensor memory = 32 weight columns
    const int col_in_tile = q * 32 + lane;
    uint32_t tile_it = 0;
    bool ok = true;
    pdl_wait();                                    // Y, the scratch and the counters may be in use by the kernel before
    for (int i = cta; i < num_items && ok; i += num_ctas, ++tile_it) {
      const Item it = item_of(p, i);
      const Layer& ly = p.L[it.layer];
      const int acc = tile_it & 1;
      if (!mbar_wait<true>(acc_full(acc), (tile_it >> 1) & 1, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const int col = it.tile * BMW + col_in_tile;
      const bool col_ok = col < ly.N;
      const bool direct = ly.chunks == 1;
      float* part = ly.partials + ((size_t)(it.tile * ly.chunks + it.chunk) * p.M) * BMW + col_in_tile;
#pragma unroll 1
      for (int c0 = 0; c0 < NT; c0 += 16) {
        if (c0 >= p.M) break;
        uint32_t r[16];
        tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + acc * 2 * NT + c0, r);
        if (it.s_hi - it.s_lo >= 2) {                // the odd stages' accumulator (empty for a one-stage item)
          uint32_t r2[16];
          tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + acc * 2 * NT + NT + c0, r2);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(r2[j]));
        }
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int token = c0 + j;
          if (token < p.M) {
            if (!direct) {
              part[(size_t)token * BMW] = __uint_as_float(r[j]);
            } else if (col_ok) {
              if (p.y_bf16) static_cast<uint16_t*>(ly.Y)[(size_t)token * ly.N + col] = bf16_rn(__uint_as_float(r[j]));
              else static_cast<float*>(ly.Y)[(size_t)token * ly.N + col] = __uint_as_float(r[j]);
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
        if (warp == 2 && lane == 0) *last_flag = (atomicAdd(ly.counters + it.tile, 1) == ly.chunks - 1) ? 1 : 0;
        epilogue_barrier();
        if (*last_flag != 0) {
          __threadfence();
          // a warp per token row, a lane per four columns; the chunk loads of two rows are in flight together
          const int c4 = lane * 4, trow0 = warp - 2;
          const bool quad_ok = it.tile * BMW + c4 < ly.N;              // N is a multiple of 8: the quad is whole
          const float* p0 = ly.partials + ((size_t)it.tile * ly.chunks * p.M) * BMW + c4;
          const size_t chunk_stride = (size_t)p.M * BMW;
          for (int token = trow0; token < p.M; token += 8) {
            float4 v[2] = {make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f)};
            for (int cb = 0; cb < ly.chunks; cb += 4) {
              float4 t[2][4];
#pragma unroll
              for (int u = 0; u < 2; ++u)
#pragma unroll
                for (int c = 0; c < 4; ++c)
                  t[u][c] = (cb + c < ly.chunks && token + 4 * u < p.M)
                                ? __ldcg(reinterpret_cast<const float4*>(p0 + (size_t)(cb + c) * chunk_stride + (size_t)(token + 4 * u) * BMW))
                                : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
              for (int u = 0; u < 2; ++u)
#pragma unroll
                for (int c = 0; c < 4; ++c) {            // chunk order: the same sum whoever computes it
                  if (cb + c < ly.chunks) { v[u].x += t[u][c].x; v[u].y += t[u][c].y; v[u].z += t[u][c].z; v[u].w += t[u][c].w; }
                }
            }
#pragma unroll
            for (int u = 0; u < 2; ++u) {
              const int tk = token + 4 * u;
              if (tk < p.M && quad_ok) {
                const size_t o = (size_t)tk * ly.N + it.tile * BMW + c4;
                if (p.y_bf16)
                  *reinterpret_cast<uint2*>(static_cast<uint16_t*>(ly.Y) + o) =
                      make_uint2(bf16_rn(v[u].x) | ((uint32_t)bf16_rn(v[u].y) << 16), bf16_rn(v[u].z) | ((uint32_t)bf16_rn(v[u].w) << 16));
                else
                  *reinterpret_cast<float4*>(static_cast<float*>(ly.Y) + o) = v[u];
              }
            }
          }
          if (warp == 2 && lane == 0) ly.counters[it.tile] = 0;      // zero again for the next call
        }
        epilogue_barrier();                         // last_flag may be rewritten only after everyone has read it
      }
    }
  } else if (warp < ISSUER_B_WARP) {
    // ------------------------------------------------------------------ converters
    const int c = threadIdx.x - 6 * 32;          // 0..767
    const int group = c >> 7, nl = c & 127;      // stage group; weight column of the tile
    const int sw = nl & 7;
    uint32_t chunk[8];                           // the row's eight 16-byte chunks after the 128-byte swizzle
#pragma unroll
    for (int i = 0; i < 8; ++i) chunk[i] = (uint32_t)(nl * 128 + ((i ^ sw) << 4));
    // the CTA's items one after the other; their K stages form one sequence of which this group takes every sixth
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
      if (!mbar_wait(pk_full(pk), (it_no / PK_SLOTS) & 1, abort_flag)) { ok = false; break; }
      if (!mbar_wait(cv_free(group), ((it_no / CV_SLOTS) & 1) ^ 1, abort_flag)) { ok = false; break; }
      const uint8_t* pkt = pk_base + pk * C::PK_SLOT_BYTES + C::X_TILE_BYTES;
      uint8_t* bt = cv_base + group * CV_TILE_BYTES;
      if (stage < ly.k_slabs) {
        const uint4 wa = *reinterpret_cast<const uint4*>(pkt + nl * 16);
        const uint4 wb = *reinterpret_cast<const uint4*>(pkt + (kTileN + nl) * 16);
        const uint32_t eb = *reinterpret_cast<const uint32_t*>(pkt + kWTileNibbleBytes + nl * 4);
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
  __syncthreads();                      // every role is done (or has given up): the flag below is final for this CTA
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

template <int NT, int PK_SLOTS>
static cudaError_t launch_nt(const TensorMaps& tmaps, const Params& p, int ctas, cudaStream_t s) {
  using C = Cfg<NT, PK_SLOTS>;
  static OncePerDevice once;
  cudaError_t e = once.run([] {
    return cudaFuncSetAttribute(gemm_tn_kernel<NT, PK_SLOTS>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
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
  return cudaLaunchKernelEx(&cfg, gemm_tn_kernel<NT, PK_SLOTS>, tmaps, p);
}

}  // namespace tn

int gemm_tn_max_layers() { return tn::MAX_LAYERS; }

cudaError_t launch_gemm_tn(const SmallGemmLayer* layers, int n, int M, bool y_bf16, DeviceStatus* st, cudaStream_t s) {
  using namespace tn;
  if (n < 1 || n > MAX_LAYERS || M < 1 || M > kSmallMaxM) return cudaErrorInvalidValue;
  EncodeTiledFn enc = encode_fn();
  if (enc == nullptr) return cudaErrorNotSupported;
  const int NT = M <= 16 ? 16 : M <= 32 ? 32 : M <= 64 ? 64 : 128;
  TensorMaps tmaps;
  Params p;
  int item_begin = 0;
  for (int i = 0; i < MAX_LAYERS; ++i) {
    const SmallGemmLayer& src = layers[i < n ? i : 0];
    const PackedMeta& m = *src.meta;
    if (m.lr_bits != layers[0].meta->lr_bits) return cudaErrorInvalidValue;
    const cuuint64_t dims[2] = {(cuuint64_t)xcat_cols(m), (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)xcat_cols(m) * 2};
    const cuuint32_t box[2] = {BK, (cuuint32_t)NT};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&tmaps.m[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(src.xcat), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
    const uint8_t* base = static_cast<const uint8_t*>(src.packed);
    Layer& ly = p.L[i];
    ly.wsec = base + m.off_w;
    ly.bsec = base + m.off_b;
    ly.Y = src.Y;
    ly.partials = src.partials;
    ly.counters = src.counters;
    ly.N = m.N; ly.K64 = m.K64;
    ly.n_tiles = m.n_tiles; ly.k_slabs = m.k_slabs; ly.r_blocks = m.r_blocks;
    ly.spt = m.k_slabs + (m.r_blocks + 1) / 2;
    ly.chunks = small_gemm_chunks(m);
    ly.chunk_stages = small_gemm_chunk_stages(m);
    ly.item_begin = item_begin;
    if (i < n) item_begin += m.n_tiles * ly.chunks;
  }
  p.n = n;
  p.num_items = item_begin;
  p.status = st;
  p.M = M;
  p.lr_shift = layers[0].meta->lr_bits - 2;
  p.y_bf16 = y_bf16 ? 1 : 0;
  p.wait_limit = wait_limit_cycles();
  p.stall = take_stall(kFamDecode) ? 1 : 0;
  const int sms = sm_count();
  if (sms < 1) return cudaErrorInvalidDevice;
  const int ctas = p.num_items < sms ? p.num_items : sms;
  switch (NT) {
    case 16: return launch_nt<16, 12>(tmaps, p, ctas, s);
    case 32: return launch_nt<32, 12>(tmaps, p, ctas, s);
    case 64: return launch_nt<64, 6>(tmaps, p, ctas, s);
    default: return launch_nt<128, 6>(tmaps, p, ctas, s);
  }
}

}  // namespace lqer
