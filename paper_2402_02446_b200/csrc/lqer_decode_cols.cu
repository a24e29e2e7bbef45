// Decode form of the layer for M <= 4 tokens (paper Section 3.1 / 3.2; Section 2.1: small-batch
// inference is memory bound):
//
//     Y[M,N] = X_q W_q + q(X_q A_q) B_q
//
// With so few tokens a tensor-core MMA would spend 16 rows of work on at most 4, and a split of K
// across CTAs would end in cross-CTA partial sums of Y.  So here a CTA owns output columns and
// the whole contraction for them: groups of 8 columns are dealt out to the CTAs in contiguous
// ranges, four groups (32 columns) per round; within a round warp w takes the slabs (64 K) w,
// w + 16, ... of those columns, and the 16 warps' sums meet in shared memory and are added in warp
// order (at one token two rounds share a barrier: the first keeps its sums in registers).  Y is
// written once, by one thread per element.
//
// A lane of a warp owns one of the round's 32 columns and takes a whole slab of it at a time: the
// four 16-blocks of the slab as two 16-byte loads plus the four exponent bytes as one word.  Per
// block: four dp4a on the raw nibbles against the int8 mantissas of X (stored in the byte order the
// nibbles unpack to), started from 1.5 * 2^23 - 8 * sum(x) (the offset-binary nibbles; the constant
// makes the integer sum the bit pattern of a float, so one subtraction converts it), scaled by
// 2^(e_x + e_w) in fp32 and accumulated per token.  The loads run four slabs ahead; they depend on
// no earlier kernel and are issued before griddepcontrol.wait.
//
// X_q and T_q = q(X_q A_q) (exact dp4a block products, scaled and summed in fp64 in a fixed order)
// reach a CTA in one of three ways:
//  - computed ahead by decode_pre_kernel for a whole stretch of independent calls and copied into
//    shared memory (the batched entry point, more than one launch);
//  - a small projection in a launch of few layers: every CTA quantises X and computes all of T
//    from a copy of A_q that cp.async stages in shared memory while the kernel before drains;
//  - otherwise up to 16 CTAs of the layer take a range of K each, leave their partial T in a
//    scratch slot of the workspace and count themselves in; every CTA streams its first round of
//    weights, then waits (bounded) for the count, adds the slots in range order and quantises T.
//    All CTAs of a launch are resident together (at most one per SM), so the count is reached
//    while the weights stream; a second counter lets the last CTA to have read the slots zero
//    both for the next call.
//
// Launches of one batched call that follow one another share no buffer and need not wait for one
// another (ChainOrder): a launch fills the SMs as the one before leaves them.
#include <algorithm>

#include "lqer_common.cuh"

namespace lqer {
namespace dcol {

constexpr int kWarps = 16;
constexpr int kThreads = kWarps * 32;
constexpr int kMaxM = 4;
constexpr int kCg = 4;            // column groups (of 8 columns) per round: one column per lane
constexpr int kSets = 4;          // slabs a warp keeps in flight
constexpr int kHoldMax = 2;       // rounds whose sums share one barrier and one pass through shared memory, at most
constexpr int kLocalTMinCtas = 24; // ... if the layer has at least this many CTAs (launches of few layers)
constexpr int kLocalTUnits = 256; // up to this many (K block, 32 rank columns) units every CTA computes T for itself
constexpr int kTRanges = 16;      // CTAs of a layer that share the work of T = X_q A_q (ranges of K), at most

constexpr int kMaxGroup = 16;  // independent layers with one M that may share a launch

struct Layer {
  const void* X;                // [M, K] of Params::x_type
  void* Y;                      // [M, N] of Params::y_type (MXINT8: mantissas [M, N], then exponent bytes [M, N / 16])
  size_t y_extent;              // bytes behind Y, for the checked build
  const uint8_t* packed;
  size_t off_w, off_b, off_a;   // sections of the packed buffer
  int K, N, K64, k_pad, k_slabs, r_blocks, n_cg;
  int cta_begin, ctas;          // this layer's CTAs in the launch (dealt out by a time model)
  int a_stage_bytes;            // shared memory for a copy of A_q (every CTA computes all of T from it), or 0
  int t_ranges;                 // the first t_ranges of them compute T, a range of K each; 0: every CTA computes all of T itself
  int t_expect;                 // arrivals the CTAs wait for: t_ranges (one more under the stall test hook)
  const uint8_t* pre;           // X_q and T_q computed ahead (decode_pre_kernel), or null: this launch computes them
  double* tslot;                // [t_ranges][M][k_pad] partial sums of T (workspace scratch)
  int* tcount;                  // arrivals, departures: zero between calls
};

struct Params {
  int cta_begin[kMaxGroup];     // first CTA of each layer (a copy, side by side: a CTA finds its layer in one cache line)
  Layer L[kMaxGroup];
  int group;                    // layers in this launch
  int order;                    // ChainOrder: where the wait for the previous kernel sits
  DeviceStatus* status;
  int M;
  int a_bits, lr_bits, exp_min, exp_max;
  int x_type, y_type;           // X: kXF32, kXBF16 or kXMXINT8; Y: kYF32, kYBF16 or kYMXINT8
  int w_bits;                   // mantissa bits of W_q: 4 (nibbles) or 2 (crumbs), one value for all layers of a launch
  long long wait_limit;         // bound of the wait for the other CTAs' partial sums, in clock cycles
};

struct SlabRegs {
  uint4 h0, h1;   // one column of a slab: blocks 0, 1 and blocks 2, 3 (16 nibbles = two words each)
  uint32_t e;     // the four exponent bytes
};
constexpr float kIntMagic = 12582912.f;          // 1.5 * 2^23: int v (|v| < 2^22) + 0x4B400000 is the bit pattern of kIntMagic + v
constexpr int kIntMagicBits = 0x4B400000;

__device__ __forceinline__ uint32_t ld_stream_u32(const void* p) {
  uint32_t v;
  asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ uint4 ld_stream_u128(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t ld_stream_u8(const void* p) {
  uint32_t v;
  asm volatile("ld.global.nc.L1::no_allocate.u8 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
// T = X_q A_q: a warp takes 32 rank columns (a lane each) of some K blocks; these many warps split the K blocks of
// one such tile of columns.
__host__ __device__ inline int t_subsets(int k_pad) {
  const int tiles = k_pad > 32 ? (k_pad + 31) / 32 : 1;
  return tiles < kWarps ? kWarps / tiles : 1;
}

struct Formats { int a_bits, lr_bits, exp_min, exp_max, x_type, w_bits; };

// X -> MXINT8 for the whole contraction, by all threads of the CTA: per row the mantissas in the byte order the nibbles
// unpack to ({0,4,1,5}, {2,6,3,7} within each 8), the block scales 2^(e_x - 6) and the dp4a seeds (bits of
// 1.5 * 2^23, minus sum(x) of the block times the offset of the stored weights: 8 for nibbles, 1 for crumbs).
__device__ __forceinline__ void quantize_x_rows(const void* X, int M, int K, int K64, const Formats& f, uint8_t* xm,
                                                float* xsc, int* xof) {
  const int tid = threadIdx.x, KB = K64 / 16;
  const int per_row = K64 / 4, total = M * per_row;             // float4 items: (row, quarter-block)
  constexpr int U = 4;                                             // loads in flight per thread
  for (int base = 0; base < total; base += kThreads * U) {
    float4 v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int item = base + u * kThreads + tid;
      const int row = item / per_row, c4 = item % per_row;
      v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (item < total && c4 * 4 < K) v[u] = load_x_quad(X, f.x_type, M, K, row, c4 * 4, f.a_bits, f.exp_min, f.exp_max);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int item = base + u * kThreads + tid;
      if (base + u * kThreads + (tid & ~31) >= total) continue;      // a whole warp past the end (the shuffles need whole warps)
      const bool valid = item < total;
      const int row = valid ? item / per_row : 0, c4 = valid ? item % per_row : 0;
      int e;
      uint32_t m8;
      uint2 unused;
      quantize_quad(v[u], f.a_bits, f.exp_min, f.exp_max, e, m8, unused);
      const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, m8, 1);
      const uint32_t perm = (c4 & 1) ? __byte_perm(other, m8, 0x7362) : __byte_perm(m8, other, 0x5140);
      int sum = __dp4a((int)m8, 0x01010101, 0);
      sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 1);
      sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 2);
      if (valid) {
        *reinterpret_cast<uint32_t*>(xm + (size_t)row * K64 + c4 * 4) = perm;
        if ((c4 & 3) == 0) {
          xsc[row * KB + (c4 >> 2)] = pow2f(e - (f.a_bits - 2));
          xof[row * KB + (c4 >> 2)] = kIntMagicBits - (f.w_bits == 2 ? 1 : 8) * sum;
        }
      }
    }
  }
}

// Partial sums of T = X_q A_q over the K blocks [kb_lo, kb_hi), by all warps of the CTA: per (16-block of K, rank column)
// an exact integer dot product (dp4a) of the mantissas, scaled in fp64.  The fp64 sums are exact too unless the block
// exponents of one row spread over more than about 30 binades, and the order of the additions is fixed in any case.
// Leaves tsub[t_subsets(k_pad)][kMaxM][k_pad]; the caller adds the subsets in order after a barrier.
template <int MT, int UNROLL, bool STAGED>
__device__ __forceinline__ void t_partial(const uint8_t* asec, int K, int K64, int k_pad, int kb_lo, int kb_hi, int M,
                                          const Formats& f, const uint8_t* xm, const float* xsc, double* tsub) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KBr = K / 16, KB = K64 / 16;
  const int NT = (k_pad + 31) / 32;                            // tiles of 32 rank columns, a lane each
  const uint8_t* a_exp = asec + (size_t)KBr * k_pad * 16;
  const int bias = -127 - (f.lr_bits - 2);                        // exponent bytes carry +127
  const int tiles_w = NT < kWarps ? NT : kWarps;                  // warps side by side on different tiles
  const int subsets = t_subsets(k_pad);                        // warps that split the K blocks of one tile
  const int sb = warp / tiles_w;
  if (sb < subsets) {
    for (int nt = warp % tiles_w; nt < NT; nt += tiles_w) {
      const int j = nt * 32 + lane;
      const bool live = j < k_pad;
      const int jc = live ? j : 0;
      double tacc[MT];
#pragma unroll
      for (int r = 0; r < MT; ++r) tacc[r] = 0.0;
#pragma unroll UNROLL
      for (int kb = kb_lo + sb; kb < kb_hi; kb += subsets) {
        // `asec` is the A_q section in global memory, or (STAGED) a copy of it in shared memory
        const uint4 a = STAGED ? *reinterpret_cast<const uint4*>(asec + ((size_t)kb * k_pad + jc) * 16)
                               : __ldg(reinterpret_cast<const uint4*>(asec + ((size_t)kb * k_pad + jc) * 16));
        const double sa = pow2d((int)(STAGED ? a_exp[(size_t)kb * k_pad + jc] : __ldg(a_exp + (size_t)kb * k_pad + jc)) + bias);
#pragma unroll
        for (int r = 0; r < MT; ++r) {
          if (r < M) {
            // the X mantissas are stored as {0,4,1,5}, {2,6,3,7} within each 8: back to the order of A_q
            const uint4 x = *reinterpret_cast<const uint4*>(xm + (size_t)r * K64 + kb * 16);
            int sm = __dp4a((int)__byte_perm(x.x, x.y, 0x6420), (int)a.x, 0);
            sm = __dp4a((int)__byte_perm(x.x, x.y, 0x7531), (int)a.y, sm);
            sm = __dp4a((int)__byte_perm(x.z, x.w, 0x6420), (int)a.z, sm);
            sm = __dp4a((int)__byte_perm(x.z, x.w, 0x7531), (int)a.w, sm);
            tacc[r] = fma((double)sm, (double)xsc[r * KB + kb] * sa, tacc[r]);
          }
        }
      }
      if (live) {
#pragma unroll
        for (int r = 0; r < MT; ++r)
          if (r < M) tsub[((size_t)sb * kMaxM + r) * k_pad + j] = tacc[r];
      }
    }
  }
}

// One value of T -> MXINT8 along the rank (16 adjacent lanes hold one block; every lane of the warp calls this).
__device__ __forceinline__ void store_tq(double tv, bool valid, int row, int col, int k_pad, const Formats& f,
                                         int8_t* tq8, float* tqs) {
  double amax = (tv != tv) ? 0.0 : fabs(tv);
#pragma unroll
  for (int sft = 1; sft < 16; sft <<= 1) amax = fmax(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, sft));
  const int e = block_exponent(amax, f.exp_min, f.exp_max);
  const int qv = quant_mantissa(tv, e, f.a_bits);
  if (valid) {
    tq8[row * k_pad + col] = (int8_t)qv;
    if ((col & 15) == 0) tqs[row * (k_pad / 16) + (col >> 4)] = pow2f(e - (f.a_bits - 2));
  }
}

// What the decode kernel needs of a layer's activations, computed ahead for many layers at once (independent calls
// of one batch): the quantised X and T_q, in the layout the decode kernel keeps them in shared memory:
//   [M][K64] mantissas, [M][K64/16] scales, [M][K64/16] dp4a seeds, [kMaxM][16] scales of T_q, [kMaxM][k_pad] T_q.
constexpr int kPreMaxCalls = 64;
struct PreCall {
  const void* X;
  const uint8_t* asec;          // A_q section of the packed buffer
  uint8_t* out;
  int M, K, K64, k_pad;
  Formats f;
};
struct PreParams {
  PreCall c[kPreMaxCalls];
  int order;                    // ChainOrder, as for the decode kernel
};
__host__ __device__ inline size_t pre_x_bytes(int M, int K64) { return (size_t)M * K64 + (size_t)M * (K64 / 16) * 8; }
__host__ __device__ inline size_t pre_t_bytes(int k_pad) { return (size_t)kMaxM * 16 * 4 + (size_t)kMaxM * (k_pad > 0 ? k_pad : 16); }

template <int MT>
__global__ void __launch_bounds__(kThreads, 1) decode_pre_kernel(const __grid_constant__ PreParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
  const PreCall& c = p.c[blockIdx.x];
  const int M = c.M, KB = c.K64 / 16, tid = threadIdx.x;
  uint8_t* xm = smem;
  float* xsc = reinterpret_cast<float*>(xm + (size_t)M * c.K64);
  int* xof = reinterpret_cast<int*>(xsc + (size_t)M * KB);
  float* tqs = reinterpret_cast<float*>(xof + (size_t)M * KB);
  int8_t* tq8 = reinterpret_cast<int8_t*>(tqs + kMaxM * 16);
  const size_t out_bytes = pre_x_bytes(M, c.K64) + pre_t_bytes(c.k_pad);
  double* tsub = reinterpret_cast<double*>(smem + ((out_bytes + 15) & ~(size_t)15));

  if (p.order != kChainFirst) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (p.order != kChainLater) asm volatile("griddepcontrol.wait;" ::: "memory");   // X may be an earlier kernel's output
  if (p.order == kChainFirst) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  quantize_x_rows(c.X, M, c.K, c.K64, c.f, xm, xsc, xof);
  for (int i = tid; i < (int)pre_t_bytes(c.k_pad) / 4; i += kThreads) reinterpret_cast<uint32_t*>(tqs)[i] = 0u;
  __syncthreads();
  if (c.k_pad > 0) {
    t_partial<MT, 8, false>(c.asec, c.K, c.K64, c.k_pad, 0, c.K / 16, M, c.f, xm, xsc, tsub);   // the whole of K: many loads in flight
    __syncthreads();
    const int subsets = t_subsets(c.k_pad), total = M * c.k_pad;
    for (int base = 0; base < total; base += kThreads) {
      const int idx = base + tid;
      const bool valid = idx < total;
      const int row = valid ? idx / c.k_pad : 0, col = valid ? idx % c.k_pad : 0;
      double tv = 0.0;
      if (valid)
        for (int q = 0; q < subsets; ++q) tv += tsub[((size_t)q * kMaxM + row) * c.k_pad + col];
      store_tq(tv, valid, row, col, c.k_pad, c.f, tq8, tqs);
    }
    __syncthreads();
  }
  for (size_t o = (size_t)tid * 16; o < out_bytes; o += (size_t)kThreads * 16)
    *reinterpret_cast<uint4*>(c.out + o) = *reinterpret_cast<const uint4*>(smem + o);
  if (p.order == kChainLater) asm volatile("griddepcontrol.wait;" ::: "memory");
}

// MT: rows the accumulators are compiled for (1 for the single-token call, kMaxM otherwise); M <= MT.
// WB: mantissa bits of W_q the kernel is compiled for: 4 (nibbles) or 2 (crumbs).  YQ: Y is MXINT8.
template <int MT, int WB, bool YQ>
__global__ void __launch_bounds__(kThreads, 1) decode_cols_kernel(const __grid_constant__ Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
  int layer = 0;
#pragma unroll
  for (int i = 1; i < kMaxGroup; ++i)
    if (i < p.group && (int)blockIdx.x >= p.cta_begin[i]) layer = i;
  const Layer& ly = p.L[layer];
  const int M = p.M, KB = ly.K64 / 16;
  uint8_t* xm = smem;                                               // [M][K64] int8 mantissas, permuted within 8
  float* xsc = reinterpret_cast<float*>(xm + (size_t)M * ly.K64);    // [M][KB] 2^(e_x - 6)
  int* xof = reinterpret_cast<int*>(xsc + (size_t)M * KB);          // [M][KB] bits of 1.5 * 2^23, minus 8 * sum(x) of the block
  float* red = reinterpret_cast<float*>(xof + (size_t)M * KB);      // two of [kHoldMax rounds][kWarps][32 columns][kMaxM], used in turn
  double* tsub = reinterpret_cast<double*>(red + 2 * kHoldMax * kWarps * kCg * 8 * kMaxM);   // [subsets][M][k_pad] per-warp-subset partials of T
  int* wait_ok = reinterpret_cast<int*>(tsub);                       // reused once T's partial sums have left: outcome of the wait
  float* tqs = reinterpret_cast<float*>(tsub + (size_t)kMaxM * ly.k_pad * t_subsets(ly.k_pad));   // [M][k_pad / 16]
  int8_t* tq8 = reinterpret_cast<int8_t*>(tqs + kMaxM * 16);        // [M][k_pad]
  uint8_t* a_stage = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(tq8) + (size_t)kMaxM * (ly.k_pad > 0 ? ly.k_pad : 16) + 15) & ~(uintptr_t)15);   // a copy of A_q

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = ly.ctas, cta = (int)blockIdx.x - ly.cta_begin;
  const void* const X = ly.X;
  void* const Y = ly.Y;
  const uint8_t* const wsec = ly.packed + ly.off_w;
  const uint8_t* const bsec = ly.packed + ly.off_b;
  const uint8_t* const asec = ly.packed + ly.off_a;
  // a CTA's columns: a range of groups of 8; for an MXINT8 Y a range of pairs of groups, so that it owns whole 16-blocks
  constexpr int cgu = YQ ? 2 : 1;
  const int cg_lo = cgu * (cta * (ly.n_cg / cgu) / G), cg_hi = cgu * ((cta + 1) * (ly.n_cg / cgu) / G);

  // This lane's column of a round (the 32 columns from column group cg0 on) and slab j: global -> registers.  Byte
  // offsets into the W section are kept per round (32 bits: the section is far below 4 GB).  Column groups past the
  // CTA's range are clamped to its last one and slabs past K to the last slab: such loads stay inside the section
  // and what they return is never used (the sums of those slabs are skipped, those columns are not stored).
  const uint32_t lane_w = (uint32_t)((lane & 7) * 16);
  constexpr uint32_t w_tile = (uint32_t)(kTileN * kSlabK * WB / 8 + kTileN * 4);   // 4608 bytes with nibbles, 2560 with crumbs
  constexpr bool crumbs = WB == 2;                                  // then a column of a slab is one 16-byte word group
  const uint32_t lane_e = (uint32_t)(kTileN * kSlabK * WB / 8 + (lane & 7) * 4);
  struct ColOff { uint32_t w, e; };
  auto col_off = [&](int cg0) -> ColOff {
    const int cg = max(min(cg0 + (lane >> 3), cg_hi - 1), 0);
    const uint32_t tile = (uint32_t)(cg >> 4) * (uint32_t)ly.k_slabs * w_tile;
    ColOff o;
    o.w = tile + (uint32_t)(cg & 15) * 128u + lane_w;
    o.e = tile + (uint32_t)(cg & 15) * 32u + lane_e;
    return o;
  };
  auto fetch = [&](SlabRegs& d, const ColOff& o, int j) {
    const uint32_t jo = (uint32_t)min(j, ly.k_slabs - 1) * w_tile;
    d.h0 = ld_stream_u128(wsec + (o.w + jo));
    if (!crumbs) d.h1 = ld_stream_u128(wsec + (o.w + jo + (uint32_t)(kTileN * 16)));
    d.e = ld_stream_u32(wsec + (o.e + jo));
  };

  // Alone: the next kernel may set up at once, and this one waits for the previous one before it reads X.  In a chain
  // of launches that share no buffer (independent layers, scratch and counters of their own): the first lets its
  // successor start only after its own wait, the later ones do not wait before they work but before they exit, so that
  // a launch fills the SMs as the one before leaves them and the kernel after the chain finds all of it complete.
  if (p.order != kChainFirst) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // this lane's column of rank block `warp` of B_q: its 16 rank values and the exponent byte
  auto fetch_rank = [&](uint4& wv, uint32_t& eb, int cg0) {
    wv = make_uint4(0u, 0u, 0u, 0u);
    eb = 127u;
    const int cg = cg0 + (lane >> 3);
    if (cg < cg_hi && warp < ly.r_blocks) {
      const int col = (cg & 15) * 8 + (lane & 7);
      const uint8_t* tile = bsec + (size_t)(cg >> 4) * ((size_t)ly.r_blocks * kTileN * 17);
      wv = ld_stream_u128(tile + ((size_t)warp * kTileN + col) * 16);
      eb = ld_stream_u8(tile + (size_t)ly.r_blocks * kTileN * 16 + warp * kTileN + col);
    }
  };

  SlabRegs regs[kSets];
  uint4 rank_w;
  uint32_t rank_e;
  // weights depend on no earlier kernel: request the first slabs, the rank blocks and this CTA's
  // share of A_q before the dependency wait
  ColOff o_cur = col_off(cg_lo), o_nxt;          // offsets of this round's and the next round's columns
#pragma unroll
  for (int s = 0; s < kSets; ++s) fetch(regs[s], o_cur, warp + kWarps * s);
  fetch_rank(rank_w, rank_e, cg_lo);
  const int KBr = ly.K / 16;
  const bool pre = ly.pre != nullptr;
  const bool t_local = !pre && ly.k_pad > 0 && ly.t_ranges == 0;     // a small projection: cheaper to repeat than to exchange
  const bool t_worker = !pre && ly.k_pad > 0 && (t_local || cta < ly.t_ranges);
  const int kb_lo = t_worker && !t_local ? cta * KBr / ly.t_ranges : 0;          // this CTA's share of K for T
  const int kb_hi = t_local ? KBr : t_worker ? (cta + 1) * KBr / ly.t_ranges : 0;
  const bool a_staged = t_local && ly.a_stage_bytes >= KBr * ly.k_pad * 17;
  if (a_staged) {                                  // all of A_q into shared memory: on its way while the kernel before drains
    const int bytes = KBr * ly.k_pad * 17;         // mantissas, then exponents: one contiguous range
    for (int o = tid * 16; o < bytes; o += kThreads * 16)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(a_stage + o)), "l"(asec + o) : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
  } else if (t_worker) {                           // this CTA's share of A_q: towards L2 while X is quantised
    const uint8_t* gm = asec + (size_t)kb_lo * ly.k_pad * 16;
    const uint8_t* ge = asec + (size_t)KBr * ly.k_pad * 16 + (size_t)kb_lo * ly.k_pad;
    const int mant = (kb_hi - kb_lo) * ly.k_pad * 16, ex = (kb_hi - kb_lo) * ly.k_pad;
    for (int o = tid * 128; o < mant; o += kThreads * 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(gm + o));
    for (int o = tid * 128; o < ex; o += kThreads * 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(ge + o));
  }

  if (p.order != kChainLater) asm volatile("griddepcontrol.wait;" ::: "memory");   // X (and the workspace) may be an earlier kernel's output
  if (p.order == kChainFirst) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // ---- X -> MXINT8 for the whole contraction: per row the mantissas in the byte order the nibbles
  //      unpack to ({0,4,1,5}, {2,6,3,7} within each 8), the block scales and the offsets 8 * sum(x)
  const Formats fmt = {p.a_bits, p.lr_bits, p.exp_min, p.exp_max, p.x_type, WB};
  if (pre) {                                       // quantised X and T_q are there already: straight into shared memory
    const int xb = (int)pre_x_bytes(M, ly.K64), tb = (int)pre_t_bytes(ly.k_pad);
    for (int o = tid * 16; o < xb; o += kThreads * 16)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(xm + o)), "l"(ly.pre + o) : "memory");
    for (int o = tid * 16; o < tb; o += kThreads * 16)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(reinterpret_cast<uint8_t*>(tqs) + o)), "l"(ly.pre + xb + o) : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
  } else {
    quantize_x_rows(X, M, ly.K, ly.K64, fmt, xm, xsc, xof);
  }
  __syncthreads();

  // ---- this CTA's share of T = X_q A_q
  if (t_worker) {
    const int subsets = t_subsets(ly.k_pad);
    if (a_staged) {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      __syncthreads();
      t_partial<MT, 4, true>(a_stage, ly.K, ly.K64, ly.k_pad, kb_lo, kb_hi, M, fmt, xm, xsc, tsub);
    } else {
      t_partial<MT, 4, false>(asec, ly.K, ly.K64, ly.k_pad, kb_lo, kb_hi, M, fmt, xm, xsc, tsub);
    }
    __syncthreads();
    if (t_local) {                                 // all of T is here: quantise it
      const int total = M * ly.k_pad;
      for (int base = 0; base < total; base += kThreads) {
        const int idx = base + tid;
        const bool valid = idx < total;
        const int row = valid ? idx / ly.k_pad : 0, col = valid ? idx % ly.k_pad : 0;
        double tv = 0.0;
        if (valid)
          for (int q = 0; q < subsets; ++q) tv += tsub[((size_t)q * kMaxM + row) * ly.k_pad + col];
        store_tq(tv, valid, row, col, ly.k_pad, fmt, tq8, tqs);
      }
    } else {
      for (int idx = tid; idx < M * ly.k_pad; idx += kThreads) {
        const int row = idx / ly.k_pad, col = idx % ly.k_pad;
        double v = 0.0;
        for (int q = 0; q < subsets; ++q) v += tsub[((size_t)q * kMaxM + row) * ly.k_pad + col];
        ly.tslot[((size_t)cta * M + row) * ly.k_pad + col] = v;
      }
    }
    __syncthreads();
    if (!t_local && tid == 0) {                    // this range of T is published; waited for before the first rank part
      __threadfence();                             // the slot (ordered before by the barrier) before the count
      atomicAdd(ly.tcount, 1);
    }
  }

  // T = sum of the ranges' partial sums (range order), then MXINT8 along the rank: 16 adjacent lanes hold one block.
  // The ranges belong to CTAs of this launch, all resident; the wait is bounded all the same.
  auto build_tq = [&]() {
    if (tid == 0) {
      int seen = 1;
      const long long t0 = clock64();
      for (;;) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ly.tcount) : "memory");
        if (v >= ly.t_expect) break;
        if (clock64() - t0 > p.wait_limit) { seen = 0; break; }
        __nanosleep(100);
      }
      if (!seen) report_error(p.status, LQER_ERR_TIMEOUT, 500, blockIdx.x);
      *wait_ok = seen;
    }
    __syncthreads();
    const bool ok = *wait_ok != 0;
    const int total = M * ly.k_pad;
    for (int base = 0; base < total; base += kThreads) {
      const int idx = base + tid;
      const bool valid = idx < total;
      const int row = valid ? idx / ly.k_pad : 0, col = valid ? idx % ly.k_pad : 0;
      double tv = 0.0;
      if (valid && ok) {
        const double* sp = ly.tslot + (size_t)row * ly.k_pad + col;
#pragma unroll 4
        for (int c = 0; c < ly.t_ranges; ++c) tv += __ldcg(sp + (size_t)c * M * ly.k_pad);
      }
      store_tq(tv, valid, row, col, ly.k_pad, fmt, tq8, tqs);
    }
    __syncthreads();
    if (tid == 0 && atomicAdd(ly.tcount + 1, 1) == G - 1) {   // every CTA of the layer has read the slots: zero for the next call
      ly.tcount[0] = 0;
      ly.tcount[1] = 0;
    }
  };
  bool tq_built = pre || t_local;
  constexpr int kHold = MT == 1 ? kHoldMax : 1;  // rounds per barrier (their sums wait in registers; four were no faster)
  constexpr int kHeld = kHold > 1 ? kHold - 1 : 1;
  int meet_no = 0, n_held = 0;
  int held_cg0[kHeld];
  float held[kHeld][MT];
#pragma unroll
  for (int h = 0; h < kHold - 1; ++h) {
    held_cg0[h] = 0;
#pragma unroll
    for (int r = 0; r < MT; ++r) held[h][r] = 0.f;
  }
  const int slabs_mine = ly.k_slabs > warp ? (ly.k_slabs - warp + kWarps - 1) / kWarps : 0;   // slabs warp, warp + 16, ...
#pragma unroll 1
  for (int cg0 = cg_lo; cg0 < cg_hi; cg0 += kCg) {
    float acc[MT];
#pragma unroll
    for (int r = 0; r < MT; ++r) acc[r] = 0.f;
    o_nxt = col_off(cg0 + kCg);

    // ---- W_q: this warp's slabs of the round's columns
#pragma unroll 1
    for (int js = 0; js < slabs_mine; js += kSets) {
#pragma unroll
      for (int s = 0; s < kSets; ++s) {
        const int j = warp + kWarps * (js + s);
        if (j < ly.k_slabs) {
          const SlabRegs d = regs[s];
          // weights as bytes in the order k {0,4,1,5}, {2,6,3,7}, {8,12,9,13}, {10,14,11,15} of each block
          uint32_t nib[16];
          if (crumbs) {
            // a word per block: (w >> 2i) & 0x03030303 holds k {2i, 2i + 8, 2i + 1, 2i + 9}; two byte permutes per pair
            const uint32_t wd[4] = {d.h0.x, d.h0.y, d.h0.z, d.h0.w};
#pragma unroll
            for (int b = 0; b < 4; ++b) {
              const uint32_t c0 = wd[b] & 0x03030303u, c1 = (wd[b] >> 2) & 0x03030303u;
              const uint32_t c2 = (wd[b] >> 4) & 0x03030303u, c3 = (wd[b] >> 6) & 0x03030303u;
              nib[4 * b] = __byte_perm(c0, c2, 0x6240);
              nib[4 * b + 1] = __byte_perm(c1, c3, 0x6240);
              nib[4 * b + 2] = __byte_perm(c0, c2, 0x7351);
              nib[4 * b + 3] = __byte_perm(c1, c3, 0x7351);
            }
          } else {
            const uint32_t wd[8] = {d.h0.x, d.h0.y, d.h0.z, d.h0.w, d.h1.x, d.h1.y, d.h1.z, d.h1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              nib[2 * i] = wd[i] & 0x0F0F0F0Fu;
              nib[2 * i + 1] = (wd[i] >> 4) & 0x0F0F0F0Fu;
            }
          }
          // 2^(e_w - (w_bits - 2)) of the four blocks: the four exponent bytes lose the mantissa's binary point at once,
          // then a byte permute brings a byte to the top of a word and a shift by one puts it into the exponent field
          float sw[4];
          const uint32_t e4w = d.e - (uint32_t)(WB - 2) * 0x01010101u;
          sw[0] = __uint_as_float(__byte_perm(e4w, 0u, 0x0444) >> 1);
          sw[1] = __uint_as_float(__byte_perm(e4w, 0u, 0x1444) >> 1);
          sw[2] = __uint_as_float(__byte_perm(e4w, 0u, 0x2444) >> 1);
          sw[3] = __uint_as_float((e4w >> 1) & 0x7F800000u);
#pragma unroll
          for (int r = 0; r < MT; ++r) {
            if (r < M) {
              const uint4* xp = reinterpret_cast<const uint4*>(xm + (size_t)r * ly.K64 + j * 64);
              const float4 sx = *reinterpret_cast<const float4*>(xsc + r * KB + j * 4);      // 2^(e_x - 6)
              const int4 seed = *reinterpret_cast<const int4*>(xof + r * KB + j * 4);
              const float sxa[4] = {sx.x, sx.y, sx.z, sx.w};
              const int seeda[4] = {seed.x, seed.y, seed.z, seed.w};
#pragma unroll
              for (int b = 0; b < 4; ++b) {
                const uint4 x = xp[b];
                int sm = __dp4a((int)x.x, (int)nib[4 * b], seeda[b]);
                sm = __dp4a((int)x.y, (int)nib[4 * b + 1], sm);
                sm = __dp4a((int)x.z, (int)nib[4 * b + 2], sm);
                sm = __dp4a((int)x.w, (int)nib[4 * b + 3], sm);
                acc[r] = fmaf(__int_as_float(sm) - kIntMagic, sxa[b] * sw[b], acc[r]);
              }
            }
          }
        }
        // refill the set: the same columns four slabs on, or - past this warp's last slabs - the
        // next round's columns from their first slabs, so that rounds follow each other without a bubble
        const bool more = js + kSets < slabs_mine;
        const int jn = more ? j + kWarps * kSets : warp + kWarps * s;
        ColOff o;
        o.w = more ? o_cur.w : o_nxt.w;
        o.e = more ? o_cur.e : o_nxt.e;
        fetch(regs[s], o, jn);
      }
    }
    o_cur = o_nxt;

    // ---- B_q against T_q: rank blocks warp, warp + 16, ...
    if (ly.k_pad > 0) {
      if (!tq_built) {
        build_tq();
        tq_built = true;
      }
      const int rbn = ly.k_pad / 16;
      if (warp < ly.r_blocks) {                   // rank block `warp` (k <= 256: at most 16 blocks); data already in registers
        const float sb = __uint_as_float((rank_e - (uint32_t)(p.lr_bits - 2)) << 23);           // 2^(e_b - 6)
#pragma unroll
        for (int r = 0; r < MT; ++r) {
          if (r < M) {
            const uint4 tw = *reinterpret_cast<const uint4*>(tq8 + r * ly.k_pad + warp * 16);
            int sm = __dp4a((int)tw.x, (int)rank_w.x, 0);
            sm = __dp4a((int)tw.y, (int)rank_w.y, sm);
            sm = __dp4a((int)tw.z, (int)rank_w.z, sm);
            sm = __dp4a((int)tw.w, (int)rank_w.w, sm);
            acc[r] = fmaf((float)sm, tqs[r * rbn + warp] * sb, acc[r]);
          }
        }
      }
      fetch_rank(rank_w, rank_e, cg0 + kCg);     // the next round's rank blocks
    }

    // ---- the 16 warps' sums of a column (fixed order), then Y.  Rounds meet kHold at a time: the earlier ones keep
    //      their sums in registers and the last brings all to shared memory, so kHold rounds cost one barrier.  Two
    //      buffers in turn: the warps that add the sums (the first four) do so while the others stream the next round;
    //      the barrier of the next meeting keeps a buffer from being rewritten before it has been read.
    if (n_held < kHold - 1 && cg0 + kCg < cg_hi) {
#pragma unroll
      for (int h = 0; h < kHold - 1; ++h)
        if (h == n_held) {
#pragma unroll
          for (int r = 0; r < MT; ++r) held[h][r] = acc[r];
          held_cg0[h] = cg0;
        }
      ++n_held;
      continue;
    }
    float* red_now = red + (meet_no & 1) * (kHoldMax * kWarps * 32 * kMaxM);
    ++meet_no;
#pragma unroll
    for (int h = 0; h < kHold - 1; ++h)
      if (h < n_held) {
#pragma unroll
        for (int r = 0; r < MT; ++r) red_now[((h * kWarps + warp) * 32 + lane) * kMaxM + r] = held[h][r];
      }
#pragma unroll
    for (int r = 0; r < MT; ++r) red_now[((n_held * kWarps + warp) * 32 + lane) * kMaxM + r] = acc[r];
    __syncthreads();
    if constexpr (YQ) {
      // a warp per token, a lane per column of the round: the two 16-blocks of the round are the two halves of the
      // warp, their maxima a butterfly over 16 lanes; the CTA's range holds whole blocks (see cg_lo)
      if (tid < 32 * kMaxM) {
        const int r = warp, col = lane;
        if (r < M) {
#pragma unroll
          for (int h = 0; h < kHold; ++h) {
            if (h <= n_held) {
              int c0 = cg0;
#pragma unroll
              for (int q = 0; q < kHold - 1; ++q)
                if (q == h && h < n_held) c0 = held_cg0[q];
              const bool live = c0 + (col >> 3) < cg_hi;
              float v = 0.f;
              if (live) {
#pragma unroll
                for (int w = 0; w < kWarps; ++w) v += red_now[((h * kWarps + w) * 32 + col) * kMaxM + r];
              }
              float amax = abs_ignore_nan(v);
#pragma unroll
              for (int sft = 1; sft < 16; sft <<= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, sft));
              const int e = block_exponent(amax, p.exp_min, p.exp_max);
              const int q8 = quant_mantissa(v, e, p.a_bits);
              const size_t idx = (size_t)r * ly.N + c0 * 8 + col;
              uint8_t* yq = static_cast<uint8_t*>(Y);
              if (live && LQER_IN_BOUNDS(p.status, (size_t)M * ly.N + idx / 16, 1, ly.y_extent, 712)) {
                yq[idx] = (uint8_t)(int8_t)q8;
                if ((col & 15) == 0) yq[(size_t)M * ly.N + idx / 16] = (uint8_t)(e + 127);
              }
            }
          }
        }
      }
    } else if (tid < 32 * kMaxM) {
      const int col = tid >> 2, r = tid & 3;
#pragma unroll
      for (int h = 0; h < kHold; ++h) {
        if (h <= n_held) {
          int c0 = cg0;
#pragma unroll
          for (int q = 0; q < kHold - 1; ++q)
            if (q == h && h < n_held) c0 = held_cg0[q];
          if (c0 + (col >> 3) < cg_hi && r < M) {
            float v = 0.f;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) v += red_now[((h * kWarps + w) * 32 + col) * kMaxM + r];
            const bool y16 = p.y_type == kYBF16;
            if (!LQER_IN_BOUNDS(p.status, ((size_t)r * ly.N + c0 * 8 + col) * (y16 ? 2 : 4), y16 ? 2 : 4, ly.y_extent, 711)) {
            } else if (y16) {
              uint32_t u = __float_as_uint(v);               // round to nearest even (NaN / inf keep their class)
              u = ((u & 0x7F800000u) == 0x7F800000u) ? ((u >> 16) | ((u & 0xFFFFu) ? 0x40u : 0u)) : ((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
              static_cast<uint16_t*>(Y)[(size_t)r * ly.N + c0 * 8 + col] = (uint16_t)u;
            } else {
              static_cast<float*>(Y)[(size_t)r * ly.N + c0 * 8 + col] = v;
            }
          }
        }
      }
    }
    n_held = 0;
  }
  if (ly.k_pad > 0 && !tq_built) build_tq();     // a CTA without columns still takes part in the counts
  if (p.order == kChainLater) asm volatile("griddepcontrol.wait;" ::: "memory");
}

}  // namespace dcol

static size_t cols_smem_bytes(const PackedMeta& m, int M) {
  using namespace dcol;
  return (size_t)M * m.K64 + (size_t)M * (m.K64 / 16) * 8 + 2 * kHoldMax * kWarps * kCg * 8 * kMaxM * 4 +
         (size_t)kMaxM * m.k_pad * 8 * t_subsets(m.k_pad) + kMaxM * 16 * 4 + (size_t)kMaxM * (m.k_pad > 0 ? m.k_pad : 16) + 256;
}
// The column-owner kernel serves M <= 4 (its dot products run on the raw nibbles or crumbs) as long as the quantised X of
// the whole contraction fits in shared memory.
bool decode_cols_fits(const PackedMeta& m, int M) { return M <= dcol::kMaxM && cols_smem_bytes(m, M) <= 200 * 1024; }

cudaError_t launch_decode_cols(const void* X, int x_type, int M, const PackedMeta& m, const void* packed, void* Y, int y_type,
                               void* workspace, cudaStream_t s) {
  const lqer_call_t one = {static_cast<const float*>(X), M, packed, static_cast<float*>(Y)};
  return launch_decode_cols_group(&one, &m, 1, workspace, 0, kChainAlone, 0, nullptr, nullptr, x_type, y_type, s);
}

int decode_cols_max_group() { return dcol::kMaxGroup; }

// n independent layers with one M (shapes may differ) in a single launch: the SMs are divided among them in proportion
// to their weight bytes, so the layers' fixed latencies (dependency wait, X quantisation, the T exchange, the final
// reduction) overlap instead of following one another.  Every layer must fit decode_cols_fits and, for n > 1, have
// at least one cluster's worth of column groups.
cudaError_t launch_decode_cols_group(const lqer_call_t* calls, const PackedMeta* metas, int n, void* workspace,
                                     size_t workspace_bytes, int order, int set, bool* fills_gpu, const uint8_t* const* pres,
                                     int x_type, int y_type, cudaStream_t s) {
  using namespace dcol;
  static OncePerDevice once;
  static bool one_cta_per_sm = true;               // false if any device could hold two CTAs of the kernel on one SM
  cudaError_t e0 = once.run([] {
    // chaining launches relies on one CTA per SM (registers): a launch on every SM then leaves room for no other
    const void* kernels[8] = {reinterpret_cast<const void*>(decode_cols_kernel<1, 4, false>), reinterpret_cast<const void*>(decode_cols_kernel<kMaxM, 4, false>),
                              reinterpret_cast<const void*>(decode_cols_kernel<1, 2, false>), reinterpret_cast<const void*>(decode_cols_kernel<kMaxM, 2, false>),
                              reinterpret_cast<const void*>(decode_cols_kernel<1, 4, true>), reinterpret_cast<const void*>(decode_cols_kernel<kMaxM, 4, true>),
                              reinterpret_cast<const void*>(decode_cols_kernel<1, 2, true>), reinterpret_cast<const void*>(decode_cols_kernel<kMaxM, 2, true>)};
    for (const void* k : kernels) {
      cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
      if (e != cudaSuccess) return e;
      int o = 2;
      if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, k, kThreads, 0) != cudaSuccess) o = 2;
      if (o != 1) one_cta_per_sm = false;
    }
    return cudaSuccess;
  });
  if (e0 != cudaSuccess) return e0;
  const int sm_count = lqer::sm_count() > 0 ? lqer::sm_count() : 1;
  if (n < 1 || n > kMaxGroup) return cudaErrorInvalidValue;
  const int M = calls[0].M;
  Params p;
  p.group = n;
  p.order = order;
  p.status = reinterpret_cast<DeviceStatus*>(workspace);
  p.M = M;
  p.a_bits = metas[0].a_bits; p.lr_bits = metas[0].lr_bits; p.exp_min = metas[0].exp_min; p.exp_max = metas[0].exp_max;
  p.x_type = x_type;
  p.w_bits = metas[0].w_bits;
  p.y_type = y_type;
  p.wait_limit = wait_limit_cycles();
  const int stall = take_stall(kFamDecode) ? 1 : 0;

  // CTAs per layer (one per SM at most, so that all of a launch are resident together): a single layer takes what
  // it can use; several share the SMs by the time their columns take
  const int max_ctas = sm_count < kDecodeMaxCtas ? sm_count : kDecodeMaxCtas;
  int ctas[kMaxGroup];
  if (n == 1) {
    ctas[0] = metas[0].N / 8 < max_ctas ? metas[0].N / 8 : max_ctas;
  } else {
    // a CTA's time is its rounds (32 columns each) times the slabs a warp streams per round plus a fixed cost per
    // round of about 1.3 slabs (measured); every layer gets one CTA, the rest go one by one where that time is largest
    if (n > max_ctas) return cudaErrorInvalidConfiguration;   // more layers than SMs
    double per_round[kMaxGroup];
    for (int g = 0; g < n; ++g) {
      ctas[g] = 1;
      per_round[g] = 1.3 + (double)((metas[g].k_slabs + kWarps - 1) / kWarps);
    }
    for (int left = max_ctas - n; left > 0; --left) {
      int best = -1;
      double worst = 0.0;
      for (int g = 0; g < n; ++g) {
        const double t = (double)(metas[g].N / 8) / (kCg * ctas[g]) * per_round[g];
        if (ctas[g] < metas[g].N / 8 && t > worst) { worst = t; best = g; }
      }
      if (best < 0) break;
      ++ctas[best];
    }
  }
  size_t head = 0;
  for (int g = 0; g < n; ++g) {
    const size_t h = (persist_bytes(metas[g]) + 255) & ~(size_t)255;
    if (h > head) head = h;
  }
  uint8_t* wsb = static_cast<uint8_t*>(workspace);
  size_t slot_off = head;
  if (set != 0) {                                       // the second set of slots lies at the end of the workspace
    size_t slots = 0;
    for (int g = 0; g < n; ++g) slots += decode_cols_slot_bytes(metas[g]);
    if (workspace_bytes < head + 2 * slots) return cudaErrorInvalidValue;
    slot_off = (workspace_bytes - slots) & ~(size_t)255;
  }

  size_t smem = 0;
  int begin = 0;
  for (int i = 0; i < kMaxGroup; ++i) {
    const int g = i < n ? i : 0;
    const PackedMeta& m = metas[g];
    if (!decode_cols_fits(m, M) || !(m.a_bits == p.a_bits && m.lr_bits == p.lr_bits && m.exp_min == p.exp_min && m.exp_max == p.exp_max))
      return cudaErrorInvalidValue;
    Layer& ly = p.L[i];
    ly.X = calls[g].X; ly.Y = calls[g].Y; ly.packed = static_cast<const uint8_t*>(calls[g].packed);
    ly.y_extent = y_bytes(y_type, (size_t)calls[g].M, (size_t)metas[g].N);
    if (kDebugBounds) ly.y_extent -= std::min(ly.y_extent, debug_y_shrink());
    ly.off_w = m.off_w; ly.off_b = m.off_b; ly.off_a = m.off_a;
    ly.K = m.K; ly.N = m.N; ly.K64 = m.K64; ly.k_pad = m.k_pad;
    ly.k_slabs = m.k_slabs; ly.r_blocks = m.r_blocks;
    ly.n_cg = m.N / 8;
    int ranges = ctas[g] < kTRanges ? ctas[g] : kTRanges;
    if (ranges > m.K / 16) ranges = m.K / 16;
    // a projection of few (K block, 32 rank columns) units costs a CTA less than the exchange of partial sums would,
    // when the layer has so many CTAs that each streams little else
    if ((long long)(m.K / 16) * ((m.k_pad + 31) / 32) <= kLocalTUnits && ctas[g] >= kLocalTMinCtas) ranges = 0;
    ly.t_ranges = ranges;
    ly.t_expect = ranges + stall;
    ly.pre = pres != nullptr ? pres[g] : nullptr;
    const size_t a_need = (size_t)(m.K / 16) * m.k_pad * 17 + 16;
    ly.a_stage_bytes = (ranges == 0 && ly.pre == nullptr && m.k_pad > 0 && cols_smem_bytes(m, M) + a_need <= 200 * 1024) ? (int)a_need : 0;
    ly.tslot = reinterpret_cast<double*>(wsb + slot_off);
    ly.tcount = reinterpret_cast<int*>(wsb + kStatusBytes) + 2 * (g + (set != 0 ? kMaxGroup : 0));
    if (i < n) slot_off += decode_cols_slot_bytes(m);
    ly.cta_begin = begin;
    p.cta_begin[i] = begin;
    ly.ctas = ctas[g];
    if (i < n) {
      begin += ctas[g];
      const size_t need = cols_smem_bytes(m, M) + ly.a_stage_bytes;
      if (need > smem) smem = need;
    }
  }

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(begin);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may start while the previous kernel drains
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (fills_gpu != nullptr) *fills_gpu = one_cta_per_sm && begin == sm_count;
  LaunchScope scope(kFamDecode, s);
  const bool yq = y_type == kYMXINT8;
  if (p.w_bits == 2) {
    if (yq) return M == 1 ? cudaLaunchKernelEx(&cfg, decode_cols_kernel<1, 2, true>, p) : cudaLaunchKernelEx(&cfg, decode_cols_kernel<kMaxM, 2, true>, p);
    return M == 1 ? cudaLaunchKernelEx(&cfg, decode_cols_kernel<1, 2, false>, p) : cudaLaunchKernelEx(&cfg, decode_cols_kernel<kMaxM, 2, false>, p);
  }
  if (yq) return M == 1 ? cudaLaunchKernelEx(&cfg, decode_cols_kernel<1, 4, true>, p) : cudaLaunchKernelEx(&cfg, decode_cols_kernel<kMaxM, 4, true>, p);
  return M == 1 ? cudaLaunchKernelEx(&cfg, decode_cols_kernel<1, 4, false>, p) : cudaLaunchKernelEx(&cfg, decode_cols_kernel<kMaxM, 4, false>, p);
}

int decode_pre_max_calls() { return dcol::kPreMaxCalls; }

// X_q and T_q of n independent decode calls (M <= 4 each, every layer fitting decode_cols_fits), one CTA per call, into
// outs[i] (decode_pre_bytes each, 256-byte aligned).
cudaError_t launch_decode_pre(const lqer_call_t* calls, const PackedMeta* metas, uint8_t* const* outs, int n, int order,
                              int x_type, cudaStream_t s) {
  using namespace dcol;
  static OncePerDevice once;
  cudaError_t e0 = once.run([] {
    cudaError_t e = cudaFuncSetAttribute(decode_pre_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(decode_pre_kernel<kMaxM>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    return e;
  });
  if (e0 != cudaSuccess) return e0;
  if (n < 1 || n > kPreMaxCalls) return cudaErrorInvalidValue;
  PreParams p;
  p.order = order;
  size_t smem = 0;
  bool single = true;
  for (int i = 0; i < kPreMaxCalls; ++i) {
    const int g = i < n ? i : 0;
    const PackedMeta& m = metas[g];
    PreCall& c = p.c[i];
    c.X = calls[g].X;
    c.asec = static_cast<const uint8_t*>(calls[g].packed) + m.off_a;
    c.out = outs[g];
    c.M = calls[g].M; c.K = m.K; c.K64 = m.K64; c.k_pad = m.k_pad;
    c.f = Formats{m.a_bits, m.lr_bits, m.exp_min, m.exp_max, x_type, m.w_bits};
    if (c.M < 1 || c.M > kMaxM) return cudaErrorInvalidValue;
    if (c.M > 1) single = false;
    const size_t need = pre_x_bytes(c.M, c.K64) + pre_t_bytes(c.k_pad) + 16 +
                        (size_t)t_subsets(c.k_pad) * kMaxM * c.k_pad * 8 + 128;
    if (need > smem) smem = need;
  }
  if (smem > 200 * 1024) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  LaunchScope scope(kFamDecode, s);
  return single ? cudaLaunchKernelEx(&cfg, decode_pre_kernel<1>, p) : cudaLaunchKernelEx(&cfg, decode_pre_kernel<kMaxM>, p);
}

}  // namespace lqer
