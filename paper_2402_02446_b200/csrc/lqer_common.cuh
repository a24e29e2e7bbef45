// Internal declarations shared by the translation units of the LQER library:
// the packed weight layout, the MXINT quantisation device routines and the
// launch wrappers of each kernel family.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "lqer.h"

namespace lqer {

// ----------------------------------------------------------------------------
// Packed weight layout
// ----------------------------------------------------------------------------
// header (256 B)
// W section: tiles [n_tile][k_slab], one tile = 128 output columns x 64 K:
//     nibbles [bp 2][n 128][16 B]   (bp = pair of 16-blocks; 16 B = 32 nibbles of one column)
//     exps    [n 128][4 B]          (the slab's four block exponents of one column)
//   Within a 32-bit word, nibble position p holds k_local = {0,2,4,6,1,3,5,7}[p] of the
//   word's eight consecutive K, offset-binary (mantissa + 8), so that
//   (w >> 4i) & 0x000F000F yields the adjacent pair (2i, 2i+1).
//   With 2-bit mantissas (w_bits == 2) a tile is 2048 bytes of crumbs [n 128][16 B] (one 32-bit word per 16-block:
//   crumb i of the low half holds k_local = 2i, crumb i of the high half k_local = 2i + 1, offset-binary
//   (mantissa + 1), so that (w >> 2i) & 0x00030003 yields the adjacent pair (2i, 2i+1)) followed by the same 512
//   exponent bytes.
// B section: per n_tile:  mantissas [rb][n 128][16 B int8]  then exps [rb][n 128]
// A section: mantissas [K/16][k_pad][16 B int8]  then exps [K/16][k_pad]
constexpr uint32_t kMagic = 0x5245514Cu;  // "LQER"
constexpr uint32_t kVersion = 2;
constexpr int kHeaderBytes = 256;
constexpr int kTileN = 128;
constexpr int kSlabK = 64;
constexpr int kWTileBytes = kTileN * kSlabK / 2 + kTileN * 4;  // 4608
constexpr int kWTileNibbleBytes = kTileN * kSlabK / 2;          // 4096
// Bytes of the mantissas of one weight tile, and of the whole tile (mantissas + 512 exponent bytes), by mantissa width.
__host__ __device__ inline int w_mant_bytes(int w_bits) { return kTileN * kSlabK * w_bits / 8; }   // 4096 (4 bit), 2048 (2 bit)
__host__ __device__ inline int w_tile_bytes(int w_bits) { return w_mant_bytes(w_bits) + kTileN * 4; }
constexpr int kStatusBytes = 256;

struct PackedMeta {
  uint32_t magic, version;
  int32_t K, N, k, k_pad;
  int32_t K64, n_tiles, k_slabs, r_blocks;
  int32_t w_bits, a_bits, lr_bits, block, exp_min, exp_max, deterministic;
  int32_t w_exp_min, w_exp_max, reserved0;      // exp_min/max: window of X and T; w_exp_min/max: of W_q, A_k, B_k
  uint64_t off_w, off_b, off_a, total_bytes;
  uint32_t checksum;
  uint32_t pad_[64 - 29];
};
static_assert(sizeof(PackedMeta) == kHeaderBytes, "header must be 256 bytes");

inline uint32_t meta_checksum(const PackedMeta& m) {
  const uint32_t* w = reinterpret_cast<const uint32_t*>(&m);
  uint32_t h = 2166136261u;
  for (int i = 0; i < 28; ++i) { h ^= w[i]; h *= 16777619u; }
  return h;
}

// Workspace layout: a persistent head of one fixed size (kPersistMaxBytes) that is all zero between calls
//   [0, 256)   status area: DeviceStatus
//   [256, ..)  the column-owner decode kernel's counters (two sets of 16 layers), the small-batch GEMM's per-tile
//              arrival counters (up to 32768 over the layers of a launch), then the counter pairs of the row tiles
//              (tensor-core prologue) or row groups (small prologue)
// followed by per-call scratch: Xcat (bf16 [M, K64 + k_pad]) with the fp64 partial sums of the prologue that runs
// and the fp32 partial sums of the small-batch or split-K GEMM, or the decode kernel's partial sums of T.
constexpr int kDecodeMaxCtas = 160;                  // CTAs of one launch of the column-owner decode kernel, at most
constexpr int kPrologueRowTiles = 512;               // an arrival and a departure counter each: batches up to 65536 rows
constexpr int kPrologueMaxCtas = 148;               // CTAs of one tensor-core prologue launch the scratch is sized for (launches use min(this, SMs))
constexpr int kGemmMaxPairs = 74;                    // CTA pairs of the pair GEMM (one per two SMs)
constexpr int kGemmSplitMaxM = 256;                  // batches up to this many rows (one row tile) may have their K range cut
constexpr size_t kPersistMaxBytes = 256 + 32768 * 4 + 16 * 256 * 8 + kPrologueRowTiles * 8;
__host__ __device__ inline size_t tacc_offset(const PackedMeta& m) {
  return (size_t)kStatusBytes + (((size_t)m.n_tiles * 4 + 255) & ~(size_t)255);
}
__host__ __device__ inline size_t pcount_offset(const PackedMeta& m) {
  return tacc_offset(m) + (size_t)16 * m.k_pad * 8;
}
// The head has one size for every layer: a workspace that serves layers of different shapes in turn then never has one
// layer's scratch (which keeps its last contents) where another layer expects zeroed counters.
__host__ __device__ inline size_t persist_bytes(const PackedMeta&) { return kPersistMaxBytes; }
// Split-K form of the pair GEMM for small batches (one row tile, so few tiles): the number of K ranges, the scratch
// for a batch of M rows, and a bound over all batches up to M_max.
inline int gemm_splitk_ranges(const PackedMeta& m, int M) {
  if (M > kGemmSplitMaxM) return 1;
  int c = kGemmMaxPairs / ((m.n_tiles + 1) / 2);
  if (c > 8) c = 8;
  if (c > m.k_slabs / 8) c = m.k_slabs / 8;      // at least eight K stages per range
  return c < 2 ? 1 : c;
}
inline size_t gemm_splitk_bytes(const PackedMeta& m, int M) {
  return ((size_t)(gemm_splitk_ranges(m, M) - 1) * M * m.N * 4 + 255) & ~(size_t)255;
}
inline size_t gemm_splitk_bound(const PackedMeta& m, int M_max) {
  return gemm_splitk_bytes(m, M_max < kGemmSplitMaxM ? M_max : kGemmSplitMaxM);
}
// Tensor-core prologue: a CTA owns 128 rows and one of `splits` ranges of K (in panels of 128 columns);
// each CTA leaves a [128, k_pad] fp64 partial sum; once all CTAs of a row tile have arrived each adds up its share of rows.
inline bool prologue_tc_rank_ok(const PackedMeta& m) { return m.k > 0 && (m.k_pad == 16 || m.k_pad == 32 || m.k_pad == 64); }
inline int prologue_tc_splits(const PackedMeta& m, int M, int max_ctas = kPrologueMaxCtas) {
  const int row_tiles = (M + 127) / 128, panels = (m.K64 + 127) / 128;
  int s = max_ctas / row_tiles;
  if (s > panels) s = panels;
  return s < 1 ? 1 : s;
}
// Upper bound of prologue_tc_scratch_bytes over every batch of up to M_max rows: the largest number of CTAs any
// such batch launches (row tiles x K ranges; beyond kPrologueMaxCtas row tiles every row tile is one CTA).
inline size_t prologue_tc_scratch_bound(const PackedMeta& m, int M_max) {
  if (!prologue_tc_rank_ok(m)) return 0;
  int rt_max = (M_max + 127) / 128;
  if (rt_max > kPrologueRowTiles) rt_max = kPrologueRowTiles;
  long long ctas = 0;
  for (int rt = 1; rt <= rt_max; ++rt) {
    const long long c = (long long)rt * prologue_tc_splits(m, rt * 128);
    if (c > ctas) ctas = c;
  }
  return (size_t)ctas * 128 * m.k_pad * 8;
}
inline size_t prologue_tc_scratch_bytes(const PackedMeta& m, int M) {
  if (!prologue_tc_rank_ok(m) || (M + 127) / 128 > kPrologueRowTiles) return 0;
  return (size_t)((M + 127) / 128) * prologue_tc_splits(m, M) * 128 * m.k_pad * 8;
}
// Small batches (up to kSmallMaxM rows): the prologue for few rows and the GEMM with the tokens on the MMA's M side
// (padded to 64 or 128 rows) and 256 weight columns on its N side.
// Everything below depends on the shape alone, never on the device or on what else shares a launch.
constexpr int kSmallMaxM = 128;
// K ranges per group of 16 rows in the small prologue (each a CTA; the last to arrive adds them up in range order).
inline int prologue_small_ranges(const PackedMeta& m, int M) {
  const int rgroups = (M + 15) / 16;
  int r = 148 / rgroups;
  if (r > 16) r = 16;
  if (r > m.K64 / 64) r = m.K64 / 64;             // at least four 16-blocks per range
  return r < 1 ? 1 : r;
}
inline size_t prologue_small_slot_bytes(const PackedMeta& m, int M) {
  return (size_t)((M + 15) / 16) * prologue_small_ranges(m, M) * 16 * m.k_pad * 8;
}
// The small-batch GEMM works on tiles of 256 output columns (two packed tiles).  K chunks per tile and weight stages
// (64 K) per chunk: as many work items per layer as fit 148 CTAs in one round, at least eight stages per chunk.
inline int small_gemm_col_tiles(const PackedMeta& m) { return (m.n_tiles + 1) / 2; }
inline int small_gemm_chunk_stages(const PackedMeta& m) {
  int c = 148 / small_gemm_col_tiles(m);
  int cap = m.k_slabs / 8;
  if (cap < 1) cap = 1;
  if (c > cap) c = cap;
  if (c < 1) c = 1;
  return (m.k_slabs + c - 1) / c;
}
inline int small_gemm_chunks(const PackedMeta& m) {
  const int cs = small_gemm_chunk_stages(m);
  return (m.k_slabs + cs - 1) / cs;
}
inline size_t small_gemm_partial_bytes(const PackedMeta& m, int M) {
  const int c = small_gemm_chunks(m);
  return c > 1 ? (size_t)small_gemm_col_tiles(m) * c * M * 256 * 4 : 0;
}
// Scratch of the column-owner decode kernel: fp64 partial sums of T, [16 ranges of K][4 rows][k_pad].
inline size_t decode_cols_slot_bytes(const PackedMeta& m) { return (size_t)16 * 4 * m.k_pad * 8; }

__host__ __device__ inline int b_tile_bytes(const PackedMeta& m) { return m.r_blocks * kTileN * 17; }
__host__ __device__ inline size_t xcat_cols(const PackedMeta& m) { return (size_t)m.K64 + (size_t)m.k_pad; }

// ----------------------------------------------------------------------------
// MXINT quantisation (value = m * 2^(e - (bits-2)), round half to even, symmetric clamp)
// ----------------------------------------------------------------------------
__device__ __forceinline__ float abs_ignore_nan(float v) { return (v != v) ? 0.0f : fabsf(v); }

// Shared exponent of a block from its maximum magnitude: the fp32 exponent field, clamped.
__device__ __forceinline__ int block_exponent(float amax, int emin, int emax) {
  int field = (int)((__float_as_uint(amax) >> 23) & 0xFFu);
  return min(max(field - 127, emin), emax);
}
__device__ __forceinline__ int block_exponent(double amax, int emin, int emax) {
  int field = (__double2hiint(amax) >> 20) & 0x7FF;
  return min(max(field - 1023, emin), emax);
}
// 2^p as fp32 / fp64 (p inside the normal range).
__device__ __forceinline__ float pow2f(int p) { return __uint_as_float((uint32_t)(p + 127) << 23); }
__device__ __forceinline__ double pow2d(int p) { return __hiloint2double((p + 1023) << 20, 0); }

__device__ __forceinline__ int quant_mantissa(float v, int e, int bits) {
  const float qmax = (float)((1 << (bits - 1)) - 1);
  float r = v * pow2f((bits - 2) - e);           // exact: power-of-two scaling
  r = fminf(fmaxf(r, -qmax), qmax);              // clamp first; +-inf saturate
  int m = __float2int_rn(r);                     // round half to even
  return (v != v) ? 0 : m;
}
__device__ __forceinline__ int quant_mantissa(double v, int e, int bits) {
  const double qmax = (double)((1 << (bits - 1)) - 1);
  double r = v * pow2d((bits - 2) - e);
  r = fmin(fmax(r, -qmax), qmax);
  int m = __double2int_rn(r);
  return (v != v) ? 0 : m;
}
// bf16 bit pattern of m * 2^p for |m| <= 127 (exact: at most 7 significant bits).
__device__ __forceinline__ uint32_t bf16_bits_of(int m, int p) {
  return __float_as_uint((float)m * pow2f(p)) >> 16;
}

// Quantise the four values a lane holds; the 16-block is spread over 4 adjacent lanes.
// Returns the four int8 mantissas packed in one word and the four exact bf16 values
// m * 2^(e - (bits-2)) packed in two words.
__device__ __forceinline__ void quantize_quad(const float4 vin, int bits, int emin, int emax, int& e, uint32_t& m8,
                                              uint2& bf) {
  // block maximum: fmaxf drops a NaN operand, so NaN counts as zero here; a block of NaNs only ends as zero too
  float amax = fmaxf(fmaxf(fabsf(vin.x), fabsf(vin.y)), fmaxf(fabsf(vin.z), fabsf(vin.w)));
  amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
  amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
  amax = fmaxf(amax, 0.0f);
  e = block_exponent(amax, emin, emax);
  const float qmax = (float)((1 << (bits - 1)) - 1);
  const float inv_step = pow2f((bits - 2) - e), step = pow2f(e - (bits - 2));
  // Adding 1.5 * 2^23 rounds a value of magnitude below 2^22 to an integer, half to even, and leaves
  // that integer (two's complement) in the low bits of the sum; (sum - 1.5 * 2^23) * step is exact.
  const float kMagic = 12582912.0f;
  const float back = -kMagic * step;
  const float v[4] = {vin.x, vin.y, vin.z, vin.w};
  uint32_t rb[4];
  float r[4];
  // The common case needs neither the clamp nor the NaN test: the lane's four values are numbers (their sum is
  // not NaN; inf - inf only sends the lane the long way round) and the block's largest scaled magnitude stays
  // below qmax + 1/2, so no element rounds past qmax (an infinite or clamped-exponent block fails this test).
  const float lane_sum = (vin.x + vin.y) + (vin.z + vin.w);
  if (lane_sum == lane_sum && amax * inv_step < qmax + 0.5f) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float s = fmaf(v[i], inv_step, kMagic);                  // exact scaling, one rounding: to the integer
      rb[i] = __float_as_uint(s);
      r[i] = fmaf(s, step, back);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float x = (v[i] == v[i]) ? v[i] : 0.0f;                  // NaN -> 0
      const float t = fminf(fmaxf(x * inv_step, -qmax), qmax);       // exact scaling, clamp (+-inf saturate)
      const float s = t + kMagic;
      rb[i] = __float_as_uint(s);
      r[i] = fmaf(s, step, back);                                    // exact: at most 7 significant bits
    }
  }
  m8 = __byte_perm(__byte_perm(rb[0], rb[1], 0x0040), __byte_perm(rb[2], rb[3], 0x0040), 0x5410);
  bf.x = __byte_perm(__float_as_uint(r[0]), __float_as_uint(r[1]), 0x7632);
  bf.y = __byte_perm(__float_as_uint(r[2]), __float_as_uint(r[3]), 0x7632);
}

// Element type of X at the layer's boundary: fp32, bf16, or MXINT (int8 mantissas [M, K] followed by the exponent bytes
// [M, K / 16], the layout the MXINT8 output has).  An MXINT X is taken at its value: the loaders below turn a block's
// mantissas into the fp32 values m * 2^(e - (bits - 2)) (exact), and the ordinary quantisers then see numbers that
// are fixed points of the quantisation (or, for a block that is not normalised, the same values renormalised).
constexpr int kXF32 = 0, kXBF16 = 1, kXMXINT8 = 2;
inline size_t x_bytes(int x_type, size_t M, size_t K) { return x_type == kXMXINT8 ? M * K + M * K / 16 : M * K * (x_type == kXBF16 ? 2 : 4); }
// Four mantissas (one word, element order) of a block with exponent byte eb -> their values.
__device__ __forceinline__ float4 mxint_quad_values(uint32_t m8, uint32_t eb, int bits, int emin, int emax) {
  const int e = min(max((int)eb - 127, emin), emax);
  const float step = pow2f(e - (bits - 2));
  const float back = -12583040.0f * step;                   // -(1.5 * 2^23 + 128) * step
  const uint32_t u = m8 ^ 0x80808080u;                       // two's complement -> offset binary
  // the bytes (u_i, 0x00, 0x40, 0x4B) are the float 1.5 * 2^23 + u_i: one byte permute converts, one fma scales (exact)
  return make_float4(fmaf(__uint_as_float(__byte_perm(u, 0x4B400000u, 0x7640)), step, back),
                     fmaf(__uint_as_float(__byte_perm(u, 0x4B400000u, 0x7641)), step, back),
                     fmaf(__uint_as_float(__byte_perm(u, 0x4B400000u, 0x7642)), step, back),
                     fmaf(__uint_as_float(__byte_perm(u, 0x4B400000u, 0x7643)), step, back));
}
// Four consecutive elements of row `row` from column `col` (a multiple of 4) of X [M, K] in any of the three types.
__device__ __forceinline__ float4 load_x_quad(const void* X, int x_type, int M, int K, int row, int col, int bits, int emin, int emax) {
  const size_t idx = (size_t)row * K + col;
  if (x_type == kXBF16) {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(X) + idx));
    return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u), __uint_as_float(v.y << 16),
                       __uint_as_float(v.y & 0xFFFF0000u));
  }
  if (x_type == kXMXINT8) {
    const uint8_t* xb = static_cast<const uint8_t*>(X);
    const uint32_t m8 = __ldg(reinterpret_cast<const uint32_t*>(xb + idx));
    const uint32_t eb = __ldg(xb + (size_t)M * K + (size_t)row * (K / 16) + (col >> 4));
    return mxint_quad_values(m8, eb, bits, emin, emax);
  }
  return __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(X) + idx));
}

// What quantize_block16 needs of the format, computed once per kernel instead of once per block.
struct QuantConsts {
  float qmax, qlim;      // 2^(bits-1) - 1, and qmax + 1/2
  int shift;             // bits - 2
  int emin, emax;
};
__device__ __forceinline__ QuantConsts quant_consts(int bits, int emin, int emax) {
  QuantConsts c;
  c.qmax = (float)((1 << (bits - 1)) - 1);
  c.qlim = c.qmax + 0.5f;
  c.shift = bits - 2;
  c.emin = emin; c.emax = emax;
  return c;
}
// The same quantisation with one lane holding a whole 16-block: no shuffles, and the exponent arithmetic is paid once
// per 16 elements.  m8 = the sixteen int8 mantissas in element order; bf0 / bf1 = the sixteen exact bf16 values.
__device__ __forceinline__ void quantize_block16(const float (&v)[16], const QuantConsts& c, int& e, uint4& m8, uint4& bf0,
                                                 uint4& bf1) {
  // Block maximum and a NaN detector, both as trees (four levels deep instead of fifteen dependent operations).
  // fmaxf drops a NaN operand, so NaN counts as zero in the maximum; the sum is NaN iff a NaN (or inf - inf) is
  // among the values, and its order does not matter because only that is asked of it.
  float mx[8], sm[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { mx[i] = fmaxf(fabsf(v[2 * i]), fabsf(v[2 * i + 1])); sm[i] = v[2 * i] + v[2 * i + 1]; }
#pragma unroll
  for (int w = 4; w > 0; w >>= 1)
#pragma unroll
    for (int i = 0; i < w; ++i) { mx[i] = fmaxf(mx[i], mx[i + w]); sm[i] += sm[i + w]; }
  float amax = mx[0];
  const float sum = sm[0];
  amax = fmaxf(amax, 0.0f);
  e = block_exponent(amax, c.emin, c.emax);
  const float inv_step = pow2f(c.shift - e), step = pow2f(e - c.shift);
  const float kMagic = 12582912.0f;                   // 1.5 * 2^23, see quantize_quad
  const float back = -kMagic * step;
  uint32_t m[4], b[8];
  if (sum == sum && amax * inv_step < c.qlim) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {                     // four elements at a time: few values alive at once
      float s4[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) s4[i] = fmaf(v[4 * q + i], inv_step, kMagic);
      m[q] = __byte_perm(__byte_perm(__float_as_uint(s4[0]), __float_as_uint(s4[1]), 0x0040),
                         __byte_perm(__float_as_uint(s4[2]), __float_as_uint(s4[3]), 0x0040), 0x5410);
      b[2 * q] = __byte_perm(__float_as_uint(fmaf(s4[0], step, back)), __float_as_uint(fmaf(s4[1], step, back)), 0x7632);
      b[2 * q + 1] = __byte_perm(__float_as_uint(fmaf(s4[2], step, back)), __float_as_uint(fmaf(s4[3], step, back)), 0x7632);
    }
  } else {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float s4[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float x = (v[4 * q + i] == v[4 * q + i]) ? v[4 * q + i] : 0.0f;
        s4[i] = fminf(fmaxf(x * inv_step, -c.qmax), c.qmax) + kMagic;
      }
      m[q] = __byte_perm(__byte_perm(__float_as_uint(s4[0]), __float_as_uint(s4[1]), 0x0040),
                         __byte_perm(__float_as_uint(s4[2]), __float_as_uint(s4[3]), 0x0040), 0x5410);
      b[2 * q] = __byte_perm(__float_as_uint(fmaf(s4[0], step, back)), __float_as_uint(fmaf(s4[1], step, back)), 0x7632);
      b[2 * q + 1] = __byte_perm(__float_as_uint(fmaf(s4[2], step, back)), __float_as_uint(fmaf(s4[3], step, back)), 0x7632);
    }
  }
  m8 = make_uint4(m[0], m[1], m[2], m[3]);
  bf0 = make_uint4(b[0], b[1], b[2], b[3]);
  bf1 = make_uint4(b[4], b[5], b[6], b[7]);
}

__device__ __forceinline__ void mma_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%7,%7,%7,%7};"
               : "=r"(c[0]), "=r"(c[1]), "=r"(c[2]), "=r"(c[3]) : "r"(a0), "r"(a1), "r"(b0), "r"(0));
}

// ----------------------------------------------------------------------------
// Device status word (head of the workspace)
// ----------------------------------------------------------------------------
struct DeviceStatus {
  int code;        // lqer_status_t, first error wins
  int where;       // kernel-specific location id
  int detail0, detail1;
};
__device__ __forceinline__ void report_error(DeviceStatus* st, int code, int where, int d0 = 0, int d1 = 0) {
  if (st != nullptr && atomicCAS(&st->code, 0, code) == 0) {
    st->where = where; st->detail0 = d0; st->detail1 = d1;
  }
}

// Checked build (-DLQER_DEBUG_BOUNDS; the library is then liblqer_dbg.so): every global store of the inference kernels,
// and every bulk copy of packed weights, first checks its byte range against the extent of the buffer it goes to
// (or comes from).  The first violation goes to the status word (LQER_ERR_BOUNDS, the site, offset and extent in
// 16-byte units) and the access is skipped: nothing traps and nothing out of range is touched.  In the ordinary build
// the macro is the constant true and the extents in the kernels' parameters are dead.
#ifdef LQER_DEBUG_BOUNDS
__device__ __forceinline__ bool in_bounds(DeviceStatus* st, size_t off, size_t len, size_t extent, int site) {
  if (off + len <= extent) return true;
  report_error(st, LQER_ERR_BOUNDS, site, (int)(off >> 4), (int)(extent >> 4));
  return false;
}
#define LQER_IN_BOUNDS(st, off, len, extent, site) ::lqer::in_bounds(st, (size_t)(off), (size_t)(len), (size_t)(extent), site)
constexpr bool kDebugBounds = true;
#else
#define LQER_IN_BOUNDS(st, off, len, extent, site) true
constexpr bool kDebugBounds = false;
#endif
// Test hook of the checked build (lqer_debug_bounds_shrink): bytes taken off the declared extent of Y at the next launches.
size_t debug_y_shrink();

// ----------------------------------------------------------------------------
// Per-device host state
// ----------------------------------------------------------------------------
// Number of SMs of the current device (cached per device; 0 if the query fails).
int sm_count();
// Runs `set` the first time it is called with a given device current: kernel attributes such as the
// dynamic shared-memory limit belong to a device, so a process that drives several GPUs sets them on each.
class OncePerDevice {
 public:
  template <class F>
  cudaError_t run(F&& set) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu_);
    if (((done_ >> dev) & 1ull) == 0) {
      if ((e = set()) != cudaSuccess) return e;
      done_ |= 1ull << dev;
    }
    return cudaSuccess;
  }
 private:
  std::mutex mu_;
  unsigned long long done_ = 0;
};
// Bound, in SM clock cycles, of every device-side wait (lqer_set_wait_limit_cycles; default about two seconds).
long long wait_limit_cycles();
// Workspace bytes the call lqer_linear_stream(X, M, packed, ...) needs on the path it would take now.
lqer_status_t call_workspace_bytes(const void* packed, int M, size_t* bytes);
// Test hook (lqer_inject_stall): true once for the next launch of `family` after it was armed; that launch then
// waits for one arrival more than will ever come, so its waits run out and it reports LQER_ERR_TIMEOUT.
bool take_stall(int family);

// ----------------------------------------------------------------------------
// Launch wrappers (each returns the cudaError_t of its launches)
// ----------------------------------------------------------------------------
// Kernel families, as reported by lqer_profile_collect.
enum KernelFamily {
  kFamPack = 0, kFamExport, kFamQuantize, kFamPrologue, kFamGemmSimt, kFamPrepare, kFamGemmTcPair, kFamDecode,
  kNumFamilies
};
// Brackets the launches of one kernel family: counts them and, while profiling is enabled,
// records a CUDA event on the stream before and after.
class LaunchScope {
 public:
  LaunchScope(int family, cudaStream_t s, int n_kernels = 1);
  ~LaunchScope();
  LaunchScope(const LaunchScope&) = delete;
  LaunchScope& operator=(const LaunchScope&) = delete;
 private:
  cudaStream_t stream_;
  cudaEvent_t stop_;
};

cudaError_t launch_pack(const float* W, const float* A, const float* B, const PackedMeta& m, void* packed,
                        cudaStream_t s);
cudaError_t launch_export(const PackedMeta& m, const void* packed, int8_t* Wm, uint8_t* We, int8_t* Am,
                          uint8_t* Ae, int8_t* Bm, uint8_t* Be, cudaStream_t s);
cudaError_t launch_quantize_x(const float* X, int M, int K, int bits, int emin, int emax, int8_t* Xm,
                              uint8_t* Xe, cudaStream_t s);
// X -> Xcat[:, 0:K64] (bf16 of the dequantised MXINT8 value) and T_q -> Xcat[:, K64:K64+k_pad];
// optional int8 / exponent exports of T_q.
cudaError_t launch_prologue(const void* X, int x_type, int M, const PackedMeta& m, const void* packed, void* xcat,
                            int8_t* Tm, uint8_t* Te, DeviceStatus* st, cudaStream_t s);
// The same prologue with the projection on the tcgen05 int8 tensor cores: ranks up to 64, large batches.
bool prologue_tc_fits(const PackedMeta& m, int M, const void* X, bool any_batch);
// `partials`: prologue_tc_scratch_bytes(m, M) of scratch; `counters`: zeroed counter pairs of the workspace head,
// one per row tile.  `order`: kChainAlone, or the place in a run of prologues that share no buffer or counter
// (each later one overlaps the tail of the one before; the kernel after the run still finds all of them complete).
enum ChainOrder { kChainAlone = 0, kChainFirst = 1, kChainLater = 2 };
cudaError_t launch_prologue_tc(const void* X, int x_type, int M, const PackedMeta& m, const void* packed, void* xcat,
                               int8_t* Tm, uint8_t* Te, DeviceStatus* st, double* partials, int* counters,
                               int order, cudaStream_t s);
// The same for up to 8 layers with one M, one k_pad and one set of formats in ONE launch (a CTA per row tile and K range
// of a layer, found by its index); prologue_tc_group_splits picks the K ranges per row tile so that the CTAs carry
// about equal work and stay within one per SM.
bool prologue_tc_group_splits(const PackedMeta* metas, int n, int M, int max_ctas, int* splits);
cudaError_t launch_prologue_tc_group(const void* const* Xs, int x_type, int M, const PackedMeta* metas, const void* const* packed,
                                     void* const* xcats, double* const* partials, int* const* counters,
                                     const int* splits, int n, int8_t* Tm, uint8_t* Te, DeviceStatus* st, int order,
                                     cudaStream_t s);
cudaError_t launch_gemm_simt(const void* xcat, int M, const PackedMeta& m, const void* packed, float* Y,
                             cudaStream_t s);
// y_type: element type of Y (kYF32, kYBF16, kYMXINT8: mantissas [M,N] then exponent bytes [M,N/16], N % 16 == 0).
constexpr int kYF32 = 0, kYBF16 = 1, kYMXINT8 = 2;
inline size_t y_bytes(int y_type, size_t M, size_t N) { return y_type == kYMXINT8 ? M * N + M * N / 16 : M * N * (y_type == kYBF16 ? 2 : 4); }
cudaError_t launch_gemm_tc2(const void* xcat, int M, const PackedMeta& m, const void* packed, void* Y, int y_type,
                            DeviceStatus* st, cudaStream_t s);
// Small batches: the layer's K range cut into gemm_splitk_ranges(m, M) ranges that run as layers of one launch;
// `partials` holds (ranges - 1) * M * N floats (gemm_splitk_bytes).
cudaError_t launch_gemm_tc2_splitk(const void* xcat, int M, const PackedMeta& m, const void* packed, void* Y, int y_type,
                                   float* partials, DeviceStatus* st, cudaStream_t s);
// Up to gemm_tc2_max_group() layers with one M in one launch (xcats, packed, Ys, metas: host arrays of n entries).
int gemm_tc2_max_group();
cudaError_t launch_gemm_tc2_group(const void* const* xcats, const void* const* packed, void* const* Ys, int y_type,
                                  const PackedMeta* metas, int n, int M, DeviceStatus* st, cudaStream_t s);
// Factor preparation (Section 3.1 / 3.2, Appendix A): A_k, B_k from W and calibration samples, by randomised subspace
// iteration with factor_sketch_rank columns; Omega [N, that many] fp32 is the caller's random test matrix.
int factor_sketch_rank(int K, int N, int k);
size_t factor_workspace_bytes(int K, int N, int k, int max_calib_rows);
cudaError_t launch_factorize(const float* W, const float* const* Xs, const int* rows, int n_samples, const float* Omega, int K,
                             int N, int k, int w_bits, int emin, int emax, float* A, float* B, void* workspace, int** status_dev,
                             float** A_used, float** B_used, cudaStream_t s);
// Small batches (M <= kSmallMaxM).  The prologue quantises X (fp32 or bf16) into Xcat and leaves T_q behind it; up to
// prologue_small_max_layers() layers with one M and one set of formats per launch.
struct SmallPrologueLayer {
  const void* X;
  const void* packed;
  const PackedMeta* meta;
  void* xcat;                 // bf16 [M, K64 + k_pad], or the fragment order below
  double* slots;              // prologue_small_slot_bytes of scratch
  int* counts;                // one zeroed counter per group of 16 rows (eight ints; in fragment order counts[kCountXq] too)
  int8_t* Tm;                 // optional exports of T_q (may be null)
  uint8_t* Te;
  int* flags;                 // fragment order: the layer's two flags (below)
};
int prologue_small_max_layers();
// Fragment order of [X_q | T_q] for up to 16 rows, as the register-operand GEMM reads it (frag_order = true; M <= 16):
// eight planes q of [slab][256 bytes], a slab being 64 columns of X_q (k_slabs of them) or 64 rank indices of T_q
// (frag_rank_slabs of them, zero beyond k_pad).  The element of row r at column c of slab s lies in plane
// q = (c % 32) / 4 at byte  s * 256 + (2 (r % 8) + c / 32) * 16 + ((c % 4) / 2 * 2 + r / 8) * 4 + (c % 2) * 2:
// 16 bytes = the four registers of one mma.sync A fragment.  Rows beyond M are written as zeros.  The prologue also
// raises two flags for the GEMM that follows it (`flags`, two ints of the layer in the workspace's status area from
// kFlagAreaOffset on, used by nothing else): flags[0] takes the launch's `epoch` once every CTA's share of X_q is in
// place (the CTAs count themselves in at counts[kCountXq]; the last one sets it back to zero), flags[1] once T_q is.
// An epoch is a number that no earlier launch on this workspace used, so a flag left by the call before never
// passes for this call's, whenever the two overlap; the GEMM's last CTA clears the flags when it leaves (a counter
// behind them counts its CTAs out), which is what a replayed graph, whose epoch repeats, relies on.
constexpr int kCountXq = 1;
constexpr int kFlagAreaOffset = 64;                 // status area bytes [64, 64 + 16 layers * 8), then the exit counter
inline int frag_rank_slabs(const PackedMeta& m) { return (m.k_pad + 63) / 64; }
inline size_t frag_bytes(const PackedMeta& m) { return (size_t)8 * (m.k_slabs + frag_rank_slabs(m)) * 256; }
cudaError_t launch_prologue_small(const SmallPrologueLayer* layers, int n, int M, int x_type, bool frag_order, int epoch,
                                  DeviceStatus* st, cudaStream_t s);
// The small-batch GEMM (tokens on the M side of a 64- or 128-row MMA, 256 weight columns on its N side); up to
// gemm_small_max_layers() layers with one M per launch.
struct SmallGemmLayer {
  const void* xcat;
  const void* packed;
  const PackedMeta* meta;
  void* Y;                    // [M, N] fp32 or bf16, or the MXINT8 pair of sections
  float* partials;            // small_gemm_partial_bytes of scratch (unused if the tiles have one chunk)
  int* counters;              // one zeroed counter per 256-column tile
  int* flags;                 // register-operand kernel: the layer's two flags, as the small prologue raises them
};
// Whether a small-batch call of M rows on these weights takes the register-operand GEMM (and with it the fragment order
// of the activations) unless the tensor-memory kernel is forced.
inline bool small_takes_mma(const PackedMeta& m, int M) { return M <= 16 && (m.w_bits == 4 || m.w_bits == 2); }
int gemm_small_max_layers();
// tensor_memory_form: keep the tcgen05 kernel also where the register-operand kernel (up to 16 rows)
// would take the launch.
cudaError_t launch_gemm_small(const SmallGemmLayer* layers, int n, int M, int y_type, bool tensor_memory_form, int epoch,
                              DeviceStatus* st, cudaStream_t s);
cudaError_t launch_decode_cols(const void* X, int x_type, int M, const PackedMeta& m, const void* packed, void* Y, int y_type,
                               void* workspace, cudaStream_t s);
bool decode_cols_fits(const PackedMeta& m, int M);
// Up to decode_cols_max_group() independent layers with one M (all fitting decode_cols_fits, N >= 32) in one launch.
// `order`, `set`: consecutive launches of a chain (ChainOrder) alternate between two sets of slots and counters: set 0
// behind the head of the workspace, set 1 at its end (`workspace_bytes`, read for set 1 only), so a chain needs
// align_up(kPersistMaxBytes, 256) plus twice the largest group's decode_cols_slot_bytes.  A launch may be chained to
// the one before only if that one reported `fills_gpu` (one CTA on every SM: at most two launches are alive then).
int decode_cols_max_group();
cudaError_t launch_decode_cols_group(const lqer_call_t* calls, const PackedMeta* metas, int n, void* workspace,
                                     size_t workspace_bytes, int order, int set, bool* fills_gpu, const uint8_t* const* pres,
                                     int x_type, int y_type, cudaStream_t s);
// The quantised activations and T_q of up to decode_pre_max_calls() independent decode calls, computed ahead (one CTA
// per call) into outs[i] (decode_pre_bytes each, 256-byte aligned); launch_decode_cols_group takes them as `pres` and
// then has no X to quantise, no T to compute and nothing to exchange.  `order` as above.
inline size_t decode_pre_bytes(const PackedMeta& m, int M) {
  const size_t b = (size_t)M * m.K64 + (size_t)M * (m.K64 / 16) * 8 + 4 * 16 * 4 + (size_t)4 * (m.k_pad > 0 ? m.k_pad : 16);
  return (b + 255) & ~(size_t)255;
}
int decode_pre_max_calls();
cudaError_t launch_decode_pre(const lqer_call_t* calls, const PackedMeta* metas, uint8_t* const* outs, int n, int order,
                              int x_type, cudaStream_t s);

}  // namespace lqer
