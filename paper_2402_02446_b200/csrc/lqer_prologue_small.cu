// Activation prologue for small batches (paper Section 4.1: X_q in MXINT8, blocks [1,16]; Section 3.1: the
// small high-precision product X A_k), built for latency: a decode step of a few tokens is a chain of short
// kernels, so this one spreads even 16 rows over many CTAs and has no wait in it.
//
//   grid = row groups (16 rows of X each) x K ranges (up to 16 per row group)
//   CTA (r, g):  X[16 rows, K range] fp32/bf16 -> MXINT8 -> exact bf16 values into Xcat[:, K range]
//                partial T = X_q A_q over its K range: one int8 mma.sync (m16n8k16, exact int32) per
//                (16-block, 8 rank columns), scaled by 2^(e_x + e_a) and summed in fp64
//                -> slot (r, g) of the scratch; then it counts itself in.
//   The CTA that arrives LAST for a row group (no one waits for anyone) adds the slots in range order,
//   re-quantises T along the rank and appends T_q to Xcat[:, K64 : K64 + k_pad].
// The results equal the other prologues' bit for bit: the block products are exact integers, the fp64 sums
// are exact unless a row's block exponents spread over more than about 30 binades, and the order of the
// additions is fixed by the ranges, which depend on the shape alone.
#include "lqer_common.cuh"

namespace lqer {
namespace psm {

constexpr int kRows = 16;                 // rows per CTA = one MMA M tile
constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kStepCols = 1024;           // columns of X a CTA quantises per step (shared-memory panel)
constexpr int kXqStride = kStepCols + 16; // bytes per row of the int8 panel (+16: conflict-free fragment loads)
constexpr int kMaxLayers = 16;

struct Layer {
  const void* X;              // [M, K] fp32 or bf16
  const uint8_t* asec;        // A_q section of the packed buffer
  uint16_t* xcat;             // [M, K64 + k_pad] bf16
  double* slots;              // [row group][range][16][k_pad] partial sums of T
  int* counts;                // [row group] arrivals, zero between calls
  int* flags;                 // fragment order: X_q ready, T_q ready (each takes the launch's epoch)
  int8_t* Tm;                 // optional exports of T_q
  uint8_t* Te;
  size_t xcat_extent, slots_extent;   // bytes behind xcat and slots, for the checked build
  int K, K64, k, k_pad;
  int ranges;                 // K ranges per row group
  int cta_begin;              // first CTA of this layer in the launch
};

struct Params {
  Layer L[kMaxLayers];
  int n;                      // layers in this launch
  int M;
  DeviceStatus* status;
  int x_type;                 // kXF32, kXBF16 or kXMXINT8
  int a_bits, lr_bits, exp_min, exp_max;
  int frag;                   // Xcat in the fragment order of the register-operand GEMM (M <= 16), with its flags
  int epoch;                  // value the flags take in this launch
};

// Byte offset of (row, column c of slab s) in the fragment order; plane: bytes of one plane.
__device__ __forceinline__ size_t frag_offset(int row, int slab, int c, size_t plane) {
  return (size_t)((c & 31) >> 2) * plane + (size_t)slab * 256 + (2 * (row & 7) + (c >> 5)) * 16 + (((c & 3) >> 1) * 2 + (row >> 3)) * 4 +
         (c & 1) * 2;
}

// TPW: rank tiles (8 columns) a warp owns: 1 for ranks up to 64, 2 up to 128, 4 up to 256.
template <int TPW>
__global__ void __launch_bounds__(kThreads, TPW == 1 ? 3 : TPW == 2 ? 2 : 1) prologue_small_kernel(const __grid_constant__ Params p) {
  __shared__ __align__(16) uint8_t s_xq[kRows * kXqStride];
  __shared__ int8_t s_xe[kRows][kStepCols / 16];
  __shared__ double s_part[kWarps][kRows * 8];        // warps that share a rank tile meet here (TPW == 1)
  __shared__ int s_last;

  int layer = 0;
#pragma unroll
  for (int i = 1; i < kMaxLayers; ++i)
    if (i < p.n && (int)blockIdx.x >= p.L[i].cta_begin) layer = i;
  const Layer& ly = p.L[layer];
  const int bid = (int)blockIdx.x - ly.cta_begin;
  const int rgroup = bid / ly.ranges, range = bid % ly.ranges;
  const int row0 = rgroup * kRows;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, tig = lane & 3;
  const int M = p.M, K = ly.K, k_pad = ly.k_pad;
  const size_t ldx = (size_t)ly.K64 + (size_t)k_pad;
  const int KB64 = ly.K64 / 16, kblocks = K / 16;
  const int kb_lo = (int)((long long)range * KB64 / ly.ranges), kb_hi = (int)((long long)(range + 1) * KB64 / ly.ranges);
  const uint8_t* a_exp = ly.asec + (size_t)kblocks * k_pad * 16;
  const int NT = k_pad / 8;                              // 8-column rank tiles
  const int WPN = NT >= kWarps ? 1 : kWarps / NT;        // warps that share one rank tile (they split the blocks)
  const bool has_rank = ly.k > 0;
  const size_t plane = (size_t)(ly.K64 / 64 + (k_pad + 63) / 64) * 256;      // fragment order: bytes of one plane
  const bool active = has_rank && (NT >= kWarps || warp < NT * WPN);
  const int bias = -127 - (p.a_bits - 2) - (p.lr_bits - 2);   // exponent bytes carry +127

  // The kernel after this one (the GEMM) may start at once: it only prefetches weights before its own wait.
  // This CTA's share of A_q depends on no earlier kernel: on its way to L2 while the kernel before drains.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (has_rank) {
    const int kr_lo = min(kb_lo, kblocks), kr_hi = min(kb_hi, kblocks);
    const uint8_t* gm = ly.asec + (size_t)kr_lo * k_pad * 16;
    const uint8_t* ge = a_exp + (size_t)kr_lo * k_pad;
    const int mant = (kr_hi - kr_lo) * k_pad * 16, ex = (kr_hi - kr_lo) * k_pad;
    for (int o = tid * 128; o < mant; o += kThreads * 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(gm + o));
    for (int o = tid * 128; o < ex; o += kThreads * 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(ge + o));
  }
  // X and the workspace may still be in use by the kernel before: wait for it.
  asm volatile("griddepcontrol.wait;" ::: "memory");

  double acc[TPW][4];
#pragma unroll
  for (int i = 0; i < TPW; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0;

  for (int kb0 = kb_lo; kb0 < kb_hi; kb0 += kStepCols / 16) {
    const int nblk = min(kStepCols / 16, kb_hi - kb0);
    // ---- quantise 16 rows x (nblk * 16) columns: bf16 to Xcat, int8 + exponents to shared memory
    const int quads_per_row = nblk * 4;
    const int n_quads = kRows * quads_per_row;                             // a multiple of 64
    for (int f0 = 0; f0 < n_quads; f0 += 4 * kThreads) {                  // whole warps: the block maximum is a shuffle
      // four loads per thread in flight, then the arithmetic: a kernel this short is a chain of memory latencies
      float4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int f = f0 + u * kThreads + tid;
        const bool live = f < n_quads;
        const int r = live ? f / quads_per_row : 0, c4 = live ? f % quads_per_row : 0;
        const int col = kb0 * 16 + c4 * 4, row = row0 + r;
        v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (live && row < M && col < K) v[u] = load_x_quad(ly.X, p.x_type, M, K, row, col, p.a_bits, p.exp_min, p.exp_max);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int f = f0 + u * kThreads + tid;
        if (f0 + u * kThreads >= n_quads) break;                           // uniform over the CTA
        const bool live = f < n_quads;
        const int r = live ? f / quads_per_row : 0, c4 = live ? f % quads_per_row : 0;
        const int col = kb0 * 16 + c4 * 4, row = row0 + r;
        int e;
        uint32_t m8;
        uint2 bf;
        quantize_quad(v[u], p.a_bits, p.exp_min, p.exp_max, e, m8, bf);
        if (live) {
          *reinterpret_cast<uint32_t*>(&s_xq[r * kXqStride + c4 * 4]) = m8;
          if ((c4 & 3) == 0) s_xe[r][c4 >> 2] = (int8_t)e;
          if (p.frag) {
            // four consecutive K of a row: the two pairs of one A fragment, 8 bytes apart (rows beyond M are zeros)
            const size_t o = frag_offset(r, col >> 6, col & 63, plane);
            if (LQER_IN_BOUNDS(p.status, o, 12, ly.xcat_extent, 311)) {
              uint8_t* dst = reinterpret_cast<uint8_t*>(ly.xcat) + o;
              *reinterpret_cast<uint32_t*>(dst) = bf.x;
              *reinterpret_cast<uint32_t*>(dst + 8) = bf.y;
            }
          } else if (row < M && LQER_IN_BOUNDS(p.status, ((size_t)row * ldx + col) * 2, 8, ly.xcat_extent, 311))
            *reinterpret_cast<uint2*>(ly.xcat + (size_t)row * ldx + col) = bf;
        }
      }
    }
    const bool last_step = kb0 + kStepCols / 16 >= kb_hi;
    if (p.frag && last_step) __threadfence();          // this CTA's share of X_q before its arrival
    __syncthreads();
    if (p.frag && last_step && tid == 0 && atomicAdd(ly.counts + kCountXq, 1) == ly.ranges - 1) {
      ly.counts[kCountXq] = 0;                         // zero again for the next call
      __threadfence();                                 // every CTA's share before the flag
      atomicExch(ly.flags, p.epoch);
    }
    // ---- partial T over these blocks (blocks beyond K are padding: zero mantissas, no A_q rows)
    if (active) {
      const int b_first = NT >= kWarps ? 0 : warp / NT;
      const int b_step = NT >= kWarps ? 1 : WPN;
      const int nt0 = NT >= kWarps ? warp : warp % NT;
      const int nreal = min(nblk, kblocks - kb0);
      // four blocks per round: their A_q words are requested together, then the MMAs run
      for (int bq = b_first; bq < nreal; bq += 4 * b_step) {
        uint32_t bw[4][TPW], ew[4][TPW];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int b = bq + u * b_step;
          const size_t kb = (size_t)(kb0 + (b < nreal ? b : bq));
#pragma unroll
          for (int i = 0; i < TPW; ++i) {
            const int nt = min(nt0 + kWarps * i, NT - 1);
            bw[u][i] = __ldg(reinterpret_cast<const uint32_t*>(ly.asec + (kb * k_pad + nt * 8 + g) * 16 + tig * 4));
            ew[u][i] = __ldg(reinterpret_cast<const uint16_t*>(a_exp + kb * k_pad + nt * 8 + tig * 2));
          }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int b = bq + u * b_step;
          if (b < nreal) {
            const uint32_t a0 = *reinterpret_cast<const uint32_t*>(&s_xq[g * kXqStride + b * 16 + tig * 4]);
            const uint32_t a1 = *reinterpret_cast<const uint32_t*>(&s_xq[(g + 8) * kXqStride + b * 16 + tig * 4]);
            const int ex0 = s_xe[g][b] + bias, ex1 = s_xe[g + 8][b] + bias;
#pragma unroll
            for (int i = 0; i < TPW; ++i) {
              if (nt0 + kWarps * i < NT) {
                int c[4];
                mma_s8(c, a0, a1, bw[u][i]);
                const int ea_lo = (int)(ew[u][i] & 0xFFu), ea_hi = (int)(ew[u][i] >> 8);
                acc[i][0] = fma((double)c[0], pow2d(ex0 + ea_lo), acc[i][0]);
                acc[i][1] = fma((double)c[1], pow2d(ex0 + ea_hi), acc[i][1]);
                acc[i][2] = fma((double)c[2], pow2d(ex1 + ea_lo), acc[i][2]);
                acc[i][3] = fma((double)c[3], pow2d(ex1 + ea_hi), acc[i][3]);
              }
            }
          }
        }
      }
    }
    __syncthreads();
  }
  if (!has_rank) return;

  // ---- this CTA's partial sums -> its slot: the warps that share a rank tile add up in warp order
  double* slot = ly.slots + ((size_t)rgroup * ly.ranges + range) * kRows * k_pad;
  if (!LQER_IN_BOUNDS(p.status, (size_t)(slot - ly.slots) * 8, (size_t)kRows * k_pad * 8, ly.slots_extent, 312)) return;
  if (NT >= kWarps) {
    if (active) {
#pragma unroll
      for (int i = 0; i < TPW; ++i) {
        const int nt = warp + kWarps * i;
        if (nt < NT) {
          *reinterpret_cast<double2*>(slot + g * k_pad + nt * 8 + tig * 2) = make_double2(acc[i][0], acc[i][1]);
          *reinterpret_cast<double2*>(slot + (g + 8) * k_pad + nt * 8 + tig * 2) = make_double2(acc[i][2], acc[i][3]);
        }
      }
    }
  } else {
    if (active) {
      double* mine = s_part[warp];
      mine[g * 8 + tig * 2] = acc[0][0];
      mine[g * 8 + tig * 2 + 1] = acc[0][1];
      mine[(g + 8) * 8 + tig * 2] = acc[0][2];
      mine[(g + 8) * 8 + tig * 2 + 1] = acc[0][3];
    }
    __syncthreads();
    for (int o = tid; o < kRows * k_pad; o += kThreads) {
      const int r = o / k_pad, j = o % k_pad, nt = j >> 3;
      double t = 0.0;
      for (int w = 0; w < WPN; ++w) t += s_part[w * NT + nt][r * 8 + (j & 7)];
      slot[r * k_pad + j] = t;
    }
  }
  __threadfence();                                   // the slot before the count
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(ly.counts + rgroup, 1) == ly.ranges - 1) ? 1 : 0;
  __syncthreads();
  if (s_last == 0) return;

  // ---- the last CTA of the row group: T = sum of the ranges (range order) -> MXINT8 along the rank -> Xcat
  __threadfence();
  const double* slots0 = ly.slots + (size_t)rgroup * ly.ranges * kRows * k_pad;
  const int n_out = kRows * k_pad;                   // a multiple of 32: 16 adjacent lanes hold one block
  for (int o = tid; o < n_out; o += kThreads) {
    const int r = o / k_pad, j = o % k_pad;
    double part[16];                                 // at most 16 ranges: all loads in flight, then the sum in range order
#pragma unroll
    for (int c = 0; c < 16; ++c) part[c] = c < ly.ranges ? __ldcg(slots0 + (size_t)c * n_out + o) : 0.0;
    double t = 0.0;
#pragma unroll
    for (int c = 0; c < 16; ++c) t += part[c];
    double amax = (t != t) ? 0.0 : fabs(t);
#pragma unroll
    for (int sft = 1; sft < 16; sft <<= 1) amax = fmax(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, sft));
    const int e = block_exponent(amax, p.exp_min, p.exp_max);
    const int q = quant_mantissa(t, e, p.a_bits);
    const int row = row0 + r;
    if (p.frag) {
      const size_t off = frag_offset(r, ly.K64 / 64 + (j >> 6), j & 63, plane);
      if (LQER_IN_BOUNDS(p.status, off, 2, ly.xcat_extent, 313))
        *reinterpret_cast<uint16_t*>(reinterpret_cast<uint8_t*>(ly.xcat) + off) = row < M ? (uint16_t)bf16_bits_of(q, e - (p.a_bits - 2)) : (uint16_t)0;
    }
    if (row < M && (p.frag || LQER_IN_BOUNDS(p.status, ((size_t)row * ldx + ly.K64 + j) * 2, 2, ly.xcat_extent, 313))) {
      if (!p.frag) ly.xcat[(size_t)row * ldx + ly.K64 + j] = (uint16_t)bf16_bits_of(q, e - (p.a_bits - 2));
      if (ly.Tm != nullptr) ly.Tm[(size_t)row * k_pad + j] = (int8_t)q;
      if (ly.Te != nullptr && (j & 15) == 0) ly.Te[(size_t)row * (k_pad / 16) + (j >> 4)] = (uint8_t)(e + 127);
    }
  }
  if (p.frag) {
    // rank indices between k_pad and the end of the last rank slab: zeros (the GEMM multiplies them with zero weights)
    const int pad = ((k_pad + 63) / 64) * 64 - k_pad;
    for (int o = tid; o < kRows * pad; o += kThreads) {
      const int r = o / pad, j = k_pad + o % pad;
      const size_t off = frag_offset(r, ly.K64 / 64 + (j >> 6), j & 63, plane);
      if (LQER_IN_BOUNDS(p.status, off, 2, ly.xcat_extent, 314)) *reinterpret_cast<uint16_t*>(reinterpret_cast<uint8_t*>(ly.xcat) + off) = 0;
    }
    __threadfence();                                 // T_q before its flag
    __syncthreads();
    if (tid == 0) atomicExch(ly.flags + 1, p.epoch);
  }
  if (tid == 0) ly.counts[rgroup] = 0;               // zero again for the next call
}

}  // namespace psm

int prologue_small_max_layers() { return psm::kMaxLayers; }

cudaError_t launch_prologue_small(const SmallPrologueLayer* layers, int n, int M, int x_type, bool frag_order, int epoch,
                                  DeviceStatus* st, cudaStream_t s) {
  using namespace psm;
  if (n < 1 || n > kMaxLayers || M < 1 || (frag_order && M > 16)) return cudaErrorInvalidValue;
  Params p;
  p.frag = frag_order ? 1 : 0;
  p.epoch = epoch;
  p.n = n;
  p.M = M;
  p.x_type = x_type;
  const PackedMeta& m0 = *layers[0].meta;
  p.status = st;
  p.a_bits = m0.a_bits; p.lr_bits = m0.lr_bits; p.exp_min = m0.exp_min; p.exp_max = m0.exp_max;
  const int rgroups = (M + kRows - 1) / kRows;
  int begin = 0, max_kpad = 0;
  for (int i = 0; i < kMaxLayers; ++i) {
    const SmallPrologueLayer& src = layers[i < n ? i : 0];
    const PackedMeta& m = *src.meta;
    if (m.a_bits != p.a_bits || m.lr_bits != p.lr_bits || m.exp_min != p.exp_min || m.exp_max != p.exp_max)
      return cudaErrorInvalidValue;
    Layer& ly = p.L[i];
    ly.X = src.X;
    ly.asec = static_cast<const uint8_t*>(src.packed) + m.off_a;
    ly.xcat = static_cast<uint16_t*>(src.xcat);
    ly.slots = src.slots;
    ly.xcat_extent = frag_order ? frag_bytes(m) : (size_t)M * xcat_cols(m) * 2;
    ly.slots_extent = prologue_small_slot_bytes(m, M);
    ly.counts = src.counts;
    ly.flags = src.flags;
    ly.Tm = src.Tm; ly.Te = src.Te;
    ly.K = m.K; ly.K64 = m.K64; ly.k = m.k; ly.k_pad = m.k_pad;
    ly.ranges = prologue_small_ranges(m, M);
    ly.cta_begin = begin;
    if (i < n) {
      begin += rgroups * ly.ranges;
      if (m.k_pad > max_kpad) max_kpad = m.k_pad;
    }
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(begin);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  LaunchScope scope(kFamPrologue, s);
  if (max_kpad <= 64) return cudaLaunchKernelEx(&cfg, prologue_small_kernel<1>, p);
  if (max_kpad <= 128) return cudaLaunchKernelEx(&cfg, prologue_small_kernel<2>, p);
  return cudaLaunchKernelEx(&cfg, prologue_small_kernel<4>, p);
}

}  // namespace lqer
