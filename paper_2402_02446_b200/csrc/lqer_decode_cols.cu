// Decode form of the layer for M <= 4 tokens (paper Section 3.1 / 3.2; Section 2.1: small-batch
// inference is memory bound):
//
//     Y[M,N] = X_q W_q + q(X_q A_q) B_q
//
// With so few tokens a tensor-core MMA would spend 16 rows of work on at most 4, and a split of K
// across CTAs would end in a round trip through global memory (slots, a fence, an arrival
// counter) that costs more than streaming the weights.  So here a CTA owns output columns and
// the whole contraction for them: groups of 8 columns are dealt out to the CTAs in contiguous
// ranges, four groups per round; within a round warp w takes the slabs (64 K) w, w + 16, ... of
// those groups, and the 16 warps' sums meet once in shared memory and are added in warp order.
// Y is written once, by one thread per element, with no global synchronisation.
//
// Lane (g, t) of a warp keeps, for column g of a group, the exact integer dot product of block t
// of the slab: four dp4a on the raw nibbles against the int8 mantissas of X (stored in the byte
// order the nibbles unpack to), minus 8 * sum(x) for the offset-binary nibbles; the block result
// is scaled by 2^(e_x + e_w) in fp32 and accumulated per token.  A warp's share of a unit (256
// bytes of nibbles + 32 exponent bytes) goes global -> registers, four slabs (16 units) ahead;
// these loads depend on no earlier kernel and are issued before griddepcontrol.wait.
//
// T = X_q A_q: every CTA adds the exact partial products of its share of K (int8 tensor-core MMA
// per 16-block, scaled in fp64) to an accumulator in the workspace at kernel start; before its
// rank part each CTA waits (bounded) until all G contributions have arrived and re-quantises T.
#include "lqer_common.cuh"

namespace lqer {
namespace dcol {

constexpr int kWarps = 16;
constexpr int kThreads = kWarps * 32;
constexpr int kMaxM = 4;
constexpr int kCg = 4;            // column groups (of 8 columns) per round
constexpr int kSets = 4;          // slabs a warp keeps in flight (x kCg units each)
constexpr long long kWaitLimitCycles = 4000000000LL;

struct Params {
  const float* X;
  float* Y;
  const uint8_t* wsec;
  const uint8_t* bsec;
  const uint8_t* asec;
  DeviceStatus* status;
  int* tcount;          // CTAs whose T contribution has arrived
  int* tdone;           // CTAs that no longer need the T accumulator
  double* tacc;         // [16][k_pad] T accumulator (all zero between calls)
  int M, K, N, K64, k_pad, k_slabs, r_blocks, n_cg;
  int a_bits, lr_bits, exp_min, exp_max;
};

struct UnitRegs {
  uint2 w;      // block t of the slab for column g: 16 nibbles
  uint32_t e;   // its exponent byte
};

__device__ __forceinline__ uint32_t ld_stream_u32(const void* p) {
  uint32_t v;
  asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ uint2 ld_stream_u64(const void* p) {
  uint2 v;
  asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t ld_stream_u8(const void* p) {
  uint32_t v;
  asm volatile("ld.global.nc.L1::no_allocate.u8 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// The T accumulator is released by every CTA once; the last one leaves it zero for the next call.
__device__ __noinline__ void release_tacc(const Params& p, int* flags) {
  const int tid = threadIdx.x, G = gridDim.x;
  if (tid == 0) flags[1] = (atomicAdd(p.tdone, 1) == G - 1) ? 1 : 0;
  __syncthreads();
  if (flags[1] != 0) {
    __threadfence();
    for (int o = tid; o < 16 * p.k_pad; o += kThreads) p.tacc[o] = 0.0;
    if (tid == 0) { *p.tcount = 0; *p.tdone = 0; }
  }
}

// T -> T_q as int8 mantissas [M][k_pad] and block scales 2^(e - 6) [M][k_pad / 16] in shared memory.
__device__ __noinline__ void build_tq(const Params& p, int* flags, int8_t* tq8, float* tqs) {
  const int tid = threadIdx.x, G = gridDim.x, M = p.M;
  if (tid == 0) {                                // bounded wait for the contributions of all CTAs
    const long long t0 = clock64();
    while (ld_acquire(p.tcount) < G) {
      __nanosleep(64);
      if (clock64() - t0 > kWaitLimitCycles) { flags[0] = 1; break; }
    }
  }
  __syncthreads();
  __threadfence();
  const int total = M * p.k_pad;                 // 16 adjacent lanes hold one block
  for (int base = 0; base < total; base += kThreads) {
    const int idx = base + tid;
    const bool valid = idx < total;
    const int row = valid ? idx / p.k_pad : 0, col = valid ? idx % p.k_pad : 0;
    const double tv = valid ? __ldcg(p.tacc + (size_t)row * p.k_pad + col) : 0.0;
    double amax = (tv != tv) ? 0.0 : fabs(tv);
#pragma unroll
    for (int sft = 1; sft < 16; sft <<= 1) amax = fmax(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, sft));
    const int e = block_exponent(amax, p.exp_min, p.exp_max);
    const int qv = quant_mantissa(tv, e, p.a_bits);
    if (valid) {
      tq8[row * p.k_pad + col] = (int8_t)qv;
      if ((col & 15) == 0) tqs[row * (p.k_pad / 16) + (col >> 4)] = pow2f(e - (p.a_bits - 2));
    }
  }
  __syncthreads();
  release_tacc(p, flags);
}

__global__ void __launch_bounds__(kThreads, 1) decode_cols_kernel(const __grid_constant__ Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
  const int M = p.M, KB = p.K64 / 16;
  uint8_t* xm = smem;                                               // [M][K64] int8 mantissas, permuted within 8
  float* xsc = reinterpret_cast<float*>(xm + (size_t)M * p.K64);    // [M][KB] 2^(e_x - 6)
  int* xof = reinterpret_cast<int*>(xsc + (size_t)M * KB);          // [M][KB] 8 * sum(x) of the block
  float* red = reinterpret_cast<float*>(xof + (size_t)M * KB);      // [kWarps][kCg][8][kMaxM]
  float* tqs = red + kWarps * kCg * 8 * kMaxM;                      // [M][k_pad / 16]
  int* flags = reinterpret_cast<int*>(tqs + kMaxM * 16);            // [0] a bounded wait ran out, [1] broadcast
  int8_t* tq8 = reinterpret_cast<int8_t*>(flags + 4);               // [M][k_pad]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int G = gridDim.x, cta = blockIdx.x;
  const int cg_lo = cta * p.n_cg / G, cg_hi = (cta + 1) * p.n_cg / G;

  // this lane's share of (column group cg, slab j): global -> registers
  auto fetch = [&](UnitRegs& d, int cg, int j) {
    d.w = make_uint2(0x88888888u, 0x88888888u);  // mantissa 0 in offset binary
    d.e = 127u;
    if (cg < cg_hi && j < p.k_slabs) {
      const int col = (cg & 15) * 8 + g;
      const uint8_t* tile = p.wsec + ((size_t)(cg >> 4) * p.k_slabs + j) * kWTileBytes;
      d.w = ld_stream_u64(tile + (t >> 1) * (kTileN * 16) + col * 16 + (t & 1) * 8);
      d.e = ld_stream_u8(tile + kWTileNibbleBytes + col * 4 + t);
    }
  };

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (tid < 4) flags[tid] = 0;

  UnitRegs regs[kSets][kCg];
  // weights depend on no earlier kernel: request the first slabs before the dependency wait
#pragma unroll
  for (int s = 0; s < kSets; ++s)
#pragma unroll
    for (int u = 0; u < kCg; ++u) fetch(regs[s][u], cg_lo + u, warp + kWarps * s);

  asm volatile("griddepcontrol.wait;" ::: "memory");   // X (and the workspace) may be an earlier kernel's output

  // ---- this CTA's share of T = X_q A_q: exact int8 MMA per (16-block of K, 8 rank columns), scaled in
  //      fp64 and added to the accumulator in the workspace (exact products; their fp64 sum is exact as
  //      well unless the block exponents of one row spread over more than about 30 binades)
  if (p.k_pad > 0) {
    const int KBr = p.K / 16, NT = p.k_pad / 8;
    const int kb_lo = cta * KBr / G, kb_hi = (cta + 1) * KBr / G;
    const uint8_t* a_exp = p.asec + (size_t)KBr * p.k_pad * 16;
    const int bias = -127 - (p.a_bits - 2) - (p.lr_bits - 2);       // exponent bytes carry +127
    const int items = (kb_hi - kb_lo) * NT;
    for (int it = warp; it < items; it += kWarps) {
      const int kb = kb_lo + it / NT, nt = it % NT;
      const float4 v0 = g < M ? __ldg(reinterpret_cast<const float4*>(p.X + (size_t)g * p.K + kb * 16 + t * 4))
                              : make_float4(0.f, 0.f, 0.f, 0.f);
      const uint32_t b0 = __ldg(reinterpret_cast<const uint32_t*>(p.asec + ((size_t)kb * p.k_pad + nt * 8 + g) * 16 + t * 4));
      const uint32_t ea2 = __ldg(reinterpret_cast<const uint16_t*>(a_exp + (size_t)kb * p.k_pad + nt * 8 + t * 2));
      int e0;
      uint32_t m0;
      uint2 unused;
      quantize_quad(v0, p.a_bits, p.exp_min, p.exp_max, e0, m0, unused);
      int c[4];
      mma_s8(c, m0, 0u, b0);
      const int tc = nt * 8 + t * 2;
      if (g < M) {
        atomicAdd(p.tacc + (size_t)g * p.k_pad + tc, (double)c[0] * pow2d(e0 + (int)(ea2 & 0xFFu) + bias));
        atomicAdd(p.tacc + (size_t)g * p.k_pad + tc + 1, (double)c[1] * pow2d(e0 + (int)(ea2 >> 8) + bias));
      }
    }
  }

  // ---- X -> MXINT8 for the whole contraction: per row the mantissas in the byte order the nibbles
  //      unpack to ({0,4,1,5}, {2,6,3,7} within each 8), the block scales and the offsets 8 * sum(x)
  {
    const int per_row = p.K64 / 4, total = M * per_row;             // float4 items: (row, quarter-block)
    for (int base = 0; base < total; base += kThreads) {
      const int item = base + tid;
      const bool valid = item < total;
      const int row = valid ? item / per_row : 0, c4 = valid ? item % per_row : 0;
      const float4 v = (valid && c4 * 4 < p.K) ? __ldg(reinterpret_cast<const float4*>(p.X + (size_t)row * p.K + c4 * 4))
                                               : make_float4(0.f, 0.f, 0.f, 0.f);
      int e;
      uint32_t m8;
      uint2 unused;
      quantize_quad(v, p.a_bits, p.exp_min, p.exp_max, e, m8, unused);
      const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, m8, 1);
      const uint32_t perm = (c4 & 1) ? __byte_perm(other, m8, 0x7362) : __byte_perm(m8, other, 0x5140);
      int sum = __dp4a((int)m8, 0x01010101, 0);
      sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 1);
      sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 2);
      if (valid) {
        *reinterpret_cast<uint32_t*>(xm + (size_t)row * p.K64 + c4 * 4) = perm;
        if ((c4 & 3) == 0) {
          xsc[row * KB + (c4 >> 2)] = pow2f(e - (p.a_bits - 2));
          xof[row * KB + (c4 >> 2)] = 8 * sum;
        }
      }
    }
  }
  __syncthreads();
  if (tid == 0 && p.k_pad > 0)                   // the T contributions of this CTA are out (ordered by the barrier)
    asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(p.tcount) : "memory");

  bool tq_built = false;
  const int slabs_mine = p.k_slabs > warp ? (p.k_slabs - warp + kWarps - 1) / kWarps : 0;   // slabs warp, warp + 16, ...
#pragma unroll 1
  for (int cg0 = cg_lo; cg0 < cg_hi; cg0 += kCg) {
    if (cg0 != cg_lo) {
#pragma unroll
      for (int s = 0; s < kSets; ++s)
#pragma unroll
        for (int u = 0; u < kCg; ++u) fetch(regs[s][u], cg0 + u, warp + kWarps * s);
    }
    float acc[kCg][kMaxM];
#pragma unroll
    for (int u = 0; u < kCg; ++u)
#pragma unroll
      for (int r = 0; r < kMaxM; ++r) acc[u][r] = 0.f;

    // ---- W_q: this warp's slabs of the round's column groups
#pragma unroll 1
    for (int js = 0; js < slabs_mine; js += kSets) {
#pragma unroll
      for (int s = 0; s < kSets; ++s) {
        const int j = warp + kWarps * (js + s);
        if (j < p.k_slabs) {
#pragma unroll
          for (int r = 0; r < kMaxM; ++r) {
            if (r < M) {
              const uint4 x = *reinterpret_cast<const uint4*>(xm + (size_t)r * p.K64 + j * 64 + t * 16);
              const float sx = xsc[r * KB + j * 4 + t];
              const int off = xof[r * KB + j * 4 + t];
#pragma unroll
              for (int u = 0; u < kCg; ++u) {
                const UnitRegs d = regs[s][u];
                // nibbles as bytes: k {0,4,1,5}, {2,6,3,7}, {8,12,9,13}, {10,14,11,15} of the block
                int sm = __dp4a((int)x.x, (int)(d.w.x & 0x0F0F0F0Fu), -off);
                sm = __dp4a((int)x.y, (int)((d.w.x >> 4) & 0x0F0F0F0Fu), sm);
                sm = __dp4a((int)x.z, (int)(d.w.y & 0x0F0F0F0Fu), sm);
                sm = __dp4a((int)x.w, (int)((d.w.y >> 4) & 0x0F0F0F0Fu), sm);
                acc[u][r] = fmaf((float)sm, sx * __uint_as_float((d.e - 2u) << 23), acc[u][r]);   // 2^(e_x - 6) 2^(e_w - 2)
              }
            }
          }
        }
#pragma unroll
        for (int u = 0; u < kCg; ++u) fetch(regs[s][u], cg0 + u, j + kWarps * kSets);
      }
    }

    // ---- B_q against T_q: rank blocks warp, warp + 16, ...
    if (p.k_pad > 0) {
      if (!tq_built) { build_tq(p, flags, tq8, tqs); tq_built = true; }
      const int rbn = p.k_pad / 16;
      for (int rb = warp; rb < p.r_blocks; rb += kWarps) {
#pragma unroll
        for (int u = 0; u < kCg; ++u) {
          const int cg = cg0 + u;
          if (cg < cg_hi) {
            const int col = (cg & 15) * 8 + g;
            const uint8_t* tile = p.bsec + (size_t)(cg >> 4) * ((size_t)p.r_blocks * kTileN * 17);
            const uint32_t wv = ld_stream_u32(tile + ((size_t)rb * kTileN + col) * 16 + t * 4);
            const uint32_t eb = ld_stream_u8(tile + (size_t)p.r_blocks * kTileN * 16 + rb * kTileN + col);
            const float sb = __uint_as_float((eb - (uint32_t)(p.lr_bits - 2)) << 23);            // 2^(e_b - 6)
#pragma unroll
            for (int r = 0; r < kMaxM; ++r) {
              if (r < M) {
                const int tw = *reinterpret_cast<const int*>(tq8 + r * p.k_pad + rb * 16 + t * 4);
                acc[u][r] = fmaf((float)__dp4a(tw, (int)wv, 0), tqs[r * rbn + rb] * sb, acc[u][r]);
              }
            }
          }
        }
      }
    }

    // ---- the four lanes of a column, then the 16 warps (fixed order), then Y
#pragma unroll
    for (int u = 0; u < kCg; ++u) {
      float mine = 0.f;
#pragma unroll
      for (int r = 0; r < kMaxM; ++r) {
        float v = acc[u][r];
        v += __shfl_xor_sync(0xFFFFFFFFu, v, 1);
        v += __shfl_xor_sync(0xFFFFFFFFu, v, 2);
        if (r == t) mine = v;
      }
      red[((warp * kCg + u) * 8 + g) * kMaxM + t] = mine;          // lane t hands row t over
    }
    __syncthreads();
    if (tid < kCg * 8 * kMaxM) {
      const int u = tid >> 5, gg = (tid >> 2) & 7, r = tid & 3;
      float v = 0.f;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) v += red[((w * kCg + u) * 8 + gg) * kMaxM + r];
      const int cg = cg0 + u;
      if (cg < cg_hi && r < M) p.Y[(size_t)r * p.N + cg * 8 + gg] = v;
    }
    __syncthreads();                             // red is rewritten by the next round
  }
  if (p.k_pad > 0 && !tq_built) release_tacc(p, flags);
  if (flags[0] != 0 && tid == 0) report_error(p.status, LQER_ERR_TIMEOUT, 600, cta);
}

}  // namespace dcol

static size_t cols_smem_bytes(const PackedMeta& m, int M) {
  using namespace dcol;
  return (size_t)M * m.K64 + (size_t)M * (m.K64 / 16) * 8 + kWarps * kCg * 8 * kMaxM * 4 + kMaxM * 16 * 4 + 16 +
         (size_t)kMaxM * (m.k_pad > 0 ? m.k_pad : 16) + 256;
}
// The column-owner kernel serves M <= 4 as long as the quantised X of the whole contraction fits in shared memory.
bool decode_cols_fits(const PackedMeta& m, int M) { return M <= dcol::kMaxM && cols_smem_bytes(m, M) <= 200 * 1024; }

cudaError_t launch_decode_cols(const float* X, int M, const PackedMeta& m, const void* packed, float* Y, void* workspace,
                               cudaStream_t s) {
  using namespace dcol;
  static int sm_count = 0;
  static bool attr_set = false;
  if (!attr_set) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
    cudaError_t e = cudaFuncSetAttribute(decode_cols_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  Params p;
  const uint8_t* base = static_cast<const uint8_t*>(packed);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  p.X = X; p.Y = Y;
  p.wsec = base + m.off_w; p.bsec = base + m.off_b; p.asec = base + m.off_a;
  p.status = reinterpret_cast<DeviceStatus*>(ws);
  p.tcount = reinterpret_cast<int*>(ws + kTCountOffset);
  p.tdone = reinterpret_cast<int*>(ws + kTDoneOffset);
  p.tacc = reinterpret_cast<double*>(ws + tacc_offset(m));
  p.M = M; p.K = m.K; p.N = m.N; p.K64 = m.K64; p.k_pad = m.k_pad;
  p.k_slabs = m.k_slabs; p.r_blocks = m.r_blocks;
  p.n_cg = m.N / 8;
  p.a_bits = m.a_bits; p.lr_bits = m.lr_bits; p.exp_min = m.exp_min; p.exp_max = m.exp_max;
  int G = p.n_cg < sm_count ? p.n_cg : sm_count;
  if (G > kDecodeMaxCtas) G = kDecodeMaxCtas;
  const size_t smem = cols_smem_bytes(m, M);
  if (!decode_cols_fits(m, M)) return cudaErrorInvalidValue;

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(G);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may start while the previous kernel drains
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  LaunchScope scope(kFamDecode, s);
  return cudaLaunchKernelEx(&cfg, decode_cols_kernel, p);
}

}  // namespace lqer
