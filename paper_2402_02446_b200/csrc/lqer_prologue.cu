// Activation prologue of the prefill path (paper Section 4.1: X_q in MXINT8, blocks [1,16];
// Section 3.1: the small high-precision product X A_k):
//   X fp32 -> per 16-block shared exponent + 8-bit mantissas (128-bit loads, 4 lanes per
//   block, two shuffle steps for the maximum), written as the exactly representable bf16
//   value m * 2^(e-6) into Xcat[:, 0:K64];
//   T = X_q A_q: one int8 tensor-core MMA (m16n8k16, exact int32) per 16-block, each block
//   result scaled by 2^(e_x + e_a) and summed in fp64 (exact for any realistic exponent
//   spread, so the re-quantisation below takes the same decisions as an fp64 reference);
//   T -> MXINT8 along the rank, appended to Xcat[:, K64:K64+k_pad].
// A CTA owns 16 rows of X and walks K in steps; the global loads of step s+1 are in flight
// while the MMAs of step s run.
#include "lqer_common.cuh"

namespace lqer {

constexpr int kRows = 16;       // rows of X per CTA = one MMA M tile
constexpr int kThreads = 256;
constexpr int kXqStride = 528;  // bytes per row of the int8 panel (512 + 16: conflict-free fragment loads)
constexpr int kPanelBytes = 1024 * 17;   // A_q panel: PB blocks x k_pad columns x (16 mantissas + 1 exponent)

// Stand-alone activation quantiser (export for bit-exact comparison).  One lane per float4.
__global__ void __launch_bounds__(256) quantize_x_kernel(const float* __restrict__ X, int M, int K, int bits,
                                                         int emin, int emax, int8_t* __restrict__ Xm,
                                                         uint8_t* __restrict__ Xe) {
  const size_t total4 = (size_t)M * (K / 4);
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  // every lane of a warp runs the same number of iterations (shuffles need all 32)
  const size_t iters = (total4 + stride - 1) / stride;
  for (size_t it = 0; it < iters; ++it) {
    const size_t idx = it * stride + (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool ok = idx < total4;
    const float4 v = ok ? reinterpret_cast<const float4*>(X)[idx] : make_float4(0.f, 0.f, 0.f, 0.f);
    int e;
    uint32_t m8;
    uint2 bf;
    quantize_quad(v, bits, emin, emax, e, m8, bf);
    if (ok) {
      if (Xm != nullptr) reinterpret_cast<uint32_t*>(Xm)[idx] = m8;
      if (Xe != nullptr && (idx & 3) == 0) Xe[idx >> 2] = (uint8_t)(e + 127);
    }
  }
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Read a double from the same shared-memory offset in another CTA of the cluster.
__device__ __forceinline__ double ld_dsmem_f64(const double* local, uint32_t cta) {
  uint32_t remote;
  double v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"((uint32_t)__cvta_generic_to_shared(local)), "r"(cta));
  asm volatile("ld.shared::cluster.f64 %0, [%1];" : "=d"(v) : "r"(remote) : "memory");
  return v;
}

// PB = 16-blocks of K per step; PB * k_pad <= 1024.  A cluster of CS CTAs shares 16 rows: CTA r
// takes the K steps s = r, r + CS, ...; the partial T sums meet through distributed shared memory.
// TPW = rank tiles one warp can own (1 for ranks up to 64): fewer accumulators, more CTAs per SM.
template <int PB, int TPW>
__global__ void __launch_bounds__(kThreads, TPW == 1 ? 3 : 2) prologue_kernel(const void* __restrict__ X, int x_type, int M, PackedMeta m,
                                                               const uint8_t* __restrict__ asec,
                                                               uint16_t* __restrict__ xcat,
                                                               int8_t* __restrict__ Tm, uint8_t* __restrict__ Te,
                                                               DeviceStatus* status) {
  constexpr int SW = PB * 16;                     // columns per step
  [[maybe_unused]] const size_t xcat_extent = (size_t)M * ((size_t)m.K64 + m.k_pad) * 2;   // bytes behind xcat, for the checked build
  constexpr int F4 = kRows * SW / 4 / kThreads;   // float4 per thread per step (PB / 4)
  __shared__ __align__(16) uint8_t s_xq[kRows * kXqStride];
  __shared__ int8_t s_xe[kRows][32];
  __shared__ __align__(16) uint8_t s_panel[2][kPanelBytes];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, tig = lane & 3;
  const int CS = (int)cluster_nctarank(), crank = (int)cluster_ctarank();
  const int row0 = (blockIdx.x / CS) * kRows;
  const size_t ldx = xcat_cols(m);
  const int kblocks = m.K / 16;
  const int steps = (m.K64 + SW - 1) / SW;
  const uint8_t* a_exp = asec + (size_t)kblocks * m.k_pad * 16;
  const int NT = m.k_pad / 8;                     // 8-column rank tiles
  const int WPN = NT >= 8 ? 1 : 8 / NT;           // warps that share one rank tile (they split the blocks)
  const bool has_rank = m.k > 0;
  const bool active = has_rank && (NT >= 8 || warp < NT * WPN);

  double acc[TPW][4];
#pragma unroll
  for (int i = 0; i < TPW; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0;

  float4 xr[F4];
  auto load_x = [&](int s) {
#pragma unroll
    for (int i = 0; i < F4; ++i) {
      const int f = tid + i * kThreads;
      const int r = f / (SW / 4), c4 = f % (SW / 4);
      const int col = s * SW + c4 * 4, row = row0 + r;
      xr[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (row < M && col < m.K) xr[i] = load_x_quad(X, x_type, M, m.K, row, col, m.a_bits, m.exp_min, m.exp_max);
    }
  };
  auto load_panel = [&](int s, int buf) {
    const int kb0 = s * PB;
    const int nblk = min(PB, kblocks - kb0);
    if (nblk > 0) {
      const int mant16 = nblk * m.k_pad;          // 16-byte units of mantissas
      const int exp16 = nblk * m.k_pad / 16;      // 16-byte units of exponents
      const uint8_t* gm = asec + (size_t)kb0 * m.k_pad * 16;
      const uint8_t* ge = a_exp + (size_t)kb0 * m.k_pad;
      for (int u = tid; u < mant16; u += kThreads) cp_async16(&s_panel[buf][u * 16], gm + (size_t)u * 16);
      for (int u = tid; u < exp16; u += kThreads) cp_async16(&s_panel[buf][PB * m.k_pad * 16 + u * 16], ge + (size_t)u * 16);
    }
  };

  if (crank < steps) {
    load_x(crank);
    if (has_rank) load_panel(crank, 0);
  }
  cp_async_commit();

  int buf = 0;
  for (int s = crank; s < steps; s += CS, buf ^= 1) {
    // ---- quantise the panel held in registers: Xcat (bf16) to global, int8 + exponents to shared
#pragma unroll
    for (int i = 0; i < F4; ++i) {
      const int f = tid + i * kThreads;
      const int r = f / (SW / 4), c4 = f % (SW / 4);
      const int col = s * SW + c4 * 4, row = row0 + r;
      int e;
      uint32_t m8;
      uint2 bf;
      quantize_quad(xr[i], m.a_bits, m.exp_min, m.exp_max, e, m8, bf);
      *reinterpret_cast<uint32_t*>(&s_xq[r * kXqStride + c4 * 4]) = m8;
      if ((c4 & 3) == 0) s_xe[r][c4 >> 2] = (int8_t)e;
      if (row < M && col < m.K64 && LQER_IN_BOUNDS(status, ((size_t)row * ldx + col) * 2, 8, xcat_extent, 321))
        *reinterpret_cast<uint2*>(xcat + (size_t)row * ldx + col) = bf;
    }
    // ---- next step's loads fly while this step's MMAs run
    if (s + CS < steps) {
      load_x(s + CS);
      if (has_rank) load_panel(s + CS, buf ^ 1);
    }
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();

    if (active) {
      const uint8_t* panel = s_panel[buf];
      const uint8_t* pexp = panel + PB * m.k_pad * 16;
      const int nblk = min(PB, kblocks - s * PB);
      const int b_first = NT >= 8 ? 0 : warp / NT;
      const int b_step = NT >= 8 ? 1 : WPN;
      const int nt0 = NT >= 8 ? warp : warp % NT;
      const int bias = -127 - (m.a_bits - 2) - (m.lr_bits - 2);   // exponent bytes carry +127
      for (int b = b_first; b < nblk; b += b_step) {
        const uint32_t a0 = *reinterpret_cast<const uint32_t*>(&s_xq[g * kXqStride + b * 16 + tig * 4]);
        const uint32_t a1 = *reinterpret_cast<const uint32_t*>(&s_xq[(g + 8) * kXqStride + b * 16 + tig * 4]);
        const int ex0 = s_xe[g][b] + bias, ex1 = s_xe[g + 8][b] + bias;
#pragma unroll
        for (int i = 0; i < TPW; ++i) {
          const int nt = nt0 + 8 * i;
          if (nt < NT) {
            const int j = nt * 8 + g;
            const uint32_t b0 = *reinterpret_cast<const uint32_t*>(panel + ((size_t)(b * m.k_pad + j) * 16) + tig * 4);
            const uint32_t ea2 = *reinterpret_cast<const uint16_t*>(pexp + b * m.k_pad + nt * 8 + tig * 2);
            int c[4];
            mma_s8(c, a0, a1, b0);
            const int ea_lo = (int)(ea2 & 0xFFu), ea_hi = (int)(ea2 >> 8);
            acc[i][0] = fma((double)c[0], pow2d(ex0 + ea_lo), acc[i][0]);
            acc[i][1] = fma((double)c[1], pow2d(ex0 + ea_hi), acc[i][1]);
            acc[i][2] = fma((double)c[2], pow2d(ex1 + ea_lo), acc[i][2]);
            acc[i][3] = fma((double)c[3], pow2d(ex1 + ea_hi), acc[i][3]);
          }
        }
      }
    }
    __syncthreads();
  }

  if (!has_rank) return;       // uniform over the cluster: nobody reaches the cluster barriers below
  // ---- partial sums of this CTA's warps -> shared memory
  cp_async_wait<0>();
  double* tpart = reinterpret_cast<double*>(&s_panel[0][0]);      // [WPN][16][k_pad]
  const int n_out = kRows * m.k_pad;
  if (active) {
    const int slot = NT >= 8 ? 0 : warp / NT;
    const int nt0 = NT >= 8 ? warp : warp % NT;
#pragma unroll
    for (int i = 0; i < TPW; ++i) {
      const int nt = nt0 + 8 * i;
      if (nt < NT) {
        double* base = tpart + (size_t)slot * n_out;
        base[g * m.k_pad + nt * 8 + tig * 2] = acc[i][0];
        base[g * m.k_pad + nt * 8 + tig * 2 + 1] = acc[i][1];
        base[(g + 8) * m.k_pad + nt * 8 + tig * 2] = acc[i][2];
        base[(g + 8) * m.k_pad + nt * 8 + tig * 2 + 1] = acc[i][3];
      }
    }
  }
  cluster_sync();
  // ---- CTA r finishes rows [r * 16/CS, (r+1) * 16/CS): sum over CTAs and warps in a fixed order,
  //      re-quantise along the rank (16 adjacent lanes hold one block), append to Xcat
  const int rows_per = kRows / CS;
  const int n_mine = rows_per * m.k_pad;           // multiple of 32
  for (int o = tid; o < n_mine; o += kThreads) {
    const int r = crank * rows_per + o / m.k_pad, j = o % m.k_pad;
    double t = 0.0;
    for (int c = 0; c < CS; ++c)
      for (int w = 0; w < WPN; ++w) t += ld_dsmem_f64(tpart + (size_t)w * n_out + r * m.k_pad + j, (uint32_t)c);
    double amax = (t != t) ? 0.0 : fabs(t);
#pragma unroll
    for (int sft = 1; sft < 16; sft <<= 1) amax = fmax(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, sft));
    const int e = block_exponent(amax, m.exp_min, m.exp_max);
    const int q = quant_mantissa(t, e, m.a_bits);
    const int row = row0 + r;
    if (row < M && LQER_IN_BOUNDS(status, ((size_t)row * ldx + m.K64 + j) * 2, 2, xcat_extent, 322)) {
      xcat[(size_t)row * ldx + m.K64 + j] = (uint16_t)bf16_bits_of(q, e - (m.a_bits - 2));
      if (Tm != nullptr) Tm[(size_t)row * m.k_pad + j] = (int8_t)q;
      if (Te != nullptr && (j & 15) == 0) Te[(size_t)row * (m.k_pad / 16) + (j >> 4)] = (uint8_t)(e + 127);
    }
  }
  cluster_sync();              // no CTA leaves while its shared memory may still be read
}

cudaError_t launch_quantize_x(const float* X, int M, int K, int bits, int emin, int emax, int8_t* Xm,
                              uint8_t* Xe, cudaStream_t s) {
  const size_t total4 = (size_t)M * (K / 4);
  int blocks = (int)((total4 + 255) / 256);
  if (blocks > sm_count() * 16) blocks = sm_count() * 16;
  if (blocks < 1) blocks = 1;
  LaunchScope scope(kFamQuantize, s);
  quantize_x_kernel<<<blocks, 256, 0, s>>>(X, M, K, bits, emin, emax, Xm, Xe);
  return cudaGetLastError();
}

template <int PB, int TPW>
static cudaError_t launch_prologue_pb(const void* X, int x_type, int M, const PackedMeta& m, const uint8_t* asec, uint16_t* xc,
                                      int8_t* Tm, uint8_t* Te, DeviceStatus* st, cudaStream_t s) {
  const int groups = (M + kRows - 1) / kRows;
  const int steps = (m.K64 + PB * 16 - 1) / (PB * 16);
  int cs = 1;
  while (cs < 8 && groups * cs < 2 * sm_count() && cs * 2 <= steps) cs *= 2;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(groups * cs);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  LaunchScope scope(kFamPrologue, s);
  return cudaLaunchKernelEx(&cfg, prologue_kernel<PB, TPW>, X, x_type, M, m, asec, xc, Tm, Te, st);
}

cudaError_t launch_prologue(const void* X, int x_type, int M, const PackedMeta& m, const void* packed, void* xcat,
                            int8_t* Tm, uint8_t* Te, DeviceStatus* st, cudaStream_t s) {
  const uint8_t* asec = static_cast<const uint8_t*>(packed) + m.off_a;
  uint16_t* xc = static_cast<uint16_t*>(xcat);
  if (m.k_pad <= 64) return launch_prologue_pb<16, 1>(X, x_type, M, m, asec, xc, Tm, Te, st, s);
  if (m.k_pad <= 128) return launch_prologue_pb<8, 2>(X, x_type, M, m, asec, xc, Tm, Te, st, s);
  return launch_prologue_pb<4, 4>(X, x_type, M, m, asec, xc, Tm, Te, st, s);
}

}  // namespace lqer
