// Activation prologue of the prefill path (paper Section 4.1: X_q in MXINT8, blocks [1,16];
// Section 3.1: the small product X A_k):
//   X fp32 -> per 16-block shared exponent + 8-bit mantissas (128-bit loads, 4 lanes per
//   block, two shuffle steps for the maximum), written as the exactly representable bf16
//   value m * 2^(e-6) into Xcat[:, 0:K64];
//   T = X_q A_q by integer dot products per block (dp4a) scaled and summed in fp64, then
//   re-quantised to MXINT8 along the rank and written into Xcat[:, K64:K64+k_pad].
#include "lqer_common.cuh"

namespace lqer {

constexpr int kRows = 8;        // rows of X per CTA
constexpr int kChunk = 512;     // K columns per pass
constexpr int kThreads = 256;
constexpr int kMaxOut = 8;      // T outputs per thread: kRows * k_pad / kThreads <= 8  (k_pad <= 256)

// Quantise the four values a lane holds; the 16-block is spread over 4 adjacent lanes.
__device__ __forceinline__ void quantize_quad(const float4 v, int bits, int emin, int emax, int& e, int (&q)[4]) {
  float amax = fmaxf(fmaxf(abs_ignore_nan(v.x), abs_ignore_nan(v.y)), fmaxf(abs_ignore_nan(v.z), abs_ignore_nan(v.w)));
  amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
  amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
  e = block_exponent(amax, emin, emax);
  q[0] = quant_mantissa(v.x, e, bits);
  q[1] = quant_mantissa(v.y, e, bits);
  q[2] = quant_mantissa(v.z, e, bits);
  q[3] = quant_mantissa(v.w, e, bits);
}

__device__ __forceinline__ uint32_t pack4_i8(const int (&q)[4]) {
  return ((uint32_t)q[0] & 0xFFu) | (((uint32_t)q[1] & 0xFFu) << 8) | (((uint32_t)q[2] & 0xFFu) << 16) |
         (((uint32_t)q[3] & 0xFFu) << 24);
}

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
    int e, q[4];
    quantize_quad(v, bits, emin, emax, e, q);
    if (ok) {
      if (Xm != nullptr) reinterpret_cast<uint32_t*>(Xm)[idx] = pack4_i8(q);
      if (Xe != nullptr && (idx & 3) == 0) Xe[idx >> 2] = (uint8_t)(e + 127);
    }
  }
}

__global__ void __launch_bounds__(kThreads) prologue_kernel(const float* __restrict__ X, int M, PackedMeta m,
                                                            const uint8_t* __restrict__ asec,
                                                            uint16_t* __restrict__ xcat,
                                                            int8_t* __restrict__ Tm, uint8_t* __restrict__ Te) {
  __shared__ __align__(16) uint32_t s_xq[kRows][kChunk / 4];   // int8 mantissas, 4 per word
  __shared__ int s_xe[kRows][kChunk / 16];

  const int tid = threadIdx.x;
  const int row0 = blockIdx.x * kRows;
  const size_t ldx = xcat_cols(m);
  const int n_out = kRows * m.k_pad;
  const uint8_t* a_exp = asec + (size_t)(m.K / 16) * m.k_pad * 16;

  double acc[kMaxOut];
#pragma unroll
  for (int i = 0; i < kMaxOut; ++i) acc[i] = 0.0;

  for (int c0 = 0; c0 < m.K64; c0 += kChunk) {
    // ---- quantise a [kRows x kChunk] panel of X
#pragma unroll
    for (int i = 0; i < kRows * (kChunk / 4) / kThreads; ++i) {
      const int idx = tid + i * kThreads;
      const int r = idx / (kChunk / 4);
      const int c4 = idx % (kChunk / 4);
      const int col = c0 + c4 * 4;
      const int row = row0 + r;
      const bool in = (row < M) && (col < m.K);
      const float4 v = in ? *reinterpret_cast<const float4*>(X + (size_t)row * m.K + col)
                          : make_float4(0.f, 0.f, 0.f, 0.f);
      int e, q[4];
      quantize_quad(v, m.a_bits, m.exp_min, m.exp_max, e, q);
      s_xq[r][c4] = pack4_i8(q);
      if ((c4 & 3) == 0) s_xe[r][c4 >> 2] = e;
      if (row < M && col < m.K64) {
        const int p = e - (m.a_bits - 2);
        uint2 o;
        o.x = bf16_bits_of(q[0], p) | (bf16_bits_of(q[1], p) << 16);
        o.y = bf16_bits_of(q[2], p) | (bf16_bits_of(q[3], p) << 16);
        *reinterpret_cast<uint2*>(xcat + (size_t)row * ldx + col) = o;
      }
    }
    __syncthreads();
    // ---- T += X_q A_q over this panel: exact integer dot per 16-block, fp64 scaling and sum
    if (m.k > 0) {
      const int kb_end = min(kChunk / 16, (m.K - c0) / 16);
#pragma unroll
      for (int i = 0; i < kMaxOut; ++i) {
        const int o = tid + i * kThreads;
        if (o < n_out) {
          const int r = o / m.k_pad, j = o % m.k_pad;
          double a = acc[i];
          for (int kb = 0; kb < kb_end; ++kb) {
            const int kbg = c0 / 16 + kb;
            const uint4 xa = *reinterpret_cast<const uint4*>(&s_xq[r][kb * 4]);
            const uint4 aa = __ldg(reinterpret_cast<const uint4*>(asec + ((size_t)kbg * m.k_pad + j) * 16));
            int d = __dp4a((int)xa.x, (int)aa.x, 0);
            d = __dp4a((int)xa.y, (int)aa.y, d);
            d = __dp4a((int)xa.z, (int)aa.z, d);
            d = __dp4a((int)xa.w, (int)aa.w, d);
            const int ea = (int)__ldg(a_exp + (size_t)kbg * m.k_pad + j) - 127;
            a = fma((double)d, pow2d(s_xe[r][kb] + ea - (m.a_bits - 2) - (m.lr_bits - 2)), a);
          }
          acc[i] = a;
        }
      }
    }
    __syncthreads();
  }

  // ---- re-quantise T along the rank (16 adjacent lanes hold one block) and append to Xcat
  if (m.k > 0) {
#pragma unroll
    for (int i = 0; i < kMaxOut; ++i) {
      const int o = tid + i * kThreads;
      if (i * kThreads < n_out) {          // uniform over the warp: n_out is a multiple of 128
        const bool ok = o < n_out;
        const double t = ok ? acc[i] : 0.0;
        double amax = (t != t) ? 0.0 : fabs(t);
#pragma unroll
        for (int s = 1; s < 16; s <<= 1) amax = fmax(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, s));
        const int e = block_exponent(amax, m.exp_min, m.exp_max);
        const int q = quant_mantissa(t, e, m.a_bits);
        const int r = o / m.k_pad, j = o % m.k_pad;
        const int row = row0 + r;
        if (ok && row < M) {
          xcat[(size_t)row * ldx + m.K64 + j] = (uint16_t)bf16_bits_of(q, e - (m.a_bits - 2));
          if (Tm != nullptr) Tm[(size_t)row * m.k_pad + j] = (int8_t)q;
          if (Te != nullptr && (j & 15) == 0) Te[(size_t)row * (m.k_pad / 16) + (j >> 4)] = (uint8_t)(e + 127);
        }
      }
    }
  }
}

cudaError_t launch_quantize_x(const float* X, int M, int K, int bits, int emin, int emax, int8_t* Xm,
                              uint8_t* Xe, cudaStream_t s) {
  const size_t total4 = (size_t)M * (K / 4);
  int blocks = (int)((total4 + 255) / 256);
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  quantize_x_kernel<<<blocks, 256, 0, s>>>(X, M, K, bits, emin, emax, Xm, Xe);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_prologue(const float* X, int M, const PackedMeta& m, const void* packed, void* xcat,
                            int8_t* Tm, uint8_t* Te, DeviceStatus* st, cudaStream_t s) {
  (void)st;
  const uint8_t* asec = static_cast<const uint8_t*>(packed) + m.off_a;
  prologue_kernel<<<(M + kRows - 1) / kRows, kThreads, 0, s>>>(X, M, m, asec, static_cast<uint16_t*>(xcat), Tm, Te);
  count_launch();
  return cudaGetLastError();
}

}  // namespace lqer
