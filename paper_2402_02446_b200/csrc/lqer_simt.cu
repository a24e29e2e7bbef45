// Plain CUDA-core form of the concatenated contraction (paper Section 3.1 / 3.2):
//   Y = [X_q | T_q] . [W_q ; B_q]
// One thread per output element, fp32 accumulation of exact products.  It exists to check
// the packed layout and the prologue end to end on small shapes; it is never selected
// automatically.
#include "lqer_common.cuh"

namespace lqer {

__device__ __forceinline__ float bf16_to_float(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }

__global__ void __launch_bounds__(256) gemm_simt_kernel(const uint16_t* __restrict__ xcat, int M, PackedMeta m,
                                                        const uint8_t* __restrict__ wsec,
                                                        const uint8_t* __restrict__ bsec, float* __restrict__ Y) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  const int row = blockIdx.y;
  if (n >= m.N || row >= M) return;
  const int nt = n / kTileN, nl = n % kTileN;
  const size_t ldx = xcat_cols(m);
  const uint16_t* x = xcat + (size_t)row * ldx;
  const int pos[8] = {0, 4, 1, 5, 2, 6, 3, 7};
  float acc = 0.0f;
  for (int kb = 0; kb < m.K64 / 16; ++kb) {
    const int ks = kb / 4, blk = kb % 4;
    const uint8_t* tile = wsec + ((size_t)nt * m.k_slabs + ks) * w_tile_bytes(m.w_bits);
    const float scale = pow2f((int)tile[w_mant_bytes(m.w_bits) + nl * 4 + blk] - 127 - (m.w_bits - 2));
    if (m.w_bits == 2) {
      const uint32_t w = *reinterpret_cast<const uint32_t*>(tile + (size_t)nl * 16 + blk * 4);
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int mant = (int)((w >> (2 * (i >> 1) + 16 * (i & 1))) & 3u) - 1;
        acc = fmaf(bf16_to_float(x[kb * 16 + i]), (float)mant * scale, acc);
      }
    } else {
      const uint2 w2 = *reinterpret_cast<const uint2*>(tile + ((size_t)((blk >> 1) * kTileN + nl) * 16) + (blk & 1) * 8);
      const uint32_t w[2] = {w2.x, w2.y};
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int mant = (int)((w[i >> 3] >> (4 * pos[i & 7])) & 0xFu) - 8;
        acc = fmaf(bf16_to_float(x[kb * 16 + i]), (float)mant * scale, acc);
      }
    }
  }
  if (m.k > 0) {
    const uint8_t* tile = bsec + (size_t)nt * (m.r_blocks * kTileN * 17);
    for (int rb = 0; rb < m.r_blocks; ++rb) {
      const int8_t* bm = reinterpret_cast<const int8_t*>(tile + ((size_t)rb * kTileN + nl) * 16);
      const float scale = pow2f((int)tile[(size_t)m.r_blocks * kTileN * 16 + rb * kTileN + nl] - 127 - (m.lr_bits - 2));
#pragma unroll
      for (int i = 0; i < 16; ++i)
        acc = fmaf(bf16_to_float(x[m.K64 + rb * 16 + i]), (float)bm[i] * scale, acc);
    }
  }
  Y[(size_t)row * m.N + n] = acc;
}

cudaError_t launch_gemm_simt(const void* xcat, int M, const PackedMeta& m, const void* packed, float* Y,
                             cudaStream_t s) {
  const uint8_t* base = static_cast<const uint8_t*>(packed);
  LaunchScope scope(kFamGemmSimt, s);
  gemm_simt_kernel<<<dim3((m.N + 255) / 256, M), 256, 0, s>>>(static_cast<const uint16_t*>(xcat), M, m,
                                                              base + m.off_w, base + m.off_b, Y);
  return cudaGetLastError();
}

}  // namespace lqer
