// Weight preparation: W -> MXINT4, A_k / B_k -> MXINT8 (paper Section 3.1, formats of
// Section 4.1), written in the tile layout the GEMM and decode kernels read, and the
// canonical read-back used for bit-exact comparison.
#include "lqer_common.cuh"

namespace lqer {

__constant__ int c_nibble_pos[8] = {0, 4, 1, 5, 2, 6, 3, 7};  // k_local -> nibble position

// One thread = one (column n, 16-block of K) of W.  grid (n_tiles, k_slabs), block 128 x 4.
__global__ void __launch_bounds__(512) pack_w_kernel(const float* __restrict__ W, PackedMeta m,
                                                     uint8_t* __restrict__ wsec) {
  const int nt = blockIdx.x, ks = blockIdx.y;
  const int nl = threadIdx.x;            // column within the tile
  const int blk = threadIdx.y;           // 16-block within the slab (0..3)
  const int n = nt * kTileN + nl;
  const int k0 = ks * kSlabK + blk * 16;
  float v[16];
  float amax = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const int k = k0 + i;
    v[i] = (n < m.N && k < m.K) ? W[(size_t)k * m.N + n] : 0.0f;
    amax = fmaxf(amax, abs_ignore_nan(v[i]));
  }
  const int e = block_exponent(amax, m.w_exp_min, m.w_exp_max);
  uint8_t* tile = wsec + ((size_t)nt * m.k_slabs + ks) * w_tile_bytes(m.w_bits);
  if (m.w_bits == 2) {
    // one word per block: even k in the low half, odd k in the high half, offset-binary crumbs
    uint32_t w = 0u;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const uint32_t c = (uint32_t)(quant_mantissa(v[i], e, 2) + 1);
      w |= c << (2 * (i >> 1) + 16 * (i & 1));
    }
    *reinterpret_cast<uint32_t*>(tile + (size_t)nl * 16 + blk * 4) = w;
  } else {
    uint32_t w[2] = {0u, 0u};
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const uint32_t nib = (uint32_t)(quant_mantissa(v[i], e, m.w_bits) + 8);
      w[i >> 3] |= nib << (4 * c_nibble_pos[i & 7]);
    }
    const int bp = blk >> 1;
    uint2* dst = reinterpret_cast<uint2*>(tile + ((size_t)(bp * kTileN + nl) * 16) + (blk & 1) * 8);
    *dst = make_uint2(w[0], w[1]);
  }
  tile[w_mant_bytes(m.w_bits) + nl * 4 + blk] = (uint8_t)(e + 127);
}

// One thread = one (16-block of K, rank column j) of A.
__global__ void pack_a_kernel(const float* __restrict__ A, PackedMeta m, uint8_t* __restrict__ asec) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  const int kb = blockIdx.y;
  if (j >= m.k_pad) return;
  float v[16];
  float amax = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    v[i] = (j < m.k) ? A[(size_t)(kb * 16 + i) * m.k + j] : 0.0f;
    amax = fmaxf(amax, abs_ignore_nan(v[i]));
  }
  const int e = block_exponent(amax, m.w_exp_min, m.w_exp_max);
  uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
  for (int i = 0; i < 16; ++i)
    w[i >> 2] |= ((uint32_t)quant_mantissa(v[i], e, m.lr_bits) & 0xFFu) << (8 * (i & 3));
  uint4* dst = reinterpret_cast<uint4*>(asec + ((size_t)kb * m.k_pad + j) * 16);
  *dst = make_uint4(w[0], w[1], w[2], w[3]);
  asec[(size_t)(m.K / 16) * m.k_pad * 16 + (size_t)kb * m.k_pad + j] = (uint8_t)(e + 127);
}

// One thread = one (rank block rb, column n) of B.  grid (n_tiles, r_blocks), block 128.
__global__ void pack_b_kernel(const float* __restrict__ B, PackedMeta m, uint8_t* __restrict__ bsec) {
  const int nt = blockIdx.x, rb = blockIdx.y, nl = threadIdx.x;
  const int n = nt * kTileN + nl;
  float v[16];
  float amax = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const int r = rb * 16 + i;
    v[i] = (n < m.N && r < m.k) ? B[(size_t)r * m.N + n] : 0.0f;
    amax = fmaxf(amax, abs_ignore_nan(v[i]));
  }
  const int e = block_exponent(amax, m.w_exp_min, m.w_exp_max);
  uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
  for (int i = 0; i < 16; ++i)
    w[i >> 2] |= ((uint32_t)quant_mantissa(v[i], e, m.lr_bits) & 0xFFu) << (8 * (i & 3));
  uint8_t* tile = bsec + (size_t)nt * (m.r_blocks * kTileN * 17);
  *reinterpret_cast<uint4*>(tile + ((size_t)rb * kTileN + nl) * 16) = make_uint4(w[0], w[1], w[2], w[3]);
  tile[(size_t)m.r_blocks * kTileN * 16 + rb * kTileN + nl] = (uint8_t)(e + 127);
}

// ---------------------------------------------------------------------------- export
__global__ void export_w_kernel(PackedMeta m, const uint8_t* __restrict__ wsec, int8_t* __restrict__ Wm,
                                uint8_t* __restrict__ We) {
  const int nt = blockIdx.x, ks = blockIdx.y, nl = threadIdx.x, blk = threadIdx.y;
  const int n = nt * kTileN + nl;
  const int k0 = ks * kSlabK + blk * 16;
  if (n >= m.N || k0 >= m.K) return;
  const uint8_t* tile = wsec + ((size_t)nt * m.k_slabs + ks) * w_tile_bytes(m.w_bits);
  if (Wm != nullptr) {
    if (m.w_bits == 2) {
      const uint32_t w = *reinterpret_cast<const uint32_t*>(tile + (size_t)nl * 16 + blk * 4);
#pragma unroll
      for (int i = 0; i < 16; ++i)
        Wm[(size_t)(k0 + i) * m.N + n] = (int8_t)((int)((w >> (2 * (i >> 1) + 16 * (i & 1))) & 3u) - 1);
    } else {
      const uint2 w2 = *reinterpret_cast<const uint2*>(tile + ((size_t)((blk >> 1) * kTileN + nl) * 16) + (blk & 1) * 8);
      const uint32_t w[2] = {w2.x, w2.y};
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int nib = (int)((w[i >> 3] >> (4 * c_nibble_pos[i & 7])) & 0xFu);
        Wm[(size_t)(k0 + i) * m.N + n] = (int8_t)(nib - 8);
      }
    }
  }
  if (We != nullptr) We[(size_t)(k0 / 16) * m.N + n] = tile[w_mant_bytes(m.w_bits) + nl * 4 + blk];
}

__global__ void export_a_kernel(PackedMeta m, const uint8_t* __restrict__ asec, int8_t* __restrict__ Am,
                                uint8_t* __restrict__ Ae) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  const int kb = blockIdx.y;
  if (j >= m.k) return;
  const int8_t* src = reinterpret_cast<const int8_t*>(asec + ((size_t)kb * m.k_pad + j) * 16);
  if (Am != nullptr)
    for (int i = 0; i < 16; ++i) Am[(size_t)(kb * 16 + i) * m.k + j] = src[i];
  if (Ae != nullptr) Ae[(size_t)kb * m.k + j] = asec[(size_t)(m.K / 16) * m.k_pad * 16 + (size_t)kb * m.k_pad + j];
}

__global__ void export_b_kernel(PackedMeta m, const uint8_t* __restrict__ bsec, int8_t* __restrict__ Bm,
                                uint8_t* __restrict__ Be) {
  const int nt = blockIdx.x, rb = blockIdx.y, nl = threadIdx.x;
  const int n = nt * kTileN + nl;
  if (n >= m.N) return;
  const uint8_t* tile = bsec + (size_t)nt * (m.r_blocks * kTileN * 17);
  const int8_t* src = reinterpret_cast<const int8_t*>(tile + ((size_t)rb * kTileN + nl) * 16);
  if (Bm != nullptr)
    for (int i = 0; i < 16; ++i) Bm[(size_t)(rb * 16 + i) * m.N + n] = src[i];
  if (Be != nullptr) Be[(size_t)rb * m.N + n] = tile[(size_t)m.r_blocks * kTileN * 16 + rb * kTileN + nl];
}

cudaError_t launch_pack(const float* W, const float* A, const float* B, const PackedMeta& m, void* packed,
                        cudaStream_t s) {
  uint8_t* base = static_cast<uint8_t*>(packed);
  LaunchScope scope(kFamPack, s, m.k > 0 ? 3 : 1);
  pack_w_kernel<<<dim3(m.n_tiles, m.k_slabs), dim3(kTileN, 4), 0, s>>>(W, m, base + m.off_w);
  if (m.k > 0) {
    pack_a_kernel<<<dim3((m.k_pad + 63) / 64, m.K / 16), 64, 0, s>>>(A, m, base + m.off_a);
    pack_b_kernel<<<dim3(m.n_tiles, m.r_blocks), kTileN, 0, s>>>(B, m, base + m.off_b);
  }
  return cudaGetLastError();
}

cudaError_t launch_export(const PackedMeta& m, const void* packed, int8_t* Wm, uint8_t* We, int8_t* Am,
                          uint8_t* Ae, int8_t* Bm, uint8_t* Be, cudaStream_t s) {
  const uint8_t* base = static_cast<const uint8_t*>(packed);
  const bool do_w = Wm != nullptr || We != nullptr;
  const bool do_a = m.k > 0 && (Am != nullptr || Ae != nullptr);
  const bool do_b = m.k > 0 && (Bm != nullptr || Be != nullptr);
  if (!do_w && !do_a && !do_b) return cudaSuccess;
  LaunchScope scope(kFamExport, s, (int)do_w + (int)do_a + (int)do_b);
  if (do_w) export_w_kernel<<<dim3(m.n_tiles, m.k_slabs), dim3(kTileN, 4), 0, s>>>(m, base + m.off_w, Wm, We);
  if (do_a) export_a_kernel<<<dim3((m.k + 63) / 64, m.K / 16), 64, 0, s>>>(m, base + m.off_a, Am, Ae);
  if (do_b) export_b_kernel<<<dim3(m.n_tiles, m.r_blocks), kTileN, 0, s>>>(m, base + m.off_b, Bm, Be);
  return cudaGetLastError();
}

}  // namespace lqer
