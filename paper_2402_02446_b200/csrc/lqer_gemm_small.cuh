// What the two small-batch GEMM kernels share: the work items (layer, 256-column tile, K chunk), the parameters of a
// launch, and the sum of a tile's chunks by the CTA whose partial arrives last (paper Section 3.1 / 3.2:
// Y = [X_q | T_q] . [W_q ; B_q] for few tokens; Section 2.1: the layer is memory bound on its weights there).
#pragma once
#include "lqer_common.cuh"

namespace lqer {
namespace sg {

constexpr int BN = 256;                    // weight columns of a work item
constexpr int MAX_LAYERS = 16;

struct Layer {
  const uint8_t* wsec;
  const uint8_t* bsec;
  const uint8_t* xfrag;        // register-operand kernel: [X_q | T_q] in fragment order (eight planes of `plane` bytes)
  int* flags;                  // ... and the prologue's two flags for this layer (X_q in place, T_q in place)
  void* Y;                     // [M, N] fp32 or bf16, or the MXINT8 sections (mantissas [M, N], exponent bytes [M, N / 16])
  float* partials;             // [tile][chunk][M][256] fp32 (tiles with more than one chunk)
  int* counters;               // [tile] arrivals, zero between calls
  size_t y_extent, partial_extent;   // bytes behind Y and behind partials, for the checked build
  size_t w_extent, b_extent;         // bytes of the packed W and B sections
  int N, K64, n_tiles, k_slabs, r_blocks;
  int plane;                   // bytes of a plane
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
  int y_type;                  // kYF32; kYBF16 (round to nearest even); kYMXINT8 (blocks of 16 along N, format below)
  int a_bits, exp_min, exp_max;// activation format, for an MXINT8 Y
  int w_bits;                  // mantissa bits of W_q: 4 or 2 (one value for all layers of a launch)
  int x_rows;                  // rows of an activation tile that TMA fills: M rounded up to 8 (the rest stay zero)
  long long wait_limit;
  int epoch;                   // register-operand kernel: the value the prologue's flags take in this call
  int* exit_count;             // ... and a zeroed counter of the CTAs that have left (the last one clears the flags)
  int stall;                   // test hook: the producer withholds the last stage of its last item
};

struct Item {
  int layer, tile, chunk, s_lo, s_hi;      // tile: index of the 256-column tile
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

__device__ __forceinline__ uint32_t bf16_rn(float v) {
  uint32_t u = __float_as_uint(v);
  if ((u & 0x7F800000u) == 0x7F800000u) return (u >> 16) | ((u & 0xFFFFu) ? 0x40u : 0u);   // inf / NaN
  u += 0x7FFFu + ((u >> 16) & 1u);                                                        // round to nearest even
  return u >> 16;
}
// Four consecutive elements of a row of Y.
__device__ __forceinline__ void store_y4(void* Y, size_t idx, float4 v, int y_type, DeviceStatus* st, size_t extent) {
  if (!LQER_IN_BOUNDS(st, idx * (y_type == kYBF16 ? 2 : 4), y_type == kYBF16 ? 8 : 16, extent, 701)) return;
  if (y_type == kYBF16)
    *reinterpret_cast<uint2*>(static_cast<uint16_t*>(Y) + idx) =
        make_uint2(bf16_rn(v.x) | (bf16_rn(v.y) << 16), bf16_rn(v.z) | (bf16_rn(v.w) << 16));
  else
    *reinterpret_cast<float4*>(static_cast<float*>(Y) + idx) = v;
}

// Y of one 256-column tile = the sum of its chunks' partials, in chunk order (the same sum whoever computes it), by
// `nthreads` threads (a multiple of 64): a thread per four columns, nthreads / 64 token rows per pass; the chunk loads
// of four rows are in flight together.
__device__ __forceinline__ void reduce_tile(const Params& p, const Layer& ly, int tile, int tid, int nthreads) {
  const int col0 = tile * BN, c4 = (tid & 63) * 4, trow0 = tid >> 6, rstep = nthreads >> 6;
  const bool quad_ok = col0 + c4 < ly.N;                                   // N is a multiple of 8: the quad is whole
  const float* p0 = ly.partials + ((size_t)tile * ly.chunks * p.M) * BN + c4;
  const size_t chunk_stride = (size_t)p.M * BN;
  for (int t0 = trow0; t0 < p.M; t0 += 4 * rstep) {
    float4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int cb = 0; cb < ly.chunks; cb += 4) {
      float4 t[4][4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int c = 0; c < 4; ++c)
          t[u][c] = (cb + c < ly.chunks && t0 + rstep * u < p.M)
                        ? __ldcg(reinterpret_cast<const float4*>(p0 + (size_t)(cb + c) * chunk_stride + (size_t)(t0 + rstep * u) * BN))
                        : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if (cb + c < ly.chunks) { v[u].x += t[u][c].x; v[u].y += t[u][c].y; v[u].z += t[u][c].z; v[u].w += t[u][c].w; }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int tk = t0 + rstep * u;
      if (p.y_type == kYMXINT8) {
        // four adjacent lanes hold a 16-block of the row (every lane of the warp takes part in the exchange)
        uint32_t m8;
        uint2 unused;
        int e;
        quantize_quad(v[u], p.a_bits, p.exp_min, p.exp_max, e, m8, unused);
        if (tk < p.M && quad_ok && LQER_IN_BOUNDS(p.status, (size_t)p.M * ly.N + ((size_t)tk * ly.N + col0 + c4) / 16, 1, ly.y_extent, 702)) {
          uint8_t* yq = static_cast<uint8_t*>(ly.Y);
          const size_t idx = (size_t)tk * ly.N + col0 + c4;
          *reinterpret_cast<uint32_t*>(yq + idx) = m8;
          if ((c4 & 15) == 0) yq[(size_t)p.M * ly.N + idx / 16] = (uint8_t)(e + 127);
        }
      } else if (tk < p.M && quad_ok) {
        store_y4(ly.Y, (size_t)tk * ly.N + col0 + c4, v[u], p.y_type, p.status, ly.y_extent);
      }
    }
  }
}

}  // namespace sg

// The register-operand form of the small-batch GEMM for up to kMmaMaxM tokens (lqer_gemm_mma.cu).
constexpr int kMmaMaxM = 16;
cudaError_t launch_gemm_mma(const sg::Params& p, cudaStream_t s);

}  // namespace lqer
