// Small-batch form of the layer's contraction for up to 16 tokens (paper Section 3.1 / 3.2:
// Y = [X_q | T_q] . [W_q ; B_q]; Section 2.1: with this few tokens the layer is bound by the bytes of its weights).
//
// The tcgen05 form of the small-batch GEMM converts every packed weight tile to bf16 in shared memory (32 KB written
// and read again per 9 KB of packed weights), and that traffic, not DRAM, sets its pace.  Here the weights never
// touch shared memory: a lane loads 16 bytes of one column straight from the packed tile into registers, turns its
// nibbles into the exact bf16 values m * 2^e there (one fma.rn.bf16x2 per pair) and feeds them to
//     D[16 tokens, 8 columns] += A[16, 16 K] . B[16 K, 8]           (mma.sync m16n8k16, bf16 -> fp32)
// as the B fragment.  The products are exact and the sums are fp32, as in the tensor-memory kernels.
//
// Which K goes where.  Operands carry their block scales, so one MMA may mix blocks, and the 16 K positions of an
// MMA may be any 16 columns of Xcat as long as both fragments agree.  A warp step covers 128 K for 32 weight columns:
// lane (g = lane / 4, t = lane % 4) owns weight column g of each of its four column octets and the 32 K
//     [128 j + 32 t, 128 j + 32 t + 32)
// of step j - exactly the 16 bytes the packed tile stores contiguously for one column and block pair.  MMA number q
// (0..7) of the step takes the lane's K 4 q .. 4 q + 3: two bf16 pairs, the halves of a converted nibble word.  The
// activations are laid out to match when a sub-chunk of Xcat (up to 2048 K) is copied into shared memory: a record of
// 512 bytes holds, for lane l, the A fragment of one MMA in register order - token rows l / 4 and l / 4 + 8 (zeros
// beyond the batch) at the lane's K 4 q, 4 q + 1, then at 4 q + 2, 4 q + 3 - so one conflict-free 16-byte load per lane
// lands in the four consecutive registers the instruction wants and serves four column octets.
//
// Work items are those of the tcgen05 form: (layer, 256-column tile, K chunk), chunks fixed by the shapes of the
// launch; a chunk's partial goes to scratch and the CTA whose partial arrives last adds the chunks in chunk order.
// A CTA has eight warps of 32 columns each; two CTAs share an SM, so that one streams while the other copies
// activations or adds up.  Nothing waits for another CTA, and there is no spin in this kernel.
#include "lqer_gemm_small.cuh"
#include "lqer_tc_ptx.cuh"

namespace lqer {
namespace mg {
using namespace sg;

constexpr int THREADS = 256;
constexpr int WARPS = THREADS / 32;
constexpr int SUB_SLABS = 32;                       // slabs of 64 K whose activations are in shared memory at a time
constexpr int STEP_BYTES = 8 * 512;                 // a step's eight records: the A fragments of its eight MMAs
constexpr int X_BYTES = (SUB_SLABS / 2) * STEP_BYTES;                // 64 KB
constexpr int SMEM_BYTES = X_BYTES + 16;
constexpr int STAGE_ROW_BYTES = BN * 4 + 32;        // a token row of a finished tile, padded
static_assert(16 * STAGE_ROW_BYTES <= X_BYTES, "a finished tile is staged in the activation buffer");

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t ld_stream4(const void* p) {
  uint32_t v;
  asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
// a: the four registers of the A fragment in order (rows g / g + 8 of the first K pair, then of the second), as one
// 16-byte load delivers them.
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint4& a, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}
// bf16 pairs (2^(e-2), 2^(e-2)) and (-136 * 2^(e-2), -136 * 2^(e-2)) of exponent byte `byte` of word e4 (eb = e + 127):
// the bf16 bits are (eb - 2) << 7 and 0x8000 | (eb + 5) << 7 | 8, i.e. eb * 0x80 plus a constant, in both halves.
__device__ __forceinline__ void w_scale_pair(uint32_t e4, int byte, uint32_t& s2, uint32_t& c2) {
  const uint32_t eb = __byte_perm(e4, 0u, 0x4440u + byte);
  s2 = eb * 0x00800080u - 0x01000100u;
  c2 = eb * 0x00800080u + 0x82888288u;
}

// (a & b) | c in one instruction, with the mask and the magic number held in registers (given as immediates the pair
// costs two instructions, because one instruction takes one immediate).
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
struct ConvConsts {
  uint32_t mask, magic;        // 0x000F000F, 0x43004300
};
__device__ __forceinline__ ConvConsts conv_consts() {
  ConvConsts k;
  asm volatile("mov.b32 %0, 0x000F000F;" : "=r"(k.mask));     // opaque to the compiler, so that they stay in registers
  asm volatile("mov.b32 %0, 0x43004300;" : "=r"(k.magic));
  return k;
}
// Eight offset-binary nibbles of one block word -> eight bf16 (n - 8) * 2^(e-2), exact: 0x4300 | n is the bf16 value
// 128 + n, and (128 + n) * s - 136 * s rounds nothing away.  Register i holds K 2 i, 2 i + 1 of the word's eight.
__device__ __forceinline__ uint4 convert_nibbles(uint32_t w, uint32_t s2, uint32_t c2, const ConvConsts& k) {
  uint4 o;
  o.x = tc::fma_bf16x2(and_or(w, k.mask, k.magic), s2, c2);
  o.y = tc::fma_bf16x2(and_or(w >> 4, k.mask, k.magic), s2, c2);
  o.z = tc::fma_bf16x2(and_or(w >> 8, k.mask, k.magic), s2, c2);
  o.w = tc::fma_bf16x2(and_or(w >> 12, k.mask, k.magic), s2, c2);
  return o;
}

// A lane's weights of one step in one column octet: 32 nibbles (one block pair) of its column, and the slab's four
// exponent bytes of that column.
struct WOct {
  uint4 w;
  uint32_t e;
};
// wp / ep: the lane's column in the packed tile of the lane's slab (nibbles of its block pair; exponent word).
__device__ __forceinline__ void load_w_oct(WOct& f, const uint8_t* wp, const uint8_t* ep) {
  f.w = ld_stream16(wp);
  f.e = ld_stream4(ep);
}

// One octet's share of a step of weight slabs: eight MMAs.  a: the step's eight A fragments; eb0: index of the first
// exponent byte of the lane's block pair in an exponent word.
__device__ __forceinline__ void compute_w_oct(float (&acc)[4], const WOct& f, const uint4 (&a)[8], int eb0, const ConvConsts& k) {
  uint32_t s2, c2;
#pragma unroll
  for (int m = 0; m < 4; ++m) {
    if ((m & 1) == 0) w_scale_pair(f.e, eb0 + (m >> 1), s2, c2);
    const uint32_t word = m == 0 ? f.w.x : m == 1 ? f.w.y : m == 2 ? f.w.z : f.w.w;
    const uint4 b = convert_nibbles(word, s2, c2, k);
    mma_bf16(acc, a[2 * m], b.x, b.y);
    mma_bf16(acc, a[2 * m + 1], b.z, b.w);
  }
}

// One octet's share of a step of the rank term: 128 rank indices, of which the lane takes two 16-blocks of B_q (rb0,
// rb0 + 1) for its column.  bt: the packed B tile of the warp's 128-column half; nl: the lane's column in it.
__device__ __forceinline__ void compute_r_oct(float (&acc)[4], const uint8_t* bt, int r_blocks, int rb0, int nl, int lr_shift,
                                              const uint8_t* xs, int lane) {
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const int rb = rb0 + u;
    uint4 w = make_uint4(0u, 0u, 0u, 0u);
    float sc = 1.f;
    if (rb < r_blocks) {
      w = ld_stream16(bt + ((size_t)rb * kTileN + nl) * 16);
      sc = pow2f((int)bt[(size_t)r_blocks * kTileN * 16 + rb * kTileN + nl] - 127 - lr_shift);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int m = 2 * u + h;
      const uint4 a0 = *reinterpret_cast<const uint4*>(xs + (2 * m) * 512 + lane * 16);
      const uint4 a1 = *reinterpret_cast<const uint4*>(xs + (2 * m + 1) * 512 + lane * 16);
      const uint4 b = tc::convert_i8x8(h ? w.z : w.x, h ? w.w : w.y, sc);
      mma_bf16(acc, a0, b.x, b.y);
      mma_bf16(acc, a1, b.z, b.w);
    }
  }
}

// Columns [c_lo, c_hi) of Xcat (a multiple of 8 each) into the records of shared memory, zeros beyond c_hi and beyond
// the batch.  A lane reads 8 K of its rows g and g + 8 and writes the A fragments of the two MMAs that take them.
__device__ __forceinline__ void fill_x(uint8_t* xs, const uint16_t* xcat, int xcat_cols, int M, int c_lo, int c_hi, int warp, int lane) {
  constexpr int kBatch = 8;                      // loads of this many passes are in flight together (the copy is bound by latency)
  const int steps = (c_hi - c_lo + 127) / 128;
  const int g = lane >> 2, t = lane & 3;
  const uint16_t* r_lo = xcat + (size_t)g * xcat_cols;
  const uint16_t* r_hi = xcat + (size_t)(g + 8) * xcat_cols;
  const bool lo_ok = g < M, hi_ok = g + 8 < M;
  for (int pr0 = warp; pr0 < steps * 4; pr0 += WARPS * kBatch) {
    uint4 lo[kBatch], hi[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int pr = pr0 + u * WARPS;
      const int col = c_lo + 128 * (pr >> 2) + 32 * t + 8 * (pr & 3);
      lo[u] = hi[u] = make_uint4(0u, 0u, 0u, 0u);
      if (pr < steps * 4 && col < c_hi) {
        if (lo_ok) lo[u] = __ldcg(reinterpret_cast<const uint4*>(r_lo + col));
        if (hi_ok) hi[u] = __ldcg(reinterpret_cast<const uint4*>(r_hi + col));
      }
    }
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int pr = pr0 + u * WARPS;
      if (pr < steps * 4) {
        uint8_t* rec = xs + ((pr >> 2) * 8 + 2 * (pr & 3)) * 512 + lane * 16;
        *reinterpret_cast<uint4*>(rec) = make_uint4(lo[u].x, hi[u].x, lo[u].y, hi[u].y);
        *reinterpret_cast<uint4*>(rec + 512) = make_uint4(lo[u].z, hi[u].z, lo[u].w, hi[u].w);
      }
    }
  }
}

// Position of 16-byte unit u of a staged row: the four units of a 16-column block are rotated by the block pair's
// index, so that the threads which later read one block each meet no bank twice.
__device__ __forceinline__ int stage_unit(int u) { return (u & ~3) | ((u & 3) ^ ((u >> 3) & 3)); }

__global__ void __launch_bounds__(THREADS, 2)
gemm_mma_kernel(const __grid_constant__ Params p) {
  extern __shared__ __align__(16) uint8_t smem[];
  uint8_t* xs = smem;
  int* last_flag = reinterpret_cast<int*>(smem + X_BYTES);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int h = warp >> 2;                       // which 128-column packed tile of the 256-column item
  const int nl = 32 * (warp & 3) + g;            // the lane's column of octet 0 in that tile
  const int eb0 = 2 * (t & 1);
  const ConvConsts kc = conv_consts();
  tc::pdl_launch_dependents();                   // the next kernel may set up (it waits for this one before it touches memory)
  bool waited = false;

  for (int i = blockIdx.x; i < p.num_items; i += gridDim.x) {
    const Item it = item_of(p, i);
    const Layer& ly = p.L[it.layer];
    const int w_lo = it.s_lo, w_hi = min(it.s_hi, ly.k_slabs);
    const bool has_rank = it.s_hi > ly.k_slabs && ly.r_blocks > 0;
    const int nt = 2 * it.tile + h;
    const bool warp_live = nt < ly.n_tiles;
    const uint8_t* tile_row = ly.wsec + (size_t)(warp_live ? nt : 0) * ly.k_slabs * kWTileBytes;
    const uint8_t* wp = tile_row + (t & 1) * 2048 + nl * 16;
    const uint8_t* ep = tile_row + kWTileNibbleBytes + nl * 4;

    float acc[4][4];
#pragma unroll
    for (int o = 0; o < 4; ++o)
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[o][q] = 0.f;

    // packed weights depend on no earlier kernel: the first step is requested before the wait for the prologue
    WOct f[4];                                   // the step's weights; an octet's registers are refilled for the next step as soon as it is done
    // The lane's slab of the step that starts at slab s is s + t / 2.  Where that is beyond the chunk (the second half of
    // an odd last step, or the step after the last) the lane reads the chunk's last slab instead: its activations in
    // shared memory are zeros there and the weights are finite, so the products vanish, and no branch is needed.
    // In the checked build a slab beyond the buffer is reported and slab w_lo read in its place.
    auto slab_of = [&](int s) {
      int slab = min(s + (t >> 1), w_hi - 1);
      if (!LQER_IN_BOUNDS(p.status, (size_t)(tile_row - ly.wsec) + (size_t)slab * kWTileBytes, kWTileBytes, ly.w_extent, 721)) slab = w_lo;
      return slab;
    };
    if (warp_live && w_lo < w_hi) {
      const size_t off = (size_t)slab_of(w_lo) * kWTileBytes;
#pragma unroll
      for (int o = 0; o < 4; ++o) load_w_oct(f[o], wp + off + o * 128, ep + off + o * 32);
    }
    if (!waited) { tc::pdl_wait(); waited = true; }

    for (int sub = w_lo; sub < w_hi; sub += SUB_SLABS) {
      const int sub_hi = min(sub + SUB_SLABS, w_hi);
      __syncthreads();                           // the records of the sub-chunk before have been read
      fill_x(xs, ly.xcat, ly.xcat_cols, p.M, sub * kSlabK, sub_hi * kSlabK, warp, lane);
      __syncthreads();
      if (warp_live) {
#pragma unroll 1
        for (int s = sub; s < sub_hi; s += 2) {
          const size_t off = (size_t)slab_of(s + 2) * kWTileBytes;
          const uint8_t* step = xs + ((s - sub) >> 1) * STEP_BYTES + lane * 16;
          uint4 a[8];                            // the step's A fragments, read once for the four octets
#pragma unroll
          for (int q = 0; q < 8; ++q) a[q] = *reinterpret_cast<const uint4*>(step + q * 512);
#pragma unroll
          for (int o = 0; o < 4; ++o) {
            compute_w_oct(acc[o], f[o], a, eb0, kc);
            load_w_oct(f[o], wp + off + o * 128, ep + off + o * 32);
          }
        }
      }
    }
    if (has_rank) {
      __syncthreads();
      fill_x(xs, ly.xcat, ly.xcat_cols, p.M, ly.K64, ly.K64 + 16 * ly.r_blocks, warp, lane);
      __syncthreads();
      if (warp_live) {
        const uint8_t* bt = ly.bsec + (size_t)nt * ly.r_blocks * kTileN * 17;
        for (int j = 0; j * 8 < ly.r_blocks; ++j)
#pragma unroll
          for (int o = 0; o < 4; ++o)
            compute_r_oct(acc[o], bt, ly.r_blocks, 8 * j + 2 * t, nl + 8 * o, p.lr_shift, xs + j * STEP_BYTES, lane);
      }
    }

    // ------------------------------------------------------------------ the item's result
    // lane (g, t) holds rows g and g + 8 of columns 32 warp + 8 o + 2 t, + 1
    const int col0 = it.tile * BN;
    if (ly.chunks > 1) {
      float* pbase = ly.partials + ((size_t)(it.tile * ly.chunks + it.chunk) * p.M) * BN;
      if (warp_live) {
#pragma unroll
        for (int o = 0; o < 4; ++o) {
          const int c = 32 * warp + 8 * o + 2 * t;
#pragma unroll
          for (int r = 0; r < 2; ++r) {
            const int row = g + 8 * r;
            float* dst = pbase + (size_t)row * BN + c;
            if (row < p.M && LQER_IN_BOUNDS(p.status, (size_t)(dst - ly.partials) * 4, 8, ly.partial_extent, 722))
              *reinterpret_cast<float2*>(dst) = make_float2(acc[o][2 * r], acc[o][2 * r + 1]);
          }
        }
      }
      // count this chunk in; whoever brings the last partial of the tile adds them all up, in chunk order
      __threadfence();
      __syncthreads();
      if (tid == 0) *last_flag = (atomicAdd(ly.counters + it.tile, 1) == ly.chunks - 1) ? 1 : 0;
      __syncthreads();
      if (*last_flag != 0) {
        __threadfence();
        reduce_tile(p, ly, it.tile, tid, THREADS);
        if (tid == 0) ly.counters[it.tile] = 0;       // zero again for the next call
      }
    } else {
      // the only chunk: through shared memory, so that a thread ends up with a whole 16-block of a row
      __syncthreads();                                // the activation records have been read
      if (warp_live) {
#pragma unroll
        for (int o = 0; o < 4; ++o) {
          const int u = 8 * warp + 2 * o + (t >> 1);
#pragma unroll
          for (int r = 0; r < 2; ++r)
            *reinterpret_cast<float2*>(xs + (g + 8 * r) * STAGE_ROW_BYTES + stage_unit(u) * 16 + (t & 1) * 8) =
                make_float2(acc[o][2 * r], acc[o][2 * r + 1]);
        }
      }
      __syncthreads();
      const int row = tid >> 4, blk = tid & 15, c = col0 + 16 * blk;
      if (row < p.M && c < ly.N) {
        float v[16];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float4 f = *reinterpret_cast<const float4*>(xs + row * STAGE_ROW_BYTES + stage_unit(4 * blk + q) * 16);
          v[4 * q] = f.x; v[4 * q + 1] = f.y; v[4 * q + 2] = f.z; v[4 * q + 3] = f.w;
        }
        const size_t idx = (size_t)row * ly.N + c;
        if (p.y_type == kYMXINT8) {                   // N is a multiple of 16 here
          const QuantConsts qc = quant_consts(p.a_bits, p.exp_min, p.exp_max);
          uint4 m8, b0, b1;
          int e;
          quantize_block16(v, qc, e, m8, b0, b1);
          uint8_t* yq = static_cast<uint8_t*>(ly.Y);
          if (LQER_IN_BOUNDS(p.status, (size_t)p.M * ly.N + idx / 16, 1, ly.y_extent, 723)) {
            *reinterpret_cast<uint4*>(yq + idx) = m8;
            yq[(size_t)p.M * ly.N + idx / 16] = (uint8_t)(e + 127);
          }
        } else {
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if (c + 4 * q < ly.N)                     // N is a multiple of 8: a quad is whole
              store_y4(ly.Y, idx + 4 * q, make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]), p.y_type, p.status, ly.y_extent);
        }
      }
    }
  }
}

static cudaError_t launch(const Params& p, int ctas, cudaStream_t s) {
  static OncePerDevice once;
  cudaError_t e = once.run([] {
    return cudaFuncSetAttribute(gemm_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  });
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(ctas);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may set up and request weights while the prologue runs
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  LaunchScope scope(kFamDecode, s);
  return cudaLaunchKernelEx(&cfg, gemm_mma_kernel, p);
}

}  // namespace mg

cudaError_t launch_gemm_mma(const sg::Params& p, cudaStream_t s) {
  if (p.M < 1 || p.M > kMmaMaxM || p.w_bits != 4) return cudaErrorInvalidValue;
  const int sms = sm_count();
  if (sms < 1) return cudaErrorInvalidDevice;
  const int ctas = p.num_items < 2 * sms ? p.num_items : 2 * sms;
  return mg::launch(p, ctas, s);
}

}  // namespace lqer
