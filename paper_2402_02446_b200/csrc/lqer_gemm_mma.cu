// Small-batch form of the layer's contraction for up to 16 tokens (paper Section 3.1 / 3.2:
// Y = [X_q | T_q] . [W_q ; B_q]; Section 2.1: with this few tokens the layer is bound by the bytes of its weights).
//
// The tcgen05 form of the small-batch GEMM converts every packed weight tile to bf16 in shared memory (32 KB written
// and read again per 9 KB of packed weights), and that traffic, not DRAM, sets its pace.  Here the weights never
// touch shared memory: a lane loads 16 bytes of one column straight from the packed tile into registers, turns its
// nibbles (or crumbs, with 2-bit weights) into the exact bf16 values m * 2^e there (one fma.rn.bf16x2 per pair) and feeds them to
//     D[16 tokens, 8 columns] += A[16, 16 K] . B[16 K, 8]           (mma.sync m16n8k16, bf16 -> fp32)
// as the B fragment.  The products are exact and the sums are fp32, as in the tensor-memory kernels.
//
// Which K goes where.  Operands carry their block scales, so one MMA may mix blocks, and the 16 K positions of an
// MMA may be any 16 columns of Xcat as long as both fragments agree.  A warp step covers 128 K for 32 weight columns:
// lane (g = lane / 4, t = lane % 4) owns weight column g of each of its four column octets and the 32 K
//     [128 j + 32 t, 128 j + 32 t + 32)
// of step j - exactly the 16 bytes the packed tile stores contiguously for one column and block pair.  MMA number q
// (0..7) of the step takes the lane's K 4 q .. 4 q + 3: two bf16 pairs, the halves of a converted nibble word.  The
// activations arrive in that order already: the small prologue writes [X_q | T_q] of its (up to) 16 rows as eight
// planes of [slab][256 bytes], 16 bytes per (row pair, block pair) = the A fragment of one MMA in register order (token
// rows l / 4 and l / 4 + 8 at the lane's K 4 q, 4 q + 1, then at 4 q + 2, 4 q + 3), so a sub-chunk of 16 slabs is
// eight bulk copies into shared memory, a lane's fragment is one conflict-free 16-byte load that lands in the four
// consecutive registers the instruction wants, and it serves four column octets.
//
// Work items are those of the tcgen05 form: (layer, 256-column tile, K chunk), chunks fixed by the shapes of the
// launch; a chunk's partial goes to scratch and the CTA whose partial arrives last adds the chunks in chunk order.
// A CTA has eight warps of 32 columns each; two CTAs share an SM.  The activations of the next sub-chunk are copied
// while the current one is multiplied (two buffers, one mbarrier each).
//
// The kernel does not wait for the prologue as a whole.  The prologue raises a flag per layer when X_q is in place
// and another when T_q is (which takes it several times longer); an item waits for the first before its first copy and
// for the second before the rank term, its last sub-chunk, so the weight stream runs while T is still being formed.
// Both waits are bounded polls of one thread.  The prologue was launched before this kernel and all its CTAs are
// resident or done by the time this one starts (the launch order of programmatic dependent launches), so it never
// depends on this kernel's progress.  The flags are raised only after the prologue's own wait for the kernels before
// it, so whatever this kernel writes after seeing a flag cannot collide with them.  A flag holds the launch's epoch, a
// number no earlier launch on the workspace used: the flag the call before left behind never passes for this call's,
// even while that call's last CTAs are still running.  The last CTA to leave clears the flags all the same, so that a
// captured graph, whose replays repeat the epoch, starts from cleared flags too.
#include "lqer_gemm_small.cuh"
#include "lqer_tc_ptx.cuh"

namespace lqer {
namespace mg {
using namespace sg;

constexpr int THREADS = 256;
constexpr int SUB_SLABS = 16;                       // slabs of 64 K per activation buffer
constexpr int PLANE_BYTES = SUB_SLABS * 256;        // a buffer's share of one of the eight planes
constexpr int BUF_BYTES = 8 * PLANE_BYTES;          // 32 KB
constexpr int OFF_BARS = 2 * BUF_BYTES;
constexpr int SMEM_BYTES = OFF_BARS + 64;
constexpr int STAGE_ROW_BYTES = BN * 4 + 32;        // a token row of a finished tile, padded
static_assert(16 * STAGE_ROW_BYTES <= BUF_BYTES, "a finished tile is staged in the first activation buffer");

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
  uint32_t mask, magic;        // 0x000F000F (nibbles) or 0x00030003 (crumbs), 0x43004300
};
template <int WB>
__device__ __forceinline__ ConvConsts conv_consts() {
  ConvConsts k;
  if (WB == 4) asm volatile("mov.b32 %0, 0x000F000F;" : "=r"(k.mask));     // opaque to the compiler, so that they stay in registers
  else asm volatile("mov.b32 %0, 0x00030003;" : "=r"(k.mask));
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
// The 2-bit format (mantissas -1, 0, 1; value m * 2^e): crumbs 4 j .. 4 j + 3 of the low and of the high half of a block
// word (K 8 j .. 8 j + 7 of the block's sixteen) -> eight bf16, exact: (128 + c) * s - 129 * s rounds nothing away.
__device__ __forceinline__ uint4 convert_crumbs(uint32_t w, int j, uint32_t s2, uint32_t c2, const ConvConsts& k) {
  uint4 o;
  o.x = tc::fma_bf16x2(and_or(w >> (8 * j), k.mask, k.magic), s2, c2);
  o.y = tc::fma_bf16x2(and_or(w >> (8 * j + 2), k.mask, k.magic), s2, c2);
  o.z = tc::fma_bf16x2(and_or(w >> (8 * j + 4), k.mask, k.magic), s2, c2);
  o.w = tc::fma_bf16x2(and_or(w >> (8 * j + 6), k.mask, k.magic), s2, c2);
  return o;
}
// bf16 pairs (2^e, 2^e) and (-129 * 2^e, -129 * 2^e) of an exponent byte of word e4: bits eb << 7 and 0x8000 | (eb + 7) << 7 | 1.
__device__ __forceinline__ void w_scale_pair2(uint32_t e4, int byte, uint32_t& s2, uint32_t& c2) {
  const uint32_t eb = __byte_perm(e4, 0u, 0x4440u + byte);
  s2 = eb * 0x00800080u;
  c2 = eb * 0x00800080u + 0x83818381u;
}

// A lane's weights of one step in one column octet: one block pair (32 K) of its column - 16 bytes of nibbles, or 8
// bytes of crumbs in w.x, w.y - and the slab's four exponent bytes of that column.
struct WOct {
  uint4 w;
  uint32_t e;
};
// wp / ep: the lane's column in the packed tile of the lane's slab (mantissas of its block pair; exponent word).
template <int WB>
__device__ __forceinline__ void load_w_oct(WOct& f, const uint8_t* wp, const uint8_t* ep) {
  if (WB == 4) {
    f.w = ld_stream16(wp);
  } else {
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];" : "=r"(f.w.x), "=r"(f.w.y) : "l"(wp));
  }
  f.e = ld_stream4(ep);
}

// One octet's share of a step of weight slabs: eight MMAs.  a: the step's eight A fragments; eb0: index of the first
// exponent byte of the lane's block pair in an exponent word.
template <int WB>
__device__ __forceinline__ void compute_w_oct(float (&acc)[4], const WOct& f, const uint4 (&a)[8], int eb0, const ConvConsts& k) {
  uint32_t s2, c2;
#pragma unroll
  for (int m = 0; m < 4; ++m) {
    if ((m & 1) == 0) {
      if (WB == 4) w_scale_pair(f.e, eb0 + (m >> 1), s2, c2);
      else w_scale_pair2(f.e, eb0 + (m >> 1), s2, c2);
    }
    uint4 b;
    if (WB == 4) {
      const uint32_t word = m == 0 ? f.w.x : m == 1 ? f.w.y : m == 2 ? f.w.z : f.w.w;
      b = convert_nibbles(word, s2, c2, k);
    } else {
      b = convert_crumbs(m < 2 ? f.w.x : f.w.y, m & 1, s2, c2, k);
    }
    mma_bf16(acc, a[2 * m], b.x, b.y);
    mma_bf16(acc, a[2 * m + 1], b.z, b.w);
  }
}

// One octet's share of a step of the rank term: 128 rank indices, of which the lane takes two 16-blocks of B_q (rb0,
// rb0 + 1) for its column.  bt: the packed B tile of the warp's 128-column half; nl: the lane's column in it; a: the
// step's eight A fragments.
__device__ __forceinline__ void compute_r_oct(float (&acc)[4], const uint8_t* bt, int r_blocks, int rb0, int nl, int lr_shift,
                                              const uint4 (&a)[8]) {
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
      const uint4 b = tc::convert_i8x8(h ? w.z : w.x, h ? w.w : w.y, sc);
      mma_bf16(acc, a[2 * m], b.x, b.y);
      mma_bf16(acc, a[2 * m + 1], b.z, b.w);
    }
  }
}

// Position of 16-byte unit u of a staged row: the four units of a 16-column block are rotated by the block pair's
// index, so that the threads which later read one block each meet no bank twice.
__device__ __forceinline__ int stage_unit(int u) { return (u & ~3) | ((u & 3) ^ ((u >> 3) & 3)); }

// Bounded poll (one thread) until a flag of the prologue holds this call's epoch.
__device__ __forceinline__ bool poll_flag(const int* flag, int epoch, volatile tc::WaitState* ws) {
  const long long t0 = clock64();
  for (;;) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
    if (v == epoch) return true;
    __nanosleep(100);
    if (ws->abort != 0) return false;
    if (clock64() - t0 > ws->limit) { ws->abort = 1; return false; }
  }
}

template <int WB>
__global__ void __launch_bounds__(THREADS, 2)
gemm_mma_kernel(const __grid_constant__ Params p) {
  constexpr int kTile = WB == 4 ? kWTileBytes : 2048 + kTileN * 4;   // bytes of a packed weight tile
  constexpr int kMant = WB == 4 ? kWTileNibbleBytes : 2048;          // of which mantissas
  extern __shared__ __align__(128) uint8_t smem[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BARS);
  int* last_flag = reinterpret_cast<int*>(smem + OFF_BARS + 16);
  volatile tc::WaitState* ws = reinterpret_cast<volatile tc::WaitState*>(smem + OFF_BARS + 32);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int h = warp >> 2;                       // which 128-column packed tile of the 256-column item
  const int nl = 32 * (warp & 3) + g;            // the lane's column of octet 0 in that tile
  const int eb0 = 2 * (t & 1);
  const uint32_t a_off = (uint32_t)((t >> 1) * 256 + (2 * g + (t & 1)) * 16);   // the lane's fragment within a step of a plane
  const ConvConsts kc = conv_consts<WB>();
  if (tid == 0) {
    tc::mbar_init(tc::smem_u32(bars), 1);
    tc::mbar_init(tc::smem_u32(bars + 1), 1);
    ws->abort = 0;
    ws->limit = p.wait_limit;
    tc::fence_barrier_init();
  }
  tc::pdl_launch_dependents();                   // the next kernel may set up (it waits for this one before it touches memory)
  uint32_t copies = 0;                           // activation copies issued so far (the same in every thread): buffer = copies & 1
  bool ok = true;

  for (int i = blockIdx.x; i < p.num_items && ok; i += gridDim.x) {
    const Item it = item_of(p, i);
    const Layer& ly = p.L[it.layer];
    const int w_lo = it.s_lo, w_hi = min(it.s_hi, ly.k_slabs);
    const bool has_rank = it.s_hi > ly.k_slabs && ly.r_blocks > 0;
    const int n_w = (w_hi - w_lo + SUB_SLABS - 1) / SUB_SLABS;
    const int n_sub = n_w + (has_rank ? 1 : 0);
    const int r_slabs = (ly.r_blocks + 3) / 4;
    const int nt = 2 * it.tile + h;
    const bool warp_live = nt < ly.n_tiles;
    const uint8_t* tile_row = ly.wsec + (size_t)(warp_live ? nt : 0) * ly.k_slabs * kTile;
    const uint8_t* wp = WB == 4 ? tile_row + (t & 1) * 2048 + nl * 16 : tile_row + nl * 16 + (t & 1) * 8;
    const uint8_t* ep = tile_row + kMant + nl * 4;

    float acc[4][4];
#pragma unroll
    for (int o = 0; o < 4; ++o)
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[o][q] = 0.f;

    WOct f[4];                                   // the step's weights; an octet's registers are refilled for the next step as soon as it is done
    // The lane's slab of the step that starts at slab s is s + t / 2.  Where that is beyond the chunk (the second half of
    // an odd last step, or the step after the last) the lane reads the chunk's last slab instead: its activations in
    // shared memory are zeros there and the weights are finite, so the products vanish, and no branch is needed.
    // In the checked build a slab beyond the buffer is reported and slab w_lo read in its place.
    auto slab_of = [&](int s) {
      int slab = min(s + (t >> 1), w_hi - 1);
      if (!LQER_IN_BOUNDS(p.status, (size_t)(tile_row - ly.wsec) + (size_t)slab * kTile, kTile, ly.w_extent, 721)) slab = w_lo;
      return slab;
    };
    // Sub-chunk n of the item: up to SUB_SLABS slabs of X_q, or (the last one of a tile's last chunk) the slabs of T_q.
    auto sub_lo = [&](int n) { return n < n_w ? w_lo + n * SUB_SLABS : ly.k_slabs; };
    auto sub_len = [&](int n) { return n < n_w ? min(SUB_SLABS, w_hi - (w_lo + n * SUB_SLABS)) : r_slabs; };
    // Thread 0: waits for what sub-chunk n needs of the prologue, then requests its eight planes as copy number `copy`
    // (buffer copy & 1).  With `ahead` (the request is made a sub-chunk early) a T_q that is not there yet is not waited
    // for: the request is put off (returns false) and made again when its turn comes, so that a short chunk's weight
    // loop runs while T is still being formed.
    auto request = [&](int n, uint32_t copy, bool ahead) -> bool {
      const int want = p.stall != 0 ? ~p.epoch : p.epoch;   // test hook: a value the flags never take
      if (n == 0 || n >= n_w) {
        const int* flag = ly.flags + (n < n_w ? 0 : 1);
        if (ahead) {
          int v;
          asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
          if (v != want) return false;
        } else if (!poll_flag(flag, want, ws)) {
          return true;                                       // given up: nothing is requested, every wait runs out
        }
        asm volatile("fence.proxy.async.global;" ::: "memory");       // what the flag vouches for, before the copies read it
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");    // this buffer's earlier readers, before the copies overwrite it
      const int len = sub_len(n);
      const uint32_t bar = tc::smem_u32(bars + (copy & 1));
      const uint32_t dst = tc::smem_u32(smem + (copy & 1) * BUF_BYTES);
      const uint8_t* src = ly.xfrag + (size_t)sub_lo(n) * 256;
      tc::mbar_expect_tx(bar, 8u * len * 256u);
#pragma unroll
      for (int q = 0; q < 8; ++q) tc::bulk_load(dst + q * PLANE_BYTES, src + (size_t)q * ly.plane, len * 256, bar);
      return true;
    };
    // Every thread: an odd sub-chunk ends in half a step; the slab after its last one reads as zeros.
    auto zero_tail = [&](int n) {
      const int len = sub_len(n);
      if ((len & 1) && tid < 128)
        *reinterpret_cast<uint4*>(smem + (copies & 1) * BUF_BYTES + (tid >> 4) * PLANE_BYTES + len * 256 + (tid & 15) * 16) = make_uint4(0u, 0u, 0u, 0u);
    };

    __syncthreads();                             // the item before has left both buffers (and the staged tile)
    if (tid == 0) request(0, copies, false);
    zero_tail(0);
    ++copies;
    bool put_off = false;                        // thread 0: the request of the next sub-chunk was put off
    // the first step's weights (after the request, whose fence would otherwise sit behind these loads)
    if (warp_live) {
      const size_t off = (size_t)slab_of(w_lo) * kTile;
#pragma unroll
      for (int o = 0; o < 4; ++o) load_w_oct<WB>(f[o], wp + off + o * 128, ep + off + o * 32);
      if (has_rank) {
        // the rank term comes last and is short: its weights are asked into L2 now, so that it does not wait for DRAM then
        const uint8_t* bt = ly.bsec + (size_t)nt * ly.r_blocks * kTileN * 17;
        if (g < 4)                                 // lane (g, t): the 128-byte line of octet g in rank blocks t, t + 4, ...
          for (int rb = t; rb < ly.r_blocks; rb += 4)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(bt + ((size_t)rb * kTileN + 32 * (warp & 3) + 8 * g) * 16));
        if (lane < ly.r_blocks) asm volatile("prefetch.global.L2 [%0];" ::"l"(bt + (size_t)ly.r_blocks * kTileN * 16 + lane * kTileN));
      }
    }

    for (int n = 0; n < n_sub; ++n) {
      __syncthreads();                           // sub-chunk n - 1 has been read: its buffer is free; zeroed tails are visible
      if (tid == 0 && put_off) {                 // this sub-chunk's own request, put off a round ago
        request(n, copies - 1, false);
        put_off = false;
      }
      if (n + 1 < n_sub) {
        if (tid == 0) put_off = !request(n + 1, copies, true);
        zero_tail(n + 1);
        ++copies;
      }
      const uint32_t mine = copies - (n + 1 < n_sub ? 2u : 1u);           // the copy that carries sub-chunk n
      ok = tc::mbar_wait<true>(tc::smem_u32(bars + (mine & 1)), (mine >> 1) & 1, ws);
      if (__syncthreads_or(ok ? 0 : 1)) { ok = false; break; }
      const uint8_t* buf = smem + (mine & 1) * BUF_BYTES + a_off;
      if (warp_live) {
        const int lo = sub_lo(n), len = sub_len(n);
        if (n < n_w) {
#pragma unroll 1
          for (int j = 0; 2 * j < len; ++j) {
            const size_t off = (size_t)slab_of(lo + 2 * j + 2) * kTile;
            uint4 a[8];                          // the step's A fragments, read once for the four octets
#pragma unroll
            for (int q = 0; q < 8; ++q) a[q] = *reinterpret_cast<const uint4*>(buf + q * PLANE_BYTES + j * 512);
#pragma unroll
            for (int o = 0; o < 4; ++o) {
              compute_w_oct<WB>(acc[o], f[o], a, eb0, kc);
              load_w_oct<WB>(f[o], wp + off + o * 128, ep + off + o * 32);
            }
          }
        } else {
          const uint8_t* bt = ly.bsec + (size_t)nt * ly.r_blocks * kTileN * 17;
          for (int j = 0; 2 * j < len; ++j) {
            uint4 a[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) a[q] = *reinterpret_cast<const uint4*>(buf + q * PLANE_BYTES + j * 512);
#pragma unroll
            for (int o = 0; o < 4; ++o) compute_r_oct(acc[o], bt, ly.r_blocks, 8 * j + 2 * t, nl + 8 * o, p.lr_shift, a);
          }
        }
      }
    }
    if (!ok) break;
    uint8_t* xs = smem;                          // the first buffer doubles as the staging area of a finished tile

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
      __syncthreads();                                // the activation buffers have been read
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
  // ------------------------------------------------------------------ leaving
  __syncthreads();
  if (tid == 0) {
    if (!ok || ws->abort != 0) {
      const long long t0 = clock64();
      while (clock64() - t0 < 400000) { }          // a copy requested before the give-up lands well within this
      report_error(p.status, LQER_ERR_TIMEOUT, 720, blockIdx.x);
    } else {
      // The last CTA to leave clears the flags.  Epochs already keep a later launch from taking them for its own; a
      // replay of a captured graph, though, repeats its epoch, and must find the flags as the first run found them.
      __threadfence();
      if (atomicAdd(p.exit_count, 1) == (int)gridDim.x - 1) {
        for (int l = 0; l < p.n; ++l) { p.L[l].flags[0] = 0; p.L[l].flags[1] = 0; }
        *p.exit_count = 0;
      }
    }
  }
}

template <int WB>
static cudaError_t launch(const Params& p, int ctas, cudaStream_t s) {
  static OncePerDevice once;
  cudaError_t e = once.run([] {
    return cudaFuncSetAttribute(gemm_mma_kernel<WB>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
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
  return cudaLaunchKernelEx(&cfg, gemm_mma_kernel<WB>, p);
}

}  // namespace mg

cudaError_t launch_gemm_mma(const sg::Params& p, cudaStream_t s) {
  if (p.M < 1 || p.M > kMmaMaxM || (p.w_bits != 4 && p.w_bits != 2)) return cudaErrorInvalidValue;
  const int sms = sm_count();
  if (sms < 1) return cudaErrorInvalidDevice;
  const int ctas = p.num_items < 2 * sms ? p.num_items : 2 * sms;
  return p.w_bits == 4 ? mg::launch<4>(p, ctas, s) : mg::launch<2>(p, ctas, s);
}

}  // namespace lqer
