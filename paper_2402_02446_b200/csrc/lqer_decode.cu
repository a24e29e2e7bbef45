// Decode form of the layer for M <= 16 tokens (paper Section 3.1 / 3.2; Section 2.1 notes that
// small-batch inference is memory bound): one fused kernel that reads the packed 4-bit weights
// exactly once and is limited by HBM bandwidth.
//
//     Y[M,N] = X_q W_q + q(X_q A_q) B_q
//
// Work decomposition.  The contraction of every 128-column tile is cut into units of 64 K
// (one packed weight tile, 4608 bytes) followed by units of 32 rank values (B_q tiles).  All
// units of all column tiles form one sequence in the order the bytes lie in memory; CTA c takes
// the contiguous range [c n / G, (c + 1) n / G), so every CTA streams the same number of bytes
// from one contiguous region.  A CTA whose range ends inside a column tile writes its partial
// sums to a slot in the workspace; the last CTA to arrive at that tile (an atomic counter, no
// waiting) adds the slots in CTA order and writes Y.
//
// T = X_q A_q needs all of K before it can be re-quantised.  Every CTA computes the exact
// partial products of its share of K (int8 tensor-core MMA per 16-block, scaled in fp64) at
// kernel start and adds them to an accumulator in the workspace; the CTAs that own rank units
// process those last and, before them, wait (bounded) until all G contributions have arrived.
//
// A kernel that lives for a few microseconds pays for every instruction-cache line it touches
// and for every hand-over between warps, so all 16 warps run the same small loop.  Warp w owns
// output columns [8 w, 8 w + 8) of the current column tile and walks all units of the CTA:
//   * its share of a unit (8 columns x 64 K = 256 bytes of nibbles + 32 exponent bytes, or
//     8 columns x 32 rank values) goes global -> shared memory by cp.async into a private ring,
//     16 units ahead, so the whole share of the CTA is requested at once; these copies depend on
//     no earlier kernel and are issued before griddepcontrol.wait (programmatic dependent launch);
//   * X is quantised to MXINT8 once per CTA, cooperatively, into one exact-bf16 tile per unit;
//   * nibbles -> exact bf16 in registers, mma.sync m16n8k16 with the tokens on the M side,
//     fp32 accumulation; no partial sums cross warps.
#include "lqer_tc_ptx.cuh"

namespace lqer {
namespace dec {
using namespace tc;

constexpr int kWarps = 16;
constexpr int kThreads = kWarps * 32;
constexpr int kXTileStride = 144;                    // bytes per row of the bf16 X tile (64 values + pad)
constexpr int kXTileBytes = 16 * kXTileStride;       // 2304
constexpr int kPhaseUnits = 40;                      // units whose X tiles are resident at a time
constexpr int kDepth = 16;                           // units a warp keeps in flight
constexpr int kSlotBytes = 288;                      // a warp's share of one unit: 256 B mantissas + 32 B exponents
constexpr int kTabUnits = kPhaseUnits + kDepth;      // window of the unit table
constexpr int kSlotFloats = 16 * kTileN;             // one partial-sum slot: 16 rows x 128 columns

struct Params {
  const float* X;
  float* Y;
  const uint8_t* wsec;
  const uint8_t* bsec;
  const uint8_t* asec;
  DeviceStatus* status;
  int* tcount;          // CTAs whose T contribution has arrived
  int* tdone;           // CTAs that no longer need the T accumulator
  int* cnt;             // per column tile: partial sums that have arrived
  double* tacc;         // [16][k_pad] T accumulator (all zero between calls)
  float* slots;         // [G][2][16][128] partial sums
  int M, K, N, k_pad;
  int n_tiles, k_slabs, r_blocks, U;   // U = units per column tile = k_slabs + rank units
  int total_units;
  int a_bits, lr_bits, exp_min, exp_max;
  long long wait_limit; // bound of the wait for the other CTAs' contributions to T, in clock cycles
  int stall;            // test hook: wait for one contribution more than will come
};

// The order in which a CTA walks its units: memory order, except that the rank units of the
// first column tile of the range (which need T_q) are moved to the very end when other column
// tiles follow, so that nothing waits for T in the middle of the stream.
struct Seq {
  int lo, hi, head_rank_lo;
  int n, n_before, rh, nt_first, nt_last, U;
  bool reordered;
  __device__ void init(int lo_, int hi_, int U_, int k_slabs) {
    lo = lo_; hi = hi_; U = U_;
    n = hi - lo;
    nt_first = lo / U;
    nt_last = n > 0 ? (hi - 1) / U : nt_first;
    rh = 0; head_rank_lo = hi; reordered = false;
    if (n > 0 && nt_first != nt_last && U > k_slabs) {
      const int rs = max(lo, nt_first * U + k_slabs);
      head_rank_lo = rs;
      rh = (nt_first + 1) * U - rs;
      reordered = rh > 0;
    }
    n_before = n - rh;
  }
  __device__ int unit(int i) const {
    if (!reordered) return lo + i;
    if (i >= n_before) return head_rank_lo + (i - n_before);
    const int u = lo + i;
    return u >= head_rank_lo ? u + rh : u;
  }
};

// First unit of CTA c's range.  32-bit arithmetic: the host refuses layers with total * G >= 2^32.
__device__ __forceinline__ int range_lo(int c, int total, int G) { return (int)((uint32_t)c * (uint32_t)total / (uint32_t)G); }
// The CTA whose range holds unit u.
__device__ __forceinline__ int cta_of(int u, int total, int G) {
  return (int)((((uint32_t)u + 1u) * (uint32_t)G + (uint32_t)total - 1u) / (uint32_t)total) - 1;
}

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

__device__ __forceinline__ void cp_async8(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async4(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// What every thread of the CTA needs to know about the CTA's range, computed once.
struct Ctx {
  int lo, hi, nt_first;
  int part_first[2], part_last[2], part_slot0[2];   // contributors of the first / last column tile of the range
  int tab_nt[kTabUnits], tab_j[kTabUnits];           // (column tile, slab or rank unit) of units [tab0, tab0 + kTabUnits)
  int pending[2];                                    // column tile + 1 whose sums sit in this CTA's slot 0 / 1
  int flags[4];                                      // [0] a bounded wait ran out, [1], [2], [3] broadcast slots
};

// Hand the sums of column tile nt over (rare path, out of line so that the unit loop stays small).
// A tile whose whole contraction this CTA covered goes straight to Y.  Otherwise the sums go to
// this CTA's slot for the tile and the tile is marked pending; nothing is waited for here.
__device__ __noinline__ void store_partial(const Params& p, Ctx* cx, int nt, float s0, float s1, float s2, float s3) {
  const int tid = threadIdx.x, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int M = p.M, cta = blockIdx.x;
  const bool complete = nt * p.U >= cx->lo && (nt + 1) * p.U <= cx->hi;
  const int cl = (tid >> 5) * 8 + t * 2, col = nt * kTileN + cl;
  if (complete) {
    if (col < p.N) {
      if (g < M) *reinterpret_cast<float2*>(p.Y + (size_t)g * p.N + col) = make_float2(s0, s1);
      if (g + 8 < M) *reinterpret_cast<float2*>(p.Y + (size_t)(g + 8) * p.N + col) = make_float2(s2, s3);
    }
    return;
  }
  const int e = nt == cx->nt_first ? 0 : 1;
  float* slot = p.slots + ((size_t)cta * 2 + e) * kSlotFloats;
  if (g < M) __stcg(reinterpret_cast<float2*>(slot + g * kTileN + cl), make_float2(s0, s1));
  if (g + 8 < M) __stcg(reinterpret_cast<float2*>(slot + (g + 8) * kTileN + cl), make_float2(s2, s3));
  if (tid == 0) cx->pending[e] = nt + 1;
}

// End of the kernel: announce the pending slots (one release-acquire increment per tile, after a
// CTA barrier that orders every thread's slot stores before it); whoever arrives last at a tile
// adds the slots of all its contributors in CTA order and writes Y.
__device__ __noinline__ void finish_tiles(const Params& p, Ctx* cx) {
  const int tid = threadIdx.x, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int M = p.M;
  __syncthreads();
  if (tid < 2) {
    int last = 0;
    const int nt = cx->pending[tid] - 1;
    if (nt >= 0) {
      int old;
      asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(p.cnt + nt) : "memory");
      last = old == cx->part_last[tid] - cx->part_first[tid];
      if (last) p.cnt[nt] = 0;                   // every contributor has arrived: ready for the next call
    }
    cx->flags[2 + tid] = last;
  }
  __syncthreads();
#pragma unroll 1
  for (int e = 0; e < 2; ++e) {
    if (cx->flags[2 + e] == 0) continue;
    __threadfence();
    const int nt = cx->pending[e] - 1;
    const int c_first = cx->part_first[e], c_last = cx->part_last[e];
    const int cl = (tid >> 5) * 8 + t * 2, col = nt * kTileN + cl;
    float2 lo = make_float2(0.f, 0.f), hi = lo;
    for (int cc = c_first; cc <= c_last; ++cc) {
      // a contributor's slot for the tile: slot 1 only if the tile is not the first of its range
      const float* src = p.slots + ((size_t)cc * 2 + (cc == c_first ? cx->part_slot0[e] : 0)) * kSlotFloats;
      if (g < M) { const float2 v = __ldcg(reinterpret_cast<const float2*>(src + g * kTileN + cl)); lo.x += v.x; lo.y += v.y; }
      if (g + 8 < M) { const float2 v = __ldcg(reinterpret_cast<const float2*>(src + (g + 8) * kTileN + cl)); hi.x += v.x; hi.y += v.y; }
    }
    if (col < p.N) {
      if (g < M) *reinterpret_cast<float2*>(p.Y + (size_t)g * p.N + col) = lo;
      if (g + 8 < M) *reinterpret_cast<float2*>(p.Y + (size_t)(g + 8) * p.N + col) = hi;
    }
  }
}

// The T accumulator is released by every CTA once; the last one leaves it zero for the next call.
__device__ __noinline__ void release_tacc(const Params& p, Ctx* cx) {
  const int tid = threadIdx.x, G = gridDim.x;
  if (tid == 0) cx->flags[1] = (atomicAdd(p.tdone, 1) == G - 1) ? 1 : 0;
  __syncthreads();
  if (cx->flags[1] != 0) {
    __threadfence();
    for (int o = tid; o < 16 * p.k_pad; o += kThreads) p.tacc[o] = 0.0;
    if (tid == 0) { *p.tcount = 0; *p.tdone = 0; }
  }
}

// T -> T_q (exact bf16, [16][k_pad + 8]) in shared memory, once, before the first rank unit.
__device__ __noinline__ void build_tq(const Params& p, Ctx* cx, uint8_t* tq) {
  const int tid = threadIdx.x, G = gridDim.x, M = p.M;
  const int tq_stride = (p.k_pad + 8) * 2;
  if (tid == 0) {                                // bounded wait for the contributions of all CTAs
    const long long t0 = clock64();
    while (ld_acquire(p.tcount) < G + p.stall) {
      __nanosleep(64);
      if (clock64() - t0 > p.wait_limit) { cx->flags[0] = 1; break; }
    }
  }
  __syncthreads();
  __threadfence();
  const int total = M * p.k_pad;                 // MXINT8 along the rank: 16 adjacent lanes hold one block
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
    if (valid) *reinterpret_cast<uint16_t*>(tq + row * tq_stride + col * 2) = (uint16_t)bf16_bits_of(qv, e - (p.a_bits - 2));
  }
  __syncthreads();
  release_tacc(p, cx);
}

__global__ void __launch_bounds__(kThreads, 1) decode_kernel(const __grid_constant__ Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
  uint8_t* xs = smem;                                               // [kPhaseUnits] bf16 X tiles
  uint8_t* ring = xs + (size_t)kPhaseUnits * kXTileBytes;           // [kWarps][kDepth][kSlotBytes]
  const int tq_stride = (p.k_pad + 8) * 2;
  uint8_t* tq = ring + (size_t)kWarps * kDepth * kSlotBytes;        // [16][k_pad + 8] bf16 T_q
  Ctx* cx = reinterpret_cast<Ctx*>(tq + ((16 * tq_stride + 127) & ~127));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int G = gridDim.x, cta = blockIdx.x;
  const int M = p.M;
  const int col = warp * 8 + g;                                     // this lane's column within a tile
  uint8_t* my_ring = ring + (size_t)warp * kDepth * kSlotBytes;

  Seq seq;
  seq.init(range_lo(cta, p.total_units, G), range_lo(cta + 1, p.total_units, G), p.U, p.k_slabs);
  const int n = seq.n;

  pdl_launch_dependents();
  if (tid < 4) cx->flags[tid] = 0;
  if (tid < 2) cx->pending[tid] = 0;
  if (tid == 0) { cx->lo = seq.lo; cx->hi = seq.hi; cx->nt_first = seq.nt_first; }
  if (tid >= 32 && tid < 34) {
    // contributors of the first / last column tile: CTAs c_first..c_last; the first of them uses its
    // slot 1 if the tile is not the first of its range (every later one starts inside the tile: slot 0)
    const int e = tid - 32, nt = e == 0 ? seq.nt_first : seq.nt_last;
    const int c_first = cta_of(nt * p.U, p.total_units, G);
    cx->part_first[e] = c_first;
    cx->part_last[e] = cta_of((nt + 1) * p.U - 1, p.total_units, G);
    cx->part_slot0[e] = (range_lo(c_first, p.total_units, G) / p.U == nt) ? 0 : 1;
  }

  // Copy of this warp's share of unit fi into its ring (nothing if the walk has ended); tab0 = first unit of the table.
  auto issue = [&](int fi, int tab0) {
    if (fi < n) {
      const int nt = cx->tab_nt[fi - tab0], j = cx->tab_j[fi - tab0];
      uint8_t* dst = my_ring + (fi % kDepth) * kSlotBytes;
      if (j < p.k_slabs) {
        // lane (g, t): block t of the slab for column g (16 nibbles); lanes t == 0: the column's four exponents
        const uint8_t* tile = p.wsec + ((size_t)nt * p.k_slabs + j) * kWTileBytes;
        cp_async8(dst + lane * 8, tile + (t >> 1) * (kTileN * 16) + col * 16 + (t & 1) * 8);
        if (t == 0) cp_async4(dst + 256 + g * 4, tile + kWTileNibbleBytes + col * 4);
      } else {
        // lane (g, t): rank values 4t..4t+3 of two rank blocks for column g; lanes 0-3: exponent bytes
        const int rb0 = (j - p.k_slabs) * 2;
        const bool two = rb0 + 1 < p.r_blocks;
        const uint8_t* tile = p.bsec + (size_t)nt * ((size_t)p.r_blocks * kTileN * 17);
        const uint8_t* ex = tile + (size_t)p.r_blocks * kTileN * 16;
        cp_async4(dst + lane * 8, tile + ((size_t)rb0 * kTileN + col) * 16 + t * 4);
        if (two) cp_async4(dst + lane * 8 + 4, tile + ((size_t)(rb0 + 1) * kTileN + col) * 16 + t * 4);
        if (lane < 2) cp_async4(dst + 256 + lane * 4, ex + rb0 * kTileN + warp * 8 + lane * 4);
        if (two && lane >= 2 && lane < 4) cp_async4(dst + 264 + (lane - 2) * 4, ex + (rb0 + 1) * kTileN + warp * 8 + (lane - 2) * 4);
      }
    }
    cp_async_commit();
  };

  float acc_a[4] = {0.f, 0.f, 0.f, 0.f}, acc_b[4] = {0.f, 0.f, 0.f, 0.f};   // two chains of MMAs, summed at the end
  float acc_head[4] = {0.f, 0.f, 0.f, 0.f};
  int cur_nt = -1;
  bool tq_built = false;

  for (int ph0 = 0; ph0 < n; ph0 += kPhaseUnits) {
    // ---- unit table of this phase (and of the units that will be requested ahead of it)
    __syncthreads();
    if (tid < kTabUnits && ph0 + tid < n) {
      const int u = seq.unit(ph0 + tid), nt = u / p.U;
      cx->tab_nt[tid] = nt;
      cx->tab_j[tid] = u - nt * p.U;
    }
    __syncthreads();
    if (ph0 == 0) {
      // weights depend on no earlier kernel: request the first kDepth units before the dependency wait
#pragma unroll 4
      for (int u = 0; u < kDepth; ++u) issue(u, 0);
      pdl_wait();                                // X (and the workspace) may be an earlier kernel's output
      // ---- this CTA's share of T = X_q A_q: exact int8 MMA per (16-block of K, 8 rank columns),
      //      scaled in fp64 and added to the accumulator in the workspace
      if (p.k_pad > 0) {
        const int KB = p.K / 16, NT = p.k_pad / 8;
        const int kb_lo = cta * KB / G, kb_hi = (cta + 1) * KB / G;
        const uint8_t* a_exp = p.asec + (size_t)KB * p.k_pad * 16;
        const int bias = -127 - (p.a_bits - 2) - (p.lr_bits - 2);   // exponent bytes carry +127
        const int items = (kb_hi - kb_lo) * NT;
        for (int it = warp; it < items; it += kWarps) {
          const int kb = kb_lo + it / NT, nt = it % NT;
          const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
          const float4 v0 = g < M ? __ldg(reinterpret_cast<const float4*>(p.X + (size_t)g * p.K + kb * 16 + t * 4)) : z;
          const float4 v1 = g + 8 < M ? __ldg(reinterpret_cast<const float4*>(p.X + (size_t)(g + 8) * p.K + kb * 16 + t * 4)) : z;
          const uint32_t b0 = __ldg(reinterpret_cast<const uint32_t*>(p.asec + ((size_t)kb * p.k_pad + nt * 8 + g) * 16 + t * 4));
          const uint32_t ea2 = __ldg(reinterpret_cast<const uint16_t*>(a_exp + (size_t)kb * p.k_pad + nt * 8 + t * 2));
          int e0, e1;
          uint32_t m0, m1;
          uint2 unused;
          quantize_quad(v0, p.a_bits, p.exp_min, p.exp_max, e0, m0, unused);
          quantize_quad(v1, p.a_bits, p.exp_min, p.exp_max, e1, m1, unused);
          int c[4];
          mma_s8(c, m0, m1, b0);
          const int ea_lo = (int)(ea2 & 0xFFu) + bias, ea_hi = (int)(ea2 >> 8) + bias;
          const int tc = nt * 8 + t * 2;
          // exact products; their fp64 sum is exact as well unless the block exponents of one row
          // spread over more than about 30 binades, so the order of the additions does not matter
          if (g < M) {
            atomicAdd(p.tacc + (size_t)g * p.k_pad + tc, (double)c[0] * pow2d(e0 + ea_lo));
            atomicAdd(p.tacc + (size_t)g * p.k_pad + tc + 1, (double)c[1] * pow2d(e0 + ea_hi));
          }
          if (g + 8 < M) {
            atomicAdd(p.tacc + (size_t)(g + 8) * p.k_pad + tc, (double)c[2] * pow2d(e1 + ea_lo));
            atomicAdd(p.tacc + (size_t)(g + 8) * p.k_pad + tc + 1, (double)c[3] * pow2d(e1 + ea_hi));
          }
        }
      }
    }
    // ---- X -> MXINT8 -> exact bf16, one 16 x 64 tile per unit of the phase
    const int cnt = min(kPhaseUnits, n - ph0);
    {
      const int per_unit = M * 16, total = cnt * per_unit;          // float4 items: (unit, row, quarter-block)
      for (int base = 0; base < total; base += kThreads) {
        const int item = base + tid;
        const bool valid = item < total;
        const int u = valid ? item / per_unit : 0, f = valid ? item % per_unit : 0;
        const int row = f >> 4, c4 = f & 15;
        const int slab = cx->tab_j[u] < p.k_slabs ? cx->tab_j[u] : -1;
        const int xc = slab * kSlabK + c4 * 4;
        const float4 v = (valid && slab >= 0 && xc < p.K) ? __ldg(reinterpret_cast<const float4*>(p.X + (size_t)row * p.K + xc))
                                                          : make_float4(0.f, 0.f, 0.f, 0.f);
        int e;
        uint32_t m8;
        uint2 bf;
        quantize_quad(v, p.a_bits, p.exp_min, p.exp_max, e, m8, bf);
        if (valid && slab >= 0) *reinterpret_cast<uint2*>(xs + (size_t)u * kXTileBytes + row * kXTileStride + c4 * 8) = bf;
      }
    }
    __syncthreads();
    if (ph0 == 0 && tid == 0 && p.k_pad > 0)     // the T contributions of this CTA are out (ordered by the barrier)
      asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(p.tcount) : "memory");

    // ---- the units of the phase, in runs that share a column tile and a kind
    int i = ph0;
    const int ph_end = ph0 + cnt;
#pragma unroll 1
    while (i < ph_end) {
      const int nt = cx->tab_nt[i - ph0], j = cx->tab_j[i - ph0];
      const bool deferred_start = seq.reordered && i == seq.n_before;
      if (nt != cur_nt || deferred_start) {
        // column-tile boundary (uniform over the CTA): the first tile's sums are kept when its rank
        // units are deferred, any other tile's sums are handed over
        if (cur_nt >= 0) {
          if (!deferred_start && seq.reordered && cur_nt == seq.nt_first) {
#pragma unroll
            for (int a = 0; a < 4; ++a) acc_head[a] = acc_a[a] + acc_b[a];
          } else {
            store_partial(p, cx, cur_nt, acc_a[0] + acc_b[0], acc_a[1] + acc_b[1], acc_a[2] + acc_b[2], acc_a[3] + acc_b[3]);
          }
#pragma unroll
          for (int a = 0; a < 4; ++a) { acc_a[a] = 0.f; acc_b[a] = 0.f; }
        }
        cur_nt = nt;
      }
      if (j < p.k_slabs) {
        // ---- a run of slabs of W_q (consecutive units): four at a time, so that their chains of
        //      shared-memory loads, conversions and MMAs overlap
        int run_end = min(ph_end, i + (p.k_slabs - j));
        if (seq.reordered && i < seq.n_before) run_end = min(run_end, seq.n_before);   // the deferred part starts there
        // 64 K of W_q: lane (g, t) holds block t of the slab for row g (A side) and column g (B side)
        auto slab = [&](int iu, float (&ca)[4], float (&cb)[4]) {
          const uint8_t* slot = my_ring + (iu % kDepth) * kSlotBytes;
          const uint8_t* xb = xs + (size_t)(iu - ph0) * kXTileBytes;
          const uint4 q0 = *reinterpret_cast<const uint4*>(xb + g * kXTileStride + t * 32);
          const uint4 q1 = *reinterpret_cast<const uint4*>(xb + g * kXTileStride + t * 32 + 16);
          uint4 r0 = make_uint4(0u, 0u, 0u, 0u), r1 = r0;
          if (M > 8) {
            r0 = *reinterpret_cast<const uint4*>(xb + (g + 8) * kXTileStride + t * 32);
            r1 = *reinterpret_cast<const uint4*>(xb + (g + 8) * kXTileStride + t * 32 + 16);
          }
          const uint2 w = *reinterpret_cast<const uint2*>(slot + lane * 8);
          uint32_t s2, c2;
          w_scales(slot[256 + lane], s2, c2);
          const uint4 b0 = convert_word(w.x, s2, c2), b1 = convert_word(w.y, s2, c2);
          mma_bf16(ca, q0.x, r0.x, q0.y, r0.y, b0.x, b0.y);
          mma_bf16(cb, q0.z, r0.z, q0.w, r0.w, b0.z, b0.w);
          mma_bf16(ca, q1.x, r1.x, q1.y, r1.y, b1.x, b1.y);
          mma_bf16(cb, q1.z, r1.z, q1.w, r1.w, b1.z, b1.w);
        };
#pragma unroll 1
        for (; i + 4 <= run_end; i += 4) {
          cp_async_wait<kDepth - 4>();
          __syncwarp();
          float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
          slab(i, acc_a, acc_b);
          slab(i + 1, c0, c1);
          slab(i + 2, acc_a, acc_b);
          slab(i + 3, c0, c1);
#pragma unroll
          for (int a = 0; a < 4; ++a) { acc_a[a] += c0[a]; acc_b[a] += c1[a]; }
          __syncwarp();                          // the four slots are free: request the units kDepth ahead
#pragma unroll 1
          for (int u = 0; u < 4; ++u) issue(i + kDepth + u, ph0);
        }
#pragma unroll 1
        for (; i < run_end; ++i) {
          cp_async_wait<kDepth - 1>();
          __syncwarp();
          slab(i, acc_a, acc_b);
          __syncwarp();
          issue(i + kDepth, ph0);
        }
      } else {
        // ---- up to 32 rank values of B_q against T_q
        if (!tq_built) { build_tq(p, cx, tq); tq_built = true; }
        cp_async_wait<kDepth - 1>();
        __syncwarp();
        const uint8_t* slot = my_ring + (i % kDepth) * kSlotBytes;
        const int rb0 = (j - p.k_slabs) * 2;
        const uint2 w = *reinterpret_cast<const uint2*>(slot + lane * 8);
        for (int rb = 0; rb < 2 && rb0 + rb < p.r_blocks; ++rb) {
          const uint2 a_lo = *reinterpret_cast<const uint2*>(tq + g * tq_stride + ((rb0 + rb) * 16 + t * 4) * 2);
          uint2 a_hi = make_uint2(0u, 0u);
          if (M > 8) a_hi = *reinterpret_cast<const uint2*>(tq + (g + 8) * tq_stride + ((rb0 + rb) * 16 + t * 4) * 2);
          const uint32_t wv = rb == 0 ? w.x : w.y;
          const float scale = pow2f((int)slot[256 + rb * 8 + g] - 127 - (p.lr_bits - 2));
          const uint32_t b0 = pack_bf16x2((float)(int8_t)(wv) * scale, (float)(int8_t)(wv >> 8) * scale);
          const uint32_t b1 = pack_bf16x2((float)(int8_t)(wv >> 16) * scale, (float)(int8_t)(wv >> 24) * scale);
          mma_bf16(acc_a, a_lo.x, a_hi.x, a_lo.y, a_hi.y, b0, b1);
        }
        __syncwarp();
        issue(i + kDepth, ph0);
        ++i;
      }
    }
  }
  if (cur_nt >= 0) {
    // with a deferred part, the last segment belongs to the first tile
    const float h0 = seq.reordered ? acc_head[0] : 0.f, h1 = seq.reordered ? acc_head[1] : 0.f;
    const float h2 = seq.reordered ? acc_head[2] : 0.f, h3 = seq.reordered ? acc_head[3] : 0.f;
    store_partial(p, cx, cur_nt, acc_a[0] + acc_b[0] + h0, acc_a[1] + acc_b[1] + h1, acc_a[2] + acc_b[2] + h2, acc_a[3] + acc_b[3] + h3);
  }
  finish_tiles(p, cx);
  if (p.k_pad > 0 && !tq_built) release_tacc(p, cx);
  cp_async_wait<0>();
  if (cx->flags[0] != 0 && tid == 0) report_error(p.status, LQER_ERR_TIMEOUT, 500, cta);
}


}  // namespace dec

int decode_max_m() { return 16; }

cudaError_t launch_decode(const float* X, int M, const PackedMeta& m, const void* packed, float* Y, void* workspace,
                          cudaStream_t s, bool force_split_k) {
  using namespace dec;
  if (decode_cols_fits(m, M) && !force_split_k) return launch_decode_cols(X, M, m, packed, Y, workspace, s);
  const size_t fixed = (size_t)kPhaseUnits * kXTileBytes + (size_t)kWarps * kDepth * kSlotBytes + sizeof(Ctx) + 256;
  static OncePerDevice once;
  cudaError_t e0 = once.run([fixed] {
    return cudaFuncSetAttribute(decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)(fixed + 16 * (256 + 8) * 2 + 128));
  });
  if (e0 != cudaSuccess) return e0;
  const int sm_count = lqer::sm_count();
  if (sm_count < 1) return cudaErrorInvalidDevice;
  Params p;
  const uint8_t* base = static_cast<const uint8_t*>(packed);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  p.X = X; p.Y = Y;
  p.wsec = base + m.off_w; p.bsec = base + m.off_b; p.asec = base + m.off_a;
  p.status = reinterpret_cast<DeviceStatus*>(ws);
  p.tcount = reinterpret_cast<int*>(ws + kTCountOffset);
  p.tdone = reinterpret_cast<int*>(ws + kTDoneOffset);
  p.cnt = reinterpret_cast<int*>(ws + kStatusBytes);
  p.tacc = reinterpret_cast<double*>(ws + tacc_offset(m));
  p.slots = reinterpret_cast<float*>(ws + ((persist_bytes(m) + 255) & ~(size_t)255));
  p.M = M; p.K = m.K; p.N = m.N; p.k_pad = m.k_pad;
  p.n_tiles = m.n_tiles; p.k_slabs = m.k_slabs; p.r_blocks = m.r_blocks;
  p.U = m.k_slabs + (m.r_blocks + 1) / 2;
  p.total_units = decode_units(m);
  p.a_bits = m.a_bits; p.lr_bits = m.lr_bits; p.exp_min = m.exp_min; p.exp_max = m.exp_max;
  p.wait_limit = wait_limit_cycles();
  p.stall = take_stall(kFamDecode) ? 1 : 0;
  const int G = decode_ctas(m, sm_count);
  if ((unsigned long long)(p.total_units + 1) * (unsigned long long)(G + 1) >= (1ull << 32)) return cudaErrorInvalidValue;
  const size_t smem = fixed + ((16 * (m.k_pad + 8) * 2 + 127) & ~127);

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
  return cudaLaunchKernelEx(&cfg, decode_kernel, p);
}

}  // namespace lqer
