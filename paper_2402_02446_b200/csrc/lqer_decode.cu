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
// Roles in a CTA (16 warps, four per scheduler):
//   warp 0       producer: bulk copies of weight tiles and of the matching X columns into a ring
//   warps 1-3    quantisers: X fp32 -> MXINT8 -> exact bf16, one 16 x 64 tile per stage
//   warps 4-7    T: partial X_q A_q, later T -> T_q (bf16) for the rank units
//   warps 8-15   consumers: nibbles -> exact bf16 in registers, mma.sync m16n8k16 (tokens are
//                the M side of the MMA, 16 output columns per warp), fp32 accumulation
// Weight copies do not depend on earlier kernels of the stream, so they are issued before
// griddepcontrol.wait: with programmatic dependent launch the next layer's weights are already
// in flight while the previous layer finishes.
#include "lqer_tc_ptx.cuh"

namespace lqer {
namespace dec {
using namespace tc;

constexpr int kQuantWarps = 3, kTWarps = 4, kConsumerWarps = 8;
constexpr int kThreads = (1 + kQuantWarps + kTWarps + kConsumerWarps) * 32;   // 512
constexpr int kXTileStride = 144;                    // bytes per row of the bf16 X tile (64 values + pad)
constexpr int kXTileBytes = 16 * kXTileStride;       // 2304
constexpr int kMaxStages = 32;
constexpr int kAChunkBytes = 16 * 1024;              // staging of A_q blocks and their X columns
constexpr int kSlotFloats = 16 * kTileN;             // one partial-sum slot: 16 rows x 128 columns
constexpr int kSmemBudget = 225 * 1024;

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
  int stages, stage_bytes, xf_bytes, a_chunk_blocks;
  int a_bits, lr_bits, exp_min, exp_max;
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

// Position in the walk: the current unit is slab / rank unit j of column tile nt.  Steps to the
// next unit by incrementing; divides only where the order jumps.
struct Walker {
  int u, nt, j;
  __device__ void set(const Seq& s, int uu) { u = uu; nt = uu / s.U; j = uu - nt * s.U; }
  __device__ void start(const Seq& s) { if (s.n > 0) set(s, s.unit(0)); else { u = 0; nt = 0; j = 0; } }
  __device__ void step(const Seq& s, int i_next) {
    if (i_next >= s.n) return;
    const int nu = s.unit(i_next);
    if (nu == u + 1) { u = nu; if (++j == s.U) { j = 0; ++nt; } }
    else set(s, nu);
  }
};

// First unit of CTA c's range (the product may exceed 32 bits; used a few times per thread only).
__device__ __forceinline__ int range_lo(int c, int total, int G) { return (int)((long long)c * total / G); }
// The CTA whose range holds unit u.
__device__ __forceinline__ int cta_of(int u, int total, int G) {
  return (int)((((long long)u + 1) * G + total - 1) / total) - 1;
}

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
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

// Wait of a whole warp on an mbarrier phase.  Only lane 0 polls, sleeping between polls, so that
// waiting warps leave the issue slots and the shared-memory pipe to the warps that have work;
// afterwards every lane observes the completed phase itself (one poll that succeeds at once).
// Bounded: gives up after WAIT_LIMIT_CYCLES or as soon as another role has given up.
template <int kSleepNs>
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  int ok = 1;
  if ((threadIdx.x & 31) == 0 && !mbar_try_wait(bar, parity)) {
    const long long t0 = clock64();
    int spins = 0;
    while (!mbar_try_wait(bar, parity)) {
      __nanosleep(kSleepNs);
      if ((++spins & 63) == 0) {
        if (*abort_flag != 0) { ok = 0; break; }
        if (clock64() - t0 > WAIT_LIMIT_CYCLES) { *abort_flag = 1; ok = 0; break; }
      }
    }
  }
  ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
  if (ok == 0) return false;
  if (!mbar_try_wait(bar, parity)) return mbar_wait<true>(bar, parity, abort_flag);
  return true;
}

// Rendezvous of the warps of one role on an mbarrier (count = number of warps), bounded like
// every other wait of the kernel.  `use` counts the rendezvous of this role so far.
__device__ __forceinline__ bool role_sync(uint32_t bar, uint32_t& use, volatile int* abort_flag) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
  const bool ok = warp_wait<32>(bar, use & 1u, abort_flag);
  ++use;
  return ok;
}

__global__ void __launch_bounds__(kThreads, 1) decode_kernel(const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
  uint8_t* stage0 = smem;
  const int tq_stride = (p.k_pad + 8) * 2;
  const int tq_bytes = (16 * tq_stride + 127) & ~127;
  uint8_t* tq = stage0 + (size_t)p.stages * p.stage_bytes;
  uint8_t* abuf = tq + tq_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(abuf + kAChunkBytes);
  int* misc = reinterpret_cast<int*>(bars + 3 * kMaxStages + 4);
  volatile int* abort_flag = misc;                 // misc[0]; misc[1], misc[2]: broadcast slots

  const uint32_t bar0 = smem_u32(bars);
  auto full = [&](int s) { return bar0 + 8u * s; };
  auto xready = [&](int s) { return bar0 + 8u * (kMaxStages + s); };
  auto empty = [&](int s) { return bar0 + 8u * (2 * kMaxStages + s); };
  const uint32_t afull = bar0 + 8u * (3 * kMaxStages);
  const uint32_t tq_ready = afull + 8u, t_bar = afull + 16u, c_bar = afull + 24u;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int G = gridDim.x, cta = blockIdx.x;
  const int S = p.stages;
  const int M = p.M;

  Seq seq;
  seq.init(range_lo(cta, p.total_units, G), range_lo(cta + 1, p.total_units, G), p.U, p.k_slabs);
  const int pre = min(seq.n, S);                   // units whose copies are issued before anything is consumed

  // ---- producer helpers (used by warp 0 only)
  Walker pw;
  auto issue_weights = [&](int st) {
    const uint32_t dst = smem_u32(stage0 + (size_t)st * p.stage_bytes);
    if (pw.j < p.k_slabs) {
      const int vc = min(kSlabK, p.K - pw.j * kSlabK);
      mbar_expect_tx(full(st), kWTileBytes + M * vc * 4);
      bulk_load(dst, p.wsec + ((size_t)pw.nt * p.k_slabs + pw.j) * kWTileBytes, kWTileBytes, full(st));
    } else {
      const int rb0 = (pw.j - p.k_slabs) * 2, nb = min(2, p.r_blocks - rb0);
      const uint8_t* tile = p.bsec + (size_t)pw.nt * ((size_t)p.r_blocks * kTileN * 17);
      mbar_expect_tx(full(st), nb * kTileN * 17);
      bulk_load(dst, tile + (size_t)rb0 * kTileN * 16, nb * kTileN * 16, full(st));
      bulk_load(dst + kWTileNibbleBytes, tile + (size_t)p.r_blocks * kTileN * 16 + rb0 * kTileN, nb * kTileN, full(st));
    }
  };
  auto issue_x = [&](int st) {                     // lane r copies row r's 64 columns of this slab
    if (pw.j < p.k_slabs && lane < M) {
      const int vc = min(kSlabK, p.K - pw.j * kSlabK);
      const uint32_t dst = smem_u32(stage0 + (size_t)st * p.stage_bytes + kWTileBytes + lane * 256);
      bulk_load(dst, p.X + (size_t)lane * p.K + (size_t)pw.j * kSlabK, vc * 4, full(st));
    }
  };

  pdl_launch_dependents();
  if (warp == 0) {
    // The producer sets the barriers up and starts the weight copies at once (they depend on no
    // earlier kernel); the other warps clear the tiles that must hold zeros meanwhile.
    if (lane == 0) {
      for (int s = 0; s < S; ++s) {
        mbar_init(full(s), 1);
        mbar_init(xready(s), kQuantWarps);
        mbar_init(empty(s), kQuantWarps + kConsumerWarps);
      }
      mbar_init(afull, 1);
      mbar_init(tq_ready, kTWarps);
      mbar_init(t_bar, kTWarps);
      mbar_init(c_bar, kConsumerWarps);
      for (int i = 0; i < 8; ++i) misc[i] = 0;
      fence_barrier_init();
      fence_proxy_async_smem();
      pw.start(seq);
      for (int i = 0; i < pre; ++i) { issue_weights(i); pw.step(seq, i + 1); }
    }
  } else {
    // rows >= M of every bf16 X tile and of T_q stay zero for the whole kernel
    const int zt = tid - 32, zn = kThreads - 32;
    for (int s = 0; s < S; ++s) {
      uint8_t* xb = stage0 + (size_t)s * p.stage_bytes + kWTileBytes + p.xf_bytes;
      for (int o = zt * 16; o < kXTileBytes; o += zn * 16) *reinterpret_cast<uint4*>(xb + o) = make_uint4(0u, 0u, 0u, 0u);
    }
    for (int o = zt * 16; o < tq_bytes; o += zn * 16) *reinterpret_cast<uint4*>(tq + o) = make_uint4(0u, 0u, 0u, 0u);
  }
  __syncthreads();

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    pdl_wait();                                                  // X may be an earlier kernel's output
    pw.start(seq);
    for (int i = 0; i < pre; ++i) { issue_x(i); pw.step(seq, i + 1); }
    int st = 0;
    uint32_t ph = 0;                                             // parity of the pass whose consumption is awaited
    for (int i = pre; i < seq.n; ++i) {
      if (!warp_wait<32>(empty(st), ph, abort_flag)) break;
      if (lane == 0) issue_weights(st);
      __syncwarp();
      issue_x(st);
      pw.step(seq, i + 1);
      if (++st == S) { st = 0; ph ^= 1; }
    }
  } else if (warp <= kQuantWarps) {
    // ------------------------------------------------------------------ quantisers
    pdl_wait();
    const int q = tid - 32;                    // 0..95
    Walker wk;
    wk.start(seq);
    int st = 0;
    uint32_t ph = 0;
    for (int i = 0; i < seq.n; ++i) {
      if (!warp_wait<32>(full(st), ph, abort_flag)) break;
      if (wk.j < p.k_slabs) {
        const int vc = min(kSlabK, p.K - wk.j * kSlabK);
        const uint8_t* xf = stage0 + (size_t)st * p.stage_bytes + kWTileBytes;
        uint8_t* xb = stage0 + (size_t)st * p.stage_bytes + kWTileBytes + p.xf_bytes;
        // one float4 (a quarter of a 16-block) per lane and pass; every lane runs every pass
        for (int f = q; f - q < M * 16; f += 32 * kQuantWarps) {
          const int row = f >> 4, c4 = f & 15;
          const bool ok = row < M;
          const float4 v = (ok && c4 * 4 < vc) ? *reinterpret_cast<const float4*>(xf + row * 256 + c4 * 16)
                                               : make_float4(0.f, 0.f, 0.f, 0.f);
          int e;
          uint32_t m8;
          uint2 bf;
          quantize_quad(v, p.a_bits, p.exp_min, p.exp_max, e, m8, bf);
          if (ok) *reinterpret_cast<uint2*>(xb + row * kXTileStride + c4 * 8) = bf;
        }
      }
      __syncwarp();
      if (lane == 0) { mbar_arrive(xready(st)); mbar_arrive(empty(st)); }
      wk.step(seq, i + 1);
      if (++st == S) { st = 0; ph ^= 1; }
    }
  } else if (warp <= kQuantWarps + kTWarps) {
    // ------------------------------------------------------------------ T = X_q A_q, then T_q
    const int tw = warp - 1 - kQuantWarps;           // 0..3
    const int tt = tid - 32 * (1 + kQuantWarps);     // 0..127
    uint32_t sync_use = 0;
    if (p.k_pad == 0) {
      pdl_wait();
    } else {
      const int KB = p.K / 16;
      const int kb_lo = (int)((long long)cta * KB / G), kb_hi = (int)((long long)(cta + 1) * KB / G);
      const int CH = p.a_chunk_blocks;
      const int NT = p.k_pad / 8;                    // 8-column rank tiles
      uint8_t* amant = abuf;
      uint8_t* aexp = abuf + (size_t)CH * p.k_pad * 16;
      uint8_t* xa = aexp + (size_t)CH * p.k_pad;     // [M][CH * 16] fp32
      const uint8_t* g_aexp = p.asec + (size_t)KB * p.k_pad * 16;
      const int bias = -127 - (p.a_bits - 2) - (p.lr_bits - 2);   // exponent bytes carry +127
      bool ok = true;
      int ci = 0;                                    // chunk loads so far (buffer hand-over, barrier parity)
      if (kb_lo >= kb_hi) pdl_wait();                // no share of K: still ordered behind earlier kernels
      // 16 rank tiles per pass (4 per warp); ranks above 128 take a second pass over the same blocks
      for (int pass = 0; pass * 16 < NT && ok && kb_lo < kb_hi; ++pass) {
        double acc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = 0.0;
        for (int c0 = kb_lo; c0 < kb_hi && ok; c0 += CH, ++ci) {
          const int nbc = min(CH, kb_hi - c0);
          if (ci > 0) ok = role_sync(t_bar, sync_use, abort_flag);      // everybody is done with the buffer
          if (tw == 0) {
            if (lane == 0) {
              mbar_expect_tx(afull, nbc * p.k_pad * 17 + M * nbc * 64);
              bulk_load(smem_u32(amant), p.asec + (size_t)c0 * p.k_pad * 16, nbc * p.k_pad * 16, afull);
              bulk_load(smem_u32(aexp), g_aexp + (size_t)c0 * p.k_pad, nbc * p.k_pad, afull);
            }
            __syncwarp();
            if (ci == 0) pdl_wait();
            if (lane < M) bulk_load(smem_u32(xa + (size_t)lane * CH * 64), p.X + (size_t)lane * p.K + (size_t)c0 * 16, nbc * 64, afull);
          } else if (ci == 0) {
            pdl_wait();
          }
          if (!warp_wait<32>(afull, ci & 1, abort_flag)) { ok = false; break; }
          for (int b = 0; b < nbc; ++b) {
            const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
            const float4 v0 = g < M ? *reinterpret_cast<const float4*>(xa + ((size_t)g * CH * 16 + b * 16 + t * 4) * 4) : z;
            const float4 v1 = g + 8 < M ? *reinterpret_cast<const float4*>(xa + ((size_t)(g + 8) * CH * 16 + b * 16 + t * 4) * 4) : z;
            int e0, e1;
            uint32_t m0, m1;
            uint2 unused;
            quantize_quad(v0, p.a_bits, p.exp_min, p.exp_max, e0, m0, unused);
            quantize_quad(v1, p.a_bits, p.exp_min, p.exp_max, e1, m1, unused);
            const int ex0 = e0 + bias, ex1 = e1 + bias;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int nt = pass * 16 + tw + 4 * i;
              if (nt < NT) {
                const uint32_t b0 = *reinterpret_cast<const uint32_t*>(amant + ((size_t)(b * p.k_pad + nt * 8 + g) * 16) + t * 4);
                const uint32_t ea2 = *reinterpret_cast<const uint16_t*>(aexp + b * p.k_pad + nt * 8 + t * 2);
                int c[4];
                mma_s8(c, m0, m1, b0);
                const int ea_lo = (int)(ea2 & 0xFFu), ea_hi = (int)(ea2 >> 8);
                acc[i][0] = fma((double)c[0], pow2d(ex0 + ea_lo), acc[i][0]);
                acc[i][1] = fma((double)c[1], pow2d(ex0 + ea_hi), acc[i][1]);
                acc[i][2] = fma((double)c[2], pow2d(ex1 + ea_lo), acc[i][2]);
                acc[i][3] = fma((double)c[3], pow2d(ex1 + ea_hi), acc[i][3]);
              }
            }
          }
        }
        // contribution of this CTA (exact partial sums; fp64 addition of them is exact as well
        // unless the block exponents of one row spread over more than about 30 binades)
        if (ok) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int nt = pass * 16 + tw + 4 * i;
            if (nt < NT) {
              const int col = nt * 8 + t * 2;
              if (g < M) { atomicAdd(p.tacc + (size_t)g * p.k_pad + col, acc[i][0]); atomicAdd(p.tacc + (size_t)g * p.k_pad + col + 1, acc[i][1]); }
              if (g + 8 < M) { atomicAdd(p.tacc + (size_t)(g + 8) * p.k_pad + col, acc[i][2]); atomicAdd(p.tacc + (size_t)(g + 8) * p.k_pad + col + 1, acc[i][3]); }
            }
          }
        }
      }
      __threadfence();
      role_sync(t_bar, sync_use, abort_flag);
      if (tt == 0) atomicAdd(p.tcount, 1);

      // does this CTA own rank units?
      bool has_rank = false;
      if (seq.n > 0) has_rank = seq.nt_first != seq.nt_last || seq.hi > seq.nt_first * p.U + p.k_slabs;
      if (has_rank) {
        if (tt == 0) {                                // bounded wait for the contributions of all CTAs
          const long long t0 = clock64();
          while (ld_acquire(p.tcount) < G) {
            __nanosleep(100);
            if (*abort_flag != 0) break;
            if (clock64() - t0 > WAIT_LIMIT_CYCLES) { *abort_flag = 2; break; }
          }
        }
        role_sync(t_bar, sync_use, abort_flag);
        __threadfence();
        // T -> MXINT8 along the rank (16 adjacent lanes hold one block) -> exact bf16 in shared memory
        const int total = M * p.k_pad;
        for (int base = 0; base < total; base += 32 * kTWarps) {
          const int idx = base + tt;
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
        __syncwarp();
        if (lane == 0) mbar_arrive(tq_ready);
      }
      // the last CTA that is done with the accumulator leaves it zero for the next call
      role_sync(t_bar, sync_use, abort_flag);
      if (tt == 0) misc[1] = (atomicAdd(p.tdone, 1) == G - 1) ? 1 : 0;
      role_sync(t_bar, sync_use, abort_flag);
      if (misc[1] != 0) {
        __threadfence();
        for (int o = tt; o < 16 * p.k_pad; o += 32 * kTWarps) p.tacc[o] = 0.0;
        if (tt == 0) { *p.tcount = 0; *p.tdone = 0; }
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers
    pdl_wait();
    const int cw = warp - 1 - kQuantWarps - kTWarps;     // 0..7: columns [16 cw, 16 cw + 16) of the tile
    const int ctid = tid - 32 * (1 + kQuantWarps + kTWarps);
    uint32_t sync_use = 0;
    float acc[2][4], acc_head[2][4];
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) { acc[i][j] = 0.f; acc_head[i][j] = 0.f; }

    // Contributors of the (at most two) column tiles this CTA covers only in part: CTAs
    // c_first..c_last, and the slot the first of them uses (every later one starts inside the
    // tile and uses its slot 0).  Computed once, while the first copies are in flight.
    int part_first[2], part_last[2], part_slot0[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int nt = e == 0 ? seq.nt_first : seq.nt_last;
      part_first[e] = cta_of(nt * p.U, p.total_units, G);
      part_last[e] = cta_of((nt + 1) * p.U - 1, p.total_units, G);
      part_slot0[e] = (range_lo(part_first[e], p.total_units, G) / p.U == nt) ? 0 : 1;
    }

    // Hand the partial sums of column tile nt over: straight to Y when this CTA covered the whole
    // contraction of the tile, otherwise through a slot; the last arriver adds the slots in CTA order.
    auto flush = [&](int nt) {
      const bool complete = nt * p.U >= seq.lo && (nt + 1) * p.U <= seq.hi;
      const int cl = cw * 16 + t * 2;                    // + 8 cg: column within the tile
      if (complete) {
#pragma unroll
        for (int cg = 0; cg < 2; ++cg) {
          const int col = nt * kTileN + cl + 8 * cg;
          if (col < p.N) {
            if (g < M) *reinterpret_cast<float2*>(p.Y + (size_t)g * p.N + col) = make_float2(acc[cg][0], acc[cg][1]);
            if (g + 8 < M) *reinterpret_cast<float2*>(p.Y + (size_t)(g + 8) * p.N + col) = make_float2(acc[cg][2], acc[cg][3]);
          }
        }
        return;
      }
      float* slot = p.slots + ((size_t)cta * 2 + (nt == seq.nt_first ? 0 : 1)) * kSlotFloats;
#pragma unroll
      for (int cg = 0; cg < 2; ++cg) {
        if (g < M) __stcg(reinterpret_cast<float2*>(slot + g * kTileN + cl + 8 * cg), make_float2(acc[cg][0], acc[cg][1]));
        if (g + 8 < M) __stcg(reinterpret_cast<float2*>(slot + (g + 8) * kTileN + cl + 8 * cg), make_float2(acc[cg][2], acc[cg][3]));
      }
      __threadfence();
      role_sync(c_bar, sync_use, abort_flag);
      const int e = nt == seq.nt_first ? 0 : 1;
      const int c_first = part_first[e], c_last = part_last[e];
      if (ctid == 0) misc[2] = (atomicAdd(p.cnt + nt, 1) == c_last - c_first) ? 1 : 0;
      role_sync(c_bar, sync_use, abort_flag);
      if (misc[2] != 0) {
        __threadfence();
        float2 s[2][2];
#pragma unroll
        for (int cg = 0; cg < 2; ++cg) { s[cg][0] = make_float2(0.f, 0.f); s[cg][1] = make_float2(0.f, 0.f); }
        for (int cc = c_first; cc <= c_last; ++cc) {
          const float* src = p.slots + ((size_t)cc * 2 + (cc == c_first ? part_slot0[e] : 0)) * kSlotFloats;
#pragma unroll
          for (int cg = 0; cg < 2; ++cg) {
            if (g < M) { const float2 v = __ldcg(reinterpret_cast<const float2*>(src + g * kTileN + cl + 8 * cg)); s[cg][0].x += v.x; s[cg][0].y += v.y; }
            if (g + 8 < M) { const float2 v = __ldcg(reinterpret_cast<const float2*>(src + (g + 8) * kTileN + cl + 8 * cg)); s[cg][1].x += v.x; s[cg][1].y += v.y; }
          }
        }
#pragma unroll
        for (int cg = 0; cg < 2; ++cg) {
          const int col = nt * kTileN + cl + 8 * cg;
          if (col < p.N) {
            if (g < M) *reinterpret_cast<float2*>(p.Y + (size_t)g * p.N + col) = s[cg][0];
            if (g + 8 < M) *reinterpret_cast<float2*>(p.Y + (size_t)(g + 8) * p.N + col) = s[cg][1];
          }
        }
        if (ctid == 0) p.cnt[nt] = 0;                  // every contributor has arrived: ready for the next call
      }
      role_sync(c_bar, sync_use, abort_flag);          // misc[2] may be rewritten after this
    };

    int cur_nt = -1;
    bool tq_waited = false;
    Walker wk;
    wk.start(seq);
    int st = 0;
    uint32_t ph = 0;
    for (int i = 0; i < seq.n; ++i) {
      const int nt = wk.nt, j = wk.j;
      if (seq.reordered && i == seq.n_before) {
        // the deferred rank units of the first column tile: finish the current tile, resume the first
        if (cur_nt >= 0) flush(cur_nt);
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
          for (int b = 0; b < 4; ++b) acc[a][b] = acc_head[a][b];
        cur_nt = nt;
      } else if (nt != cur_nt) {
        if (cur_nt >= 0) {
          if (seq.reordered && cur_nt == seq.nt_first) {
#pragma unroll
            for (int a = 0; a < 2; ++a)
#pragma unroll
              for (int b = 0; b < 4; ++b) acc_head[a][b] = acc[a][b];
          } else {
            flush(cur_nt);
          }
        }
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
          for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
        cur_nt = nt;
      }
      if (!warp_wait<20>(full(st), ph, abort_flag)) break;
      if (!warp_wait<20>(xready(st), ph, abort_flag)) break;
      const uint8_t* stage = stage0 + (size_t)st * p.stage_bytes;
      if (j < p.k_slabs) {
        // ---- 64 K of W_q: lane (g, t) holds block t of the slab for row g (A side) and column g (B side)
        const uint8_t* xb = stage + kWTileBytes + p.xf_bytes;
        const uint4 q0 = *reinterpret_cast<const uint4*>(xb + g * kXTileStride + t * 32);
        const uint4 q1 = *reinterpret_cast<const uint4*>(xb + g * kXTileStride + t * 32 + 16);
        uint4 r0 = make_uint4(0u, 0u, 0u, 0u), r1 = r0;
        if (M > 8) {
          r0 = *reinterpret_cast<const uint4*>(xb + (g + 8) * kXTileStride + t * 32);
          r1 = *reinterpret_cast<const uint4*>(xb + (g + 8) * kXTileStride + t * 32 + 16);
        }
#pragma unroll
        for (int cg = 0; cg < 2; ++cg) {
          const int col = cw * 16 + cg * 8 + g;
          const uint2 w = *reinterpret_cast<const uint2*>(stage + (t >> 1) * (kTileN * 16) + col * 16 + (t & 1) * 8);
          const uint32_t eb = stage[kWTileNibbleBytes + col * 4 + t];
          uint32_t s2, c2;
          w_scales(eb, s2, c2);
          const uint4 b0 = convert_word(w.x, s2, c2), b1 = convert_word(w.y, s2, c2);
          mma_bf16(acc[cg], q0.x, r0.x, q0.y, r0.y, b0.x, b0.y);
          mma_bf16(acc[cg], q0.z, r0.z, q0.w, r0.w, b0.z, b0.w);
          mma_bf16(acc[cg], q1.x, r1.x, q1.y, r1.y, b1.x, b1.y);
          mma_bf16(acc[cg], q1.z, r1.z, q1.w, r1.w, b1.z, b1.w);
        }
      } else {
        // ---- 32 rank values of B_q against T_q
        if (!tq_waited) {
          if (!warp_wait<32>(tq_ready, 0u, abort_flag)) break;
          tq_waited = true;
        }
        const int rb0 = (j - p.k_slabs) * 2, nb = min(2, p.r_blocks - rb0);
        for (int rb = 0; rb < nb; ++rb) {
          const uint2 a_lo = *reinterpret_cast<const uint2*>(tq + g * tq_stride + ((rb0 + rb) * 16 + t * 4) * 2);
          uint2 a_hi = make_uint2(0u, 0u);
          if (M > 8) a_hi = *reinterpret_cast<const uint2*>(tq + (g + 8) * tq_stride + ((rb0 + rb) * 16 + t * 4) * 2);
#pragma unroll
          for (int cg = 0; cg < 2; ++cg) {
            const int col = cw * 16 + cg * 8 + g;
            const uint32_t wv = *reinterpret_cast<const uint32_t*>(stage + (rb * kTileN + col) * 16 + t * 4);
            const float scale = pow2f((int)stage[kWTileNibbleBytes + rb * kTileN + col] - 127 - (p.lr_bits - 2));
            const uint32_t b0 = pack_bf16x2((float)(int8_t)(wv) * scale, (float)(int8_t)(wv >> 8) * scale);
            const uint32_t b1 = pack_bf16x2((float)(int8_t)(wv >> 16) * scale, (float)(int8_t)(wv >> 24) * scale);
            mma_bf16(acc[cg], a_lo.x, a_hi.x, a_lo.y, a_hi.y, b0, b1);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty(st));
      wk.step(seq, i + 1);
      if (++st == S) { st = 0; ph ^= 1; }
    }
    if (cur_nt >= 0 && *abort_flag == 0) flush(cur_nt);
  }

  // ------------------------------------------------------------------ teardown
  __syncthreads();
  if (*abort_flag != 0) {
    // a wait ran out: give copies that may still be in flight time to land before shared memory goes away
    const long long t0 = clock64();
    while (clock64() - t0 < 400000) { }
    if (tid == 0) report_error(p.status, LQER_ERR_TIMEOUT, 500 + *abort_flag, cta);
  }
}

}  // namespace dec

int decode_max_m() { return 16; }

cudaError_t launch_decode(const float* X, int M, const PackedMeta& m, const void* packed, float* Y, void* workspace,
                          cudaStream_t s) {
  using namespace dec;
  static int sm_count = 0;
  static bool attr_set = false;
  if (!attr_set) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
    cudaError_t e = cudaFuncSetAttribute(decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
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
  p.cnt = reinterpret_cast<int*>(ws + kStatusBytes);
  p.tacc = reinterpret_cast<double*>(ws + tacc_offset(m));
  p.slots = reinterpret_cast<float*>(ws + ((persist_bytes(m) + 255) & ~(size_t)255));
  p.M = M; p.K = m.K; p.N = m.N; p.k_pad = m.k_pad;
  p.n_tiles = m.n_tiles; p.k_slabs = m.k_slabs; p.r_blocks = m.r_blocks;
  p.U = m.k_slabs + (m.r_blocks + 1) / 2;
  p.total_units = decode_units(m);
  p.a_bits = m.a_bits; p.lr_bits = m.lr_bits; p.exp_min = m.exp_min; p.exp_max = m.exp_max;

  const int G = decode_ctas(m, sm_count);
  p.xf_bytes = M * 256;
  p.stage_bytes = kWTileBytes + p.xf_bytes + kXTileBytes;
  const int tq_bytes = (16 * (m.k_pad + 8) * 2 + 127) & ~127;
  const int fixed = tq_bytes + kAChunkBytes + (3 * kMaxStages + 4) * 8 + 64 + 128;
  const int per_cta = (p.total_units + G - 1) / G;
  int stages = (kSmemBudget - fixed) / p.stage_bytes;
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages > per_cta) stages = per_cta;
  if (stages < 1) return cudaErrorInvalidValue;
  p.stages = stages;
  p.a_chunk_blocks = 1;
  if (m.k_pad > 0) {
    const int KB = m.K / 16;
    const int need = (KB + G - 1) / G;
    const int fit = kAChunkBytes / (m.k_pad * 17 + M * 64);
    if (fit < 1) return cudaErrorInvalidValue;
    p.a_chunk_blocks = need < fit ? need : fit;
  }
  const size_t smem = (size_t)stages * p.stage_bytes + fixed;

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
