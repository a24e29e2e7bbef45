// Activation prologue of the prefill path for large batches, with the projection on the
// 5th-generation tensor cores (paper Section 4.1: X_q in MXINT8, blocks [1,16]; Section 3.1:
// the small high-precision product X A_k).
//
// Same results as prologue_kernel (bit for bit in X_q and T_q); what differs is where the work
// runs.  A CTA owns 128 rows of X and one of `splits` ranges of K; the CTAs of a row tile leave
// fp64 partial sums in global scratch and, once all have arrived, each adds up a share of the rows
// in a fixed order.
//   scalers      read the int32 block products from tensor memory, scale each by 2^(e_x + e_a)
//                and sum in fp64 (exact for any realistic exponent spread)
//   quantisers   take X (fp32 or bf16) from a shared-memory ring that TMA fills, a whole 16-block per lane, write
//                the exact bf16 values m * 2^(e-6) to Xcat, the int8 mantissas to shared memory in the K-major
//                128-byte-swizzled layout the MMA reads, and the block exponents beside them
//   panel warp   A_q panels: 16-byte asynchronous copies into a block-diagonal operand
//   issuer warp  one lane issues tcgen05.mma kind::i8 (M=128, N=2*k_pad, K=32)
//   TMA warp     one lane keeps the ring of X full (128 rows x 64 columns per stage, in 128-byte-wide swizzled boxes)
// Each 16-block needs its own integer product, because its scale differs from its neighbour's.
// The int8 MMA contracts 32 values, so the B operand of a block pair is laid out as
//     rows 0..k_pad-1:        [A_b | 0]        rows k_pad..2 k_pad-1:  [0 | A_{b+1}]
// and one MMA yields X_b A_b in the first k_pad accumulator columns and X_{b+1} A_{b+1} in the
// next k_pad.  The zero halves are written once; only the diagonal chunks change per panel.
#include "lqer_tc_ptx.cuh"

namespace lqer {
namespace ptc {

using namespace tc;

constexpr int ROWS = 128;                    // rows of X per CTA = one MMA M tile
constexpr int STAGE_COLS = 64;               // columns of X per stage: 4 blocks = 2 block pairs
constexpr int RAW_SLOTS = 4;                 // fp32 ring
constexpr int RAW_BYTES = ROWS * STAGE_COLS * 4;   // 32768
constexpr int X_SLOTS = 4;                   // int8 ring of stages; two stages share one 128-byte-row buffer
constexpr int XBUF_BYTES = ROWS * 128;       // 16384: 128 rows x 128 int8 (8 blocks), swizzled
constexpr int PANELS = 3;                    // ring of A_q panels (8 blocks each)
constexpr int WORK_WARPS = 24;               // scalers + quantisers
constexpr int NUM_WARPS = WORK_WARPS + 3;
constexpr int NUM_THREADS = NUM_WARPS * 32;  // 864
constexpr int MAX_TMEM_SLOTS = 8;
constexpr unsigned kNapNs = 100;              // sleep between polls of the roles that run ahead of the scalers

template <int KP>
struct Cfg {
  static constexpr int SCALER_WARPS = KP >= 32 ? 16 : 8;     // four lane quarters x column groups
  static constexpr int QUANT_WARPS = WORK_WARPS - SCALER_WARPS;
  static constexpr int CPW = KP / (SCALER_WARPS / 4);        // rank columns per scaler warp
  static constexpr int BPL = ROWS / (QUANT_WARPS * 8);       // 16-blocks per quantiser lane and stage (a warp: 8 rows x 4 blocks)
  static constexpr int SLOT_COLS = 2 * KP;                   // accumulator columns per block pair
  static constexpr int TMEM_SLOTS = (512 / SLOT_COLS) < MAX_TMEM_SLOTS ? (512 / SLOT_COLS) : MAX_TMEM_SLOTS;
  static constexpr int TMEM_COLS = 512;
  // The quantisers hand registers to the scalers (whole warpgroups each; the CTA was launched with 27 x 72 per lane):
  // 8 x 88 + 16 x 64 + 3 x 72 with 8 scaler warps (k_pad 16), 16 x 80 + 8 x 56 + 3 x 72 with 16 scaler warps of 16
  // columns (k_pad 64).  At k_pad 32 (16 scaler warps of 8 columns) nobody is short of registers and the shift only
  // slowed the quantisers.
  static constexpr bool REG_SHIFT = CPW == 16 || SCALER_WARPS == 8;
  static constexpr int SCALER_REGS = SCALER_WARPS == 8 ? 88 : 80;
  static constexpr int QUANT_REGS = SCALER_WARPS == 8 ? 64 : 56;
  static constexpr int PANEL_BYTES = 2 * KP * 128;           // 2 k_pad rows x 128 bytes
  static constexpr int OFF_XQ = RAW_SLOTS * RAW_BYTES;
  static constexpr int OFF_PANEL = OFF_XQ + (X_SLOTS / 2) * XBUF_BYTES;
  static constexpr int OFF_XE = OFF_PANEL + PANELS * PANEL_BYTES;   // [X_SLOTS][ROWS][4] block exponents
  static constexpr int OFF_HIA = OFF_XE + X_SLOTS * ROWS * 4;       // [PANELS][8][KP] high words of 2^(e_a + bias)
  static constexpr int OFF_BARS = OFF_HIA + PANELS * 8 * KP * 4;
  static constexpr int NUM_BARS = 2 * RAW_SLOTS + 2 * X_SLOTS + 2 * PANELS + 2 * MAX_TMEM_SLOTS;
  static constexpr int SMEM_BYTES = OFF_BARS + NUM_BARS * 8 + 32 + 1024;
  static_assert(CPW % 8 == 0 && CPW <= 16, "scaler registers");
  static_assert(ROWS % (QUANT_WARPS * 8) == 0, "quantiser passes");
  static_assert(PANEL_BYTES % 1024 == 0, "swizzle atoms need 1024-byte bases");
  static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
};

struct Params {
  const uint8_t* asec;      // A_q section of the packed buffer: mantissas then exponents
  uint16_t* xcat;
  int8_t* Tm;               // optional exports of T_q
  uint8_t* Te;
  DeviceStatus* status;
  double* partials;         // [row tile][split][128][k_pad]
  int* counters;            // [row tile][arrivals, departures], zero between calls
  int M, K, K64;
  int kblocks;              // K / 16
  int panels;               // ceil(K64 / 128)
  int splits;               // CTAs per row tile
  int expect;               // arrivals a row tile waits for: splits (one more under the stall test hook)
  long long wait_limit;     // bound of every wait, in clock cycles
  int a_bits, lr_bits, exp_min, exp_max;
  int order;                // ChainOrder: where the wait for the previous kernel sits
  int x_type;               // kXF32 (a stage of the ring holds 32 KB), kXBF16 (16 KB) or kXMXINT8 (8 KB of mantissas)
  const uint8_t* x_exp;     // MXINT X: its exponent bytes [M, K / 16]
  size_t ldx;               // columns of Xcat
  size_t xcat_extent, partials_extent;   // bytes behind xcat and partials, for the checked build
};

// Up to kMaxLayers independent layers with one M, one rank padding and one set of formats may share a launch: a
// CTA finds its layer by its index (cta_begin) and then works as in a launch of that layer alone.
constexpr int kMaxLayers = 8;
struct GroupParams {
  Params L[kMaxLayers];
  int cta_begin[kMaxLayers];
  int n;
};
struct TensorMaps {
  CUtensorMap m[kMaxLayers];   // X of each layer: [M, K], box 128 bytes (32 fp32 or 64 bf16) x 128 rows, 128-byte swizzle
};

// int8 x int8 -> int32, both operands K-major, M = m, N = n.
__host__ __device__ constexpr uint32_t make_idesc_i8(int m, int n) {
  return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
// D = A B (the accumulator is overwritten).
__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, 0, 0;\n tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr) : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// try_wait with a suspend-time hint: the hardware parks the thread until the phase completes or the hint
// (nanoseconds) runs out, so a waiting role takes few issue slots from the working ones.
__device__ __forceinline__ bool mbar_try_wait_parked(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok) : "r"(bar), "r"(parity), "r"(20000u) : "memory");
  return ok != 0;
}
// Bounded like tc::mbar_wait: gives up after the launch's wait limit or as soon as another role has given up.
// nap_ns > 0: the role is ahead of the one it waits for, so it sleeps between polls and leaves the issue slots to
// the roles that work (a polling warp is eligible every cycle and competes with them).
__device__ __forceinline__ bool parked_wait(uint32_t bar, uint32_t parity, volatile WaitState* abort_flag, unsigned nap_ns = 0) {
  if (mbar_try_wait_parked(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait_parked(bar, parity)) {
    if (nap_ns) __nanosleep(nap_ns);
    if (abort_flag->abort != 0) return false;
    if (clock64() - t0 > abort_flag->limit) { abort_flag->abort = 1; return false; }
  }
  return true;
}
// A wait whose outcome every lane of the warp shares (the code after it shuffles or touches tensor memory as a warp).
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, volatile WaitState* abort_flag, unsigned nap_ns = 0) {
  return __all_sync(0xFFFFFFFFu, parked_wait(bar, parity, abort_flag, nap_ns)) != 0;
}

template <int KP>
__global__ void __launch_bounds__(NUM_THREADS, 1) prologue_tc_kernel(const __grid_constant__ TensorMaps tmaps,
                                                                     const __grid_constant__ GroupParams gp) {
  using C = Cfg<KP>;
  int layer = 0;
#pragma unroll
  for (int i = 1; i < kMaxLayers; ++i)
    if (i < gp.n && (int)blockIdx.x >= gp.cta_begin[i]) layer = i;
  const Params& p = gp.L[layer];
  const CUtensorMap* const tmap_x = &tmaps.m[layer];
  const int bid = (int)blockIdx.x - gp.cta_begin[layer];          // index within the layer's CTAs
  constexpr int SW = C::SCALER_WARPS, QW = C::QUANT_WARPS, CPW = C::CPW;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* raw_base = smem;
  uint8_t* xq_base = smem + C::OFF_XQ;
  uint8_t* panel_base = smem + C::OFF_PANEL;
  int8_t* s_xe = reinterpret_cast<int8_t*>(smem + C::OFF_XE);
  int* s_hia = reinterpret_cast<int*>(smem + C::OFF_HIA);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BARS);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + C::NUM_BARS);
  int* last_flag = reinterpret_cast<int*>(tmem_slot + 1);
  volatile WaitState* abort_flag = reinterpret_cast<volatile WaitState*>(tmem_slot + 2);

  const uint32_t bar0 = smem_u32(bars);
  auto raw_full = [&](int s) { return bar0 + 8u * s; };
  auto raw_empty = [&](int s) { return bar0 + 8u * (RAW_SLOTS + s); };
  auto xq_full = [&](int s) { return bar0 + 8u * (2 * RAW_SLOTS + s); };
  auto xq_empty = [&](int s) { return bar0 + 8u * (2 * RAW_SLOTS + X_SLOTS + s); };
  auto panel_full = [&](int s) { return bar0 + 8u * (2 * RAW_SLOTS + 2 * X_SLOTS + s); };
  auto panel_empty = [&](int s) { return bar0 + 8u * (2 * RAW_SLOTS + 2 * X_SLOTS + PANELS + s); };
  auto slot_full = [&](int s) { return bar0 + 8u * (2 * RAW_SLOTS + 2 * X_SLOTS + 2 * PANELS + s); };
  auto slot_empty = [&](int s) { return bar0 + 8u * (2 * RAW_SLOTS + 2 * X_SLOTS + 2 * PANELS + MAX_TMEM_SLOTS + s); };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int row_tile = bid / p.splits, split = bid % p.splits;
  const int row0 = row_tile * ROWS;
  const int pan_lo = (int)((long long)split * p.panels / p.splits);
  const int pan_hi = (int)((long long)(split + 1) * p.panels / p.splits);
  const int n_stages = 2 * (pan_hi - pan_lo);
  const uint8_t* a_exp = p.asec + (size_t)p.kblocks * KP * 16;

  // zero halves of the block-diagonal panels (never written again)
  for (int i = tid; i < PANELS * C::PANEL_BYTES / 16; i += NUM_THREADS)
    reinterpret_cast<uint4*>(panel_base)[i] = make_uint4(0u, 0u, 0u, 0u);
  if (tid == 0) {
    for (int s = 0; s < RAW_SLOTS; ++s) { mbar_init(raw_full(s), 1); mbar_init(raw_empty(s), QW); }
    for (int s = 0; s < X_SLOTS; ++s) { mbar_init(xq_full(s), QW); mbar_init(xq_empty(s), SW + 1); }
    for (int s = 0; s < PANELS; ++s) { mbar_init(panel_full(s), 1); mbar_init(panel_empty(s), SW + 1); }
    for (int s = 0; s < MAX_TMEM_SLOTS; ++s) { mbar_init(slot_full(s), 1); mbar_init(slot_empty(s), SW); }
    abort_flag->abort = 0;
    abort_flag->limit = p.wait_limit;
    fence_barrier_init();
  }
  fence_proxy_async_smem();
  if (warp == WORK_WARPS + 1) tmem_alloc(smem_u32(tmem_slot), C::TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Set up.  Alone: the next kernel may start its own setup at once; X, Xcat and the scratch may still be in use by
  // an earlier kernel, so the work waits for it.  First of a group of independent prologues: the next one starts
  // only once the earlier kernels are done, since it does not wait before it works.  Later in a group: nothing here
  // is shared with the prologue before, so the work starts at once and only the exit waits for it (a kernel after
  // the group then finds all of them complete).
  if (p.order == kChainFirst) {
    pdl_wait();
    pdl_launch_dependents();
  } else {
    pdl_launch_dependents();
    if (p.order == kChainAlone) pdl_wait();
  }

  if (warp < SW) {
    // ------------------------------------------------------------------ scalers
    if (C::REG_SHIFT) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(C::SCALER_REGS) : "memory");   // registers the quantisers gave up
    const int q = warp & 3, h = warp >> 2;
    const int row = q * 32 + lane;
    double acc[CPW];
#pragma unroll
    for (int i = 0; i < CPW; ++i) acc[i] = 0.0;
    bool ok = true;
    for (int s = 0; s < n_stages && ok; ++s) {
      const int xs = s % X_SLOTS, pp = s >> 1, pb = pp % PANELS;
      if ((s & 1) == 0 && !warp_wait(panel_full(pb), (pp / PANELS) & 1, abort_flag)) { ok = false; break; }
      if (!warp_wait(xq_full(xs), (s / X_SLOTS) & 1, abort_flag)) { ok = false; break; }
      const uint32_t e4 = *reinterpret_cast<const uint32_t*>(s_xe + (xs * ROWS + row) * 4);
      __syncwarp();
      if (lane == 0) mbar_arrive(xq_empty(xs));
      const int* hia = s_hia + (pb * 8 + (s & 1) * 4) * KP;
#pragma unroll 1
      for (int j = 0; j < 2; ++j) {
        const int u = 2 * s + j, slot = u % C::TMEM_SLOTS;
        if (!warp_wait(slot_full(slot), (u / C::TMEM_SLOTS) & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        // As few round trips to tensor memory as the registers allow: with 8 columns per warp both blocks of the
        // slot are loaded together and waited for once, with 16 a block at a time.  The slot is free again as soon
        // as its last values are in registers, before the arithmetic on them.
        constexpr int LB = CPW == 8 ? 2 : 1;                              // blocks per round trip
        const double kMagic = 4503601774854144.0;                         // 2^52 + 2^31
#pragma unroll
        for (int trip = 0; trip < 2 / LB; ++trip) {
          uint32_t c[LB][CPW];
#pragma unroll
          for (int lb = 0; lb < LB; ++lb) {
            const int blk = trip * LB + lb;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + slot * C::SLOT_COLS + blk * KP + h * CPW;
#pragma unroll
            for (int g8 = 0; g8 < CPW / 8; ++g8) tmem_ld8(taddr + g8 * 8, c[lb] + g8 * 8);
          }
          tmem_ld_wait();
          if (trip == 2 / LB - 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(slot_empty(slot));
          }
#pragma unroll
          for (int lb = 0; lb < LB; ++lb) {
            const int bi = 2 * j + trip * LB + lb;                        // block within the stage
            const int ehi = (int)(int8_t)(e4 >> (8 * bi)) * (1 << 20);
            const int* hrow = hia + bi * KP + h * CPW;
#pragma unroll
            for (int g = 0; g < CPW / 4; ++g) {
              const int4 hv = *reinterpret_cast<const int4*>(hrow + 4 * g);
              double* a = acc + 4 * g;
              const uint32_t* cc = c[lb] + 4 * g;
              // int32 -> fp64 without the conversion unit: 2^52 + 2^31 + c has the bits (0x43300000, c ^ 2^31)
              a[0] = fma(__hiloint2double(0x43300000, (int)(cc[0] ^ 0x80000000u)) - kMagic, __hiloint2double(hv.x + ehi, 0), a[0]);
              a[1] = fma(__hiloint2double(0x43300000, (int)(cc[1] ^ 0x80000000u)) - kMagic, __hiloint2double(hv.y + ehi, 0), a[1]);
              a[2] = fma(__hiloint2double(0x43300000, (int)(cc[2] ^ 0x80000000u)) - kMagic, __hiloint2double(hv.z + ehi, 0), a[2]);
              a[3] = fma(__hiloint2double(0x43300000, (int)(cc[3] ^ 0x80000000u)) - kMagic, __hiloint2double(hv.w + ehi, 0), a[3]);
            }
          }
        }
      }
      if (ok && (s & 1)) {                                              // done with the panel's exponent table
        __syncwarp();
        if (lane == 0) mbar_arrive(panel_empty(pb));
      }
    }
    // partial sums of this CTA's K range -> global scratch
    double* dst = p.partials + ((size_t)bid * ROWS + row) * KP + h * CPW;
    if (LQER_IN_BOUNDS(p.status, (size_t)(dst - p.partials) * 8, CPW * 8, p.partials_extent, 302)) {
#pragma unroll
      for (int i = 0; i < CPW; i += 2) *reinterpret_cast<double2*>(dst + i) = make_double2(acc[i], acc[i + 1]);
    }
  } else if (warp < WORK_WARPS) {
    // ------------------------------------------------------------------ quantisers
    // A lane owns a whole 16-block of a row: lanes 0-7 of a warp take block 0 of eight consecutive rows, lanes 8-15
    // block 1, and so on, so that every quarter warp reads and writes eight different 16-byte chunks of the swizzled
    // tiles (no bank conflicts) and the warp stores 8 rows x 128 contiguous bytes of Xcat.
    if (C::REG_SHIFT) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(C::QUANT_REGS) : "memory");
    const int qwarp = warp - SW;
    const int blk = lane >> 3;                         // 16-block within the 64-column stage
    const int r0 = qwarp * 8 + (lane & 7);             // first row (then + 8 * QW per pass)
    const uint32_t swz = (uint32_t)(lane & 7);         // row & 7: the rows of a pass differ by multiples of 8
    const QuantConsts qc = quant_consts(p.a_bits, p.exp_min, p.exp_max);
    uint16_t* cp = p.xcat + (size_t)(row0 + r0) * p.ldx + pan_lo * 2 * STAGE_COLS + blk * 16;
    const size_t c_step = (size_t)(8 * QW) * p.ldx;
    const int rows_ok = p.M - (row0 + r0);              // pass i is a real row while 8 * QW * i < rows_ok
    // offsets of the lane's block within a raw slot: fp32 = two half tiles of 32 columns (16 KB each, rows of 128
    // bytes), the block is four chunks; bf16 = one tile of 64 columns, the block is two chunks
    // an MXINT X: the tile is 128 rows of 64 mantissa bytes (64-byte swizzle: chunk ^ (row / 2 mod 4)), the block one chunk
    const uint32_t raw_off = p.x_type == kXMXINT8 ? (uint32_t)(r0 * 64)
                             : p.x_type == kXBF16 ? (uint32_t)(r0 * 128) : (uint32_t)((blk >> 1) * (RAW_BYTES / 2) + r0 * 128);
    const uint32_t chunk0 = p.x_type == kXBF16 ? (uint32_t)(blk * 2) : (uint32_t)((blk & 1) * 4);
    const uint32_t swz64 = (uint32_t)((lane >> 1) & 3);   // (row >> 1) & 3: the rows of a pass differ by multiples of 8
    const int kb_row = p.K / 16;
    bool ok = true;
    for (int s = 0; s < n_stages && ok; ++s) {
      const int rs = s % RAW_SLOTS, xs = s % X_SLOTS;
      if (!warp_wait(raw_full(rs), (s / RAW_SLOTS) & 1, abort_flag, kNapNs)) { ok = false; break; }
      if (!warp_wait(xq_empty(xs), ((s / X_SLOTS) & 1) ^ 1, abort_flag, kNapNs)) { ok = false; break; }
      const uint8_t* src = raw_base + rs * RAW_BYTES + raw_off;
      const uint32_t chunk = (uint32_t)((xs & 1) * 4 + blk);     // 16-byte chunk of the 128-byte row of mantissas
      uint8_t* xdst = xq_base + (xs >> 1) * XBUF_BYTES + r0 * 128 + ((chunk ^ swz) << 4);
      int8_t* xe_dst = s_xe + (xs * ROWS + r0) * 4 + blk;
      const bool store_ok = (pan_lo * 2 + s) * STAGE_COLS < p.K64;
      uint16_t* cd = cp + (size_t)s * STAGE_COLS;
#pragma unroll
      for (int i = 0; i < C::BPL; ++i) {
        const uint8_t* row = src + i * (8 * QW) * 128;
        uint4 m8, bf0, bf1;
        int e;
        if (p.x_type == kXMXINT8) {
          // the block is quantised already: its mantissas are the MMA's operand as they stand, its values m * 2^(e - 6)
          // go to Xcat (a block that is not normalised gives the same values, hence the same T and Y, as its normal form)
          m8 = *reinterpret_cast<const uint4*>(src + i * (8 * QW) * 64 + ((blk ^ swz64) << 4));
          const int grow = row0 + r0 + i * (8 * QW), kb = (pan_lo * 2 + s) * 4 + blk;
          const uint32_t eb = (grow < p.M && kb < kb_row) ? (uint32_t)__ldg(p.x_exp + (size_t)grow * kb_row + kb) : 127u;
          if (i == C::BPL - 1) {
            __syncwarp();
            if (lane == 0) mbar_arrive(raw_empty(rs));
          }
          e = min(max((int)eb - 127, p.exp_min), p.exp_max);
          const uint32_t ww[4] = {m8.x, m8.y, m8.z, m8.w};
          uint32_t b[8];
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            const float4 q = mxint_quad_values(ww[t], eb, p.a_bits, p.exp_min, p.exp_max);
            b[2 * t] = __byte_perm(__float_as_uint(q.x), __float_as_uint(q.y), 0x7632);
            b[2 * t + 1] = __byte_perm(__float_as_uint(q.z), __float_as_uint(q.w), 0x7632);
          }
          bf0 = make_uint4(b[0], b[1], b[2], b[3]);
          bf1 = make_uint4(b[4], b[5], b[6], b[7]);
        } else {
          float v[16];
          if (p.x_type == kXBF16) {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
              const uint4 w = *reinterpret_cast<const uint4*>(row + (((chunk0 + j) ^ swz) << 4));
              const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
              for (int t = 0; t < 4; ++t) {
                v[8 * j + 2 * t] = __uint_as_float(ww[t] << 16);
                v[8 * j + 2 * t + 1] = __uint_as_float(ww[t] & 0xFFFF0000u);
              }
            }
          } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float4 w = *reinterpret_cast<const float4*>(row + (((chunk0 + j) ^ swz) << 4));
              v[4 * j] = w.x; v[4 * j + 1] = w.y; v[4 * j + 2] = w.z; v[4 * j + 3] = w.w;
            }
          }
          if (i == C::BPL - 1) {                       // the stage's values are in registers: the slot can be refilled
            __syncwarp();
            if (lane == 0) mbar_arrive(raw_empty(rs));
          }
          quantize_block16(v, qc, e, m8, bf0, bf1);
        }
        *reinterpret_cast<uint4*>(xdst + i * (8 * QW) * 128) = m8;
        xe_dst[i * (8 * QW) * 4] = (int8_t)e;
        if (store_ok && 8 * QW * i < rows_ok &&
            LQER_IN_BOUNDS(p.status, (size_t)(cd + i * c_step - p.xcat) * 2, 32, p.xcat_extent, 301)) {
          uint4* g = reinterpret_cast<uint4*>(cd + i * c_step);
          g[0] = bf0;
          g[1] = bf1;
        }
      }
      fence_proxy_async_smem();                      // generic-proxy writes -> visible to the MMA's async proxy
      __syncwarp();
      if (lane == 0) mbar_arrive(xq_full(xs));
    }
  } else if (warp == WORK_WARPS) {
    // ------------------------------------------------------------------ A_q panels
    const int n_pan = pan_hi - pan_lo;
    const int cbias = -127 - (p.a_bits - 2) - (p.lr_bits - 2) + 1023;
    constexpr int EPL = 8 * KP / 32;                  // table entries per lane and panel
    bool ok = true;
    // exponent bytes of a panel, one load ahead of their use
    int eb[EPL];
    auto load_exps = [&](int pp) {
      const int b0 = (pan_lo + pp) * 8;
#pragma unroll
      for (int t = 0; t < EPL; ++t) {
        const int i = lane + 32 * t;
        eb[t] = (pp < n_pan && b0 + i / KP < p.kblocks) ? (int)__ldg(a_exp + (size_t)b0 * KP + i) : 1023 - cbias;
      }
    };
    auto publish = [&](int pp) {
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(panel_full(pp % PANELS));
    };
    load_exps(0);
    for (int pp = 0; pp < n_pan && ok; ++pp) {
      const int pb = pp % PANELS;
      if (!warp_wait(panel_empty(pb), ((pp / PANELS) & 1) ^ 1, abort_flag, kNapNs)) { ok = false; break; }
      const int b0 = (pan_lo + pp) * 8;
      const uint32_t dst0 = smem_u32(panel_base + pb * C::PANEL_BYTES);
      for (int i = lane; i < 8 * KP; i += 32) {
        const int c = i / KP, j = i % KP;              // block within the panel, rank column
        if (b0 + c < p.kblocks) {
          const int prow = (c & 1) * KP + j;           // even blocks: first k_pad rows; odd: the rest
          cp_async16(dst0 + prow * 128 + ((c ^ (prow & 7)) << 4), p.asec + ((size_t)(b0 + c) * KP + j) * 16);
        }
      }
      cp_async_commit();
      // high words of 2^(e_a - 127 - shifts) per block and rank column, for the scalers
#pragma unroll
      for (int t = 0; t < EPL; ++t) s_hia[pb * 8 * KP + lane + 32 * t] = (eb[t] + cbias) << 20;
      load_exps(pp + 1);
      // the first panel goes out as soon as it has landed; later ones one panel behind their copies
      if (pp == 0) { cp_async_wait<0>(); publish(0); }
      else if (pp >= 2) { cp_async_wait<1>(); publish(pp - 1); }
    }
    cp_async_wait<0>();
    if (ok && n_pan > 1) publish(n_pan - 1);
  } else if (warp == WORK_WARPS + 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = make_idesc_i8(ROWS, C::SLOT_COLS);
      bool ok = true;
      for (int s = 0; s < n_stages && ok; ++s) {
        const int xs = s % X_SLOTS, pp = s >> 1, pb = pp % PANELS;
        if (!parked_wait(xq_full(xs), (s / X_SLOTS) & 1, abort_flag, kNapNs)) { ok = false; break; }
        if ((s & 1) == 0 && !parked_wait(panel_full(pb), (pp / PANELS) & 1, abort_flag, kNapNs)) { ok = false; break; }
        const uint64_t a_desc = make_desc(smem_u32(xq_base + (xs >> 1) * XBUF_BYTES));
        const uint64_t b_desc = make_desc(smem_u32(panel_base + pb * C::PANEL_BYTES));
        for (int j = 0; j < 2; ++j) {
          const int u = 2 * s + j, slot = u % C::TMEM_SLOTS;
          if (!parked_wait(slot_empty(slot), ((u / C::TMEM_SLOTS) & 1) ^ 1, abort_flag, kNapNs)) { ok = false; break; }
          tc_fence_after();
          const int kstep = (s & 1) * 2 + j;           // 32 bytes along the swizzled row: +2 in the address field
          umma_i8(tmem_base + slot * C::SLOT_COLS, a_desc + 2 * kstep, b_desc + 2 * kstep, idesc);
          umma_commit(slot_full(slot));
        }
        if (!ok) break;
        umma_commit(xq_empty(xs));
        if (s & 1) umma_commit(panel_empty(pb));
      }
    }
  } else {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      for (int s = 0; s < n_stages; ++s) {
        const int rs = s % RAW_SLOTS;
        if (!parked_wait(raw_empty(rs), ((s / RAW_SLOTS) & 1) ^ 1, abort_flag, kNapNs)) break;
        mbar_expect_tx(raw_full(rs), p.x_type == kXMXINT8 ? RAW_BYTES / 4 : p.x_type == kXBF16 ? RAW_BYTES / 2 : RAW_BYTES);   // rows and columns outside X arrive as zeros
        const uint32_t dst = smem_u32(raw_base + rs * RAW_BYTES);
        const int col = (pan_lo * 2 + s) * STAGE_COLS;
        tma_load_2d(dst, tmap_x, col, row0, raw_full(rs));                         // a box is 128 bytes wide (swizzled rows):
        if (p.x_type == kXF32) tma_load_2d(dst + RAW_BYTES / 2, tmap_x, col + STAGE_COLS / 2, row0, raw_full(rs));   // fp32 takes two
      }
    }
  }

  // ------------------------------------------------------------------ the CTAs of a row tile finish T together
  __syncthreads();                 // every role is done (or has given up): the flag below is final for this CTA
  if (abort_flag->abort != 0) {
    const long long t0 = clock64();
    while (clock64() - t0 < 400000) { }
    if (tid == 0) report_error(p.status, LQER_ERR_TIMEOUT, 400, blockIdx.x);
  }
  __threadfence();                 // this CTA's partial sums before its arrival
  tc_fence_before();
  __syncthreads();
  if (warp == WORK_WARPS + 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
  // Every CTA of the row tile finishes a share of its rows once all partial sums are there.  The CTAs of a launch
  // fit the GPU together (at most one per SM), so the wait below ends as soon as the last of them has run; it is
  // bounded all the same.  Two counters per row tile: arrivals, and departures (the last to leave zeroes both).
  int* arrive_cnt = p.counters + 2 * row_tile;
  int* depart_cnt = arrive_cnt + 1;
  if (tid == 0) {
    atomicAdd(arrive_cnt, 1);
    int seen = 1;
    const long long t0 = clock64();
    for (;;) {
      int v;
      asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(arrive_cnt) : "memory");
      if (v >= p.expect) break;
      if (clock64() - t0 > p.wait_limit) { seen = 0; break; }
      __nanosleep(100);
    }
    if (!seen) report_error(p.status, LQER_ERR_TIMEOUT, 401, blockIdx.x);
    *last_flag = seen;
  }
  __syncthreads();
  if (*last_flag != 0) {
    // rows [r_lo, r_hi) of the tile: sum over the K ranges in a fixed order, re-quantise along the rank (16 adjacent
    // lanes hold one block), append to Xcat
    const int r_lo = split * ROWS / p.splits, r_hi = (split + 1) * ROWS / p.splits;
    const int n_out = (r_hi - r_lo) * KP;                                  // a multiple of 16
    const double* part0 = p.partials + (size_t)row_tile * p.splits * ROWS * KP + (size_t)r_lo * KP;
    for (int o0 = warp * 32; o0 < n_out; o0 += NUM_THREADS) {              // whole warps: the shuffles need every lane
      const int o = o0 + lane;
      const bool live = o < n_out;
      double t = 0.0;
      if (live) {
        const double* pc = part0 + o;
#pragma unroll 4
        for (int c = 0; c < p.splits; ++c) t += __ldcg(pc + (size_t)c * ROWS * KP);
      }
      double amax = (t != t) ? 0.0 : fabs(t);
#pragma unroll
      for (int sft = 1; sft < 16; sft <<= 1) amax = fmax(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, sft));
      const int e = block_exponent(amax, p.exp_min, p.exp_max);
      const int qv = quant_mantissa(t, e, p.a_bits);
      const int r = r_lo + o / KP, j = o % KP;
      const int row = row0 + r;
      if (live && row < p.M && LQER_IN_BOUNDS(p.status, ((size_t)row * p.ldx + p.K64 + j) * 2, 2, p.xcat_extent, 303)) {
        p.xcat[(size_t)row * p.ldx + p.K64 + j] = (uint16_t)bf16_bits_of(qv, e - (p.a_bits - 2));
        if (p.Tm != nullptr) p.Tm[(size_t)row * KP + j] = (int8_t)qv;
        if (p.Te != nullptr && (j & 15) == 0) p.Te[(size_t)row * (KP / 16) + (j >> 4)] = (uint8_t)(e + 127);
      }
    }
  }
  __syncthreads();
  if (tid == 0 && atomicAdd(depart_cnt, 1) == p.splits - 1) {              // everyone has read the counters: zero for the next call
    *arrive_cnt = 0;
    *depart_cnt = 0;
  }
  if (p.order == kChainLater) pdl_wait();
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &f, 12000, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

template <int KP>
static cudaError_t launch_kp(const TensorMaps& tmaps, const GroupParams& gp, int ctas, cudaStream_t s) {
  using C = Cfg<KP>;
  static OncePerDevice once;
  cudaError_t e = once.run([] {
    return cudaFuncSetAttribute(prologue_tc_kernel<KP>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
  });
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(ctas);
  cfg.blockDim = dim3(NUM_THREADS);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may set up while the previous kernel drains
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  LaunchScope scope(kFamPrologue, s);
  return cudaLaunchKernelEx(&cfg, prologue_tc_kernel<KP>, tmaps, gp);
}

}  // namespace ptc

// The tensor-core prologue serves ranks padded to 16, 32 or 64 and batches large enough to give most SMs a CTA.
bool prologue_tc_fits(const PackedMeta& m, int M, const void* X, bool any_batch) {
  if (!prologue_tc_rank_ok(m) || (M + 127) / 128 > kPrologueRowTiles) return false;
  if ((reinterpret_cast<uintptr_t>(X) & 15) != 0) return false;
  return any_batch || M >= 1024;
}

// K ranges per row tile for each of n layers that share a launch: about as many panels (128 columns of X) per CTA
// everywhere, at most max_ctas CTAs in all (one per SM: the CTAs of a row tile wait for one another).  Returns whether
// ranges had to be taken away to stay within max_ctas (the work per CTA may then be unequal).
bool prologue_tc_group_splits(const PackedMeta* metas, int n, int M, int max_ctas, int* splits) {
  const int row_tiles = (M + 127) / 128;
  long long total = 0;
  int panels[ptc::kMaxLayers];
  for (int g = 0; g < n; ++g) {
    panels[g] = (metas[g].K64 + 127) / 128;
    total += (long long)row_tiles * panels[g];
  }
  const double per = (double)total / max_ctas;
  int ctas = 0;
  for (int g = 0; g < n; ++g) {
    int sp = (int)((double)panels[g] / per + 0.5);
    const int cap = prologue_tc_splits(metas[g], M);              // what the scratch is sized for
    if (sp > cap) sp = cap;
    if (sp > panels[g]) sp = panels[g];
    if (sp < 1) sp = 1;
    splits[g] = sp;
    ctas += row_tiles * sp;
  }
  bool squeezed = false;
  while (ctas > max_ctas) {                                       // take a range away where the ranges are shortest
    squeezed = true;
    int best = -1;
    double shortest = 0.0;
    for (int g = 0; g < n; ++g) {
      const double len = (double)panels[g] / splits[g];
      if (splits[g] > 1 && (best < 0 || len < shortest)) { best = g; shortest = len; }
    }
    if (best < 0) break;
    --splits[best];
    ctas -= row_tiles;
  }
  return squeezed;
}

// n layers (one M, one k_pad, one set of formats) in ONE launch.  splits[g] K ranges per row tile of layer g; the
// caller sees to it that the CTAs (row tiles x splits, summed) are at most one per SM.  Tm / Te: for n == 1 only.
cudaError_t launch_prologue_tc_group(const void* const* Xs, int x_type, int M, const PackedMeta* metas, const void* const* packed,
                                     void* const* xcats, double* const* partials, int* const* counters,
                                     const int* splits, int n, int8_t* Tm, uint8_t* Te, DeviceStatus* st, int order,
                                     cudaStream_t s) {
  using namespace ptc;
  EncodeTiledFn enc = encode_fn();
  if (enc == nullptr) return cudaErrorNotSupported;
  if (n < 1 || n > kMaxLayers) return cudaErrorInvalidValue;
  TensorMaps tmaps;
  GroupParams gp;
  gp.n = n;
  int begin = 0;
  const long long limit = wait_limit_cycles();
  const int stall = take_stall(kFamPrologue) ? 1 : 0;
  for (int i = 0; i < kMaxLayers; ++i) {
    const int g = i < n ? i : 0;
    const PackedMeta& m = metas[g];
    if (m.k_pad != metas[0].k_pad) return cudaErrorInvalidValue;
    const cuuint64_t dims[2] = {(cuuint64_t)m.K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)m.K * (x_type == kXMXINT8 ? 1 : x_type == kXBF16 ? 2 : 4)};
    // a box is one swizzled row wide: 128 bytes of fp32 (half a stage) or bf16, 64 bytes of MXINT mantissas
    const cuuint32_t box[2] = {(cuuint32_t)(x_type == kXF32 ? STAGE_COLS / 2 : STAGE_COLS), ROWS};
    const CUtensorMapDataType x_dt = x_type == kXMXINT8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                     : x_type == kXBF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&tmaps.m[i], x_dt, 2, const_cast<void*>(Xs[g]), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, x_type == kXMXINT8 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorInvalidValue;
    Params& p = gp.L[i];
    p.asec = static_cast<const uint8_t*>(packed[g]) + m.off_a;
    p.xcat = static_cast<uint16_t*>(xcats[g]);
    p.Tm = n == 1 ? Tm : nullptr; p.Te = n == 1 ? Te : nullptr; p.status = st;
    p.partials = partials[g]; p.counters = counters[g];
    p.M = M; p.K = m.K; p.K64 = m.K64;
    p.kblocks = m.K / 16;
    p.panels = (m.K64 + 127) / 128;
    p.splits = splits[g];
    p.expect = splits[g] + stall;
    p.wait_limit = limit;
    p.a_bits = m.a_bits; p.lr_bits = m.lr_bits; p.exp_min = m.exp_min; p.exp_max = m.exp_max;
    p.order = order;
    p.x_type = x_type;
    p.x_exp = static_cast<const uint8_t*>(Xs[g]) + (size_t)M * m.K;
    p.ldx = xcat_cols(m);
    p.xcat_extent = (size_t)M * xcat_cols(m) * 2;
    p.partials_extent = (size_t)((M + ROWS - 1) / ROWS) * splits[g] * ROWS * m.k_pad * 8;
    gp.cta_begin[i] = begin;
    if (i < n) begin += ((M + ROWS - 1) / ROWS) * p.splits;
  }
  switch (metas[0].k_pad) {
    case 16: return launch_kp<16>(tmaps, gp, begin, s);
    case 32: return launch_kp<32>(tmaps, gp, begin, s);
    case 64: return launch_kp<64>(tmaps, gp, begin, s);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_prologue_tc(const void* X, int x_type, int M, const PackedMeta& m, const void* packed, void* xcat,
                               int8_t* Tm, uint8_t* Te, DeviceStatus* st, double* partials, int* counters,
                               int order, cudaStream_t s) {
  const int sms = sm_count();
  const int splits = prologue_tc_splits(m, M, sms > 0 && sms < kPrologueMaxCtas ? sms : kPrologueMaxCtas);
  return launch_prologue_tc_group(&X, x_type, M, &m, &packed, &xcat, &partials, &counters, &splits, 1, Tm, Te, st, order, s);
}

}  // namespace lqer
