// Inline-PTX wrappers shared by the tensor-core GEMM kernels: mbarriers with bounded waits,
// TMA / bulk copies, tcgen05 (tensor memory, MMA, commit), and the exact int4 / int8 -> bf16
// operand conversion.
#pragma once

#include <cuda.h>

#include "lqer_common.cuh"

namespace lqer {
namespace tc {

// What the bounded waits of a CTA share (shared memory): a flag that any role sets when it gives up, and the bound
// in clock cycles (a launch parameter: wait_limit_cycles()).
struct WaitState {
  int abort;
  int unused;
  long long limit;
};
constexpr int UMMA_M = 128;                                  // rows of the MMA tile per CTA

// ---------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: gives up after ws->limit cycles or as soon as another role has given up.
// kBackoff: sleep between polls (for roles that are not on the critical path, so that their
// polling does not take issue slots from the MMA issuer).
template <bool kBackoff = false>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile WaitState* ws) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  int spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if (kBackoff) __nanosleep(64);
    if ((++spins & 255) == 0) {
      if (ws->abort != 0) return false;
      if (clock64() - t0 > ws->limit) { ws->abort = 1; return false; }
    }
  }
  return true;
}
// True in exactly one lane of a fully converged warp.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n .reg .pred p;\n elect.sync _|p, 0xFFFFFFFF;\n selp.u32 %0, 1, 0, p;\n}\n" : "=r"(pred));
  return pred != 0;
}
// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may start while its
// predecessor drains; what it does before pdl_wait() must not touch anything an earlier kernel reads or writes.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);       // start address
  d |= (uint64_t)1 << 16;                         // leading byte offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                         // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                         // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = m, N = n.
__host__ __device__ constexpr uint32_t make_idesc(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

__device__ __forceinline__ uint32_t fma_bf16x2(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
// Eight offset-binary nibbles of one block word -> eight bf16 (n - 8) * 2^(e-2), exact:
// 0x4300 | n is the bf16 value 128 + n, and (128 + n) * s - 136 * s rounds nothing away.
__device__ __forceinline__ uint4 convert_word(uint32_t w, uint32_t s2, uint32_t c2) {
  uint4 o;
  o.x = fma_bf16x2((w & 0x000F000Fu) | 0x43004300u, s2, c2);
  o.y = fma_bf16x2(((w >> 4) & 0x000F000Fu) | 0x43004300u, s2, c2);
  o.z = fma_bf16x2(((w >> 8) & 0x000F000Fu) | 0x43004300u, s2, c2);
  o.w = fma_bf16x2(((w >> 12) & 0x000F000Fu) | 0x43004300u, s2, c2);
  return o;
}
__device__ __forceinline__ void w_scales(uint32_t eb, uint32_t& s2, uint32_t& c2) {
  const uint32_t s = (eb - 2u) << 7;                       // bf16 bits of 2^(e-2), eb = e + 127
  const uint32_t c = 0x8000u | ((eb + 5u) << 7) | 8u;      // bf16 bits of -136 * 2^(e-2)
  s2 = s | (s << 16);
  c2 = c | (c << 16);
}
// The 2-bit format (mantissas -1, 0, 1; value = m * 2^e): sixteen offset-binary crumbs of one block word -> sixteen
// bf16, exact: 0x4300 | c is the bf16 value 128 + c, and (128 + c) * s - 129 * s rounds nothing away.
__device__ __forceinline__ void convert_word2(uint32_t w, uint32_t s2, uint32_t c2, uint4& lo, uint4& hi) {
  lo.x = fma_bf16x2((w & 0x00030003u) | 0x43004300u, s2, c2);
  lo.y = fma_bf16x2(((w >> 2) & 0x00030003u) | 0x43004300u, s2, c2);
  lo.z = fma_bf16x2(((w >> 4) & 0x00030003u) | 0x43004300u, s2, c2);
  lo.w = fma_bf16x2(((w >> 6) & 0x00030003u) | 0x43004300u, s2, c2);
  hi.x = fma_bf16x2(((w >> 8) & 0x00030003u) | 0x43004300u, s2, c2);
  hi.y = fma_bf16x2(((w >> 10) & 0x00030003u) | 0x43004300u, s2, c2);
  hi.z = fma_bf16x2(((w >> 12) & 0x00030003u) | 0x43004300u, s2, c2);
  hi.w = fma_bf16x2(((w >> 14) & 0x00030003u) | 0x43004300u, s2, c2);
}
__device__ __forceinline__ void w_scales2(uint32_t eb, uint32_t& s2, uint32_t& c2) {
  const uint32_t s = eb << 7;                              // bf16 bits of 2^e, eb = e + 127
  const uint32_t c = 0x8000u | ((eb + 7u) << 7) | 1u;      // bf16 bits of -129 * 2^e
  s2 = s | (s << 16);
  c2 = c | (c << 16);
}
// One weight column of a 64-K stage from its packed form (pk: the column's mantissas at mant_off + nl * 16 resp.
// the two block pairs of the 4-bit layout, exponents at exp_off + nl * 4) into its eight swizzled 16-byte chunks.
__device__ __forceinline__ void convert_column(const uint8_t* pk, int nl, int w_bits, uint8_t* bt, const uint32_t (&chunk)[8]) {
  uint32_t s2, c2;
  if (w_bits == 2) {
    const uint4 wv = *reinterpret_cast<const uint4*>(pk + nl * 16);
    const uint32_t eb = *reinterpret_cast<const uint32_t*>(pk + 2048 + nl * 4);
    uint4 lo, hi;
    w_scales2(eb & 0xFFu, s2, c2);
    convert_word2(wv.x, s2, c2, lo, hi);
    *reinterpret_cast<uint4*>(bt + chunk[0]) = lo;
    *reinterpret_cast<uint4*>(bt + chunk[1]) = hi;
    w_scales2((eb >> 8) & 0xFFu, s2, c2);
    convert_word2(wv.y, s2, c2, lo, hi);
    *reinterpret_cast<uint4*>(bt + chunk[2]) = lo;
    *reinterpret_cast<uint4*>(bt + chunk[3]) = hi;
    w_scales2((eb >> 16) & 0xFFu, s2, c2);
    convert_word2(wv.z, s2, c2, lo, hi);
    *reinterpret_cast<uint4*>(bt + chunk[4]) = lo;
    *reinterpret_cast<uint4*>(bt + chunk[5]) = hi;
    w_scales2(eb >> 24, s2, c2);
    convert_word2(wv.w, s2, c2, lo, hi);
    *reinterpret_cast<uint4*>(bt + chunk[6]) = lo;
    *reinterpret_cast<uint4*>(bt + chunk[7]) = hi;
  } else {
    const uint4 wa = *reinterpret_cast<const uint4*>(pk + nl * 16);
    const uint4 wb = *reinterpret_cast<const uint4*>(pk + (kTileN + nl) * 16);
    const uint32_t eb = *reinterpret_cast<const uint32_t*>(pk + kWTileNibbleBytes + nl * 4);
    w_scales(eb & 0xFFu, s2, c2);
    *reinterpret_cast<uint4*>(bt + chunk[0]) = convert_word(wa.x, s2, c2);
    *reinterpret_cast<uint4*>(bt + chunk[1]) = convert_word(wa.y, s2, c2);
    w_scales((eb >> 8) & 0xFFu, s2, c2);
    *reinterpret_cast<uint4*>(bt + chunk[2]) = convert_word(wa.z, s2, c2);
    *reinterpret_cast<uint4*>(bt + chunk[3]) = convert_word(wa.w, s2, c2);
    w_scales((eb >> 16) & 0xFFu, s2, c2);
    *reinterpret_cast<uint4*>(bt + chunk[4]) = convert_word(wb.x, s2, c2);
    *reinterpret_cast<uint4*>(bt + chunk[5]) = convert_word(wb.y, s2, c2);
    w_scales(eb >> 24, s2, c2);
    *reinterpret_cast<uint4*>(bt + chunk[6]) = convert_word(wb.z, s2, c2);
    *reinterpret_cast<uint4*>(bt + chunk[7]) = convert_word(wb.w, s2, c2);
  }
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  return (__float_as_uint(lo) >> 16) | (__float_as_uint(hi) & 0xFFFF0000u);   // exact values: truncation loses nothing
}
__device__ __forceinline__ uint4 convert_i8x8(uint32_t w0, uint32_t w1, float scale) {
  uint4 o;
  o.x = pack_bf16x2((float)(int8_t)(w0) * scale, (float)(int8_t)(w0 >> 8) * scale);
  o.y = pack_bf16x2((float)(int8_t)(w0 >> 16) * scale, (float)(int8_t)(w0 >> 24) * scale);
  o.z = pack_bf16x2((float)(int8_t)(w1) * scale, (float)(int8_t)(w1 >> 8) * scale);
  o.w = pack_bf16x2((float)(int8_t)(w1 >> 16) * scale, (float)(int8_t)(w1 >> 24) * scale);
  return o;
}


// ---------------------------------------------------------------------------- CTA-pair (cta_group::2) forms
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive on the barrier at the same shared-memory offset in CTA `cta` of the cluster.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t bar, uint32_t cta) {
  asm volatile(
      "{\n .reg .b32 ra;\n mapa.shared::cluster.u32 ra, %0, %1;\n"
      " mbarrier.arrive.shared::cluster.b64 _, [ra];\n}\n" ::"r"(bar), "r"(cta) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// Arrives (once the MMAs issued so far have finished) on the barrier at this offset in both CTAs of the pair.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}

}  // namespace tc
}  // namespace lqer
