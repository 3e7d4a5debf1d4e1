// Pieces shared by the fp16 sparse-convolution kernels (sm_100a): the thread-tile geometry, PTX wrappers
// (mbarrier, bulk copies, matrix loads, tensor memory) and the per-pattern multiply-add code of a consumer thread.
#pragma once
#include <cuda.h>
#include "common.cuh"

namespace pat {
namespace fast16 {

constexpr int TR = 2, TC = 14;          // pixel tile of a thread
constexpr int LX = 4, LY = 8;           // tiles of a warp: 4 column slots x 8 tile rows
constexpr int CB = kChanTile;           // channels per pipeline stage (16)
constexpr int RF = 2;                   // filters per consumer warp
constexpr int NCW = 16;                // consumer warps of a block
constexpr int FG = NCW * RF;            // filters per work item (32)
static_assert(FG == kExecGroup, "a work item is one execution group of the blob");
constexpr int SEGB = 32;                // bytes of a segment: 16 px (cols -1..14) of one channel
constexpr int ROWB = LX * SEGB;         // 128
constexpr int LAUNCH_REGS = 96;         // registers per thread at launch (the pool that setmaxnreg redistributes)
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr unsigned long long kWaitNs = 2000000000ull;   // 2 s: far beyond any healthy wait
constexpr int kFillSleepNs = 200;                       // pause between polls of a waiting fill / store warp

// ------------------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_n(uint32_t bar, uint32_t n) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(n) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: gives up after limit_ns of wall time (or kSpinLimit polls), raises the block-wide abort flag
// and returns false; also returns false as soon as another thread of the block has given up.
// SLEEP_NS > 0: sleep between polls.  The fill and store warps wait that way: a polling warp takes issue
// slots from the four consumer warps of its SM partition, and those warps have slack (they work ahead by up
// to three ring slots).  Consumers poll without sleeping: they rarely wait, and must restart at once.
template <int SLEEP_NS>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned long long limit_ns = kWaitNs) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
    if (SLEEP_NS > 0) __nanosleep(SLEEP_NS);
    if (mbar_try_wait(bar, parity)) return true;
    if ((spin & 31u) == 31u) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > limit_ns) break;
    }
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, int c2, int c3, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& a, uint32_t& b, uint32_t& c, uint32_t& d) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(addr) : "memory");
}
__device__ __forceinline__ void stmatrix_x4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1,%2,%3,%4};"
               ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void lds128(uint32_t addr, uint32_t& a, uint32_t& b, uint32_t& c, uint32_t& d) {
  asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(addr));
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void sts16(uint32_t addr, unsigned short a) {
  asm volatile("st.shared.b16 [%0], %1;" ::"r"(addr), "h"(a) : "memory");
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t a) {
  asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr), "r"(a) : "memory");
}
__device__ __forceinline__ void fma_f32_f16(float& acc, unsigned short a, unsigned short b) {
  asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc) : "h"(a), "h"(b));
}
__device__ __forceinline__ void split_h2(uint32_t v, unsigned short& lo, unsigned short& hi) {
  asm("mov.b32 {%0,%1}, %2;" : "=h"(lo), "=h"(hi) : "r"(v));
}

// ---- tensor memory (256 KB per SM, 128 lanes x 512 columns of 32 bits).  No tensor-core instruction is used
// here: the memory only parks the accumulators of the filter a warp is not working on, so that the per-pattern
// code exists once (for one set of accumulator registers) and stays inside the instruction cache.  A warp may
// touch the 32 lanes of its own quarter (warp index % 4); thread i of the warp reads / writes lane i.
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {      // whole warp; ncols: power of two >= 32
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {         // whole warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// 32 consecutive columns of the thread's lane <-> 32 registers: rows Y0 and Y0 + 1 of an accumulator tile
// (28 values + 4 unused).  The _rows functions only issue the transfer; tmem_wait_st / tmem_wait_ld complete it.
template <int T, int Y0>
__device__ __forceinline__ void tmem_store_rows(uint32_t taddr, const float (&a)[T][TC]) {
  static_assert(TC == 14 && Y0 + 1 < T, "two rows of 14 values");
  const float z = 0.0f;
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%29,%29,%29};"
      ::"r"(taddr),
        "f"(a[Y0][0]), "f"(a[Y0][1]), "f"(a[Y0][2]), "f"(a[Y0][3]), "f"(a[Y0][4]), "f"(a[Y0][5]), "f"(a[Y0][6]),
        "f"(a[Y0][7]), "f"(a[Y0][8]), "f"(a[Y0][9]), "f"(a[Y0][10]), "f"(a[Y0][11]), "f"(a[Y0][12]), "f"(a[Y0][13]),
        "f"(a[Y0 + 1][0]), "f"(a[Y0 + 1][1]), "f"(a[Y0 + 1][2]), "f"(a[Y0 + 1][3]), "f"(a[Y0 + 1][4]), "f"(a[Y0 + 1][5]), "f"(a[Y0 + 1][6]),
        "f"(a[Y0 + 1][7]), "f"(a[Y0 + 1][8]), "f"(a[Y0 + 1][9]), "f"(a[Y0 + 1][10]), "f"(a[Y0 + 1][11]), "f"(a[Y0 + 1][12]), "f"(a[Y0 + 1][13]),
        "f"(z)
      : "memory");
}
template <int T, int Y0>
__device__ __forceinline__ void tmem_load_rows(uint32_t taddr, float (&a)[T][TC]) {
  static_assert(TC == 14 && Y0 + 1 < T, "two rows of 14 values");
  float d0, d1, d2, d3;
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=f"(a[Y0][0]), "=f"(a[Y0][1]), "=f"(a[Y0][2]), "=f"(a[Y0][3]), "=f"(a[Y0][4]), "=f"(a[Y0][5]), "=f"(a[Y0][6]),
        "=f"(a[Y0][7]), "=f"(a[Y0][8]), "=f"(a[Y0][9]), "=f"(a[Y0][10]), "=f"(a[Y0][11]), "=f"(a[Y0][12]), "=f"(a[Y0][13]),
        "=f"(a[Y0 + 1][0]), "=f"(a[Y0 + 1][1]), "=f"(a[Y0 + 1][2]), "=f"(a[Y0 + 1][3]), "=f"(a[Y0 + 1][4]), "=f"(a[Y0 + 1][5]), "=f"(a[Y0 + 1][6]),
        "=f"(a[Y0 + 1][7]), "=f"(a[Y0 + 1][8]), "=f"(a[Y0 + 1][9]), "=f"(a[Y0 + 1][10]), "=f"(a[Y0 + 1][11]), "=f"(a[Y0 + 1][12]), "=f"(a[Y0 + 1][13]),
        "=f"(d0), "=f"(d1), "=f"(d2), "=f"(d3)
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_store32(uint32_t taddr, const float (&a)[TR][TC]) {
  tmem_store_rows<TR, 0>(taddr, a);
  tmem_wait_st();
}
__device__ __forceinline__ void tmem_load32(uint32_t taddr, float (&a)[TR][TC]) {
  tmem_load_rows<TR, 0>(taddr, a);
  tmem_wait_ld();
}

template <int REGS>
__device__ __forceinline__ void set_warp_registers() {
  if constexpr (REGS > LAUNCH_REGS) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS));
  else if constexpr (REGS < LAUNCH_REGS) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS));
}

// ------------------------------------------------------------------------------------------ consumer math
// One tap of one kept kernel at kernel position B = 3*r + s:  acc[y][x] += w * in[y + r][x + s], where `in` is
// the thread's (TR+2) x 16 window (row 0 / column 0 = the halo above / left of the tile).  B is a template
// argument, so every register index below is fixed at compile time (Section 6.2: access code per pattern
// position known ahead of time); the code of a tap is shared by all patterns that contain it.
template <int B>
__device__ __forceinline__ void tap_body(float (&acc)[TR][TC], const unsigned short (&h)[TR + 2][16], unsigned short w) {
  constexpr int r = B / 3, s = B % 3;
#pragma unroll
  for (int y = 0; y < TR; ++y)
#pragma unroll
    for (int x = 0; x < TC; ++x) fma_f32_f16(acc[y][x], h[y + r][x + s], w);
}

__device__ __forceinline__ void load_row(unsigned short (&hrow)[16], uint32_t a0, uint32_t a1) {
  uint32_t q[8];
  lds128(a0, q[0], q[1], q[2], q[3]);   // logical chunk 0: cols -1..6
  lds128(a1, q[4], q[5], q[6], q[7]);   // logical chunk 1: cols 7..14
#pragma unroll
  for (int e = 0; e < 8; ++e) split_h2(q[e], hrow[2 * e], hrow[2 * e + 1]);
}

template <uint32_t MASK>
__device__ __forceinline__ void pattern_body(float (&acc)[TR][TC], const unsigned short (&h)[TR + 2][16], uint32_t w01, uint32_t w23) {
  unsigned short w0, w1, w2, w3;
  split_h2(w01, w0, w1);
  split_h2(w23, w2, w3);
  tap_body<nth_bit(MASK, 0)>(acc, h, w0);
  tap_body<nth_bit(MASK, 1)>(acc, h, w1);
  tap_body<nth_bit(MASK, 2)>(acc, h, w2);
  tap_body<nth_bit(MASK, 3)>(acc, h, w3);
}

// One kept kernel.  meta = descriptor word (see pattern_word); w01 / w23 = its four taps (fp16) in ascending
// position order; baseA / baseB = the lane's two chunk addresses of window row 0 in the kernel's channel plane.
// Every branch is warp-uniform (the whole warp works on the same kernel).
__device__ __forceinline__ void one_kernel(float (&acc)[TR][TC], uint32_t baseA, uint32_t baseB, uint32_t meta,
                                           uint32_t w01, uint32_t w23) {
  static_assert(TR == 2, "window addressing below is written for two-row tiles");
  unsigned short h[TR + 2][16];
  // window rows shift .. shift+2 (physical chunk = logical chunk ^ ((row >> 1) & 1) ^ lane swizzle)
  const uint32_t sh = (meta >> 17) & 1u;
  const uint32_t rb = sh * ROWB;
  load_row(h[0], baseA + rb, baseB + rb);                                   // row 0 or 1: u = 0
  load_row(h[1], (sh ? baseB : baseA) + rb + ROWB, (sh ? baseA : baseB) + rb + ROWB);   // row 1 (u = 0) or 2 (u = 1)
  load_row(h[2], baseB + rb + 2 * ROWB, baseA + rb + 2 * ROWB);             // row 2 or 3: u = 1
  // Warp-uniform dispatch on the code as a tree of direct branches (an indexed jump costs far more here: the
  // target address comes from a table in memory, and nothing can be fetched until it has arrived).
  const uint32_t code = (meta >> 13) & 15u;
#define PAT_ROW3() load_row(h[3], baseB + 3 * ROWB, baseA + 3 * ROWB)
  if (code & 8u) {
    if (code & 4u) {
      // any other pattern: a warp-uniform test of each of the nine positions guards the code of that position
      PAT_ROW3();
#define PAT_TAP(B)                                                   \
  if (meta & (16u << (B))) {                                         \
    tap_body<B>(acc, h, (unsigned short)(w01 & 0xFFFFu));            \
    w01 = __funnelshift_r(w01, w23, 16);                             \
    w23 >>= 16;                                                      \
  }
      PAT_TAP(0) PAT_TAP(1) PAT_TAP(2) PAT_TAP(3) PAT_TAP(4) PAT_TAP(5) PAT_TAP(6) PAT_TAP(7) PAT_TAP(8)
#undef PAT_TAP
    } else if (code & 1u) {
      pattern_body<code_mask(9)>(acc, h, w01, w23);
    } else {
      PAT_ROW3(); pattern_body<code_mask(8)>(acc, h, w01, w23);
    }
  } else if (code & 4u) {
    if (code & 2u) {
      if (code & 1u) pattern_body<code_mask(7)>(acc, h, w01, w23);
      else { PAT_ROW3(); pattern_body<code_mask(6)>(acc, h, w01, w23); }
    } else {
      if (code & 1u) pattern_body<code_mask(5)>(acc, h, w01, w23);
      else pattern_body<code_mask(4)>(acc, h, w01, w23);
    }
  } else {
    if (code & 2u) {
      PAT_ROW3();
      if (code & 1u) pattern_body<code_mask(3)>(acc, h, w01, w23);
      else pattern_body<code_mask(2)>(acc, h, w01, w23);
    } else {
      if (code & 1u) pattern_body<code_mask(1)>(acc, h, w01, w23);
      else pattern_body<code_mask(0)>(acc, h, w01, w23);
    }
  }
#undef PAT_ROW3
}

// ---- 4 x 14 pixel tiles (56 accumulators)
constexpr int TR4 = 4;
static_assert(ROWB == kImgRowBytes, "the descriptors' window offsets are written for this row pitch");
__host__ __device__ constexpr int last_tap_row(uint32_t mask) { return (mask >> 6) ? 2 : ((mask >> 3) ? 1 : 0); }

// A tile in tensor memory: 56 consecutive columns of the thread's lane, value (y, x) at column 14 y + x, moved by
// three transfers of 32, 16 and 8 columns whose register lists are the tile in that order (no padding values, so
// the accumulators can stay where they are).  tmem_store_tile / tmem_load_tile only issue the transfers;
// tmem_wait_st / tmem_wait_ld complete them.
#define PAT_F(i) "f"(a[(i) / TC][(i) % TC])
#define PAT_O(i) "=f"(a[(i) / TC][(i) % TC])
__device__ __forceinline__ void tmem_store_tile(uint32_t taddr, const float (&a)[TR4][TC]) {
  static_assert(TR4 * TC == 56, "32 + 16 + 8 columns");
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), PAT_F(0), PAT_F(1), PAT_F(2), PAT_F(3), PAT_F(4), PAT_F(5), PAT_F(6), PAT_F(7), PAT_F(8), PAT_F(9), PAT_F(10),
        PAT_F(11), PAT_F(12), PAT_F(13), PAT_F(14), PAT_F(15), PAT_F(16), PAT_F(17), PAT_F(18), PAT_F(19), PAT_F(20), PAT_F(21),
        PAT_F(22), PAT_F(23), PAT_F(24), PAT_F(25), PAT_F(26), PAT_F(27), PAT_F(28), PAT_F(29), PAT_F(30), PAT_F(31)
      : "memory");
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr + 32u), PAT_F(32), PAT_F(33), PAT_F(34), PAT_F(35), PAT_F(36), PAT_F(37), PAT_F(38), PAT_F(39), PAT_F(40),
        PAT_F(41), PAT_F(42), PAT_F(43), PAT_F(44), PAT_F(45), PAT_F(46), PAT_F(47)
      : "memory");
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
      ::"r"(taddr + 48u), PAT_F(48), PAT_F(49), PAT_F(50), PAT_F(51), PAT_F(52), PAT_F(53), PAT_F(54), PAT_F(55)
      : "memory");
}
__device__ __forceinline__ void tmem_load_tile(uint32_t taddr, float (&a)[TR4][TC]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : PAT_O(0), PAT_O(1), PAT_O(2), PAT_O(3), PAT_O(4), PAT_O(5), PAT_O(6), PAT_O(7), PAT_O(8), PAT_O(9), PAT_O(10),
        PAT_O(11), PAT_O(12), PAT_O(13), PAT_O(14), PAT_O(15), PAT_O(16), PAT_O(17), PAT_O(18), PAT_O(19), PAT_O(20), PAT_O(21),
        PAT_O(22), PAT_O(23), PAT_O(24), PAT_O(25), PAT_O(26), PAT_O(27), PAT_O(28), PAT_O(29), PAT_O(30), PAT_O(31)
      : "r"(taddr) : "memory");
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : PAT_O(32), PAT_O(33), PAT_O(34), PAT_O(35), PAT_O(36), PAT_O(37), PAT_O(38), PAT_O(39), PAT_O(40),
        PAT_O(41), PAT_O(42), PAT_O(43), PAT_O(44), PAT_O(45), PAT_O(46), PAT_O(47)
      : "r"(taddr + 32u) : "memory");
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
      : PAT_O(48), PAT_O(49), PAT_O(50), PAT_O(51), PAT_O(52), PAT_O(53), PAT_O(54), PAT_O(55)
      : "r"(taddr + 48u) : "memory");
}
#undef PAT_F
#undef PAT_O

// One multiply-add whose fp16 operands are halves of 32-bit registers (no instruction is spent on taking a
// register apart: the halves are operand selectors of the multiply-add itself).
template <int VHI, int WHI>
__device__ __forceinline__ void fma_half_of(float& acc, uint32_t v, uint32_t w) {
  unsigned short a, b, u0, u1;
  if (VHI) asm("mov.b32 {%0,%1}, %2;" : "=h"(u0), "=h"(a) : "r"(v)); else asm("mov.b32 {%0,%1}, %2;" : "=h"(a), "=h"(u0) : "r"(v));
  if (WHI) asm("mov.b32 {%0,%1}, %2;" : "=h"(u1), "=h"(b) : "r"(w)); else asm("mov.b32 {%0,%1}, %2;" : "=h"(b), "=h"(u1) : "r"(w));
  asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc) : "h"(a), "h"(b));
}
__device__ __forceinline__ void lds_row(uint32_t (&q)[8], uint32_t a0, uint32_t a1) {
  lds128(a0, q[0], q[1], q[2], q[3]);   // logical chunk 0: cols -1..6
  lds128(a1, q[4], q[5], q[6], q[7]);   // logical chunk 1: cols 7..14
}
template <int B>
__device__ __forceinline__ void tap_row(float (&acc)[TC], const uint32_t (&q)[8], uint32_t w01, uint32_t w23, int t) {
  // tap number t (0..3, compile time after unrolling) of the pattern sits at kernel column B % 3
  constexpr int c = B % 3;
#pragma unroll
  for (int x = 0; x < TC; ++x) {
    const uint32_t v = q[(x + c) >> 1];
    const uint32_t w = t < 2 ? w01 : w23;
    if ((x + c) & 1) { if (t & 1) fma_half_of<1, 1>(acc[x], v, w); else fma_half_of<1, 0>(acc[x], v, w); }
    else             { if (t & 1) fma_half_of<0, 1>(acc[x], v, w); else fma_half_of<0, 0>(acc[x], v, w); }
  }
}

// The code of one pattern: it walks down the thread's window one row of 16 pixels at a time, and every row
// serves all taps that read it.  MASK is a compiled code (first tap in kernel row 0); a0 / a1 = the lane's
// addresses of logical chunks 0 / 1 of window row `sh`, the first row the code reads; r0 / r1 = that row and the
// next one, loaded by the caller before it branched here.  The two chunks of a segment trade places every four
// image rows, i.e. from window row 4 on.
template <uint32_t MASK>
__device__ __forceinline__ void pattern_body4(float (&acc)[TR4][TC], uint32_t a0, uint32_t a1, uint32_t sh, uint32_t w01, uint32_t w23,
                                              const uint32_t (&r0)[8], const uint32_t (&r1)[8]) {
  constexpr int NR = last_tap_row(MASK) + TR4;      // rows of the window this code reads
#pragma unroll
  for (int j = 0; j < NR; ++j) {
    uint32_t q[8];
    if (j == 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i) q[i] = r0[i];
    } else if (j == 1) {
#pragma unroll
      for (int i = 0; i < 8; ++i) q[i] = r1[i];
    } else {
      uint32_t p0 = a0 + j * ROWB, p1 = a1 + j * ROWB;
      if (j >= 4) { const uint32_t t = p0; p0 = p1; p1 = t; }
      else if (j == 3) { const uint32_t q0 = sh ? p1 : p0, q1 = sh ? p0 : p1; p0 = q0; p1 = q1; }
      lds_row(q, p0, p1);
    }
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      constexpr uint32_t M = MASK;
      const int b = nth_bit(M, t);
      const int y = j - b / 3;
      if (y >= 0 && y < TR4) {
        switch (b) {   // b is a compile-time constant after unrolling
          case 0: tap_row<0>(acc[y], q, w01, w23, t); break;
          case 1: tap_row<1>(acc[y], q, w01, w23, t); break;
          case 2: tap_row<2>(acc[y], q, w01, w23, t); break;
          case 3: tap_row<3>(acc[y], q, w01, w23, t); break;
          case 4: tap_row<4>(acc[y], q, w01, w23, t); break;
          case 5: tap_row<5>(acc[y], q, w01, w23, t); break;
          case 6: tap_row<6>(acc[y], q, w01, w23, t); break;
          case 7: tap_row<7>(acc[y], q, w01, w23, t); break;
          default: tap_row<8>(acc[y], q, w01, w23, t); break;
        }
      }
    }
  }
}

// One kept kernel on a 4-row tile.  plane = the lane's address of logical chunk 0 of window row 0 in channel
// plane 0 of the stage; meta / w01 / w23 / off = the kernel's descriptor (off = byte offset of its channel plane
// plus its window row shift).  Every branch is warp-uniform.  NCODES = number of compiled pattern codes the
// library can produce (6 for the eight patterns of Section 4.2, 10 for the twelve), GENERIC = the library holds
// patterns without compiled code: a kernel compiled for a smaller set carries less code and fewer live registers.
template <int NCODES, bool GENERIC>
__device__ __forceinline__ void one_kernel4(float (&acc)[TR4][TC], uint32_t plane, uint32_t meta, uint32_t w01, uint32_t w23,
                                            uint32_t off, const uint32_t (&r0)[8], const uint32_t (&r1)[8]) {
  static_assert(NCODES == 6 || NCODES == kNumCodes, "code sets with compiled dispatch trees");
  static_assert(kGenericCode == 15, "the generic code is the last leaf of the tree");
  const uint32_t sh = (meta >> 17) & 1u;
  const uint32_t a0 = plane + off, a1 = a0 ^ 16u;
  const uint32_t code = (meta >> 13) & 15u;
  if ((NCODES > 8 || GENERIC) && (code & 8u)) {
    if (code & 4u) {
      if constexpr (GENERIC) {
        // any other pattern: position by position, each with its own pass over the window rows it reads
        const uint32_t baseA = a0 - sh * ROWB, baseB = baseA ^ 16u;
#define PAT_TAP4(B)                                                                          \
  if (meta & (16u << (B))) {                                                                 \
    _Pragma("unroll")                                                                        \
    for (int y = 0; y < TR4; ++y) {                                                          \
      uint32_t q[8];                                                                         \
      const int jr = y + (B) / 3;                                                            \
      const uint32_t q0 = baseA + jr * ROWB, q1 = baseB + jr * ROWB;                         \
      if (jr >= 4) lds_row(q, q1, q0); else lds_row(q, q0, q1);                              \
      tap_row<B>(acc[y], q, w01, w23, 0);                                                    \
    }                                                                                        \
    w01 = __funnelshift_r(w01, w23, 16);                                                     \
    w23 >>= 16;                                                                              \
  }
        PAT_TAP4(0) PAT_TAP4(1) PAT_TAP4(2) PAT_TAP4(3) PAT_TAP4(4) PAT_TAP4(5) PAT_TAP4(6) PAT_TAP4(7) PAT_TAP4(8)
#undef PAT_TAP4
      }
    } else if constexpr (NCODES > 8) {
      if (code & 1u) pattern_body4<code_mask(9)>(acc, a0, a1, sh, w01, w23, r0, r1);
      else pattern_body4<code_mask(8)>(acc, a0, a1, sh, w01, w23, r0, r1);
    }
  } else if (code & 4u) {
    if (NCODES > 6 && (code & 2u)) {
      if constexpr (NCODES > 6) {
        if (code & 1u) pattern_body4<code_mask(7)>(acc, a0, a1, sh, w01, w23, r0, r1);
        else pattern_body4<code_mask(6)>(acc, a0, a1, sh, w01, w23, r0, r1);
      }
    } else {
      if (code & 1u) pattern_body4<code_mask(5)>(acc, a0, a1, sh, w01, w23, r0, r1);
      else pattern_body4<code_mask(4)>(acc, a0, a1, sh, w01, w23, r0, r1);
    }
  } else {
    if (code & 2u) {
      if (code & 1u) pattern_body4<code_mask(3)>(acc, a0, a1, sh, w01, w23, r0, r1);
      else pattern_body4<code_mask(2)>(acc, a0, a1, sh, w01, w23, r0, r1);
    } else {
      if (code & 1u) pattern_body4<code_mask(1)>(acc, a0, a1, sh, w01, w23, r0, r1);
      else pattern_body4<code_mask(0)>(acc, a0, a1, sh, w01, w23, r0, r1);
    }
  }
}

}  // namespace fast16
}  // namespace pat
