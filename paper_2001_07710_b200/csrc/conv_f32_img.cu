// Sparse 3x3 convolution for fp32 storage and accumulation (sm_100a): the workspace path of conv_f16_img.cu for
// 4-byte activations (stride 2 likewise: computed like stride 1, the results at even rows and columns written).  The same three kernels and the same protocol (stage images built once per call, a
// persistent warp-specialised kernel fed by bulk copies through a ring of shared-memory slots, flat pack-time
// operation lists, one accumulator tile in registers and one parked in tensor memory, cut items reduced by a third
// kernel); what differs:
//  * a stage holds 8 input channels (the same 72 KB): channel-planar [8 ch][36 rows][4 segments][16 px] floats, a
//    segment = four 16-byte chunks.  Physical chunk = logical chunk ^ (segment / 2 + 2 x parity of the tile row whose
//    window starts in that row's group of four), so the eight lanes that share a wavefront of a 16-byte load
//    (four column slots x two tile rows) touch eight different bank groups;
//  * an operation is 32 bytes (four fp32 taps), a window row is four 16-byte loads and plain fp32 multiply-adds;
//  * the results leave in two rounds (tile rows 0-1, then 2-3): a slot takes one tile row of fp32 results.
#include <algorithm>
#include "img_geometry.cuh"

namespace pat {
namespace img32 {
using namespace fast16;
using namespace imggeo;

constexpr int NTHREADS = 640;              // 16 consumer warps, producer warp, three idle warps (register donors)
constexpr int W_PRODUCER = NCW;
constexpr int CBI = kChanStageF32;         // channels per ring stage (8)
constexpr int SEGF = 64;                   // bytes of a segment: 16 px of one channel
constexpr int ROWF = LX * SEGF;            // 256
constexpr int CHPF = MAXROWS * ROWF;       // channel plane pitch (9216)
constexpr int IMG_BYTES = CBI * CHPF;      // 73728
static_assert(ROWF == kImgRowBytesF32 && CHPF == kImgPlaneBytesF32 && NCW == kBlockWarps, "the descriptor blocks are written for this geometry");
constexpr int MAX_NS = 3;
constexpr int OPB = 32;                    // bytes of an operation
constexpr int MAXE3 = 108;                 // operations of a descriptor block that still allow three slots
constexpr int DBLK3 = kBlockHeaderBytes + MAXE3 * OPB;                       // 3584
constexpr int DBLK2 = kBlockHeaderBytes + (FG * CBI + kBlockWarps + 4) * OPB; // largest possible block and spare slots (8960)
constexpr int OFF_SLOTS = 256;
constexpr int SMEM_BYTES = OFF_SLOTS + 3 * (IMG_BYTES + DBLK3);
static_assert(OFF_SLOTS + 2 * (IMG_BYTES + DBLK2) <= SMEM_BYTES, "the two-slot layout fits too");
static_assert(IMG_BYTES % 128 == 0 && DBLK3 % 128 == 0 && DBLK2 % 128 == 0 && SMEM_BYTES <= 232448, "shared memory budget of one SM");
constexpr int OUT_PITCH = FG * 4 + 4;      // output staging inside a slot: [448 px][32 channels] fp32, pixel pitch 132 B
constexpr int OUT_ROW = 32 * TC * OUT_PITCH;   // one row of every thread tile (59136)
static_assert(OUT_ROW <= IMG_BYTES, "one tile row of results fits a slot");
constexpr int CONSUMER_REGS = 112, OTHER_REGS = 32;
static_assert(NCW * 32 * CONSUMER_REGS + (NTHREADS / 32 - NCW) * 32 * OTHER_REGS <= NTHREADS * LAUNCH_REGS, "register pool of the block");
constexpr uint32_t TMEM_COLS = 512;

struct Params : ImgGeometry {   // geometry, work items and cut items: see img_geometry.cuh (nct = stages of 8 channels)
  const float* x;
  float* y;
  char* images;            // stage images: [region][stage of 8 channels][IMG_BYTES]
  const int32_t* xfilt;    // execution position -> original filter
  const uint32_t* dboff;   // descriptor block -> offset in 16-byte units
  const char* dblk;
  const BlobHeader* hdr;
  int* status;
  int K;
  long long n_keep;
  uint16_t masks[256];
};

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// ------------------------------------------------------------------------------------------ stage images
// One block per (region, stage of 8 channels).  Image layout: byte ch * CHPF + row * ROWF + seg * SEGF +
// ((px >> 2) ^ sw) * 16 + (px & 3) * 4 with px = 0..15 <-> image column 14 * (tile column) - 1 + px and
// sw = seg / 2 + 2 * (parity of the tile row, counted through both bands, whose window starts in that row's group of four).
constexpr int SI_THREADS = 256;
constexpr int SI_PITCH = CHPF + 16;        // the two channel quads a warp writes at once fall into different bank halves
constexpr int SI_SMEM = CBI * SI_PITCH;
__global__ void __launch_bounds__(SI_THREADS) k_stage_images_f32(const Params p) {
  extern __shared__ __align__(16) unsigned char img[];
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // see conv_f16_img.cu
  const int st8 = (int)(blockIdx.x % (unsigned)p.nct);
  const int reg = (int)(blockIdx.x / (unsigned)p.nct);
  const Region r = decode_region(p, reg);
  const int rows0 = TR4 * r.n0 + 2;
  const int txe_shift = (p.TXe == 4) ? 2 : (p.TXe == 2 ? 1 : 0);
  // a unit = one pixel x one channel quad: one 16-byte load, four 4-byte stores
  constexpr int UNITS = MAXROWS * LX * 16 * 2, PER_THREAD = UNITS / SI_THREADS;   // 18 per thread
  static_assert(UNITS % SI_THREADS == 0, "units per thread");
  uint4 v[PER_THREAD];
#pragma unroll
  for (int i = 0; i < PER_THREAD; ++i) {
    const int u = (int)threadIdx.x + SI_THREADS * i;
    const int quad = u & 1, k = (u >> 1) & 15, seg = (u >> 5) & 3, pr = u >> 7;
    v[i] = make_uint4(0u, 0u, 0u, 0u);
    if (pr < r.nrows) {
      const int b = (pr >= rows0) ? 1 : 0;
      const int yy = b ? (pr - rows0 - 1) : (TR4 * r.ta0 - 1 + pr);
      const int ni = seg >> txe_shift, tx = seg & (p.TXe - 1);
      const int n_img = (r.ig0 + b) * p.NI + ni;
      const int xx = (r.cg * p.TXe + tx) * TC - 1 + k;
      if (yy >= 0 && yy < p.H && n_img < p.N && xx >= 0 && xx < p.W)
        v[i] = __ldg(reinterpret_cast<const uint4*>(p.x + (((size_t)n_img * p.H + yy) * p.W + xx) * p.C + st8 * CBI + quad * 4));
    }
  }
#pragma unroll
  for (int i = 0; i < PER_THREAD; ++i) {
    const int u = (int)threadIdx.x + SI_THREADS * i;
    const int quad = u & 1, k = (u >> 1) & 15, seg = (u >> 5) & 3, pr = u >> 7;
    const int b = (pr >= rows0) ? 1 : 0;
    const int par = ((((b ? pr - rows0 : pr) >> 2) + (b ? r.n0 : 0)) & 1);
    const int sw = (seg >> 1) | (par << 1);
    const uint32_t o = (uint32_t)(pr * ROWF + seg * SEGF + (((k >> 2) ^ sw) << 4) + (k & 3) * 4);
    *reinterpret_cast<uint32_t*>(img + (quad * 4 + 0) * SI_PITCH + o) = v[i].x;
    *reinterpret_cast<uint32_t*>(img + (quad * 4 + 1) * SI_PITCH + o) = v[i].y;
    *reinterpret_cast<uint32_t*>(img + (quad * 4 + 2) * SI_PITCH + o) = v[i].z;
    *reinterpret_cast<uint32_t*>(img + (quad * 4 + 3) * SI_PITCH + o) = v[i].w;
  }
  // the planes leave by bulk copies (one per channel; the plane pitch keeps them 16-byte aligned), see conv_f16_img.cu
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  if (threadIdx.x < CBI) {
    char* dst = p.images + (size_t)blockIdx.x * IMG_BYTES + (size_t)threadIdx.x * CHPF;
    const uint32_t src = smem_u32(img + threadIdx.x * SI_PITCH);
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"((uint32_t)CHPF) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
  }
}

// ------------------------------------------------------------------------------------------ consumer math
__device__ __forceinline__ void lds_row_f32(float (&h)[16], uint32_t a, uint32_t x) {
  // a = address of logical chunk 0 of the row (64-byte aligned), x = the lane's chunk swizzle for this row (bits 4-5)
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    uint32_t q0, q1, q2, q3;
    lds128((a + 16u * c) ^ x, q0, q1, q2, q3);
    h[4 * c] = __uint_as_float(q0); h[4 * c + 1] = __uint_as_float(q1); h[4 * c + 2] = __uint_as_float(q2); h[4 * c + 3] = __uint_as_float(q3);
  }
}

// The code of one pattern on a 4 x 14 tile (see pattern_body4 in f16_tile.cuh): a0 = address of logical chunk 0 of
// window row `sh`, swb = the lane's chunk swizzle (bits 4-5) for window rows 0-3; from window row 4 on the rows
// belong to the next tile row's group, whose parity bit is the other one.
// S2 (stride 2): only the results at even rows and columns of the tile are wanted (tiles start at even image
// coordinates), so the multiply-adds of the other three quarters and the window rows only they read are left out.
__host__ __device__ constexpr bool row_used(uint32_t mask, int j, bool s2) {
  for (int t = 0; t < 4; ++t) {
    const int y = j - nth_bit(mask, t) / 3;
    if (y >= 0 && y < TR4 && (!s2 || (y & 1) == 0)) return true;
  }
  return false;
}
template <uint32_t MASK, bool S2>
__device__ __forceinline__ void pattern_body4f(float (&acc)[TR4][TC], uint32_t a0, uint32_t sh, uint32_t swb, const float (&w)[4],
                                               const float (&r0)[16]) {
  constexpr int NR = last_tap_row(MASK) + TR4;
#pragma unroll
  for (int j = 0; j < NR; ++j) {
    if (!row_used(MASK, j, S2)) continue;
    uint32_t x = swb;
    if (j >= 4) x ^= 32u;
    else if (j == 3) x ^= sh << 5;
    float h[16];
    if (j == 0) {
#pragma unroll
      for (int i = 0; i < 16; ++i) h[i] = r0[i];       // loaded by the caller before it branched here
    } else {
      lds_row_f32(h, a0 + j * ROWF, x);
    }
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const int b = nth_bit(MASK, t);
      const int y = j - b / 3, c = b % 3;
      if (y >= 0 && y < TR4 && (!S2 || (y & 1) == 0)) {
#pragma unroll
        for (int xx = 0; xx < TC; xx += (S2 ? 2 : 1)) acc[y][xx] = fmaf(h[xx + c], w[t], acc[y][xx]);
      }
    }
  }
}

template <int NCODES, bool GENERIC, bool S2>
__device__ __forceinline__ void one_kernel4f(float (&acc)[TR4][TC], uint32_t plane, uint32_t swb, uint32_t meta, uint32_t off,
                                             float (&w)[4], const float (&r0)[16]) {
  static_assert(NCODES == 6 || NCODES == kNumCodes, "code sets with compiled dispatch trees");
  const uint32_t sh = (meta >> 17) & 1u;
  const uint32_t a0 = plane + off;
  const uint32_t code = (meta >> 13) & 15u;
  if ((NCODES > 8 || GENERIC) && (code & 8u)) {
    if (code & 4u) {
      if constexpr (GENERIC) {
        // any other pattern: position by position, each with its own pass over the window rows it reads
        const uint32_t base = a0 - sh * ROWF;
#define PAT_TAP4F(B)                                                                         \
  if (meta & (16u << (B))) {                                                                 \
    _Pragma("unroll")                                                                        \
    for (int y = 0; y < TR4; y += (S2 ? 2 : 1)) {                                            \
      float h[16];                                                                           \
      const int jr = y + (B) / 3;                                                            \
      lds_row_f32(h, base + jr * ROWF, jr >= 4 ? (swb ^ 32u) : swb);                         \
      _Pragma("unroll")                                                                      \
      for (int xx = 0; xx < TC; xx += (S2 ? 2 : 1)) acc[y][xx] = fmaf(h[xx + (B) % 3], w[0], acc[y][xx]);  \
    }                                                                                        \
    w[0] = w[1]; w[1] = w[2]; w[2] = w[3];                                                   \
  }
        PAT_TAP4F(0) PAT_TAP4F(1) PAT_TAP4F(2) PAT_TAP4F(3) PAT_TAP4F(4) PAT_TAP4F(5) PAT_TAP4F(6) PAT_TAP4F(7) PAT_TAP4F(8)
#undef PAT_TAP4F
      }
    } else if constexpr (NCODES > 8) {
      if (code & 1u) pattern_body4f<code_mask(9), S2>(acc, a0, sh, swb, w, r0);
      else pattern_body4f<code_mask(8), S2>(acc, a0, sh, swb, w, r0);
    }
  } else if (code & 4u) {
    if (NCODES > 6 && (code & 2u)) {
      if constexpr (NCODES > 6) {
        if (code & 1u) pattern_body4f<code_mask(7), S2>(acc, a0, sh, swb, w, r0);
        else pattern_body4f<code_mask(6), S2>(acc, a0, sh, swb, w, r0);
      }
    } else {
      if (code & 1u) pattern_body4f<code_mask(5), S2>(acc, a0, sh, swb, w, r0);
      else pattern_body4f<code_mask(4), S2>(acc, a0, sh, swb, w, r0);
    }
  } else {
    if (code & 2u) {
      if (code & 1u) pattern_body4f<code_mask(3), S2>(acc, a0, sh, swb, w, r0);
      else pattern_body4f<code_mask(2), S2>(acc, a0, sh, swb, w, r0);
    } else {
      if (code & 1u) pattern_body4f<code_mask(1), S2>(acc, a0, sh, swb, w, r0);
      else pattern_body4f<code_mask(0), S2>(acc, a0, sh, swb, w, r0);
    }
  }
}

// ------------------------------------------------------------------------------------------ the convolution
// Ring protocol as in conv_f16_img.cu: per work item nst stages of 8 channels, then two output stages whose slots
// the consumers use as staging for the results - here twice (tile rows 0-1, then 2-3), with a block-wide barrier
// after writing and after copying out the first pair of rows.
template <bool SPARSE, int NCODES, bool GENERIC, bool S2>
__device__ __forceinline__ void conv_body(const Params& p, unsigned char* smem) {
  constexpr int NS = SPARSE ? 3 : 2;
  constexpr uint32_t SLOT = (uint32_t)IMG_BYTES + (uint32_t)(SPARSE ? DBLK3 : DBLK2);
  const uint32_t sbase = smem_u32(smem);
  auto slot_full = [&](int s) { return sbase + 8u * s; };
  auto slot_empty = [&](int s) { return sbase + 8u * (MAX_NS + s); };
  auto out_ready = [&](int s) { return sbase + 8u * (2 * MAX_NS + s); };   // 0: results written, 1: first rows copied out
  static_assert(8 * 3 * MAX_NS + 8 <= OFF_SLOTS, "barrier block and control words");
  int& s_abort = *reinterpret_cast<int*>(smem + 8 * 3 * MAX_NS);
  uint32_t& s_tmem = *reinterpret_cast<uint32_t*>(smem + 8 * 3 * MAX_NS + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t slot0 = sbase + OFF_SLOTS;

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < MAX_NS; ++s) { mbar_init(slot_full(s), 1); mbar_init(slot_empty(s), NCW); mbar_init(out_ready(s), NCW); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) tmem_alloc(smem_u32(&s_tmem), TMEM_COLS);
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  volatile int* abort_flag = &s_abort;
  const uint32_t tmem_base = s_tmem;

  const int n_my_whole = (p.n_whole > (int)blockIdx.x) ? (p.n_whole - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  const int n_my_items = n_my_whole + ((p.parts > 1 && (int)blockIdx.x < p.n_split * p.parts) ? 1 : 0);
  const int nst = p.nct;
  auto item_of = [&](int it_idx) {
    return it_idx < n_my_whole ? (int)blockIdx.x + it_idx * (int)gridDim.x : p.n_whole + (int)blockIdx.x / p.parts;
  };
  auto piece_of = [&](int it_idx, int& c0, int& c1) {
    if (it_idx < n_my_whole) { c0 = 0; c1 = nst; return false; }
    const int q = (int)blockIdx.x % p.parts;
    c0 = q * nst / p.parts; c1 = (q + 1) * nst / p.parts;
    return true;
  };

  if (warp >= NCW) {
    set_warp_registers<OTHER_REGS>();
    if (warp == W_PRODUCER) {
      // ========================================================================= producer warp
      int pslot = 0;
      uint32_t epar = 1u;
      uint32_t armed = 0u, armed_par = 0u;
      bool alive = true;
      for (int it_idx = 0; it_idx < n_my_items && alive; ++it_idx) {
        const int item = item_of(it_idx);
        const int g = item % p.NG, reg = item / p.NG;
        const char* img = p.images + (size_t)reg * nst * IMG_BYTES;
        const uint32_t* bo = p.dboff + (size_t)g * nst;
        int c0, c1;
        const bool piece = piece_of(it_idx, c0, c1);
        uint32_t o0 = __ldg(bo + c0);
        for (int cb = c0; cb < c1 && alive; ++cb) {
          const uint32_t o1 = __ldg(bo + cb + 1);
          if (!mbar_wait<kFillSleepNs>(slot_empty(pslot), epar, abort_flag)) { alive = false; break; }
          if (lane == 0) {
            const uint32_t dbytes = (o1 - o0) * 16u;
            const uint32_t dst = slot0 + (uint32_t)pslot * SLOT;
            mbar_arrive_expect_tx(slot_full(pslot), (uint32_t)IMG_BYTES + dbytes);
            bulk_load(dst + IMG_BYTES, p.dblk + (size_t)o0 * 16, dbytes, slot_full(pslot));
            bulk_load(dst, img + (size_t)cb * IMG_BYTES, (uint32_t)IMG_BYTES, slot_full(pslot));
          }
          armed |= 1u << pslot;
          armed_par = (armed_par & ~(1u << pslot)) | ((epar ^ 1u) << pslot);
          o0 = o1;
          if (++pslot == NS) { pslot = 0; epar ^= 1u; }
        }
        // output stages: hand the next two slots to the consumers as they become free (a piece has none)
        for (int o = 0; o < 2 && alive && !piece; ++o) {
          if (!mbar_wait<kFillSleepNs>(slot_empty(pslot), epar, abort_flag)) { alive = false; break; }
          if (lane == 0) mbar_arrive(slot_full(pslot));
          armed &= ~(1u << pslot);
          if (++pslot == NS) { pslot = 0; epar ^= 1u; }
        }
      }
      if (!alive && lane == 0) {
        const unsigned long long t0 = global_ns();
        for (int s = 0; s < NS; ++s) {
          if (!((armed >> s) & 1u)) continue;
          for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
            if (mbar_try_wait(slot_full(s), (armed_par >> s) & 1u)) break;
            if (global_ns() - t0 > kWaitNs) break;
          }
        }
        atomicExch(p.status, PAT_ERR_TIMEOUT);
      }
    }
  } else {
    // =========================================================================== consumer warps
    set_warp_registers<CONSUMER_REGS>();
    const uint32_t tm0 = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 128);
    auto park = [&](uint32_t f, const float (&a)[TR4][TC]) {
      tmem_store_tile(tm0 + f * 64u, a);
      tmem_wait_st();
    };
    auto fetch = [&](uint32_t f, float (&a)[TR4][TC]) {
      tmem_load_tile(tm0 + f * 64u, a);
      tmem_wait_ld();
    };
    int pslot = 0;
    uint32_t fpar = 0u;
    bool alive = true;
    for (int it_idx = 0; it_idx < n_my_items && alive; ++it_idx) {
      const int item = item_of(it_idx);
      const Region it = decode_region(p, item / p.NG);
      const int ly = lane >> 2, lx = lane & 3;
      const int band = (ly < it.n0) ? 0 : 1;
      // the lane's address of logical chunk 0 of window row 0, relative to a channel plane, and its chunk swizzle
      const uint32_t offA = (uint32_t)((TR4 * ly + 2 * band) * ROWF + lx * SEGF);
      const uint32_t swb = (uint32_t)(((lx >> 1) | ((ly & 1) << 1)) << 4);
      float acc[TR4][TC];
#pragma unroll
      for (int y = 0; y < TR4; ++y)
#pragma unroll
        for (int x = 0; x < TC; ++x) acc[y][x] = 0.0f;
      int c0, c1;
      const bool piece = piece_of(it_idx, c0, c1);
      if (!mbar_wait<0>(slot_full(pslot), fpar, abort_flag)) { alive = false; break; }
      uint32_t sl = slot0 + (uint32_t)pslot * SLOT;
      uint32_t pl0 = sl + offA;
      const uint32_t hw = lds32(sl + IMG_BYTES + (uint32_t)warp * 4u);
      uint32_t cur = hw >> 31;           // which of the two filters the registers hold (both tiles are zero now)
      park(cur ^ 1u, acc);
      uint32_t e = sl + IMG_BYTES + kBlockHeaderBytes + (hw & 0xFFFFu) * 16u;
      uint32_t m0, off, w0, w1, w2, w3, pad0, pad1;
      lds128(e, m0, off, w0, w1);
      lds128(e + 16u, w2, w3, pad0, pad1);
      int cb = c0;
#pragma unroll 1
      for (;;) {
        // all lanes hold the same descriptor word; the warp-wide reduction makes that known to the compiler, so that
        // the branches of this visit are uniform branches without reconvergence bookkeeping (see conv_f16_img.cu)
        const uint32_t cm = __reduce_or_sync(0xFFFFFFFFu, m0), coff = off;
        float w[4] = {__uint_as_float(w0), __uint_as_float(w1), __uint_as_float(w2), __uint_as_float(w3)};
        float r0[16];                      // the first window row of this kernel (window rows 0-3 share the lane's swizzle)
        lds_row_f32(r0, pl0 + coff, swb);
        e += OPB;
        lds128(e, m0, off, w0, w1);        // the next operation
        lds128(e + 16u, w2, w3, pad0, pad1);
        if (cm & (kOpSwap | kOpNop)) {     // one test for the two rare cases
          if (cm & kOpNop) goto stage_end;
          park(cur, acc);
          cur ^= 1u;
          fetch(cur, acc);
        }
        one_kernel4f<NCODES, GENERIC, S2>(acc, pl0, swb, cm, coff, w, r0);
      stage_end:
        if (cm & kOpEnd) {
          __syncwarp();
          if (lane == 0) mbar_arrive(slot_empty(pslot));
          if (++pslot == NS) { pslot = 0; fpar ^= 1u; }
          if (++cb == c1) break;
          if (!mbar_wait<0>(slot_full(pslot), fpar, abort_flag)) { alive = false; break; }
          sl = slot0 + (uint32_t)pslot * SLOT;
          pl0 = sl + offA;
          e = sl + IMG_BYTES + kBlockHeaderBytes + (cm >> kOpNextShift) * 16u;
          lds128(e, m0, off, w0, w1);
          lds128(e + 16u, w2, w3, pad0, pad1);
        }
      }
      if (!alive) break;

      if (piece) {
        // partial sums of a cut item: one 128-byte line per value and warp
        float* dst = p.partials + (size_t)blockIdx.x * (FG * TR4 * TC * 32) + lane;
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
          float* d = dst + (size_t)(cur ? FG - 1 - warp : warp) * (TR4 * TC * 32);
#pragma unroll
          for (int y = 0; y < TR4; ++y)
#pragma unroll
            for (int x = 0; x < TC; ++x) d[(y * TC + x) * 32] = acc[y][x];
          if (half == 0) {
            cur ^= 1u;
            fetch(cur, acc);
          }
        }
        continue;
      }

      // results, two rounds: tile row 2 r into the first output slot, 2 r + 1 into the second, as [pixel][32 channels];
      // once all 16 warps have written, every warp copies those rows of two thread tiles to global memory
      const int g_out = item % p.NG;
      const uint32_t cposA = ((uint32_t)__ldg(p.xfilt + g_out * FG + warp) & (uint32_t)(FG - 1)) * 4u;
      const uint32_t cposB = ((uint32_t)__ldg(p.xfilt + g_out * FG + FG - 1 - warp) & (uint32_t)(FG - 1)) * 4u;
      const int s0 = pslot, s1 = (pslot + 1 == NS) ? 0 : pslot + 1;
      const uint32_t par1 = (pslot + 1 == NS) ? (fpar ^ 1u) : fpar;
      if (!mbar_wait<0>(slot_full(s0), fpar, abort_flag)) { alive = false; break; }
      if (!mbar_wait<0>(slot_full(s1), par1, abort_flag)) { alive = false; break; }
      const uint32_t ob0 = slot0 + (uint32_t)s0 * SLOT, ob1 = slot0 + (uint32_t)s1 * SLOT;
      const int txe_shift = (p.TXe == 4) ? 2 : (p.TXe == 2 ? 1 : 0);
      // tiles 16-31 sit one word further on: lanes l and l + 16 would otherwise store to the same banks
      const uint32_t ol = (uint32_t)(lane * TC) * OUT_PITCH + (uint32_t)(lane >> 4) * 4u;
#pragma unroll 1
      for (int round = 0; round < 2 && alive; ++round) {
        // this round's two rows of both filters: the one in registers first, then the other one
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
          const uint32_t cp = ol + (cur ? cposB : cposA);
          if (p.relu) {                      // the fused rectifier (a tile parked between the rounds is clamped twice: harmless)
#pragma unroll
            for (int y = 0; y < TR4; ++y)
#pragma unroll
              for (int x = 0; x < TC; ++x) acc[y][x] = fmaxf(acc[y][x], 0.0f);
          }
          if (p.relu == 2) {
            // rectifier and 2 x 2 max pooling: a thread tile starts at an even row and column, so the pooling windows
            // of this round's two rows lie in this lane's registers; the seven pooled values take the first slot
#pragma unroll
            for (int xx = 0; xx < TC / 2; ++xx) {
              const float top = round ? fmaxf(acc[2][2 * xx], acc[2][2 * xx + 1]) : fmaxf(acc[0][2 * xx], acc[0][2 * xx + 1]);
              const float bot = round ? fmaxf(acc[3][2 * xx], acc[3][2 * xx + 1]) : fmaxf(acc[1][2 * xx], acc[1][2 * xx + 1]);
              sts32(ob0 + (uint32_t)(xx * OUT_PITCH) + cp, __float_as_uint(fmaxf(fmaxf(top, bot), 0.0f)));
            }
          } else {
#pragma unroll
            for (int x = 0; x < TC; ++x) {
              sts32(ob0 + (uint32_t)(x * OUT_PITCH) + cp, __float_as_uint(round ? acc[2][x] : acc[0][x]));
              sts32(ob1 + (uint32_t)(x * OUT_PITCH) + cp, __float_as_uint(round ? acc[3][x] : acc[1][x]));
            }
          }
          if (half == 0) {
            if (round == 0) park(cur, acc);     // its rows 2-3 are still to come
            cur ^= 1u;
            fetch(cur, acc);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(out_ready(0));
        if (!mbar_wait<0>(out_ready(0), (uint32_t)round, abort_flag)) { alive = false; break; }
        // 14 pixels x 8 chunks of 4 channels per tile row: eight consecutive lanes write one pixel's 128 bytes
        const uint32_t slc = (uint32_t)(lane >> 3) * OUT_PITCH + (uint32_t)(lane & 7) * 16u;
#pragma unroll 1
        for (int k = 0; k < 32 / NCW; ++k) {
          const int t = warp * (32 / NCW) + k;
          const int tly = t >> 2, tlx = t & 3;
          const int b = (tly < it.n0) ? 0 : 1;
          const int ni = tlx >> txe_shift, tx = tlx & (p.TXe - 1);
          const int ig = it.ig0 + b;
          const int ty = b ? (tly - it.n0) : (it.ta0 + tly);
          const int n_img = ig * p.NI + ni;
          if (!((b == 0 || it.band1) && ig < p.NIG && n_img < p.N)) continue;
          const int col0 = (it.cg * p.TXe + tx) * TC;
          const uint32_t src = slc + (uint32_t)(t * TC) * OUT_PITCH + (uint32_t)(t >> 4) * 4u;
          if (p.relu == 2) {
            // this round's pooled row of the tile: seven pixels of 128 bytes in the image of half the height and width
            const int prow = (TR4 / 2) * ty + round, pcol = (col0 >> 1) + (lane >> 3);
            float* dst = p.y + ((size_t)n_img * p.Ho + prow) * p.Wo * p.F + g_out * FG + (lane & 7) * 4;
            uint4 pv[2];
#pragma unroll
            for (int i = 0; i < 2; ++i)
              if (4 * i + (lane >> 3) < TC / 2) {
                const uint32_t a = ob0 + src + (uint32_t)(4 * i) * OUT_PITCH;
                pv[i].x = lds32(a); pv[i].y = lds32(a + 4); pv[i].z = lds32(a + 8); pv[i].w = lds32(a + 12);
              }
#pragma unroll
            for (int i = 0; i < 2; ++i)
              if (4 * i + (lane >> 3) < TC / 2 && prow < p.Ho && pcol + 4 * i < p.Wo)
                *reinterpret_cast<uint4*>(dst + (size_t)(pcol + 4 * i) * p.F) = pv[i];
            continue;
          }
#pragma unroll
          for (int yy = 0; yy < 2; ++yy) {
            const int row = TR4 * ty + 2 * round + yy;
            const int colp = col0 + (lane >> 3);
            float* dst = p.y + ((size_t)n_img * p.Ho + (row >> p.sub)) * p.Wo * p.F + g_out * FG + (lane & 7) * 4;
            uint4 v[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
              if (4 * i + (lane >> 3) < TC) {
                const uint32_t a = (yy ? ob1 : ob0) + src + (uint32_t)(4 * i) * OUT_PITCH;
                v[i].x = lds32(a); v[i].y = lds32(a + 4); v[i].z = lds32(a + 8); v[i].w = lds32(a + 12);
              }
#pragma unroll
            for (int i = 0; i < 4; ++i)
              if (4 * i + (lane >> 3) < TC && row < p.H && colp + 4 * i < p.W && ((row | (colp + 4 * i)) & p.sub) == 0)
                *reinterpret_cast<uint4*>(dst + (size_t)((colp + 4 * i) >> p.sub) * p.F) = v[i];
          }
        }
        if (round == 0) {
          // the second pair of rows overwrites the staging: every warp must have copied the first pair out
          __syncwarp();
          if (lane == 0) mbar_arrive(out_ready(1));
          if (!mbar_wait<0>(out_ready(1), (uint32_t)(it_idx & 1), abort_flag)) { alive = false; break; }
        }
      }
      if (!alive) break;
      // the slots are refilled by bulk copies next: order this warp's accesses to them before those writes
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) { mbar_arrive(slot_empty(s0)); mbar_arrive(slot_empty(s1)); }
      for (int o = 0; o < 2; ++o)
        if (++pslot == NS) { pslot = 0; fpar ^= 1u; }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, TMEM_COLS);
}

// The blob was packed with the parameters of this call (every thread reads the same header: a uniform decision).
__device__ __forceinline__ bool blob_matches(const Params& p) {
  const BlobHeader* bh = p.hdr;
  bool ok = bh->magic == kBlobMagic && bh->version == kBlobVersion && bh->F == p.F && bh->C == p.C &&
            bh->K == p.K && bh->dtype == PAT_F32 && bh->n_keep == p.n_keep &&
            bh->max_block_entries >= 0 && bh->max_block_entries <= FG * CBI + kBlockWarps;
  for (int j = 0; ok && j < p.K; ++j) ok = bh->masks[j] == p.masks[j];
  return ok;
}

// The same decision taken by a whole thread block at once (all loads in flight together, the masks spread over the
// threads): one memory round trip at the start of a short kernel instead of a chain of them.
__device__ __forceinline__ bool blob_matches_block(const Params& p) {
  const BlobHeader* bh = p.hdr;
  bool ok = bh->magic == kBlobMagic && bh->version == kBlobVersion && bh->F == p.F && bh->C == p.C &&
            bh->K == p.K && bh->dtype == PAT_F32 && bh->n_keep == p.n_keep;
  for (int j = threadIdx.x; j < p.K; j += blockDim.x) ok = ok && bh->masks[j] == p.masks[j];
  return __syncthreads_and(ok) != 0;
}

// S2: the stride-2 variant (a quarter of the multiply-adds, see pattern_body4f)
template <int NCODES, bool GENERIC, bool S2>
__global__ void __launch_bounds__(NTHREADS, 1)
k_conv_f32_img(const Params p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  // refuse a blob packed with other parameters (uniform decision: every thread reads the same header)
  const BlobHeader* bh = p.hdr;
  if (!blob_matches(p)) {
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicExch(p.status, PAT_ERR_BLOB);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    return;
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (bh->max_block_entries + 1 <= MAXE3) conv_body<true, NCODES, GENERIC, S2>(p, smem);
  else conv_body<false, NCODES, GENERIC, S2>(p, smem);
}

// ------------------------------------------------------------------------------------------ cut items
// Adds the partial sums of the pieces of a cut item (piece 0 first) and writes the results.  One block per
// (cut item, value of the thread tile); thread = (filter position, lane).
constexpr int RP_THREADS = 1024;
__global__ void __launch_bounds__(RP_THREADS) k_reduce_parts_f32(const Params p) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (!blob_matches_block(p)) return;                    // the convolution kernel refused the blob and wrote no partial sums
  const int v = (int)blockIdx.x % (TR4 * TC), li = (int)blockIdx.x / (TR4 * TC);
  const int item = p.n_whole + li;
  const int g = item % p.NG;
  const Region it = decode_region(p, item / p.NG);
  const int lane = threadIdx.x & 31, slot = threadIdx.x >> 5;
  const float* src = p.partials + (size_t)li * p.parts * PIECE_FLOATS + ((size_t)slot * (TR4 * TC) + v) * 32 + lane;
  float sum = 0.0f;
  for (int q = 0; q < p.parts; ++q) sum += __ldg(src + (size_t)q * PIECE_FLOATS);   // piece 0 first
  const int txe_shift = (p.TXe == 4) ? 2 : (p.TXe == 2 ? 1 : 0);
  const int ly = lane >> 2, lx = lane & 3;
  const int b = (ly < it.n0) ? 0 : 1;
  const int ni = lx >> txe_shift, tx = lx & (p.TXe - 1);
  const int ig = it.ig0 + b;
  const int ty = b ? (ly - it.n0) : (it.ta0 + ly);
  const int n_img = ig * p.NI + ni;
  const int row = TR4 * ty + v / TC, col = (it.cg * p.TXe + tx) * TC + v % TC;
  if (!((b == 0 || it.band1) && ig < p.NIG && n_img < p.N) || row >= p.H || col >= p.W || ((row | col) & p.sub) != 0) return;
  p.y[(((size_t)n_img * p.Ho + (row >> p.sub)) * p.Wo + (col >> p.sub)) * p.F + __ldg(p.xfilt + g * FG + slot)] = p.relu ? fmaxf(sum, 0.0f) : sum;
}

// The same for a call with rectifier and 2 x 2 max pooling: one block per (cut item, pooled value of the thread
// tile); the four sums of the pooling window are formed piece by piece in the same fixed order, then clamped and compared.
__global__ void __launch_bounds__(RP_THREADS) k_reduce_parts_pool_f32(const Params p) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (!blob_matches_block(p)) return;
  constexpr int PV = (TR4 / 2) * (TC / 2);
  const int v = (int)blockIdx.x % PV, li = (int)blockIdx.x / PV;
  const int yy = v / (TC / 2), xx = v % (TC / 2);
  const int item = p.n_whole + li;
  const int g = item % p.NG;
  const Region it = decode_region(p, item / p.NG);
  const int lane = threadIdx.x & 31, slot = threadIdx.x >> 5;
  const float* src = p.partials + (size_t)li * p.parts * PIECE_FLOATS + (size_t)slot * (TR4 * TC) * 32 + lane;
  float m = 0.0f;                                          // the rectifier's floor
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    const float* s = src + (size_t)((2 * yy + (w >> 1)) * TC + 2 * xx + (w & 1)) * 32;
    float sum = 0.0f;
    for (int q = 0; q < p.parts; ++q) sum += __ldg(s + (size_t)q * PIECE_FLOATS);   // piece 0 first
    m = fmaxf(m, sum);
  }
  const int txe_shift = (p.TXe == 4) ? 2 : (p.TXe == 2 ? 1 : 0);
  const int ly = lane >> 2, lx = lane & 3;
  const int b = (ly < it.n0) ? 0 : 1;
  const int ni = lx >> txe_shift, tx = lx & (p.TXe - 1);
  const int ig = it.ig0 + b;
  const int ty = b ? (ly - it.n0) : (it.ta0 + ly);
  const int n_img = ig * p.NI + ni;
  const int prow = (TR4 / 2) * ty + yy, pcol = ((it.cg * p.TXe + tx) * TC >> 1) + xx;
  if (!((b == 0 || it.band1) && ig < p.NIG && n_img < p.N) || prow >= p.Ho || pcol >= p.Wo) return;
  p.y[(((size_t)n_img * p.Ho + prow) * p.Wo + pcol) * p.F + __ldg(p.xfilt + g * FG + slot)] = m;
}

// ------------------------------------------------------------------------------------------ host side
static bool fill_geometry(Params& p, int F, int C, int N, int H, int W) { return imggeo::fill_geometry(p, F, C, N, H, W, CBI); }

}  // namespace img32

// True when the fp32 stage-image kernels cover this layer.
bool conv_f32_img_supported(int F, int C, int dtype, int N, int H, int W, int stride) {
  using namespace img32;
  return dtype == PAT_F32 && shape_supported(F, C, N, H, W, stride, kChanTile, CBI);
}

size_t conv_f32_img_workspace(int F, int C, int dtype, int N, int H, int W, int stride) {
  using namespace img32;
  if (!conv_f32_img_supported(F, C, dtype, N, H, W, stride)) return 0;
  Params p;
  if (!fill_geometry(p, F, C, N, H, W)) return 0;
  return align256((size_t)p.n_regions * p.nct * IMG_BYTES) + MAX_PIECES * PIECE_FLOATS * sizeof(float);
}

int conv_f32_img(const void* blob, int F, int C, const uint16_t* masks, int K, int64_t n_keep,
                 const void* x, void* y, int N, int H, int W, int stride, int relu, void* workspace, cudaStream_t st) {
  using namespace img32;
  const BlobLayout L = blob_layout(F, C, K, n_keep, PAT_F32);
  const char* b = static_cast<const char*>(blob);
  Params p;
  if (!fill_geometry(p, F, C, N, H, W) || L.nblk == 0) return set_error(PAT_ERR_SHAPE, "pat_conv3x3: layer not covered by the stage-image kernels");
  p.x = static_cast<const float*>(x);
  p.y = static_cast<float*>(y);
  p.images = static_cast<char*>(workspace);
  p.hdr = reinterpret_cast<const BlobHeader*>(b);
  p.xfilt = reinterpret_cast<const int32_t*>(b + L.xfilt);
  p.dboff = reinterpret_cast<const uint32_t*>(b + L.dboff);
  p.dblk = b + L.dblk;
  p.status = status_word();
  if (!p.status) return set_error(PAT_ERR_CUDA, "pat_conv3x3: cannot resolve the status word");
  p.K = K; p.n_keep = n_keep;
  p.sub = stride - 1; p.Ho = (H - 1) / stride + 1; p.Wo = (W - 1) / stride + 1; p.relu = relu;
  if (relu == 2) {   // rectifier and 2 x 2 max pooling: the pooled image is written
    if (stride != 1 || (H & 1) || (W & 1)) return set_error(PAT_ERR_SHAPE, "pat_conv3x3_ws_act: pooling needs stride 1 and even H and W");
    p.Ho = H / 2; p.Wo = W / 2;
  }
  for (int j = 0; j < 256; ++j) p.masks[j] = (j < K) ? masks[j] : (uint16_t)0;

  int variant = 0;
  for (int j = 0; j < K; ++j) {
    const int code = (int)((pattern_word(masks[j]) >> 13) & 15u);
    variant = std::max(variant, code == kGenericCode ? 2 : (code >= 6 ? 1 : 0));
  }
  using KernelFn = void (*)(const Params);
  // [stride - 1][code set]
  static const KernelFn kernels[6] = {k_conv_f32_img<6, false, false>, k_conv_f32_img<kNumCodes, false, false>, k_conv_f32_img<kNumCodes, true, false>,
                                      k_conv_f32_img<6, false, true>, k_conv_f32_img<kNumCodes, false, true>, k_conv_f32_img<kNumCodes, true, true>};

  static thread_local DeviceSlot slots[kMaxDevices];
  DeviceSlot* dv = device_slot(slots);
  if (!dv) return set_error(PAT_ERR_CUDA, "pat_conv3x3: cannot query the current device");
  const int sm_count = dv->sms;
  if (!dv->ready) {
    if (int rc = check_cuda(cudaFuncSetAttribute(k_stage_images_f32, cudaFuncAttributeMaxDynamicSharedMemorySize, SI_SMEM), "set shared memory size")) return rc;
    for (KernelFn fn : kernels) {
      if (int rc = check_cuda(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES), "set shared memory size")) return rc;
      cudaFuncAttributes fa;
      if (int rc = check_cuda(cudaFuncGetAttributes(&fa, fn), "query kernel attributes")) return rc;
      if (fa.numRegs < LAUNCH_REGS)
        return set_error(PAT_ERR_CUDA, "pat_conv3x3: kernel was compiled with %d registers per thread, the register split needs %d", fa.numRegs, LAUNCH_REGS);
    }
    dv->ready = true;
  }
  const int grid = plan_items(p, sm_count, CBI, reinterpret_cast<float*>(static_cast<char*>(workspace) + align256((size_t)p.n_regions * p.nct * IMG_BYTES)));
  k_stage_images_f32<<<(unsigned)(p.n_regions * p.nct), SI_THREADS, SI_SMEM, st>>>(p);
  cudaLaunchAttribute pdl;
  pdl.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  pdl.val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.stream = st; cfg.attrs = &pdl; cfg.numAttrs = 1;
  cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(NTHREADS); cfg.dynamicSmemBytes = SMEM_BYTES;
  if (int rc = check_cuda(cudaLaunchKernelEx(&cfg, kernels[3 * p.sub + variant], p), "pat_conv3x3 launch")) return rc;
  count_launches(2);
  if (p.parts > 1) {
    cfg.gridDim = dim3((unsigned)(p.n_split * (relu == 2 ? (TR4 / 2) * (TC / 2) : TR4 * TC))); cfg.blockDim = dim3(RP_THREADS); cfg.dynamicSmemBytes = 0;
    if (int rc = check_cuda(cudaLaunchKernelEx(&cfg, relu == 2 ? k_reduce_parts_pool_f32 : k_reduce_parts_f32, p), "pat_conv3x3 launch")) return rc;
    count_launches(1);
  }
  return check_cuda(cudaGetLastError(), "pat_conv3x3 launch");
}

}  // namespace pat
