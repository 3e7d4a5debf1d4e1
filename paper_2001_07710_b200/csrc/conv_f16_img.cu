// Sparse 3x3 convolution for fp16 storage / fp32 accumulation, stride 1 (sm_100a): two kernels.
//
//  1. k_stage_images re-arranges the NHWC activations once per call into "stage images": for every region
//     (8 tile rows x 4 column slots of 2 x 14 pixel tiles) and every block of 16 input channels one contiguous
//     40 KB piece laid out exactly as the convolution kernel wants it in shared memory - channel-planar
//     [16 ch][20 rows][4 segments][16 px], halo pixels duplicated, zero padding written out, 16-byte chunks of a
//     segment swapped on every other row pair so that the 16-byte window loads of a warp touch every bank once.
//     This is plain streaming work (reads the input once, writes 1.43 x its size) and it is done once per region,
//     whereas a kernel that transposes inside its pipeline repeats it for every group of 32 filters.
//  2. k_conv_f16_img is the persistent, warp-specialised convolution kernel (one block per SM).  A work item is one
//     region x one group of 32 filters.  One producer thread streams the item's stage images and the matching
//     kernel-descriptor blocks of the packed weights (both contiguous, one bulk copy each per stage) into a ring of
//     4 or 5 shared-memory slots; 16 consumer warps (two filters each, 2 x 14 pixels per thread, one accumulator
//     tile in registers and the other parked in tensor memory) run the per-pattern multiply-add code (Section 6.2);
//     results leave through two extra ring stages per item and a store warp, as 64-byte runs of NHWC output.
//     With nothing but two bulk copies per stage on the producer side the ring can be deeper, and the consumer
//     warps, whose per-stage work differs (two or three kernels per filter and channel block at 12.5 % density),
//     seldom wait for each other.  Every wait is bounded; tensor memory is released on every path.
#include <algorithm>
#include "f16_tile.cuh"

namespace pat {
namespace img16 {
using namespace fast16;

constexpr int NTHREADS = 640;              // 16 consumer warps, producer warp, store warp, two idle warps (register donors)
constexpr int W_PRODUCER = NCW, W_STORE = NCW + 1;
constexpr int MAXROWS = LY * TR + 4;       // two bands, each with a top and a bottom halo row
constexpr int CHP = MAXROWS * ROWB;        // channel plane pitch (2560)
constexpr int IMG_BYTES = CB * CHP;        // 40960
constexpr int OFF_SLOTS = 256;             // barriers sit in front of the ring
constexpr int SMEM_BYTES = 232448 - 1024;  // dynamic shared memory (the rest covers the static variables)
constexpr int MAX_PS = 5;
// ring geometry: five slots when every descriptor block of the blob fits the smaller descriptor area, else four
constexpr int DSLOT5 = ((SMEM_BYTES - OFF_SLOTS) / 5 - IMG_BYTES) / 128 * 128;
constexpr int DSLOT4 = kBlockHeaderBytes + FG * CB * 16;
constexpr int MAXE5 = (DSLOT5 - kBlockHeaderBytes) / 16;
static_assert(OFF_SLOTS + 5 * (IMG_BYTES + DSLOT5) <= SMEM_BYTES, "five-slot ring");
static_assert(OFF_SLOTS + 4 * (IMG_BYTES + DSLOT4) <= SMEM_BYTES, "four-slot ring");
static_assert(DSLOT4 % 128 == 0 && DSLOT5 > kBlockHeaderBytes, "descriptor areas");
constexpr int OUT_PITCH = FG * 2 + 4;      // output staging inside a slot: [448 px][32 channels] fp16, pixel pitch 68 B
static_assert(32 * TC * OUT_PITCH <= IMG_BYTES, "one tile row of results fits a slot");
constexpr int CONSUMER_REGS = 88, OTHER_REGS = 64;
static_assert(NCW * 32 * CONSUMER_REGS + (NTHREADS / 32 - NCW) * 32 * OTHER_REGS <= NTHREADS * LAUNCH_REGS, "register pool of the block");
constexpr uint32_t TMEM_COLS = 256;        // 4 consumer warps per lane quarter x 2 filters x 32 columns

struct Params {
  const __half* x;
  __half* y;
  char* images;            // stage images: [region][channel block][IMG_BYTES]
  const int32_t* xfilt;    // execution position -> original filter
  const uint32_t* dboff;   // descriptor block -> offset in 16-byte units
  const char* dblk;
  const BlobHeader* hdr;
  int* status;
  int N, H, W, C, F, K, nct;
  long long n_keep;
  int TY;                  // tile rows per image (H / 2)
  int TXe, NI;             // tile columns per region, images side by side
  int CG, NIG;             // column groups per image, image groups
  int NG;                  // filter groups (F / 32)
  int n_regions, n_items;  // n_items = n_regions * NG
  uint16_t masks[256];     // the library (checked against the blob header)
};

// A region = LY consecutive tile rows x LX column slots.  Tile rows are numbered through all image groups
// (group g, tile row t -> g * TY + t), so a region may straddle two image groups: it then has two bands,
// each with its own halo rows.
struct Region {
  int cg;           // column group
  int ig0, ta0, n0; // band 0: image group, first tile row, number of tile rows
  bool band1;       // band 1 exists (image group ig0 + 1, tile rows 0 .. LY - n0)
  int nrows;        // image rows in use
};

__device__ __forceinline__ Region decode_region(const Params& p, int reg) {
  Region r;
  r.cg = reg % p.CG;
  const int gt0 = (reg / p.CG) * LY;
  r.ig0 = gt0 / p.TY;
  r.ta0 = gt0 % p.TY;
  r.n0 = min(LY, p.TY - r.ta0);
  r.band1 = (r.n0 < LY) && (r.ig0 + 1 < p.NIG);
  r.nrows = r.band1 ? MAXROWS : 2 * r.n0 + 2;
  return r;
}

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// ------------------------------------------------------------------------------------------ stage images
// One block per (region, channel block), channel block fastest so that blocks running together read the same
// pixels.  Image layout: byte ch * CHP + row * ROWB + seg * SEGB + (chunk ^ ((row >> 1) & 1)) * 16 + (px & 7) * 2
// with chunk = px >> 3, px = 0..15 <-> image column 14 * (tile column) - 1 + px.
__global__ void __launch_bounds__(256) k_stage_images(const Params p) {
  // channel planes are built with a pitch of 2568 bytes: the two channel octets a warp writes at once then fall
  // into different halves of the banks
  constexpr int SP = CHP + 8;
  __shared__ __align__(16) unsigned char img[CB * SP];
  const int cb = (int)(blockIdx.x % (unsigned)p.nct);
  const int reg = (int)(blockIdx.x / (unsigned)p.nct);
  const Region r = decode_region(p, reg);
  const int rows0 = 2 * r.n0 + 2;
  const int txe_shift = (p.TXe == 4) ? 2 : (p.TXe == 2 ? 1 : 0);
  // a unit = one pixel pair x one channel octet: two 16-byte loads, eight 4-byte stores
  constexpr int UNITS = MAXROWS * LX * 8 * 2, PER_THREAD = UNITS / 256;
  static_assert(UNITS % 256 == 0, "units per thread");
  uint4 va[PER_THREAD], vb[PER_THREAD];
#pragma unroll
  for (int i = 0; i < PER_THREAD; ++i) {
    const int u = (int)threadIdx.x + 256 * i;
    const int half = u & 1, kp = (u >> 1) & 7, seg = (u >> 4) & 3, pr = u >> 6;
    va[i] = make_uint4(0u, 0u, 0u, 0u);
    vb[i] = make_uint4(0u, 0u, 0u, 0u);
    if (pr < r.nrows) {
      const int b = (pr >= rows0) ? 1 : 0;
      const int yy = b ? (pr - rows0 - 1) : (2 * r.ta0 - 1 + pr);
      const int ni = seg >> txe_shift, tx = seg & (p.TXe - 1);
      const int n_img = (r.ig0 + b) * p.NI + ni;
      const int xx = (r.cg * p.TXe + tx) * TC - 1 + 2 * kp;
      if (yy >= 0 && yy < p.H && n_img < p.N) {
        const __half* src = p.x + (((size_t)n_img * p.H + yy) * p.W + xx) * p.C + cb * CB + half * 8;
        if (xx >= 0 && xx < p.W) va[i] = __ldg(reinterpret_cast<const uint4*>(src));
        if (xx + 1 >= 0 && xx + 1 < p.W) vb[i] = __ldg(reinterpret_cast<const uint4*>(src + p.C));
      }
    }
  }
#pragma unroll
  for (int i = 0; i < PER_THREAD; ++i) {
    const int u = (int)threadIdx.x + 256 * i;
    const int half = u & 1, kp = (u >> 1) & 7, seg = (u >> 4) & 3, pr = u >> 6;
    const uint32_t o = (uint32_t)(pr * ROWB + seg * SEGB + (((kp >> 2) ^ ((pr >> 1) & 1)) << 4) + (kp & 3) * 4);
    const uint32_t a[4] = {va[i].x, va[i].y, va[i].z, va[i].w};
    const uint32_t c[4] = {vb[i].x, vb[i].y, vb[i].z, vb[i].w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      *reinterpret_cast<uint32_t*>(img + (half * 8 + 2 * j) * SP + o) = __byte_perm(a[j], c[j], 0x5410);
      *reinterpret_cast<uint32_t*>(img + (half * 8 + 2 * j + 1) * SP + o) = __byte_perm(a[j], c[j], 0x7632);
    }
  }
  __syncthreads();
  uint2* dst = reinterpret_cast<uint2*>(p.images + (size_t)blockIdx.x * IMG_BYTES);
  for (int i = threadIdx.x; i < IMG_BYTES / 8; i += 256) {
    const int ch = i / (CHP / 8), w = i % (CHP / 8);
    dst[i] = *reinterpret_cast<const uint2*>(img + ch * SP + w * 8);
  }
}

// ------------------------------------------------------------------------------------------ the convolution
// Ring protocol.  Every work item takes nct "real" ring stages (one channel block each) followed by two
// "output" stages.  Stage number s uses slot s % PS.
//   real stage:    the producer waits slot_empty, arms slot_full with the byte count and issues two bulk copies;
//                  consumers wait slot_full, compute, arrive slot_empty (16 arrivals).
//   output stage:  the producer waits slot_empty and arrives slot_full at once (the slot is free to be written);
//                  consumers wait slot_full, write one tile row of results, arrive out_ready (16 arrivals);
//                  the store warp waits out_ready, copies the slot to global memory and arrives slot_empty
//                  with a count of 16 in the consumers' place.
__global__ void __launch_bounds__(NTHREADS, 1)
k_conv_f16_img(const Params p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ int s_abort;
  __shared__ uint32_t s_tmem;            // base address of the block's tensor-memory columns
  const uint32_t sbase = smem_u32(smem);
  auto slot_full = [&](int s) { return sbase + 8u * s; };
  auto slot_empty = [&](int s) { return sbase + 8u * (MAX_PS + s); };
  auto out_ready = [&](int s) { return sbase + 8u * (2 * MAX_PS + s); };
  static_assert(8 * 3 * MAX_PS <= OFF_SLOTS, "barrier block");

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // refuse a blob packed with other parameters (uniform decision: every thread reads the same header)
  const BlobHeader* bh = p.hdr;
  {
    bool ok = bh->magic == kBlobMagic && bh->version == kBlobVersion && bh->F == p.F && bh->C == p.C &&
              bh->K == p.K && bh->dtype == PAT_F16 && bh->n_keep == p.n_keep &&
              bh->max_block_entries >= 0 && bh->max_block_entries <= FG * CB;
    for (int j = 0; ok && j < p.K; ++j) ok = bh->masks[j] == p.masks[j];
    if (!ok) {
      if (threadIdx.x == 0 && blockIdx.x == 0) atomicExch(p.status, PAT_ERR_BLOB);
      return;
    }
  }
  const int PS = (bh->max_block_entries <= MAXE5) ? 5 : 4;
  const uint32_t SLOT = (uint32_t)IMG_BYTES + (uint32_t)(PS == 5 ? DSLOT5 : DSLOT4);
  const uint32_t slot0 = sbase + OFF_SLOTS;

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < MAX_PS; ++s) { mbar_init(slot_full(s), 1); mbar_init(slot_empty(s), NCW); mbar_init(out_ready(s), NCW); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) tmem_alloc(smem_u32(&s_tmem), TMEM_COLS);
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  volatile int* abort_flag = &s_abort;
  const uint32_t tmem_base = s_tmem;

  const int n_my_items = (p.n_items > (int)blockIdx.x) ? (p.n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  const int nct = p.nct;
  auto item_of = [&](int it_idx) { return (int)blockIdx.x + it_idx * (int)gridDim.x; };   // item = region * NG + filter group

  if (warp >= NCW) {
    set_warp_registers<OTHER_REGS>();
    if (warp == W_PRODUCER) {
      // ========================================================================= producer warp
      int pslot = 0;
      uint32_t epar = 1u;                  // parity to wait for on slot_empty of the current slot
      uint32_t armed = 0u, armed_par = 0u; // slots with a copy that may still be in flight, and the phase it completes
      bool alive = true;
      for (int it_idx = 0; it_idx < n_my_items && alive; ++it_idx) {
        const int item = item_of(it_idx);
        const int g = item % p.NG, reg = item / p.NG;
        const char* img = p.images + (size_t)reg * nct * IMG_BYTES;
        const uint32_t* bo = p.dboff + (size_t)g * nct;
        uint32_t o0 = __ldg(bo);
        for (int cb = 0; cb < nct && alive; ++cb) {
          const uint32_t o1 = __ldg(bo + cb + 1);
          if (!mbar_wait<kFillSleepNs>(slot_empty(pslot), epar, abort_flag)) { alive = false; break; }
          if (lane == 0) {
            const uint32_t dbytes = (o1 - o0) * 16u;
            const uint32_t dst = slot0 + (uint32_t)pslot * SLOT;
            mbar_arrive_expect_tx(slot_full(pslot), (uint32_t)IMG_BYTES + dbytes);
            bulk_load(dst, img + (size_t)cb * IMG_BYTES, (uint32_t)IMG_BYTES, slot_full(pslot));
            bulk_load(dst + IMG_BYTES, p.dblk + (size_t)o0 * 16, dbytes, slot_full(pslot));
          }
          armed |= 1u << pslot;
          armed_par = (armed_par & ~(1u << pslot)) | ((epar ^ 1u) << pslot);
          o0 = o1;
          if (++pslot == PS) { pslot = 0; epar ^= 1u; }
        }
        // output stages: hand the next TR slots to the consumers as they become free
        for (int y = 0; y < TR && alive; ++y) {
          if (!mbar_wait<kFillSleepNs>(slot_empty(pslot), epar, abort_flag)) { alive = false; break; }
          if (lane == 0) mbar_arrive(slot_full(pslot));
          armed &= ~(1u << pslot);
          if (++pslot == PS) { pslot = 0; epar ^= 1u; }
        }
      }
      if (!alive && lane == 0) {
        // copies already issued still write into this block's shared memory: give them (bounded) time to land
        const unsigned long long t0 = global_ns();
        for (int s = 0; s < PS; ++s) {
          if (!((armed >> s) & 1u)) continue;
          for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
            if (mbar_try_wait(slot_full(s), (armed_par >> s) & 1u)) break;
            if (global_ns() - t0 > kWaitNs) break;
          }
        }
        atomicExch(p.status, PAT_ERR_TIMEOUT);
      }
    } else if (warp == W_STORE) {
      // ========================================================================= store warp
      const int txe_shift = (p.TXe == 4) ? 2 : (p.TXe == 2 ? 1 : 0);
      uint32_t opar = 0;                           // phase parity of out_ready, one bit per slot
      bool alive = true;
      int pslot = 0;
      for (int it_idx = 0; it_idx < n_my_items && alive; ++it_idx) {
        const int item = item_of(it_idx);
        const int g = item % p.NG;
        const Region it = decode_region(p, item / p.NG);
        pslot = (pslot + nct) % PS;                // skip the real stages of the item
        for (int y = 0; y < TR && alive; ++y) {
          if (!mbar_wait<kFillSleepNs>(out_ready(pslot), (opar >> pslot) & 1u, abort_flag)) { alive = false; break; }
          opar ^= 1u << pslot;
          const uint32_t o0 = slot0 + (uint32_t)pslot * SLOT;
          // one thread tile (= one consumer lane) at a time: 14 pixels x 4 chunks of 8 channels; consecutive lanes
          // take consecutive chunks, so every pixel is written as one 64-byte run
          for (int t = 0; t < 32; ++t) {
            const int ly = t >> 2, lx = t & 3;
            const int b = (ly < it.n0) ? 0 : 1;
            const int ni = lx >> txe_shift, tx = lx & (p.TXe - 1);
            const int ig = it.ig0 + b;
            const int ty = b ? (ly - it.n0) : (it.ta0 + ly);
            const int n_img = ig * p.NI + ni;
            if (!((b == 0 || it.band1) && ig < p.NIG && n_img < p.N)) continue;
            const int col0 = (it.cg * p.TXe + tx) * TC;
            __half* dst_tile = p.y + (((size_t)n_img * p.H + (TR * ty + y)) * p.W + col0) * p.F + g * FG;
            const uint32_t src_tile = o0 + (uint32_t)(t * TC) * OUT_PITCH;
#pragma unroll
            for (int q0 = 0; q0 < TC * 4; q0 += 32) {
              const int q = q0 + lane;
              if (q < TC * 4) {
                const int x = q >> 2, j = q & 3;
                const uint32_t src = src_tile + x * OUT_PITCH + j * 16;
                uint4 v;
                v.x = lds32(src); v.y = lds32(src + 4); v.z = lds32(src + 8); v.w = lds32(src + 12);
                *reinterpret_cast<uint4*>(dst_tile + (size_t)x * p.F + j * 8) = v;
              }
            }
          }
          // the slot is refilled by a bulk copy next: order this warp's reads of it before that write
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive_n(slot_empty(pslot), NCW);   // the slot goes back to the ring
          if (++pslot == PS) pslot = 0;
        }
      }
    }
    // the two remaining warps only lend their registers
  } else {
    // =========================================================================== consumer warps
    set_warp_registers<CONSUMER_REGS>();
    const int ly = lane >> 2, lx = lane & 3;
    // Warp w owns filter slots w and 31 - w of the group (the most loaded filter with the least loaded one, ...).
    // Only one of the two accumulator tiles is in registers at a time; the other is parked in tensor memory:
    // columns [64 * (w / 4) + 32 * f, +32) of the lanes of quarter w % 4.
    const uint32_t tm0 = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 64);
    int pslot = 0;
    uint32_t fpar = 0u;                    // parity to wait for on slot_full of the current slot
    bool alive = true;
    for (int it_idx = 0; it_idx < n_my_items && alive; ++it_idx) {
      uint32_t offA, offB;               // the lane's two chunk addresses of window row 0, relative to a channel plane
      uint32_t cposA, cposB;             // byte offsets of filters 0 / 1 inside the group of 32 output channels
      {
        const int item = item_of(it_idx);
        const int g = item % p.NG;
        const Region it = decode_region(p, item / p.NG);
        const int b = (ly < it.n0) ? 0 : 1;                  // band of this lane's tile row
        const uint32_t lane_off = (uint32_t)((2 * ly + 2 * b) * ROWB + lx * SEGB);
        const int swl = (ly + b) & 1;
        offA = lane_off + (uint32_t)(swl << 4);
        offB = lane_off + (uint32_t)((swl ^ 1) << 4);
        cposA = ((uint32_t)__ldg(p.xfilt + g * FG + warp) & (uint32_t)(FG - 1)) * 2u;
        cposB = ((uint32_t)__ldg(p.xfilt + g * FG + FG - 1 - warp) & (uint32_t)(FG - 1)) * 2u;
      }
      float acc[TR][TC];
#pragma unroll
      for (int y = 0; y < TR; ++y)
#pragma unroll
        for (int x = 0; x < TC; ++x) acc[y][x] = 0.0f;
      tmem_store32(tm0 + 32u, acc);      // filter 1 starts from zero in tensor memory, filter 0 in registers
      uint32_t cur = 0u;                 // which of the two filters the registers hold

      // the kernels of filter f in the current stage
      auto run_filter = [&](uint32_t f, uint32_t pl0, uint32_t d0) {
        const uint32_t slot = f ? (uint32_t)(FG - 1 - warp) : (uint32_t)warp;
        const uint32_t hw = lds32(d0 + slot * 4);
        const int nk = (int)(hw >> 16);
        uint32_t e = d0 + kBlockHeaderBytes + (hw & 0xFFFFu) * 16u;
        for (int k = 0; k < nk; ++k, e += 16) {
          uint32_t m0, w01, w23, pad;
          lds128(e, m0, w01, w23, pad);
          const uint32_t base = pl0 + (m0 & 15u) * CHP;
          one_kernel(acc, base + offA, base + offB, m0, w01, w23);
        }
      };

      for (int cb = 0; cb < nct; ++cb) {
        if (!mbar_wait<0>(slot_full(pslot), fpar, abort_flag)) { alive = false; break; }
        const uint32_t pl0 = slot0 + (uint32_t)pslot * SLOT;
        const uint32_t d0 = pl0 + IMG_BYTES;
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
          run_filter(cur, pl0, d0);
          if (half == 0) {               // swap: park this filter, fetch the other
            tmem_store32(tm0 + cur * 32u, acc);
            cur ^= 1u;
            tmem_load32(tm0 + cur * 32u, acc);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(slot_empty(pslot));
        if (++pslot == PS) { pslot = 0; fpar ^= 1u; }
      }
      if (!alive) break;

      // results: fp32 -> fp16 (round to nearest even) into the two output stages, one tile row each
#pragma unroll 1
      for (int y = 0; y < TR; ++y) {
        if (!mbar_wait<0>(slot_full(pslot), fpar, abort_flag)) { alive = false; break; }
        const uint32_t o0 = slot0 + (uint32_t)pslot * SLOT + (uint32_t)(lane * TC) * OUT_PITCH;
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
          const uint32_t cp = cur ? cposB : cposA;
          if (y == 0) {
#pragma unroll
            for (int x = 0; x < TC; ++x) sts16(o0 + x * OUT_PITCH + cp, __half_as_ushort(__float2half_rn(acc[0][x])));
          } else {
#pragma unroll
            for (int x = 0; x < TC; ++x) sts16(o0 + x * OUT_PITCH + cp, __half_as_ushort(__float2half_rn(acc[1][x])));
          }
          if (half == 0) {
            if (y == 0) tmem_store32(tm0 + cur * 32u, acc);   // still needed for the second tile row
            cur ^= 1u;
            tmem_load32(tm0 + cur * 32u, acc);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(out_ready(pslot));
        if (++pslot == PS) { pslot = 0; fpar ^= 1u; }
      }
    }
  }
  // every warp comes here, also after a failed wait: the tensor memory must be given back before the block ends
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, TMEM_COLS);
}

// ------------------------------------------------------------------------------------------ host side
static bool fill_geometry(Params& p, int F, int C, int N, int H, int W) {
  p.N = N; p.H = H; p.W = W; p.C = C; p.F = F;
  p.nct = C / CB;
  p.TY = H / TR;
  const int TX = W / TC;
  p.TXe = TX >= LX ? LX : TX;
  p.NI = LX / p.TXe;
  p.CG = TX / p.TXe;
  p.NIG = (N + p.NI - 1) / p.NI;
  p.NG = F / FG;
  const long long row_blocks = ((long long)p.NIG * p.TY + LY - 1) / LY;
  const long long regions = row_blocks * p.CG;
  const long long items = regions * p.NG;
  if (items > 0x7FFFFFFFll || regions * p.nct > 0x7FFFFFFFll) return false;
  p.n_regions = (int)regions;
  p.n_items = (int)items;
  return true;
}

}  // namespace img16

// True when the stage-image kernels cover this layer.
bool conv_f16_img_supported(int F, int C, int dtype, int N, int H, int W, int stride) {
  using namespace img16;
  if (dtype != PAT_F16 || stride != 1) return false;
  if (W % TC != 0 || H % TR != 0 || H < 2 * (LY - 1)) return false;
  const int TX = W / TC;
  if (!(TX == 1 || TX == 2 || TX % 4 == 0)) return false;
  if (C % CB != 0 || F % FG != 0) return false;
  Params p;
  return N >= 1 && fill_geometry(p, F, C, N, H, W);
}

// Bytes of workspace (the stage images) for a layer the kernels cover; 0 otherwise.
size_t conv_f16_img_workspace(int F, int C, int dtype, int N, int H, int W, int stride) {
  using namespace img16;
  if (!conv_f16_img_supported(F, C, dtype, N, H, W, stride)) return 0;
  Params p;
  fill_geometry(p, F, C, N, H, W);
  return (size_t)p.n_regions * p.nct * IMG_BYTES;
}

int conv_f16_img(const void* blob, int F, int C, const uint16_t* masks, int K, int64_t n_keep,
                 const void* x, void* y, int N, int H, int W, void* workspace, cudaStream_t st) {
  using namespace img16;
  const BlobLayout L = blob_layout(F, C, K, n_keep, PAT_F16);
  const char* b = static_cast<const char*>(blob);
  Params p;
  if (!fill_geometry(p, F, C, N, H, W) || L.nblk == 0) return set_error(PAT_ERR_SHAPE, "pat_conv3x3: layer not covered by the stage-image kernels");
  p.x = static_cast<const __half*>(x);
  p.y = static_cast<__half*>(y);
  p.images = static_cast<char*>(workspace);
  p.hdr = reinterpret_cast<const BlobHeader*>(b);
  p.xfilt = reinterpret_cast<const int32_t*>(b + L.xfilt);
  p.dboff = reinterpret_cast<const uint32_t*>(b + L.dboff);
  p.dblk = b + L.dblk;
  p.status = status_word();
  if (!p.status) return set_error(PAT_ERR_CUDA, "pat_conv3x3: cannot resolve the status word");
  p.K = K; p.n_keep = n_keep;
  for (int j = 0; j < 256; ++j) p.masks[j] = (j < K) ? masks[j] : (uint16_t)0;

  static thread_local int sm_count = 0;
  static thread_local bool attr_set = false;
  if (!attr_set) {
    int dev = 0;
    if (int rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice")) return rc;
    if (int rc = check_cuda(cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev), "query SM count")) return rc;
    if (int rc = check_cuda(cudaFuncSetAttribute(k_conv_f16_img, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES), "set shared memory size")) return rc;
    cudaFuncAttributes fa;
    if (int rc = check_cuda(cudaFuncGetAttributes(&fa, k_conv_f16_img), "query kernel attributes")) return rc;
    if (fa.numRegs < LAUNCH_REGS)
      return set_error(PAT_ERR_CUDA, "pat_conv3x3: kernel was compiled with %d registers per thread, the register split needs %d", fa.numRegs, LAUNCH_REGS);
    attr_set = true;
  }
  k_stage_images<<<(unsigned)(p.n_regions * p.nct), 256, 0, st>>>(p);
  const int grid = std::min(p.n_items, sm_count);
  k_conv_f16_img<<<grid, NTHREADS, SMEM_BYTES, st>>>(p);
  count_launches(2);
  return check_cuda(cudaGetLastError(), "pat_conv3x3 launch");
}

}  // namespace pat
