// Sparse 3x3 convolution for fp16 storage / fp32 accumulation (sm_100a): three kernels.  Stride 2 is computed like
// stride 1 and only the results at even rows and columns are written.
//
//  1. k_stage_images re-arranges the NHWC activations once per call into "stage images": for every region
//     (8 tile rows x 4 column slots of 4 x 14 pixel tiles) and every block of 16 input channels one contiguous
//     72 KB piece laid out exactly as the convolution kernel wants it in shared memory - channel-planar
//     [16 ch][36 rows][4 segments][16 px], halo pixels duplicated, zero padding written out, the two 16-byte chunks
//     of a segment trading places from one tile row to the next so that the 16-byte window loads of a warp touch
//     every bank once.  This is plain streaming work (reads the input once, writes 1.3 x its size) and it is done
//     once per region, whereas a kernel that transposes inside its pipeline repeats it for every group of 32 filters.
//  2. k_conv_f16_img is the persistent, warp-specialised convolution kernel (one block per SM).  A work item is one
//     region x one group of 32 filters.  One producer thread streams the item's stage images and the matching
//     descriptor blocks of the packed weights (both contiguous, one bulk copy each per stage) into a ring of three
//     shared-memory slots (two when the blob is dense); 16 consumer warps (two filters each, 4 x 14 pixels per
//     thread, one accumulator tile of 56 values in registers and the other parked in tensor memory) run the
//     per-pattern multiply-add code (Section 6.2) over flat operation lists written at pack time; the results leave
//     through two extra ring stages per item: the consumer warps stage them as [pixel][32 channels] and copy them
//     out as 64-byte runs of NHWC output.  The tall thread tile is what the multiply-add rate hangs on: a kernel
//     costs about the same number of other instructions (descriptor, addresses, branch) and 1.5 x the window loads
//     of a 2 x 14 tile for twice the multiply-adds.  Every wait is bounded; tensor memory is released on every path.
//  3. k_reduce_parts adds, in a fixed order, the fp32 partial sums of work items that were cut along the input
//     channels (the items of a last, mostly idle round; every item when there are fewer items than half the SMs).
#include <algorithm>
#include "img_geometry.cuh"

namespace pat {
namespace img16 {
using namespace fast16;
using namespace imggeo;

constexpr int NTHREADS = 640;              // 16 consumer warps, producer warp, three idle warps (register donors)
constexpr int W_PRODUCER = NCW;
constexpr int CBI = kChanTile;             // channels per ring stage (16)
constexpr int CHP = MAXROWS * ROWB;        // channel plane pitch (4608)
constexpr int IMG_BYTES = CBI * CHP;       // 73728
// Ring slots hold one stage each: the stage image and the kernel-descriptor block of the same 16 channels.
// Three slots when every block of the blob has at most MAXE3 kernels (the sparse case), else two.
constexpr int MAX_NS = 3;
constexpr int MAXE3 = 152;
constexpr int DBLK3 = kBlockHeaderBytes + MAXE3 * 16;           // 2560
constexpr int DBLK2 = kBlockHeaderBytes + (FG * kChanTile + kBlockWarps + 8) * 16;  // largest possible block and spare slots up to a multiple of 128 (8704)
constexpr int OFF_SLOTS = 256;             // barriers and two control words sit in front of the ring
constexpr int SMEM_BYTES = OFF_SLOTS + 3 * (IMG_BYTES + DBLK3);
static_assert(OFF_SLOTS + 2 * (IMG_BYTES + DBLK2) <= SMEM_BYTES, "the two-slot layout fits too");
static_assert(IMG_BYTES % 128 == 0 && DBLK3 % 128 == 0 && DBLK2 % 128 == 0 && SMEM_BYTES <= 232448, "shared memory budget of one SM");
static_assert(CHP == kImgPlaneBytes && NCW == kBlockWarps, "the descriptor blocks are written for this geometry");
constexpr int OUT_PITCH = FG * 2 + 4;      // output staging inside a slot: [448 px][32 channels] fp16, pixel pitch 68 B
constexpr int OUT_ROW = 32 * TC * OUT_PITCH;   // one row of every thread tile (30464)
static_assert(2 * OUT_ROW <= IMG_BYTES && 32 % NCW == 0, "two tile rows of results fit a slot");
static_assert(OUT_PITCH - FG * 2 >= 4, "the last pixel's padding takes the one-word shift of tiles 16-31");
constexpr int CONSUMER_REGS = 112, OTHER_REGS = 32;
static_assert(NCW * 32 * CONSUMER_REGS + (NTHREADS / 32 - NCW) * 32 * OTHER_REGS <= NTHREADS * LAUNCH_REGS, "register pool of the block");
constexpr uint32_t TMEM_COLS = 512;        // 4 consumer warps per lane quarter x 2 filters x 64 columns

struct Params : ImgGeometry {   // geometry, work items and cut items: see img_geometry.cuh (nct = channel blocks of 16)
  const __half* x;
  __half* y;
  char* images;            // stage images: [region][channel block][IMG_BYTES]
  const int32_t* xfilt;    // execution position -> original filter
  const uint32_t* dboff;   // descriptor block -> offset in 16-byte units
  const char* dblk;
  const BlobHeader* hdr;
  int* status;
  int K;
  long long n_keep;
  unsigned long long wait_ns;   // limit of every wait of the convolution kernel
  int test_skip;           // test hook: the producer never issues the copies of this stage number (-1: none)
  uint16_t masks[256];     // the library (checked against the blob header)
};

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// ------------------------------------------------------------------------------------------ stage images
// One block per (region, 16 input channels), channels fastest so that blocks running together read
// the same pixels.  Image layout: byte ch * CHP + row * ROWB + seg * SEGB + (chunk ^ swz(row)) * 16 + (px & 7) * 2
// with chunk = px >> 3, px = 0..15 <-> image column 14 * (tile column) - 1 + px, and swz(row) = parity of the tile
// row (counted through both bands) whose window starts in that row's group of four.
constexpr int SI_THREADS = 256;
// Channel planes in shared memory: dense (the bulk copies that write them out want 16-byte aligned, contiguous
// sources), the upper octet 64 bytes further on so that the two channel octets a warp writes at once fall into
// different bank halves.
constexpr int SI_SMEM = CBI * CHP + 64;
__device__ __forceinline__ uint32_t si_plane(int ch) { return (uint32_t)(ch * CHP + (ch >> 3) * 64); }
__global__ void __launch_bounds__(SI_THREADS) k_stage_images(const Params p) {
  extern __shared__ __align__(16) unsigned char img[];
  // the convolution kernel is launched as a programmatic dependent: its blocks may take over SMs as this grid's
  // last blocks finish, and wait (griddepcontrol.wait) for the whole grid before they read a stage image
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int cb16 = (int)(blockIdx.x % (unsigned)p.nct);
  const int reg = (int)(blockIdx.x / (unsigned)p.nct);
  const Region r = decode_region(p, reg);
  const int rows0 = TR4 * r.n0 + 2;
  const int txe_shift = (p.TXe == 4) ? 2 : (p.TXe == 2 ? 1 : 0);
  // a unit = one pixel pair x one channel octet: two 16-byte loads, eight 4-byte stores
  constexpr int UNITS = MAXROWS * LX * 8 * 2, PER_THREAD = UNITS / SI_THREADS;
  static_assert(UNITS % SI_THREADS == 0, "units per thread");
  uint4 va[PER_THREAD], vb[PER_THREAD];
#pragma unroll
  for (int i = 0; i < PER_THREAD; ++i) {
    const int u = (int)threadIdx.x + SI_THREADS * i;
    const int half = u & 1, kp = (u >> 1) & 7, seg = (u >> 4) & 3, pr = u >> 6;
    va[i] = make_uint4(0u, 0u, 0u, 0u);
    vb[i] = make_uint4(0u, 0u, 0u, 0u);
    if (pr < r.nrows) {
      const int b = (pr >= rows0) ? 1 : 0;
      const int yy = b ? (pr - rows0 - 1) : (TR4 * r.ta0 - 1 + pr);
      const int ni = seg >> txe_shift, tx = seg & (p.TXe - 1);
      const int n_img = (r.ig0 + b) * p.NI + ni;
      const int xx = (r.cg * p.TXe + tx) * TC - 1 + 2 * kp;
      if (yy >= 0 && yy < p.H && n_img < p.N) {
        const __half* src = p.x + (((size_t)n_img * p.H + yy) * p.W + xx) * p.C + cb16 * 16 + half * 8;
        if (xx >= 0 && xx < p.W) va[i] = __ldg(reinterpret_cast<const uint4*>(src));
        if (xx + 1 < p.W) vb[i] = __ldg(reinterpret_cast<const uint4*>(src + p.C));
      }
    }
  }
#pragma unroll
  for (int i = 0; i < PER_THREAD; ++i) {
    const int u = (int)threadIdx.x + SI_THREADS * i;
    const int half = u & 1, kp = (u >> 1) & 7, seg = (u >> 4) & 3, pr = u >> 6;
    const int b = (pr >= rows0) ? 1 : 0;
    const int swz = ((((b ? pr - rows0 : pr) >> 2) + (b ? r.n0 : 0)) & 1);
    const uint32_t o = (uint32_t)(pr * ROWB + seg * SEGB + (((kp >> 2) ^ swz) << 4) + (kp & 3) * 4);
    const uint32_t a[4] = {va[i].x, va[i].y, va[i].z, va[i].w};
    const uint32_t c[4] = {vb[i].x, vb[i].y, vb[i].z, vb[i].w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      *reinterpret_cast<uint32_t*>(img + si_plane(half * 8 + 2 * j) + o) = __byte_perm(a[j], c[j], 0x5410);
      *reinterpret_cast<uint32_t*>(img + si_plane(half * 8 + 2 * j + 1) + o) = __byte_perm(a[j], c[j], 0x7632);
    }
  }
  // the planes leave by bulk copies (one per channel, issued by sixteen threads): no thread spends load / store
  // pairs on them, and the block only waits until its shared memory has been read
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the stores above, before the copy engine reads them
  __syncthreads();
  if (threadIdx.x < CBI) {
    char* dst = p.images + (size_t)blockIdx.x * IMG_BYTES + (size_t)threadIdx.x * CHP;
    const uint32_t src = smem_u32(img + si_plane((int)threadIdx.x));
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"((uint32_t)CHP) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
  }
}

// ------------------------------------------------------------------------------------------ the convolution
// Ring protocol.  Every work item takes nct "real" ring stages (16 channels each) followed by two "output"
// stages.  Stage number s uses slot s % NS.
//   real stage:    the producer waits slot_empty, arms slot_full with the byte count and issues two bulk copies
//                  (image, descriptor block); consumers wait slot_full, compute, arrive slot_empty (16 arrivals).
//   output stages: the producer waits slot_empty and arrives slot_full at once (the slot is free to be written);
//                  consumers wait slot_full of both, write their results (tile rows 0-1 into the first, 2-3 into
//                  the second slot), arrive out_ready and wait for it (16 arrivals: every warp has written),
//                  copy two thread tiles each to global memory and arrive slot_empty of both slots.
//                  (A separate store warp shares the issue slots of its SM partition with four consumer warps and
//                  needed longer for a slot than the consumers for two stages: the ring stood still meanwhile.)
// In a real stage a consumer warp runs the operations of its list in the stage's descriptor block: the kernels of the
// filter whose tile it holds, a swap of the two accumulator tiles through tensor memory if its other filter has
// kernels in this stage, and those kernels; the next stage starts with the tile it then holds.
template <bool SPARSE, int NCODES, bool GENERIC, int ACT>
__device__ __forceinline__ void conv_body(const Params& p, unsigned char* smem) {
  constexpr int NS = SPARSE ? 3 : 2;
  constexpr uint32_t SLOT = (uint32_t)IMG_BYTES + (uint32_t)(SPARSE ? DBLK3 : DBLK2);
  const uint32_t sbase = smem_u32(smem);
  auto slot_full = [&](int s) { return sbase + 8u * s; };
  auto slot_empty = [&](int s) { return sbase + 8u * (MAX_NS + s); };
  auto out_ready = [&](int s) { return sbase + 8u * (2 * MAX_NS + s); };
  static_assert(8 * 3 * MAX_NS + 8 <= OFF_SLOTS, "barrier block and control words");
  int& s_abort = *reinterpret_cast<int*>(smem + 8 * 3 * MAX_NS);                 // a wait has given up
  uint32_t& s_tmem = *reinterpret_cast<uint32_t*>(smem + 8 * 3 * MAX_NS + 4);    // base address of the block's tensor-memory columns

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

  // work units of this block: whole items (item = region * NG + filter group), then at most one piece of a cut item
  const int n_my_whole = (p.n_whole > (int)blockIdx.x) ? (p.n_whole - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  const int n_my_items = n_my_whole + ((p.parts > 1 && (int)blockIdx.x < p.n_split * p.parts) ? 1 : 0);
  const int nct = p.nct;
  auto item_of = [&](int it_idx) {
    return it_idx < n_my_whole ? (int)blockIdx.x + it_idx * (int)gridDim.x : p.n_whole + (int)blockIdx.x / p.parts;
  };
  auto piece_of = [&](int it_idx, int& c0, int& c1) {   // channel blocks [c0, c1) of the unit; true for a piece
    if (it_idx < n_my_whole) { c0 = 0; c1 = nct; return false; }
    const int q = (int)blockIdx.x % p.parts;
    c0 = q * nct / p.parts; c1 = (q + 1) * nct / p.parts;
    return true;
  };

  if (warp >= NCW) {
    set_warp_registers<OTHER_REGS>();
    if (warp == W_PRODUCER) {
      // ========================================================================= producer warp
      int pslot = 0, stage_no = 0;
      uint32_t epar = 1u;                  // parity to wait for on slot_empty of the current slot
      uint32_t armed = 0u, armed_par = 0u; // slots with a copy that may still be in flight, and the phase it completes
      bool alive = true;
      for (int it_idx = 0; it_idx < n_my_items && alive; ++it_idx) {
        const int item = item_of(it_idx);
        const int reg = p.d_NG.div(item), g = item - reg * p.NG;
        const char* img = p.images + (size_t)reg * nct * IMG_BYTES;
        const uint32_t* bo = p.dboff + (size_t)g * nct;
        int c0, c1;
        const bool piece = piece_of(it_idx, c0, c1);
        uint32_t o0 = __ldg(bo + c0);
        for (int cb = c0; cb < c1 && alive; ++cb) {
          const uint32_t o1 = __ldg(bo + cb + 1);
          if (!mbar_wait<kFillSleepNs>(slot_empty(pslot), epar, abort_flag, p.wait_ns)) { alive = false; break; }
          if (lane == 0) {
            const uint32_t dbytes = (o1 - o0) * 16u;
            const uint32_t dst = slot0 + (uint32_t)pslot * SLOT;
            mbar_arrive_expect_tx(slot_full(pslot), (uint32_t)IMG_BYTES + dbytes);
            if (stage_no != p.test_skip) {
              bulk_load(dst + IMG_BYTES, p.dblk + (size_t)o0 * 16, dbytes, slot_full(pslot));
              bulk_load(dst, img + (size_t)cb * IMG_BYTES, (uint32_t)IMG_BYTES, slot_full(pslot));
            }
          }
          ++stage_no;
          armed |= 1u << pslot;
          armed_par = (armed_par & ~(1u << pslot)) | ((epar ^ 1u) << pslot);
          o0 = o1;
          if (++pslot == NS) { pslot = 0; epar ^= 1u; }
        }
        // output stages: hand the next two slots to the consumers as they become free (a piece has none)
        for (int o = 0; o < TR4 / 2 && alive && !piece; ++o) {
          if (!mbar_wait<kFillSleepNs>(slot_empty(pslot), epar, abort_flag, p.wait_ns)) { alive = false; break; }
          if (lane == 0) mbar_arrive(slot_full(pslot));
          armed &= ~(1u << pslot);
          if (++pslot == NS) { pslot = 0; epar ^= 1u; }
        }
      }
      if (!alive && lane == 0) {
        // copies already issued still write into this block's shared memory: give them (bounded) time to land
        const unsigned long long t0 = global_ns();
        for (int s = 0; s < NS; ++s) {
          if (!((armed >> s) & 1u)) continue;
          for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
            if (mbar_try_wait(slot_full(s), (armed_par >> s) & 1u)) break;
            if (global_ns() - t0 > p.wait_ns) break;
          }
        }
        atomicExch(p.status, PAT_ERR_TIMEOUT);
      }
    }
    // the other three warps only lend their registers
  } else {
    // =========================================================================== consumer warps
    set_warp_registers<CONSUMER_REGS>();
    // Warp w owns filter slots w and 31 - w of the group (the most loaded filter with the least loaded one, ...).
    // Only one of the two accumulator tiles is in registers at a time; the other is parked in tensor memory:
    // columns [128 * (w / 4) + 64 * f, +64) of the lanes of quarter w % 4.
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
    uint32_t fpar = 0u;                    // parity to wait for on slot_full of the current slot
    bool alive = true;
    for (int it_idx = 0; it_idx < n_my_items && alive; ++it_idx) {
      uint32_t offA;                     // the lane's address of logical chunk 0 of window row 0, relative to a channel plane
      {                                  // (logical chunk 1 sits at offA ^ 16)
        const Region it = decode_region(p, p.d_NG.div(item_of(it_idx)));
        const int ly = lane >> 2, lx = lane & 3;
        const int b = (ly < it.n0) ? 0 : 1;                  // band of this lane's tile row
        offA = (uint32_t)((TR4 * ly + 2 * b) * ROWB + lx * SEGB + ((ly & 1) << 4));
      }
      float acc[TR4][TC];
#pragma unroll
      for (int y = 0; y < TR4; ++y)
#pragma unroll
        for (int x = 0; x < TC; ++x) acc[y][x] = 0.0f;
      int c0, c1;
      const bool piece = piece_of(it_idx, c0, c1);
      // A stage is one flat list of operations per warp, written at pack time: kernels of the filter whose tile
      // the warp holds, then (flag kOpSwap) the other filter's; the last one carries kOpEnd and the place of the
      // warp's list in the next stage's block.  The next operation and the first two window rows of the current
      // one are loaded before the pattern's code runs.
      if (!mbar_wait<0>(slot_full(pslot), fpar, abort_flag, p.wait_ns)) { alive = false; break; }
      uint32_t sl = slot0 + (uint32_t)pslot * SLOT;
      uint32_t pl0 = sl + offA;
      const uint32_t hw = lds32(sl + IMG_BYTES + (uint32_t)warp * 4u);
      uint32_t cur = hw >> 31;           // which of the two filters the registers hold (both tiles are zero now)
      park(cur ^ 1u, acc);
      uint32_t e = sl + IMG_BYTES + kBlockHeaderBytes + (hw & 0xFFFFu) * 16u;
      uint32_t m0, w01, w23, off;
      lds128(e, m0, w01, w23, off);
      int cb = c0;
      uint32_t where = 0u;               // output channels of the warp's two filters (read from the last stage's block)
#pragma unroll 1
      for (;;) {
        const uint32_t a0 = pl0 + off;
        uint32_t r0[8], r1[8];
        lds_row(r0, a0, a0 ^ 16u);
        lds_row(r1, a0 + ROWB, (a0 ^ 16u) + ROWB);
        // The descriptor word decides every branch of this visit.  All lanes have loaded the same word, but only a
        // warp-wide reduction tells the compiler so: its result is warp-uniform, the branches on it become uniform
        // branches, and the reconvergence bookkeeping around them (about a tenth of the loop's other instructions)
        // disappears.  The taps and the window offset stay per-lane values: they are operands of the multiply-adds
        // and of the loads.
        const uint32_t cm = __reduce_or_sync(0xFFFFFFFFu, m0), c01 = w01, c23 = w23, coff = off;
        e += 16u;
        lds128(e, m0, w01, w23, off);
        if (cm & (kOpSwap | kOpNop)) {   // one test for the two rare cases
          if (cm & kOpNop) goto stage_end;
          park(cur, acc);
          cur ^= 1u;
          fetch(cur, acc);
        }
        one_kernel4<NCODES, GENERIC>(acc, pl0, cm, c01, c23, coff, r0, r1);
      stage_end:
        if (cm & kOpEnd) {
          if (cb + 1 == c1) where = lds32(sl + IMG_BYTES + (uint32_t)(kBlockWarps + warp) * 4u);
          __syncwarp();
          if (lane == 0) mbar_arrive(slot_empty(pslot));
          if (++pslot == NS) { pslot = 0; fpar ^= 1u; }
          if (++cb == c1) break;
          if (!mbar_wait<0>(slot_full(pslot), fpar, abort_flag, p.wait_ns)) { alive = false; break; }
          sl = slot0 + (uint32_t)pslot * SLOT;
          pl0 = sl + offA;
          e = sl + IMG_BYTES + kBlockHeaderBytes + (cm >> kOpNextShift) * 16u;
          lds128(e, m0, w01, w23, off);
        }
      }
      if (!alive) break;

      if (piece) {
        // partial sums of a cut item: fp32, one 128-byte line per value and warp
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

      // results: fp32 -> fp16 (round to nearest even) into the two output stages (tile rows 0-1 and 2-3), then,
      // once all 16 warps have written, every warp copies two thread tiles to global memory
      const int item = item_of(it_idx);
      const int g_out = p.d_NG.mod(item);
      // byte offsets of filters 0 / 1 inside the group of 32 output channels
      const uint32_t cposA = (where & 0xFFu) * 2u, cposB = ((where >> 8) & 0xFFu) * 2u;
      const int s0 = pslot, s1 = (pslot + 1 == NS) ? 0 : pslot + 1;
      const uint32_t par1 = (pslot + 1 == NS) ? (fpar ^ 1u) : fpar;
      if (!mbar_wait<0>(slot_full(s0), fpar, abort_flag, p.wait_ns)) { alive = false; break; }
      if (!mbar_wait<0>(slot_full(s1), par1, abort_flag, p.wait_ns)) { alive = false; break; }
      const uint32_t ob0 = slot0 + (uint32_t)s0 * SLOT, ob1 = slot0 + (uint32_t)s1 * SLOT;
      {
        // tiles 16-31 sit one word further on: lanes l and l + 16 would otherwise store to the same banks
        const uint32_t ol = (uint32_t)(lane * TC) * OUT_PITCH + (uint32_t)(lane >> 4) * 4u;
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
          const uint32_t cp = ol + (cur ? cposB : cposA);
          if constexpr (ACT == 1) {          // the fused rectifier: a kernel of its own, so that the plain one pays nothing
#pragma unroll
            for (int y = 0; y < TR4; ++y)
#pragma unroll
              for (int x = 0; x < TC; ++x) acc[y][x] = fmaxf(acc[y][x], 0.0f);
          }
          if constexpr (ACT == 2) {
            // rectifier and 2 x 2 max pooling: a thread tile starts at an even row and column, so every pooling window
            // lies inside one lane's registers; the 2 x 7 pooled values take the first output stage (rounding is
            // monotone: the maximum of the fp32 sums rounds to the maximum of the rounded results)
#pragma unroll
            for (int yy = 0; yy < TR4 / 2; ++yy)
#pragma unroll
              for (int xx = 0; xx < TC / 2; ++xx) {
                const float m = fmaxf(fmaxf(fmaxf(acc[2 * yy][2 * xx], acc[2 * yy][2 * xx + 1]),
                                            fmaxf(acc[2 * yy + 1][2 * xx], acc[2 * yy + 1][2 * xx + 1])), 0.0f);
                sts16(ob0 + (uint32_t)(yy * OUT_ROW + xx * OUT_PITCH) + cp, __half_as_ushort(__float2half_rn(m)));
              }
          } else {
#pragma unroll
            for (int y = 0; y < TR4; ++y)
#pragma unroll
              for (int x = 0; x < TC; ++x)
                sts16((y < 2 ? ob0 : ob1) + (uint32_t)((y & 1) * OUT_ROW + x * OUT_PITCH) + cp, __half_as_ushort(__float2half_rn(acc[y][x])));
          }
          if (half == 0) {
            cur ^= 1u;
            fetch(cur, acc);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(out_ready(0));
      if (!mbar_wait<0>(out_ready(0), (uint32_t)(it_idx & 1), abort_flag, p.wait_ns)) { alive = false; break; }
      {
        const Region it = decode_region(p, p.d_NG.div(item));
        const int txe_shift = (p.TXe == 4) ? 2 : (p.TXe == 2 ? 1 : 0);
        // 14 pixels x 4 chunks of 8 channels per tile row: consecutive lanes take consecutive chunks, so every pixel
        // is written as one 64-byte run; all loads of a tile are issued before its stores
        const uint32_t sl = (uint32_t)(lane >> 2) * OUT_PITCH + (uint32_t)(lane & 3) * 16u;
#pragma unroll 1
        for (int k = 0; k < 32 / NCW; ++k) {
          const int t = warp * (32 / NCW) + k;
          const int ly = t >> 2, lx = t & 3;
          const int b = (ly < it.n0) ? 0 : 1;
          const int ni = lx >> txe_shift, tx = lx & (p.TXe - 1);
          const int ig = it.ig0 + b;
          const int ty = b ? (ly - it.n0) : (it.ta0 + ly);
          const int n_img = ig * p.NI + ni;
          if (!((b == 0 || it.band1) && ig < p.NIG && n_img < p.N)) continue;
          const int col0 = (it.cg * p.TXe + tx) * TC;
          const int row0 = TR4 * ty, colp = col0 + (lane >> 2);
          __half* dst = p.y + (size_t)n_img * p.Ho * p.Wo * p.F + g_out * FG + (lane & 3) * 8;
          const uint32_t src = sl + (uint32_t)(t * TC) * OUT_PITCH + (uint32_t)(t >> 4) * 4u;
          if constexpr (ACT == 2) {
            // pooled tile: 2 rows x 7 pixels, each pixel one 64-byte run of the image of half the height and width
            const int prow0 = row0 >> 1, pcol = (col0 >> 1) + (lane >> 2);
            uint4 pv[TR4 / 2];
#pragma unroll
            for (int yy = 0; yy < TR4 / 2; ++yy)
              if (lane < 4 * (TC / 2)) {
                const uint32_t a = ob0 + src + (uint32_t)(yy * OUT_ROW);
                pv[yy].x = lds32(a); pv[yy].y = lds32(a + 4); pv[yy].z = lds32(a + 8); pv[yy].w = lds32(a + 12);
              }
#pragma unroll
            for (int yy = 0; yy < TR4 / 2; ++yy)
              if (lane < 4 * (TC / 2) && prow0 + yy < p.Ho && pcol < p.Wo)
                *reinterpret_cast<uint4*>(dst + ((size_t)(prow0 + yy) * p.Wo + pcol) * p.F) = pv[yy];
            continue;
          }
          uint4 v[TR4][2];
#pragma unroll
          for (int y = 0; y < TR4; ++y)
#pragma unroll
            for (int part = 0; part < 2; ++part)
              if (part == 0 || lane < 4 * (TC - 8)) {
                const uint32_t a = (y < 2 ? ob0 : ob1) + src + (uint32_t)((y & 1) * OUT_ROW + part * (8 * OUT_PITCH));
                v[y][part].x = lds32(a); v[y][part].y = lds32(a + 4); v[y][part].z = lds32(a + 8); v[y][part].w = lds32(a + 12);
              }
#pragma unroll
          for (int y = 0; y < TR4; ++y)
#pragma unroll
            for (int part = 0; part < 2; ++part)
              if ((part == 0 || lane < 4 * (TC - 8)) && row0 + y < p.H && colp + 8 * part < p.W && (((row0 + y) | (colp + 8 * part)) & p.sub) == 0)
                *reinterpret_cast<uint4*>(dst + ((size_t)((row0 + y) >> p.sub) * p.Wo + ((colp + 8 * part) >> p.sub)) * p.F) = v[y][part];
        }
      }
      // the slots are refilled by bulk copies next: order this warp's reads of them before those writes
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) { mbar_arrive(slot_empty(s0)); mbar_arrive(slot_empty(s1)); }
      for (int o = 0; o < TR4 / 2; ++o)
        if (++pslot == NS) { pslot = 0; fpar ^= 1u; }
    }
  }
  // every warp comes here, also after a failed wait: the tensor memory must be given back before the block ends
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, TMEM_COLS);
}

// The blob was packed with the parameters of this call (every thread reads the same header: a uniform decision).
__device__ __forceinline__ bool blob_matches(const Params& p) {
  const BlobHeader* bh = p.hdr;
  bool ok = bh->magic == kBlobMagic && bh->version == kBlobVersion && bh->F == p.F && bh->C == p.C &&
            bh->K == p.K && bh->dtype == PAT_F16 && bh->n_keep == p.n_keep &&
            bh->max_block_entries >= 0 && bh->max_block_entries <= FG * kChanTile + kBlockWarps;
  for (int j = 0; ok && j < p.K; ++j) ok = bh->masks[j] == p.masks[j];
  return ok;
}

// The same decision taken by a whole thread block at once (all loads in flight together, the masks spread over the
// threads): one memory round trip at the start of a short kernel instead of a chain of them.
__device__ __forceinline__ bool blob_matches_block(const Params& p) {
  const BlobHeader* bh = p.hdr;
  bool ok = bh->magic == kBlobMagic && bh->version == kBlobVersion && bh->F == p.F && bh->C == p.C &&
            bh->K == p.K && bh->dtype == PAT_F16 && bh->n_keep == p.n_keep;
  for (int j = threadIdx.x; j < p.K; j += blockDim.x) ok = ok && bh->masks[j] == p.masks[j];
  return __syncthreads_and(ok) != 0;
}

// NCODES / GENERIC: the pattern codes the kernel carries code for (see one_kernel4); the host picks the smallest
// set that covers the library.  ACT: 1 - results below zero are written as zero; 2 - that, then the maximum of every
// 2 x 2 block of results is written (the pooled image has half the height and width).
template <int NCODES, bool GENERIC, int ACT>
__global__ void __launch_bounds__(NTHREADS, 1)
k_conv_f16_img(const Params p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  // refuse a blob packed with other parameters (uniform decision: every thread reads the same header)
  const BlobHeader* bh = p.hdr;
  const bool ok = blob_matches(p);
  if (!ok) {
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicExch(p.status, PAT_ERR_BLOB);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    return;
  }
  // everything below reads the stage images or writes the output: the stage-image grid must be complete
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // ring geometry by the size of the largest descriptor block (see MAX_NS above)
  if (bh->max_block_entries + 1 <= MAXE3) conv_body<true, NCODES, GENERIC, ACT>(p, smem);
  else conv_body<false, NCODES, GENERIC, ACT>(p, smem);
}

// ------------------------------------------------------------------------------------------ cut items
// Adds the partial sums of the pieces of a cut item (piece 0 first) and writes the fp16 results.  One block per
// (cut item, row of the thread tiles): the sums go through shared memory as [448 px][32 channels] and leave as
// 64-byte runs, like the results of a whole item.  One block per (cut item, row of the thread tiles, half of the
// tile columns).
constexpr int RP_THREADS = 1024, RP_XH = TC / 2;
__global__ void __launch_bounds__(RP_THREADS) k_reduce_parts(const Params p) {
  asm volatile("griddepcontrol.wait;" ::: "memory");   // launched as a programmatic dependent of the convolution kernel
  if (!blob_matches_block(p)) return;                    // the convolution kernel refused the blob and wrote no partial sums
  __shared__ __align__(16) unsigned char stage[OUT_ROW];
  // block = (cut item, row of the thread tiles, left or right half of the tile columns)
  const int xh = (int)blockIdx.x & 1, y = ((int)blockIdx.x >> 1) % TR4, li = (int)blockIdx.x / (2 * TR4);
  const int item = p.n_whole + li;
  const int g = p.d_NG.mod(item);
  const Region it = decode_region(p, p.d_NG.div(item));
  const float* src = p.partials + (size_t)li * p.parts * PIECE_FLOATS;
  constexpr int PER_THREAD = FG * RP_XH * 32 / RP_THREADS;   // 7
  static_assert(FG * RP_XH * 32 % RP_THREADS == 0, "elements per thread");
  float v[PER_THREAD][MAX_PARTS];
#pragma unroll
  for (int i = 0; i < PER_THREAD; ++i) {                      // all loads in flight
    const int idx = (int)threadIdx.x + i * RP_THREADS;
    const int lane = idx & 31, x = xh * RP_XH + (idx >> 5) % RP_XH, slot = idx / (32 * RP_XH);
    const size_t e = ((size_t)slot * (TR4 * TC) + (size_t)(y * TC + x)) * 32 + lane;
#pragma unroll
    for (int q = 0; q < MAX_PARTS; ++q) v[i][q] = (q < p.parts) ? __ldg(src + (size_t)q * PIECE_FLOATS + e) : 0.0f;
  }
#pragma unroll
  for (int i = 0; i < PER_THREAD; ++i) {
    const int idx = (int)threadIdx.x + i * RP_THREADS;
    const int lane = idx & 31, x = xh * RP_XH + (idx >> 5) % RP_XH, slot = idx / (32 * RP_XH);
    float sum = 0.0f;
#pragma unroll
    for (int q = 0; q < MAX_PARTS; ++q) sum += v[i][q];       // piece 0 first
    const int cpos = (__ldg(p.xfilt + g * FG + slot) & (FG - 1)) * 2;
    *reinterpret_cast<__half*>(stage + (lane * TC + x) * OUT_PITCH + cpos) = __float2half_rn(p.relu ? fmaxf(sum, 0.0f) : sum);
  }
  __syncthreads();
  const int txe_shift = (p.TXe == 4) ? 2 : (p.TXe == 2 ? 1 : 0);
  const int t = threadIdx.x >> 5, lane = threadIdx.x & 31;    // one warp per thread tile
  static_assert(RP_THREADS == 32 * 32 && RP_XH * 4 <= 32, "one warp per tile, one lane per 16-byte chunk");
  const int ly = t >> 2, lx = t & 3;
  const int b = (ly < it.n0) ? 0 : 1;
  const int ni = lx >> txe_shift, tx = lx & (p.TXe - 1);
  const int ig = it.ig0 + b;
  const int ty = b ? (ly - it.n0) : (it.ta0 + ly);
  const int n_img = ig * p.NI + ni;
  if (!((b == 0 || it.band1) && ig < p.NIG && n_img < p.N) || TR4 * ty + y >= p.H) return;
  const int col0 = (it.cg * p.TXe + tx) * TC;
  const int row = TR4 * ty + y;
  if (lane < RP_XH * 4 && col0 + xh * RP_XH + (lane >> 2) < p.W) {
    const int x = xh * RP_XH + (lane >> 2), j = lane & 3;
    if (((row | (col0 + x)) & p.sub) != 0) return;           // stride 2: even rows and columns only
    const uint32_t* sp = reinterpret_cast<const uint32_t*>(stage + (t * TC + x) * OUT_PITCH + j * 16);
    __half* dst = p.y + (((size_t)n_img * p.Ho + (row >> p.sub)) * p.Wo + ((col0 + x) >> p.sub)) * p.F + g * FG + j * 8;
    *reinterpret_cast<uint4*>(dst) = make_uint4(sp[0], sp[1], sp[2], sp[3]);
  }
}

// The same for a call with rectifier and 2 x 2 max pooling: one block per (cut item, pooled row of the thread
// tiles); the four sums of a pooling window are formed piece by piece in the same fixed order, then clamped and
// compared.  The pooled values go through shared memory as [32 tiles x 7 px][32 channels] and leave as 64-byte runs.
__global__ void __launch_bounds__(RP_THREADS) k_reduce_parts_pool(const Params p) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (!blob_matches_block(p)) return;
  __shared__ __align__(16) unsigned char stage[OUT_ROW];
  constexpr int PX = TC / 2;                                  // pooled pixels of a tile row
  const int yy = (int)blockIdx.x % (TR4 / 2), li = (int)blockIdx.x / (TR4 / 2);
  const int item = p.n_whole + li;
  const int g = p.d_NG.mod(item);
  const Region it = decode_region(p, p.d_NG.div(item));
  const float* src = p.partials + (size_t)li * p.parts * PIECE_FLOATS;
  static_assert(FG * PX * 32 % RP_THREADS == 0, "elements per thread");
#pragma unroll 1
  for (int i = 0; i < FG * PX * 32 / RP_THREADS; ++i) {
    const int idx = (int)threadIdx.x + i * RP_THREADS;
    const int lane = idx & 31, xx = (idx >> 5) % PX, slot = idx / (32 * PX);
    float m = 0.0f;                                           // the rectifier's floor
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const int y = 2 * yy + (w >> 1), x = 2 * xx + (w & 1);
      const size_t e = ((size_t)slot * (TR4 * TC) + (size_t)(y * TC + x)) * 32 + lane;
      float sum = 0.0f;
      for (int q = 0; q < p.parts; ++q) sum += __ldg(src + (size_t)q * PIECE_FLOATS + e);   // piece 0 first
      m = fmaxf(m, sum);
    }
    const int cpos = (__ldg(p.xfilt + g * FG + slot) & (FG - 1)) * 2;
    *reinterpret_cast<__half*>(stage + (lane * TC + xx) * OUT_PITCH + cpos) = __float2half_rn(m);
  }
  __syncthreads();
  const int txe_shift = (p.TXe == 4) ? 2 : (p.TXe == 2 ? 1 : 0);
  const int t = threadIdx.x >> 5, lane = threadIdx.x & 31;    // one warp per thread tile
  const int ly = t >> 2, lx = t & 3;
  const int b = (ly < it.n0) ? 0 : 1;
  const int ni = lx >> txe_shift, tx = lx & (p.TXe - 1);
  const int ig = it.ig0 + b;
  const int ty = b ? (ly - it.n0) : (it.ta0 + ly);
  const int n_img = ig * p.NI + ni;
  if (!((b == 0 || it.band1) && ig < p.NIG && n_img < p.N)) return;
  const int prow = (TR4 / 2) * ty + yy, pcol = ((it.cg * p.TXe + tx) * TC >> 1) + (lane >> 2);
  if (lane < 4 * PX && prow < p.Ho && pcol < p.Wo) {
    const int j = lane & 3;
    const uint32_t* sp = reinterpret_cast<const uint32_t*>(stage + (t * TC + (lane >> 2)) * OUT_PITCH + j * 16);
    __half* dst = p.y + (((size_t)n_img * p.Ho + prow) * p.Wo + pcol) * p.F + g * FG + j * 8;
    *reinterpret_cast<uint4*>(dst) = make_uint4(sp[0], sp[1], sp[2], sp[3]);
  }
}

// ------------------------------------------------------------------------------------------ host side
static bool fill_geometry(Params& p, int F, int C, int N, int H, int W) { return imggeo::fill_geometry(p, F, C, N, H, W, CBI); }

}  // namespace img16

// test hooks of the bounded waits (see pat_debug_set)
static unsigned long long g_wait_ns = fast16::kWaitNs;
static int g_test_skip = -1;
int conv_f16_img_debug(int what, long long value) {
  if (what == 0) g_wait_ns = value > 0 ? (unsigned long long)value : fast16::kWaitNs;
  else if (what == 1) g_test_skip = value < 0 ? -1 : (int)value;
  else return set_error(PAT_ERR_INVALID_ARG, "pat_debug_set: unknown switch %d", what);
  return PAT_OK;
}

// True when the stage-image kernels cover this layer.
bool conv_f16_img_supported(int F, int C, int dtype, int N, int H, int W, int stride) {
  using namespace img16;
  return dtype == PAT_F16 && shape_supported(F, C, N, H, W, stride, kChanTile, CBI);
}

// Bytes of workspace (the stage images) for a layer the kernels cover; 0 otherwise.
size_t conv_f16_img_workspace(int F, int C, int dtype, int N, int H, int W, int stride) {
  using namespace img16;
  if (!conv_f16_img_supported(F, C, dtype, N, H, W, stride)) return 0;
  Params p;
  if (!fill_geometry(p, F, C, N, H, W)) return 0;
  return align256((size_t)p.n_regions * p.nct * IMG_BYTES) + MAX_PIECES * PIECE_FLOATS * sizeof(float);
}

int conv_f16_img(const void* blob, int F, int C, const uint16_t* masks, int K, int64_t n_keep,
                 const void* x, void* y, int N, int H, int W, int stride, int relu, void* workspace, cudaStream_t st) {
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
  p.wait_ns = g_wait_ns; p.test_skip = g_test_skip;
  p.sub = stride - 1; p.Ho = (H - 1) / stride + 1; p.Wo = (W - 1) / stride + 1; p.relu = relu;
  if (relu == 2) {   // rectifier and 2 x 2 max pooling: the pooled image is written
    if (stride != 1 || (H & 1) || (W & 1)) return set_error(PAT_ERR_SHAPE, "pat_conv3x3_ws_act: pooling needs stride 1 and even H and W");
    p.Ho = H / 2; p.Wo = W / 2;
  }
  for (int j = 0; j < 256; ++j) p.masks[j] = (j < K) ? masks[j] : (uint16_t)0;

  // the smallest set of compiled pattern codes that covers the library
  int variant = 0;
  for (int j = 0; j < K; ++j) {
    const int code = (int)((pattern_word(masks[j]) >> 13) & 15u);
    variant = std::max(variant, code == kGenericCode ? 2 : (code >= 6 ? 1 : 0));
  }
  using KernelFn = void (*)(const Params);
  static const KernelFn kernels[9] = {k_conv_f16_img<6, false, 0>, k_conv_f16_img<kNumCodes, false, 0>, k_conv_f16_img<kNumCodes, true, 0>,
                                      k_conv_f16_img<6, false, 1>, k_conv_f16_img<kNumCodes, false, 1>, k_conv_f16_img<kNumCodes, true, 1>,
                                      k_conv_f16_img<6, false, 2>, k_conv_f16_img<kNumCodes, false, 2>, k_conv_f16_img<kNumCodes, true, 2>};

  static thread_local DeviceSlot slots[kMaxDevices];
  DeviceSlot* dv = device_slot(slots);
  if (!dv) return set_error(PAT_ERR_CUDA, "pat_conv3x3: cannot query the current device");
  const int sm_count = dv->sms;
  if (!dv->ready) {
    if (int rc = check_cuda(cudaFuncSetAttribute(k_stage_images, cudaFuncAttributeMaxDynamicSharedMemorySize, SI_SMEM), "set shared memory size")) return rc;
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
  k_stage_images<<<(unsigned)(p.n_regions * p.nct), SI_THREADS, SI_SMEM, st>>>(p);
  // the two kernels that follow are programmatic dependents of their predecessor: the launch itself overlaps the
  // predecessor's tail, the kernels wait for its completion before they touch its results
  cudaLaunchAttribute pdl;
  pdl.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  pdl.val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.stream = st; cfg.attrs = &pdl; cfg.numAttrs = 1;
  cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(NTHREADS); cfg.dynamicSmemBytes = SMEM_BYTES;
  if (int rc = check_cuda(cudaLaunchKernelEx(&cfg, kernels[variant + 3 * relu], p), "pat_conv3x3 launch")) return rc;
  count_launches(2);
  if (p.parts > 1) {
    cfg.gridDim = dim3((unsigned)(relu == 2 ? p.n_split * (TR4 / 2) : p.n_split * TR4 * 2)); cfg.blockDim = dim3(RP_THREADS); cfg.dynamicSmemBytes = 0;
    if (int rc = check_cuda(cudaLaunchKernelEx(&cfg, relu == 2 ? k_reduce_parts_pool : k_reduce_parts, p), "pat_conv3x3 launch")) return rc;
    count_launches(1);
  }
  return check_cuda(cudaGetLastError(), "pat_conv3x3 launch");
}

}  // namespace pat
