// Tuned sparse 3x3 convolution for fp16 storage / fp32 accumulation, stride 1 (sm_100a).
//
// What Section 6.2 asks of the execution code - one branch-free code path per pattern with the tap positions
// known ahead of time, kernels of a filter grouped, filters balanced across thread groups - mapped to B200:
//
//  * persistent, warp-specialised thread blocks (one per SM): 16 consumer warps + 4 producer warps; the
//    producers hand most of their registers to the consumers (setmaxnreg);
//  * activations come from NHWC global memory by TMA (one tiled copy per tile row, 16 channels deep, zero
//    fill outside the image = the padding), land as [row][pixel][16 ch], and are transposed by the producer
//    warps (ldmatrix.trans -> stmatrix) into a channel-planar layout [ch][row][segment][16 px] in which every
//    thread finds the 14 pixels of its tile row plus both halo pixels in two 16-byte loads;
//  * a consumer thread owns a 2 x 14 pixel tile of R = 2 filters (56 fp32 accumulators); lanes of a warp are 32
//    different tiles of the same filter, so weights are warp-uniform; the 16 warps cover 32 filters;
//  * per kept kernel: the 16-pixel-wide window of its channel is loaded with 16-byte loads, then one
//    warp-uniform jump on the pattern selects fully unrolled code whose register offsets are immediates
//    (patterns that are a built-in pattern shifted down one row share its code; other libraries run through
//    nine guarded per-position bodies); the multiply-adds are fma.rn.f32.f16 (fp16 x fp16 products are
//    exact in fp32, the sum is fp32), so no conversion instruction sits in the loop;
//  * channel blocks flow through a 3-deep planar ring and a 2-deep raw ring guarded by mbarriers, so warps
//    with more kernels in one channel block catch up in the next; every wait is bounded;
//  * the output of a work item goes through the same ring: two extra ring stages per item receive the fp16
//    results (one row of every thread tile each) in a [pixel][32 channels] layout, and a store warp writes
//    them to NHWC global memory as full 64-byte runs (the 32 adjacent output channels of the filter group).
#include <algorithm>
#include "f16_tile.cuh"

namespace pat {
namespace fast16 {

constexpr int NFW = 3, NSW = 1;           // fill (producer) warps, store warp
constexpr int NPW = NFW + NSW;
constexpr int PS = 3, RS = 2;           // planar / raw ring depth
constexpr int NTHREADS = (NCW + NPW) * 32;
constexpr int MAXROWS = LY * TR + 4;    // two bands, each with a top and a bottom halo row
constexpr int CHP = MAXROWS * ROWB + 16;  // channel plane pitch (odd multiple of 16 B: conflict-free stmatrix)
constexpr int PLANAR_STAGE = CB * CHP;    // 41216
constexpr int RAW_POS = 64;               // positions per raw row (58, 60 or 64 used)
constexpr int RAW_STAGE = MAXROWS * RAW_POS * CB * 2;  // 40960
constexpr int NMAPS = LY;                 // one tensor map per band height (2n + 2 rows, n = 1..8 tile rows)
// kernel descriptors of a stage: per filter slot a count, the original filter id, and up to 16 entries of
// 16 bytes {channel-in-block | 4 tap codes << 4, taps 0-1 (fp16 x2), taps 2-3 (fp16 x2), unused}
constexpr int DESC_HDR = FG * 8;
constexpr int DESC_STAGE = DESC_HDR + FG * CB * 16;   // 8448
constexpr int OFF_RAW = PS * PLANAR_STAGE;
constexpr int OFF_DESC = OFF_RAW + RS * RAW_STAGE;
constexpr int OFF_BAR = OFF_DESC + PS * DESC_STAGE;
constexpr int SMEM_BYTES = OFF_BAR + 128;
// output staging inside a planar slot: [448 pixels of a tile row set][32 channels] fp16, pixel pitch 68 bytes
constexpr int OUT_PITCH = FG * 2 + 4;
constexpr int OUT_PIX = 32 * TC;
static_assert(OUT_PIX * OUT_PITCH <= PLANAR_STAGE, "a half tile of results fits one planar slot");
static_assert(SMEM_BYTES <= 232448, "shared memory budget of one SM");
// Register split between the warp groups.  The pool is what the block got at launch (threads x registers per
// thread as compiled), so the split must fit inside it or the increase would wait forever; the host checks the
// compiled count before launching.
constexpr int CONSUMER_REGS = 88, PRODUCER_REGS = 128;
static_assert(NCW * 32 * CONSUMER_REGS + NPW * 32 * PRODUCER_REGS <= NTHREADS * LAUNCH_REGS, "register pool of the block");
constexpr uint32_t TMEM_COLS = 256;        // 4 consumer warps per lane quarter x 2 filters x 32 columns

// One tiled copy brings a whole band (all its rows, all images side by side), because issuing a copy costs far
// more than the copy engine needs per row; the box height is part of a tensor map, hence one map per height.
struct alignas(64) TmapSet { CUtensorMap m[NMAPS]; };

struct Params {
  const __half* x;
  __half* y;
  const int32_t* xfilt;    // execution position -> original filter
  const int32_t* tptr;     // [F][nct+1], execution order
  const uint32_t* tmeta;   // channel | pattern << 16
  const uint2* tw4;        // four fp16 taps per kernel
  const BlobHeader* hdr;
  int* status;
  int N, H, W, C, F, K, nct;
  long long n_keep;
  int TY;                  // tile rows per image (H / 2)
  int TXe, NI, BW;         // tile columns per region, images side by side, box width (pixels)
  int CG, NIG;             // column groups per image, image groups
  int NG;                  // filter groups (F / 32)
  int n_items;             // regions * NG
  int n_row_blocks;        // ceil(NIG * TY / LY)
  uint16_t masks[256];     // the library (checked against the blob header)
  uint32_t pword[256];     // pattern id -> descriptor word (mask, compiled code, window shift)
};

// ------------------------------------------------------------------------------------------ work items
// A work item = one region (8 tile rows x 4 column slots = 32 thread tiles) x one group of 32 filters.
// Tile rows are numbered through all image groups (group g, tile row t -> g * TY + t), so a region may
// straddle two image groups: it then has two bands, each with its own halo rows in shared memory.
struct Item {
  int g;            // filter group
  int cg;           // column group
  int ig0, ta0, n0; // band 0: image group, first tile row, number of tile rows
  bool band1;       // band 1 exists (image group ig0 + 1, tile rows 0 .. LY - n0)
  int nrows;        // shared-memory rows in use
};

__device__ __forceinline__ Item decode_item(const Params& p, int item) {
  Item it;
  it.g = item % p.NG;
  const int reg = item / p.NG;
  it.cg = reg % p.CG;
  const int rb = reg / p.CG;
  const int gt0 = rb * LY;
  it.ig0 = gt0 / p.TY;
  it.ta0 = gt0 % p.TY;
  it.n0 = min(LY, p.TY - it.ta0);
  it.band1 = (it.n0 < LY) && (it.ig0 + 1 < p.NIG);
  it.nrows = it.band1 ? MAXROWS : 2 * it.n0 + 2;
  return it;
}

// ------------------------------------------------------------------------------------------ the kernel
// Ring protocol.  Every work item takes nct "real" ring stages (one channel block each) followed by two
// "output" stages.  Stage number s uses planar slot s % PS in phase s / PS.
//   real stage:    fill warps wait pl_empty, transpose + write descriptors, arrive pl_full (3 arrivals);
//                  consumers wait pl_full, compute, arrive pl_empty (16 arrivals).
//   output stage:  fill warps wait pl_empty and arrive pl_full at once (the slot is free to be written);
//                  consumers wait pl_full, write one tile row of results, arrive out_ready (16 arrivals);
//                  the store warp waits out_ready, copies the slot to global memory and arrives pl_empty
//                  with a count of 16 in the consumers' place.
__global__ void __launch_bounds__(NTHREADS, 1)
k_conv_f16_s1(const __grid_constant__ TmapSet tms, const Params p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ int s_abort;
  __shared__ uint32_t s_tmem;            // base address of the block's tensor-memory columns
  __shared__ int s_rawdone[RS];          // fill warps that have finished reading a raw slot
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar0 = sbase + OFF_BAR;
  auto raw_full = [&](int s) { return bar0 + 8u * s; };
  auto pl_full = [&](int s) { return bar0 + 8u * (2 * RS + s); };
  auto pl_empty = [&](int s) { return bar0 + 8u * (2 * RS + PS + s); };
  auto out_ready = [&](int s) { return bar0 + 8u * (2 * RS + 2 * PS + s); };
  static_assert(8 * (2 * RS + 3 * PS) <= 128, "barrier block");

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // refuse a blob packed with other parameters (uniform decision: every thread reads the same header)
  {
    const BlobHeader* h = p.hdr;
    bool ok = h->magic == kBlobMagic && h->version == kBlobVersion && h->F == p.F && h->C == p.C &&
              h->K == p.K && h->dtype == PAT_F16 && h->n_keep == p.n_keep;
    for (int j = 0; ok && j < p.K; ++j) ok = h->masks[j] == p.masks[j];
    if (!ok) {
      if (threadIdx.x == 0 && blockIdx.x == 0) atomicExch(p.status, PAT_ERR_BLOB);
      return;
    }
  }

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < RS; ++s) { mbar_init(raw_full(s), 1); s_rawdone[s] = 0; }
    for (int s = 0; s < PS; ++s) { mbar_init(pl_full(s), NFW); mbar_init(pl_empty(s), NCW); mbar_init(out_ready(s), NCW); }
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
  auto item_of = [&](int it_idx) { return decode_item(p, (int)blockIdx.x + it_idx * (int)gridDim.x); };

  if (warp >= NCW) {
    set_warp_registers<PRODUCER_REGS>();
    const int txe_shift = (p.TXe == 4) ? 2 : (p.TXe == 2 ? 1 : 0);
    if (warp < NCW + NFW) {
      // ========================================================================= fill warps
      // These warps share the issue slots of their SM partition with four consumer warps, so every instruction
      // here is paid for with multiply-add slots: ring positions are kept incrementally, addresses are lane
      // constants plus small per-row terms, and item geometry is decoded once per item.
      const int pw = warp - NCW;
      // lane constants of the transposition: lane -> (matrix m = lane / 8, row i = lane % 8) for both ld and st
      const int m = lane >> 3, i8 = lane & 7;
      const int hch = m >> 1, oct = m & 1;                     // pixel chunk (0/1), channel octet (0/1)
      // raw layout of a band: [image slot][row][pixel -1 .. BW-2][16 channels]
      const uint32_t rowpitch = (uint32_t)(p.BW * CB * 2);
      uint32_t ldoff[LX];                                      // per segment: offset of the lane's matrix row inside a raw row
#pragma unroll
      for (int seg = 0; seg < LX; ++seg) {
        const int tx = seg & (p.TXe - 1);
        ldoff[seg] = (uint32_t)((TC * tx + 8 * hch + i8) * (CB * 2) + oct * 16);
      }
      const uint32_t st_lane = (uint32_t)((oct * 8 + i8) * CHP);
      const uint32_t stoff0 = st_lane + (uint32_t)(hch << 4), stoff1 = st_lane + (uint32_t)((hch ^ 1) << 4);
      const int row_bytes = p.NI * p.BW * CB * 2;              // bytes one row copy brings in
      // lane roles for the kernel descriptors: 3 lanes per filter slot over the 96 fill lanes
      const int dslot = (pw * 32 + lane) / 3, dj = (pw * 32 + lane) % 3;
      static_assert(NFW * 32 / 3 == FG, "three lanes per filter slot");
      static_assert(MAXROWS <= 32, "one lane per row copy");

      // Issue cursor: the (item, channel block) whose copies go out next; it runs RS real stages ahead of the
      // stage being transposed.  Lane 0 holds the coordinates of band 0 of the cursor's item, lane 1 those of band 1.
      int cur_it = 0, cur_cb = 0, cur_y = 0, cur_n = 0, cur_x = 0, cur_rows = 0, cur_map = -1;
      uint32_t cur_dst = 0;
      auto cursor_load = [&]() {
        if (cur_it < n_my_items) {
          const Item ci = item_of(cur_it);
          const int rows0 = 2 * ci.n0 + 2;
          cur_rows = ci.nrows;
          cur_x = ci.cg * p.TXe * TC - 1;
          cur_map = -1;
          if (lane == 0) { cur_y = 2 * ci.ta0 - 1; cur_n = ci.ig0 * p.NI; cur_dst = 0u; cur_map = ci.n0 - 1; }
          if (lane == 1 && ci.band1) { cur_y = -1; cur_n = (ci.ig0 + 1) * p.NI; cur_dst = (uint32_t)(p.NI * rows0) * rowpitch; cur_map = LY - ci.n0 - 1; }
        }
      };
      auto cursor_advance = [&]() {
        if (++cur_cb == nct) { cur_cb = 0; ++cur_it; cursor_load(); }
      };
      auto cursor_issue = [&](int slot) {                     // whole warp: lanes 0 and 1 each copy one band
        if (lane == 0) mbar_arrive_expect_tx(raw_full(slot), (uint32_t)(cur_rows * row_bytes));
        __syncwarp();
        if (cur_map >= 0)
          tma_load_4d(sbase + OFF_RAW + slot * RAW_STAGE + cur_dst, &tms.m[cur_map], cur_cb * CB, cur_x, cur_y, cur_n, raw_full(slot));
      };
      const int n_real = n_my_items * nct;         // real stages (raw ring positions)
      cursor_load();
      for (int s = 0; s < RS && s < n_real; ++s) {   // prologue: fill warp 0 issues, every warp advances its cursor
        if (pw == 0) cursor_issue(s);
        cursor_advance();
      }
      // kernel range of this lane's filter slot in a channel block (global loads; prefetched one block ahead)
      auto load_range = [&](int g, int cb, int& kb, int& ke) {
        const int32_t* row = p.tptr + (size_t)(g * FG + dslot) * (nct + 1) + cb;
        kb = __ldg(row); ke = __ldg(row + 1);
      };

      bool alive = true;
      int rstage = 0, landed = 0;                  // real stages done / whose copies this warp has seen land
      int pslot = 0, rslot = 0;
      uint32_t ppar = 1u, rpar = 0u;               // parity to wait for: pl_empty of the slot, raw_full of the raw slot
      int kb = 0, ke = 0;
      for (int it_idx = 0; it_idx < n_my_items && alive; ++it_idx) {
        int g, nrows, rows0;
        { const Item it = item_of(it_idx); g = it.g; nrows = it.nrows; rows0 = 2 * it.n0 + 2; }
        // per band: where image slot ni of the band starts in the raw buffer (segments of a row may belong to different slots)
        uint32_t nioff[2][LX];
#pragma unroll
        for (int seg = 0; seg < LX; ++seg) {
          const uint32_t ni = (uint32_t)(seg >> txe_shift);
          nioff[0][seg] = ni * (uint32_t)rows0 * rowpitch + ldoff[seg];
          nioff[1][seg] = (uint32_t)(p.NI * rows0) * rowpitch + ni * (uint32_t)(nrows - rows0) * rowpitch + ldoff[seg];
        }
        load_range(g, 0, kb, ke);
        const int forig = __ldg(p.xfilt + g * FG + dslot);
        for (int cb = 0; cb < nct && alive; ++cb, ++rstage) {
          // descriptors of this block: issue the global loads of the first entries now, use them after the transposition
          const int nk = ke - kb, kb_cur = kb;
          uint32_t dmeta[2] = {0u, 0u};
          uint2 dw[2] = {make_uint2(0u, 0u), make_uint2(0u, 0u)};
#pragma unroll
          for (int u = 0; u < 2; ++u)
            if (dj + 3 * u < nk) { dmeta[u] = __ldg(p.tmeta + kb + dj + 3 * u); dw[u] = __ldg(p.tw4 + kb + dj + 3 * u); }
          if (cb + 1 < nct) load_range(g, cb + 1, kb, ke);

          if (!mbar_wait<kFillSleepNs>(raw_full(rslot), rpar, abort_flag)) { alive = false; break; }
          landed = rstage + 1;
          if (!mbar_wait<kFillSleepNs>(pl_empty(pslot), ppar, abort_flag)) { alive = false; break; }
          const uint32_t raw0 = sbase + OFF_RAW + rslot * RAW_STAGE;
          const uint32_t pl0 = sbase + pslot * PLANAR_STAGE;
          // transposition, one shared-memory row (4 segments) at a time: four independent loads, then their stores
          auto load_prow = [&](int pr, uint32_t (&v)[LX][4]) {
            const bool b1 = pr >= rows0;
            const uint32_t lr = raw0 + (uint32_t)(b1 ? pr - rows0 : pr) * rowpitch;
#pragma unroll
            for (int seg = 0; seg < LX; ++seg) {
              // the copies are written with the 32-byte swizzle (16-byte chunk index ^= address bit 7), which
              // spreads the eight 32-byte-strided rows of a matrix over all banks
              const uint32_t la = lr + (b1 ? nioff[1][seg] : nioff[0][seg]);
              ldmatrix_x4_trans(la ^ ((la >> 3) & 16u), v[seg][0], v[seg][1], v[seg][2], v[seg][3]);
            }
          };
          auto store_prow = [&](int pr, const uint32_t (&v)[LX][4]) {
            const uint32_t sr = pl0 + pr * ROWB + ((pr & 2) ? stoff1 : stoff0);   // chunk swizzle by (row >> 1) & 1
#pragma unroll
            for (int seg = 0; seg < LX; ++seg) stmatrix_x4(sr + seg * SEGB, v[seg][0], v[seg][1], v[seg][2], v[seg][3]);
          };
          for (int pr = pw; pr < nrows; pr += NFW) {
            uint32_t va[LX][4];
            load_prow(pr, va);
            store_prow(pr, va);
          }
          // kernel descriptors
          {
            const uint32_t d0 = sbase + OFF_DESC + pslot * DESC_STAGE;
            if (dj == 0) { sts32(d0 + dslot * 4, (uint32_t)nk); sts32(d0 + FG * 4 + dslot * 4, (uint32_t)forig); }
            auto put = [&](int e, uint32_t mt, uint2 wv) {
              const uint32_t cl = (mt & 0xFFFFu) - (uint32_t)(cb * CB);
              const uint32_t mm = cl | p.pword[mt >> 16];
              sts128(d0 + DESC_HDR + (dslot * CB + e) * 16, mm, wv.x, wv.y, 0u);
            };
#pragma unroll
            for (int u = 0; u < 2; ++u)
              if (dj + 3 * u < nk) put(dj + 3 * u, dmeta[u], dw[u]);
            for (int e = dj + 6; e < nk; e += 3) put(e, __ldg(p.tmeta + kb_cur + e), __ldg(p.tw4 + kb_cur + e));   // more than 6 kernels: rare
          }
          __syncwarp();
          // the fill warp that is last to finish with the raw slot refills it
          int last = 0;
          if (lane == 0) {
            mbar_arrive(pl_full(pslot));
            last = (atomicAdd(&s_rawdone[rslot], 1) == NFW - 1) ? 1 : 0;
            if (last) s_rawdone[rslot] = 0;
          }
          last = __shfl_sync(0xFFFFFFFFu, last, 0);
          if (rstage + RS < n_real) {
            if (last) cursor_issue(rslot);
            cursor_advance();
          }
          if (++pslot == PS) { pslot = 0; ppar ^= 1u; }
          if (++rslot == RS) { rslot = 0; rpar ^= 1u; }
        }
        // output stages: hand the next TR slots to the consumers as they become free
        for (int y = 0; y < TR && alive; ++y) {
          if (!mbar_wait<kFillSleepNs>(pl_empty(pslot), ppar, abort_flag)) { alive = false; break; }
          if (lane == 0) mbar_arrive(pl_full(pslot));
          if (++pslot == PS) { pslot = 0; ppar ^= 1u; }
        }
      }
      if (!alive && pw == 0 && lane == 0) {
        // copies already issued still write into this block's shared memory: give them (bounded) time to land
        const unsigned long long t0 = global_ns();
        for (int s = landed; s < landed + RS && s < n_real; ++s)   // issued or not: a copy that was issued lands long before the limit
          for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
            if (mbar_try_wait(raw_full(s % RS), (uint32_t)((s / RS) & 1))) break;
            if (global_ns() - t0 > kWaitNs) break;
          }
        atomicExch(p.status, PAT_ERR_TIMEOUT);
      }
    } else {
      // ========================================================================= store warp
      uint32_t opar = 0;                           // phase parity of out_ready, one bit per planar slot
      bool alive = true;
      int pslot = 0;
      for (int it_idx = 0; it_idx < n_my_items && alive; ++it_idx) {
        const Item it = item_of(it_idx);
        pslot = (pslot + nct) % PS;                // skip the real stages of the item
        for (int y = 0; y < TR && alive; ++y) {
          if (!mbar_wait<kFillSleepNs>(out_ready(pslot), (opar >> pslot) & 1u, abort_flag)) { alive = false; break; }
          opar ^= 1u << pslot;
          const uint32_t o0 = sbase + pslot * PLANAR_STAGE;
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
            __half* dst_tile = p.y + (((size_t)n_img * p.H + (TR * ty + y)) * p.W + col0) * p.F + it.g * FG;
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
          __syncwarp();
          if (lane == 0) mbar_arrive_n(pl_empty(pslot), NCW);   // the slot goes back to the ring
          if (++pslot == PS) pslot = 0;
        }
      }
    }
  } else {
    // =========================================================================== consumer warps
    set_warp_registers<CONSUMER_REGS>();
    const int ly = lane >> 2, lx = lane & 3;
    // Warp w owns filter slots w and 31 - w of the group (the most loaded filter with the least loaded one, ...).
    // Only one of the two accumulator tiles is in registers at a time; the other is parked in tensor memory:
    // columns [64 * (w / 4) + 32 * f, +32) of the lanes of quarter w % 4.
    const uint32_t tm0 = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 64);
    int pslot = 0;
    uint32_t fpar = 0u;                    // parity to wait for on pl_full of the current slot
    bool alive = true;
    for (int it_idx = 0; it_idx < n_my_items && alive; ++it_idx) {
      uint32_t offA, offB;               // the lane's two chunk addresses of window row 0, relative to a channel plane
      {
        const Item it = item_of(it_idx);
        const int b = (ly < it.n0) ? 0 : 1;                  // band of this lane's tile row
        const uint32_t lane_off = (uint32_t)((2 * ly + 2 * b) * ROWB + lx * SEGB);
        const int swl = (ly + b) & 1;
        offA = lane_off + (uint32_t)(swl << 4);
        offB = lane_off + (uint32_t)((swl ^ 1) << 4);
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
        const int nk = (int)lds32(d0 + slot * 4);
        uint32_t e = d0 + DESC_HDR + slot * (CB * 16);
        for (int k = 0; k < nk; ++k, e += 16) {
          uint32_t m0, w01, w23, pad;
          lds128(e, m0, w01, w23, pad);
          const uint32_t base = pl0 + (m0 & 15u) * CHP;
          one_kernel(acc, base + offA, base + offB, m0, w01, w23);
        }
      };

      uint32_t cposA = 0u, cposB = 0u;   // byte offsets of filters 0 / 1 inside the group of 32 output channels
      for (int cb = 0; cb < nct; ++cb) {
        if (!mbar_wait<0>(pl_full(pslot), fpar, abort_flag)) { alive = false; break; }
        const uint32_t pl0 = sbase + pslot * PLANAR_STAGE;
        const uint32_t d0 = sbase + OFF_DESC + pslot * DESC_STAGE;
        if (cb == nct - 1) {
          cposA = (lds32(d0 + FG * 4 + (uint32_t)warp * 4) & (uint32_t)(FG - 1)) * 2u;
          cposB = (lds32(d0 + FG * 4 + (uint32_t)(FG - 1 - warp) * 4) & (uint32_t)(FG - 1)) * 2u;
        }
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
        if (lane == 0) mbar_arrive(pl_empty(pslot));
        if (++pslot == PS) { pslot = 0; fpar ^= 1u; }
      }
      if (!alive) break;

      // results: fp32 -> fp16 (round to nearest even) into the two output stages, one tile row each
#pragma unroll 1
      for (int y = 0; y < TR; ++y) {
        if (!mbar_wait<0>(pl_full(pslot), fpar, abort_flag)) { alive = false; break; }
        const uint32_t o0 = sbase + pslot * PLANAR_STAGE + (uint32_t)(lane * TC) * OUT_PITCH;
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
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

}  // namespace fast16

// True when the tuned kernel covers this layer.
bool conv_f16_fast_supported(int F, int C, const uint16_t* masks, int K, int dtype, int N, int H, int W, int stride) {
  using namespace fast16;
  if (dtype != PAT_F16 || stride != 1) return false;
  if (W % TC != 0 || H % TR != 0 || H < 2 * (LY - 1)) return false;
  const int TX = W / TC;
  if (!(TX == 1 || TX == 2 || TX % 4 == 0)) return false;
  if (C % CB != 0 || F % FG != 0) return false;
  (void)N; (void)masks; (void)K;
  return encode_fn() != nullptr;
}

int conv_f16_fast(const void* blob, int F, int C, const uint16_t* masks, int K, int64_t n_keep,
                  const void* x, void* y, int N, int H, int W, cudaStream_t st) {
  using namespace fast16;
  const BlobLayout L = blob_layout(F, C, K, n_keep, PAT_F16);
  const char* b = static_cast<const char*>(blob);
  Params p;
  p.x = static_cast<const __half*>(x);
  p.y = static_cast<__half*>(y);
  p.hdr = reinterpret_cast<const BlobHeader*>(b);
  p.tptr = reinterpret_cast<const int32_t*>(b + L.tptr);
  p.tmeta = reinterpret_cast<const uint32_t*>(b + L.tmeta);
  p.tw4 = reinterpret_cast<const uint2*>(b + L.tw4);
  p.xfilt = reinterpret_cast<const int32_t*>(b + L.xfilt);
  p.status = status_word();
  if (!p.status) return set_error(PAT_ERR_CUDA, "pat_conv3x3: cannot resolve the status word");
  p.N = N; p.H = H; p.W = W; p.C = C; p.F = F; p.K = K; p.nct = L.nct; p.n_keep = n_keep;
  p.TY = H / TR;
  const int TX = W / TC;
  p.TXe = TX >= LX ? LX : TX;
  p.NI = LX / p.TXe;
  p.BW = p.TXe * TC + 2;
  p.CG = TX / p.TXe;
  p.NIG = (N + p.NI - 1) / p.NI;
  p.NG = F / FG;
  p.n_row_blocks = (int)(((long long)p.NIG * p.TY + LY - 1) / LY);
  const long long items = (long long)p.n_row_blocks * p.CG * p.NG;
  if (items > 0x7FFFFFFFll) return set_error(PAT_ERR_SHAPE, "pat_conv3x3: too many work items");
  p.n_items = (int)items;
  for (int j = 0; j < 256; ++j) {
    p.masks[j] = (j < K) ? masks[j] : (uint16_t)0;
    p.pword[j] = (j < K) ? pattern_word(masks[j]) : 0u;
  }

  TmapSet tm;
  const cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
  const cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  for (int n = 1; n <= NMAPS; ++n) {          // band of n tile rows: 2n rows + a halo row above and below
    const cuuint32_t box[4] = {(cuuint32_t)CB, (cuuint32_t)p.BW, (cuuint32_t)(TR * n + 2), (cuuint32_t)p.NI};
    const CUresult cr = encode_fn()(&tm.m[n - 1], CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<void*>(x), dims, strides, box, estr,
                                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_32B,
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return set_error(PAT_ERR_CUDA, "pat_conv3x3: cuTensorMapEncodeTiled failed (%d)", (int)cr);
  }

  static thread_local DeviceSlot slots[kMaxDevices];
  DeviceSlot* dv = device_slot(slots);
  if (!dv) return set_error(PAT_ERR_CUDA, "pat_conv3x3: cannot query the current device");
  const int sm_count = dv->sms;
  if (!dv->ready) {
    if (int rc = check_cuda(cudaFuncSetAttribute(k_conv_f16_s1, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES), "set shared memory size")) return rc;
    cudaFuncAttributes fa;
    if (int rc = check_cuda(cudaFuncGetAttributes(&fa, k_conv_f16_s1), "query kernel attributes")) return rc;
    if (fa.numRegs < LAUNCH_REGS)
      return set_error(PAT_ERR_CUDA, "pat_conv3x3: kernel was compiled with %d registers per thread, the register split needs %d", fa.numRegs, LAUNCH_REGS);
    dv->ready = true;
  }
  const int grid = (int)std::min<long long>(items, sm_count);
  k_conv_f16_s1<<<grid, NTHREADS, SMEM_BYTES, st>>>(tm, p);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "pat_conv3x3 launch");
}

}  // namespace pat
