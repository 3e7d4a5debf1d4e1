// pat_pack / pat_unpack: compressed, re-ordered weight storage.
//
// Section 6.2 re-orders filters so that filters with similar kernels sit together (balanced work per thread
// group) and groups, inside each filter, the kernels that share a pattern (one code path per group, no
// branches inside it).  The blob holds a canonical section in exactly that order and an execution section in
// which each filter's kernels are re-sorted by blocks of 16 input channels (the unit in which the convolution
// kernels stage activations), then pattern, then channel.  The execution section has its own filter order:
// filters stay inside their aligned group of 32 original filters (so that a thread block that owns a group
// writes 32 adjacent output channels) and are sorted inside the group by kept-kernel count, descending, so
// that pairing position i with position 31 - i gives every warp the same amount of work.
#include "common.cuh"

namespace pat {
namespace {

struct BlobPtrs {
  BlobHeader* hdr;
  int32_t *perm, *fptr, *pptr;
  uint16_t* chan;
  void* w4;
  int32_t* xfilt;      // execution position -> original filter
  int32_t* tptr;
  uint32_t* tmeta;
  void* tw4;
  uint32_t* dboff;     // descriptor block -> offset inside dblk, in 16-byte units (nblk + 1 entries)
  char* dblk;
  int32_t *hist, *cnt, *inv, *xinv, *xbase;
};

__host__ __device__ inline BlobPtrs blob_ptrs(void* blob, const BlobLayout& L, int F, int K) {
  char* b = static_cast<char*>(blob);
  BlobPtrs p;
  p.hdr = reinterpret_cast<BlobHeader*>(b);
  p.perm = reinterpret_cast<int32_t*>(b + L.perm);
  p.fptr = reinterpret_cast<int32_t*>(b + L.fptr);
  p.pptr = reinterpret_cast<int32_t*>(b + L.pptr);
  p.chan = reinterpret_cast<uint16_t*>(b + L.chan);
  p.w4 = b + L.w4;
  p.xfilt = reinterpret_cast<int32_t*>(b + L.xfilt);
  p.tptr = reinterpret_cast<int32_t*>(b + L.tptr);
  p.tmeta = reinterpret_cast<uint32_t*>(b + L.tmeta);
  p.tw4 = b + L.tw4;
  p.dboff = reinterpret_cast<uint32_t*>(b + L.dboff);
  p.dblk = b + L.dblk;
  p.hist = reinterpret_cast<int32_t*>(b + L.scratch);
  p.cnt = p.hist + (size_t)F * K;
  p.inv = p.cnt + F;
  p.xinv = p.inv + F;
  p.xbase = p.xinv + F;
  return p;
}

// One block per original filter: per-pattern counts and kept count.
__global__ void __launch_bounds__(256) k_pack_count(const uint8_t* __restrict__ pid, int C, int K, BlobPtrs bp, int* status) {
  pdl_wait();
  extern __shared__ int sh[];   // K counters
  const int f = blockIdx.x;
  for (int j = threadIdx.x; j < K; j += blockDim.x) sh[j] = 0;
  __syncthreads();
  for (int c = threadIdx.x; c < C; c += blockDim.x) {
    const int p = pid[(size_t)f * C + c];
    if (p == PAT_PRUNED) continue;
    if (p >= K) { atomicExch(status, PAT_ERR_BLOB); continue; }
    atomicAdd(&sh[p], 1);
  }
  __syncthreads();
  int tot = 0;
  for (int j = threadIdx.x; j < K; j += blockDim.x) bp.hist[(size_t)f * K + j] = sh[j];
  if (threadIdx.x == 0) {
    for (int j = 0; j < K; ++j) tot += sh[j];
    bp.cnt[f] = tot;
  }
}

// One block per filter: position = number of filters that come before it in the ordering
// (kept count descending, per-pattern counts lexicographically descending, original index ascending);
// the threads of the block share the comparisons.
__global__ void __launch_bounds__(128) k_pack_rank(int F, int K, BlobPtrs bp) {
  pdl_wait();
  __shared__ int s_rank, s_xrank;
  const int f = blockIdx.x;
  if (threadIdx.x == 0) { s_rank = 0; s_xrank = 0; }
  __syncthreads();
  const int nf = bp.cnt[f];
  const int32_t* hf = bp.hist + (size_t)f * K;
  const int g0 = (f / kExecGroup) * kExecGroup, g1 = min(F, g0 + kExecGroup);
  int rank = 0, xr = 0;
  for (int g = threadIdx.x; g < F; g += blockDim.x) {
    if (g == f) continue;
    const int ng = bp.cnt[g];
    bool before;
    if (ng != nf) before = ng > nf;
    else {
      const int32_t* hg = bp.hist + (size_t)g * K;
      int j = 0;
      while (j < K && hg[j] == hf[j]) ++j;
      before = (j < K) ? (hg[j] > hf[j]) : (g < f);
    }
    rank += before ? 1 : 0;
    // execution order: inside the aligned group of 32 original filters, by kept count (descending), then index
    if (g >= g0 && g < g1) xr += (ng > nf || (ng == nf && g < f)) ? 1 : 0;
  }
  atomicAdd(&s_rank, rank);
  atomicAdd(&s_xrank, xr);
  __syncthreads();
  if (threadIdx.x == 0) {
    bp.perm[s_rank] = f;
    bp.inv[f] = s_rank;
    bp.xfilt[g0 + s_xrank] = f;
    bp.xinv[f] = g0 + s_xrank;
  }
}

// Inclusive scan over the threads of a block (up to 1024; warp_tot: 32 words), thread 0 first: shuffles inside a
// warp, the warp totals through shared memory.
__device__ inline int block_scan_int(int v, int* warp_tot) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int u = __shfl_up_sync(0xFFFFFFFFu, v, off);
    if (lane >= off) v += u;
  }
  if (lane == 31) warp_tot[wid] = v;
  __syncthreads();
  int add = 0;
  for (int q = 0; q < wid; ++q) add += warp_tot[q];
  __syncthreads();
  return v + add;
}

// One block: fptr = exclusive scan of kept counts in the new order; pattern segment pointers; header.
constexpr int kPtrsThreads = 512;
__global__ void __launch_bounds__(kPtrsThreads) k_pack_ptrs(int F, int C, int K, long long n_keep, int dtype, MaskTable lib,
                                                            unsigned long long total_bytes, BlobPtrs bp, int* status) {
  pdl_wait();
  __shared__ int warp_tot[32];
  __shared__ int s_total;
  int carry = 0;                           // kept kernels of the filters in earlier chunks (the same in every thread)
  for (int base = 0; base < F; base += kPtrsThreads) {
    const int q = base + threadIdx.x;
    const int v = (q < F) ? bp.cnt[bp.perm[q]] : 0;
    const int incl = block_scan_int(v, warp_tot);
    if (q < F) {
      const int start = carry + incl - v;
      bp.fptr[q] = start;
      const int32_t* h = bp.hist + (size_t)bp.perm[q] * K;
      int pos = start;
      for (int j = 0; j < K; ++j) { bp.pptr[(size_t)q * (K + 1) + j] = pos; pos += h[j]; }
      bp.pptr[(size_t)q * (K + 1) + K] = pos;
    }
    if (threadIdx.x == kPtrsThreads - 1) s_total = incl;
    __syncthreads();
    carry += s_total;
    __syncthreads();
  }
  const int total = carry;
  // same scan in execution order
  carry = 0;
  for (int base = 0; base < F; base += kPtrsThreads) {
    const int e = base + threadIdx.x;
    const int v = (e < F) ? bp.cnt[bp.xfilt[e]] : 0;
    const int incl = block_scan_int(v, warp_tot);
    if (e < F) bp.xbase[e] = carry + incl - v;
    if (threadIdx.x == kPtrsThreads - 1) s_total = incl;
    __syncthreads();
    carry += s_total;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    bp.fptr[F] = total;
    const bool ok = (long long)total == n_keep;
    if (!ok) atomicExch(status, PAT_ERR_BLOB);
    BlobHeader* h = bp.hdr;
    h->magic = ok ? kBlobMagic : 0u;
    h->version = kBlobVersion;
    h->F = F; h->C = C; h->K = K; h->dtype = dtype;
    h->n_keep = n_keep;
    h->total_bytes = total_bytes;
    for (int j = 0; j <= kMaxK; ++j) h->masks[j] = lib.m[j];
    h->max_block_entries = 0;   // raised by k_pack_blocks
  }
}

template <typename T> __device__ inline T cvt_weight(float v);
template <> __device__ inline float cvt_weight<float>(float v) { return v; }
template <> __device__ inline __half cvt_weight<__half>(float v) { return __float2half_rn(v); }

// One block per original filter: place every kept kernel in the canonical and in the execution order.
// Positions are counted, never searched: per (16-channel tile, pattern) counts in shared memory give, after
// prefix sums over the tiles, the start of every (pattern) run in the canonical order and of every tile in the
// execution order; the rank of a kernel inside its tile needs a look at the 16 channels of that tile only.
// TABLE = false (tile x pattern table too large for shared memory): the counts are taken by direct loops.
template <typename T, bool TABLE>
__global__ void __launch_bounds__(256) k_pack_scatter(const float* __restrict__ wm, const uint8_t* __restrict__ pid,
                                                      int C, int K, int nct, MaskTable lib, BlobPtrs bp) {
  pdl_wait();
  // k_pack_ptrs refused the inputs (pattern_id keeps another number of kernels than n_keep): the positions computed
  // below would leave the sections sized by n_keep, so nothing is written
  if (bp.hdr->magic != kBlobMagic) return;
  extern __shared__ __align__(16) uint8_t sm_raw[];
  int* tile_pat = reinterpret_cast<int*>(sm_raw);                          // [nct][K] (TABLE only)
  int* tile_start = tile_pat + (TABLE ? nct * K : 0);                      // [nct + 1] kept kernels before tile t
  uint8_t* spid = reinterpret_cast<uint8_t*>(tile_start + nct + 1);        // C pattern ids of this filter
  const int f = blockIdx.x;
  const int q = bp.inv[f];
  for (int c = threadIdx.x; c < C; c += blockDim.x) spid[c] = pid[(size_t)f * C + c];
  if (TABLE)
    for (int i = threadIdx.x; i < nct * K; i += blockDim.x) tile_pat[i] = 0;
  __syncthreads();
  // kept kernels per tile (and per tile and pattern)
  for (int t = threadIdx.x; t < nct; t += blockDim.x) {
    int n = 0;
    const int c0 = t * kChanTile, c1 = min(c0 + kChanTile, C);
    for (int c = c0; c < c1; ++c) {
      const int j = spid[c];
      if (j == PAT_PRUNED || j >= K) continue;
      ++n;
      if (TABLE) tile_pat[t * K + j] += 1;        // one thread per tile: no race
    }
    tile_start[t + 1] = n;
  }
  __syncthreads();
  // exclusive prefix sums over the tiles: one thread per pattern column, one more for the tile totals
  if (TABLE) {
    for (int j = threadIdx.x; j < K; j += blockDim.x) {
      int run = 0;
      for (int t = 0; t < nct; ++t) { const int v = tile_pat[t * K + j]; tile_pat[t * K + j] = run; run += v; }
    }
  }
  if (threadIdx.x == blockDim.x - 1) {
    int run = 0;
    tile_start[0] = 0;
    for (int t = 0; t < nct; ++t) { const int v = tile_start[t + 1]; tile_start[t + 1] = run + v; run += v; }
  }
  __syncthreads();
  const int xe = bp.xinv[f];
  const int f0 = bp.xbase[xe];
  for (int t = threadIdx.x; t <= nct; t += blockDim.x) bp.tptr[(size_t)xe * (nct + 1) + t] = f0 + tile_start[t];
  T* w4 = static_cast<T*>(bp.w4);
  T* tw4 = static_cast<T*>(bp.tw4);
  for (int c = threadIdx.x; c < C; c += blockDim.x) {
    const int j = spid[c];
    if (j == PAT_PRUNED || j >= K) continue;
    const int tile = c / kChanTile;
    const int c0 = tile * kChanTile, c1 = min(c0 + kChanTile, C);
    int same_in_tile = 0;     // kernels of the same pattern on lower channels of this tile
    int exec_in_tile = 0;     // kernels of this tile ordered before (pattern, channel)
    for (int d = c0; d < c1; ++d) {
      const int pd = spid[d];
      if (pd == PAT_PRUNED || pd >= K) continue;
      same_in_tile += (pd == j && d < c) ? 1 : 0;
      exec_in_tile += (pd < j || (pd == j && d < c)) ? 1 : 0;
    }
    int same_before;          // kernels of the same pattern on lower channels (canonical order)
    if (TABLE) same_before = tile_pat[tile * K + j] + same_in_tile;
    else {
      same_before = same_in_tile;
      for (int d = 0; d < c0; ++d) same_before += (spid[d] == j) ? 1 : 0;
    }
    const int pos = bp.pptr[(size_t)q * (K + 1) + j] + same_before;
    const int tpos = f0 + tile_start[tile] + exec_in_tile;
    bp.chan[pos] = (uint16_t)c;
    bp.tmeta[tpos] = (uint32_t)c | ((uint32_t)j << 16);
    int bits[4];
    mask_bits(lib.m[j], bits);
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const T v = cvt_weight<T>(wm[((size_t)f * C + c) * 9 + bits[t]]);
      w4[(size_t)pos * 4 + t] = v;
      tw4[(size_t)tpos * 4 + t] = v;
    }
  }
}

// Descriptor blocks of the fp16 convolution kernel that copies its work lists with one bulk copy per pipeline
// stage.  One block per (group of 32 filters in execution order, 16-channel tile), groups major.  A block is the
// work of the kernel's 16 consumer warps in that stage; warp w owns filter slots w ("A") and 31 - w ("B") of the
// group and keeps one accumulator tile in registers, the other parked.  The order of a warp's operations is fixed
// here, at pack time: starting from the tile it holds when the stage begins (A at the first tile; afterwards
// whatever the previous stage left), first the kernels of that filter, then - only if the other filter has kernels
// in this tile - a swap and the other filter's kernels.
//   header   32 words; word w < 16: first operation of warp w (bits 0-15) | filter whose tile is in registers when
//            the stage begins (bit 31).  Word 16 + w: the output channels (inside the group of 32) of warp w's filters.
//   lists    16 bytes per operation, warp after warp, every list one slot longer than the warp's kernels:
//            {channel inside the tile | pattern_word(mask) | flags, taps 0-1 (fp16 x2), taps 2-3 (fp16 x2),
//             byte offset of the kernel's window in a stage image: channel plane + window row shift}
//            flags: kOpSwap on the first kernel after the swap, kOpEnd on the warp's last operation, together with
//            the start of the warp's list in the next tile's block (bits 21-31).  A warp without kernels in the
//            tile gets one operation with the flag kOpNop; otherwise the spare slot stays unused.
// Inside a filter the kernels are in (pattern, channel) order.  dboff[b] is the block's offset in 16-byte units.
// Launched with one warp per block (lane = consumer warp, lanes 16-31 idle apart from the shuffles).
__global__ void __launch_bounds__(32) k_pack_blocks(int nct, int nblk, MaskTable lib, BlobPtrs bp) {
  pdl_wait();
  if (bp.hdr->magic != kBlobMagic) return;   // refused by k_pack_ptrs, see k_pack_scatter
  const int blk = blockIdx.x, lane = threadIdx.x;
  const int g = blk / nct, cb = blk % nct;
  const bool active = lane < kBlockWarps;
  const int w = active ? lane : 0;
  const int32_t* rowA = bp.tptr + (size_t)(g * kExecGroup + w) * (nct + 1);
  const int32_t* rowB = bp.tptr + (size_t)(g * kExecGroup + kExecGroup - 1 - w) * (nct + 1);
  // which tile the warp holds when this stage begins
  int cur = 0;
  {
    // both rows are read whatever `cur` is: the loads do not wait for the decision of the tile before
    int pa = rowA[0], pb = rowB[0];
    for (int t = 0; t < cb; ++t) {
      const int na = rowA[t + 1], nb = rowB[t + 1];
      const int nother = cur ? na - pa : nb - pb;
      if (nother > 0) cur ^= 1;
      pa = na; pb = nb;
    }
  }
  const int aA = rowA[cb], nA = rowA[cb + 1] - aA, aB = rowB[cb], nB = rowB[cb + 1] - aB;
  const int cap = active ? nA + nB + 1 : 0;                       // list slots of this warp in this block
  const int cap_next = (active && cb + 1 < nct) ? (rowA[cb + 2] - rowA[cb + 1]) + (rowB[cb + 2] - rowB[cb + 1]) + 1 : 0;
  int incl = cap, incl_next = cap_next;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int v = __shfl_up_sync(0xFFFFFFFFu, incl, off), vn = __shfl_up_sync(0xFFFFFFFFu, incl_next, off);
    if (lane >= off) { incl += v; incl_next += vn; }
  }
  const int start = incl - cap, start_next = incl_next - cap_next;
  const int tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
  // kernels of this group in earlier tiles (all 32 filter slots)
  const int32_t* row = bp.tptr + (size_t)(g * kExecGroup + lane) * (nct + 1);
  int before = row[cb] - row[0];
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) before += __shfl_xor_sync(0xFFFFFFFFu, before, off);
  const uint32_t group_first = (uint32_t)bp.tptr[(size_t)(g * kExecGroup) * (nct + 1)];   // kernels of earlier groups
  const uint32_t off16 = (uint32_t)blk * (uint32_t)(kBlockHeaderBytes / 16 + kBlockWarps) + group_first + (uint32_t)before;
  if (lane == 0) {
    bp.dboff[blk] = off16;
    if (blk == nblk - 1) bp.dboff[nblk] = off16 + kBlockHeaderBytes / 16 + (uint32_t)tot;
    atomicMax(&bp.hdr->max_block_entries, tot);
  }
  char* base = bp.dblk + (size_t)off16 * 16;
  // words 16-31: for consumer warp lane - 16, where the results of its two filters go inside the group's 32 output
  // channels (original filter index modulo 32, filter A in bits 0-7, filter B in bits 8-15)
  const int wo = lane - kBlockWarps;
  const uint32_t where = active ? 0u
      : ((uint32_t)bp.xfilt[g * kExecGroup + wo] & (uint32_t)(kExecGroup - 1)) |
        (((uint32_t)bp.xfilt[g * kExecGroup + kExecGroup - 1 - wo] & (uint32_t)(kExecGroup - 1)) << 8);
  reinterpret_cast<uint32_t*>(base)[lane] = active ? ((uint32_t)start | ((uint32_t)cur << 31)) : where;
  if (!active) return;
  uint4* ent = reinterpret_cast<uint4*>(base + kBlockHeaderBytes) + start;
  const uint2* tw4 = static_cast<const uint2*>(bp.tw4);
  const int n_first = cur ? nB : nA, a_first = cur ? aB : aA;
  const int n_second = cur ? nA : nB, a_second = cur ? aA : aB;
  const int n_ops = n_first + n_second;
  const uint32_t end_flags = kOpEnd | ((uint32_t)start_next << kOpNextShift);
  if (n_ops == 0) {
    ent[0] = make_uint4(kOpNop | end_flags, 0u, 0u, 0u);
    return;
  }
  for (int k = 0; k < n_ops; ++k) {
    const int src = k < n_first ? a_first + k : a_second + (k - n_first);
    const uint32_t mt = bp.tmeta[src];
    const uint2 wv = tw4[src];
    const uint32_t ch = (mt & 0xFFFFu) - (uint32_t)(cb * kChanTile);
    const uint32_t pw = pattern_word(lib.m[mt >> 16]);
    uint32_t flags = 0u;
    if (k == n_first) flags |= kOpSwap;
    if (k == n_ops - 1) flags |= end_flags;
    ent[k] = make_uint4(ch | pw | flags, wv.x, wv.y, ch * (uint32_t)kImgPlaneBytes + ((pw >> 17) & 1u) * (uint32_t)kImgRowBytes);
  }
}

// Descriptor blocks of fp32 blobs: the same lists for stages of 8 channels (a tile of 16 channels of the
// execution section gives two stages: its kernels with channel 0-7 and 8-15, each in (pattern, channel) order) and
// 32-byte operations:
//   {channel inside the stage | pattern_word(mask) | flags, byte offset of the window in an fp32 stage image, taps 0-1}
//   {taps 2-3, 0, 0}
// Offsets (header words, "next list", dboff) count 16-byte units as in fp16 blobs, so an operation is two units.
__global__ void __launch_bounds__(32) k_pack_blocks_f32(int nct, int nblk, MaskTable lib, BlobPtrs bp) {
  pdl_wait();
  if (bp.hdr->magic != kBlobMagic) return;   // refused by k_pack_ptrs, see k_pack_scatter
  const int blk = blockIdx.x, lane = threadIdx.x;
  const int nst = 2 * nct;                                   // stages of 8 channels
  const int g = blk / nst, st8 = blk % nst;
  const bool active = lane < kBlockWarps;
  const int w = active ? lane : 0;
  const int32_t* rowA = bp.tptr + (size_t)(g * kExecGroup + w) * (nct + 1);
  const int32_t* rowB = bp.tptr + (size_t)(g * kExecGroup + kExecGroup - 1 - w) * (nct + 1);
  // kernels of a filter slot in stage s: those of tile s / 2 whose channel lies in half s % 2
  auto count = [&](const int32_t* row, int s) {
    const int t = s >> 1, half = s & 1;
    int n = 0;
    for (int k = row[t]; k < row[t + 1]; ++k) n += ((int)(((bp.tmeta[k] & 0xFFFFu) >> 3) & 1u) == half) ? 1 : 0;
    return n;
  };
  int cur = 0;                                               // which tile the warp holds when this stage begins
  for (int s = 0; s < st8; ++s)
    if (count(cur ? rowA : rowB, s) > 0) cur ^= 1;
  const int nA = count(rowA, st8), nB = count(rowB, st8);
  const int cap = active ? nA + nB + 1 : 0;
  const int cap_next = (active && st8 + 1 < nst) ? count(rowA, st8 + 1) + count(rowB, st8 + 1) + 1 : 0;
  int incl = cap, incl_next = cap_next;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int v = __shfl_up_sync(0xFFFFFFFFu, incl, off), vn = __shfl_up_sync(0xFFFFFFFFu, incl_next, off);
    if (lane >= off) { incl += v; incl_next += vn; }
  }
  const int start = incl - cap, start_next = incl_next - cap_next;
  const int tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
  // kernels of this group in earlier stages (all 32 filter slots)
  const int32_t* row = bp.tptr + (size_t)(g * kExecGroup + lane) * (nct + 1);
  int before = row[st8 >> 1] - row[0] + ((st8 & 1) ? count(row, st8 - 1) : 0);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) before += __shfl_xor_sync(0xFFFFFFFFu, before, off);
  const uint32_t group_first = (uint32_t)bp.tptr[(size_t)(g * kExecGroup) * (nct + 1)];
  const uint32_t off16 = (uint32_t)blk * (uint32_t)(kBlockHeaderBytes / 16 + 2 * kBlockWarps) + 2u * (group_first + (uint32_t)before);
  if (lane == 0) {
    bp.dboff[blk] = off16;
    if (blk == nblk - 1) bp.dboff[nblk] = off16 + kBlockHeaderBytes / 16 + 2u * (uint32_t)tot;
    atomicMax(&bp.hdr->max_block_entries, tot);
  }
  char* base = bp.dblk + (size_t)off16 * 16;
  reinterpret_cast<uint32_t*>(base)[lane] = active ? ((uint32_t)(2 * start) | ((uint32_t)cur << 31)) : 0u;
  if (!active) return;
  uint4* ent = reinterpret_cast<uint4*>(base + kBlockHeaderBytes) + 2 * start;
  const uint4* tw4 = static_cast<const uint4*>(bp.tw4);       // four fp32 taps per kernel
  const int n_first = cur ? nB : nA, n_second = cur ? nA : nB;
  const int n_ops = n_first + n_second;
  const uint32_t end_flags = kOpEnd | ((uint32_t)(2 * start_next) << kOpNextShift);
  if (n_ops == 0) {
    ent[0] = make_uint4(kOpNop | end_flags, 0u, 0u, 0u);
    ent[1] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  const int t16 = st8 >> 1, half = st8 & 1;
  int k_out = 0;
  for (int pass = 0; pass < 2; ++pass) {
    const int32_t* r = (pass == 0) == (cur == 0) ? rowA : rowB;   // first the filter whose tile is held
    for (int k = r[t16]; k < r[t16 + 1]; ++k) {
      const uint32_t mt = bp.tmeta[k];
      const uint32_t ch16 = (mt & 0xFFFFu) - (uint32_t)(t16 * kChanTile);
      if ((int)(ch16 >> 3) != half) continue;
      const uint32_t ch = ch16 & 7u;
      const uint32_t pw = pattern_word(lib.m[mt >> 16]);
      uint32_t flags = 0u;
      if (k_out == n_first) flags |= kOpSwap;
      if (k_out == n_ops - 1) flags |= end_flags;
      const uint4 wv = tw4[k];
      ent[2 * k_out] = make_uint4(ch | pw | flags, ch * (uint32_t)kImgPlaneBytesF32 + ((pw >> 17) & 1u) * (uint32_t)kImgRowBytesF32, wv.x, wv.y);
      ent[2 * k_out + 1] = make_uint4(wv.z, wv.w, 0u, 0u);
      ++k_out;
    }
  }
}

__device__ inline bool header_matches(const BlobHeader* h, int F, int C, int K, long long n_keep, int dtype, const MaskTable& lib) {
  if (h->magic != kBlobMagic || h->version != kBlobVersion) return false;
  if (h->F != F || h->C != C || h->K != K || h->dtype != dtype || h->n_keep != n_keep) return false;
  for (int j = 0; j < K; ++j) if (h->masks[j] != lib.m[j]) return false;
  return true;
}

// One block per re-ordered filter: write its kept entries into the (pre-zeroed) dense tensor.
template <typename T>
__global__ void __launch_bounds__(128) k_unpack(BlobPtrs bp, int F, int C, int K, long long n_keep, int dtype, MaskTable lib,
                                                float* __restrict__ out, int* status) {
  if (!header_matches(bp.hdr, F, C, K, n_keep, dtype, lib)) {
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicExch(status, PAT_ERR_BLOB);
    return;
  }
  const int q = blockIdx.x;
  const int f = bp.perm[q];
  const T* w4 = static_cast<const T*>(bp.w4);
  for (int j = 0; j < K; ++j) {
    int bits[4];
    mask_bits(lib.m[j], bits);
    const int a = bp.pptr[(size_t)q * (K + 1) + j], b = bp.pptr[(size_t)q * (K + 1) + j + 1];
    for (int k = a + threadIdx.x; k < b; k += blockDim.x) {
      const int c = bp.chan[k];
#pragma unroll
      for (int t = 0; t < 4; ++t) out[((size_t)f * C + c) * 9 + bits[t]] = (float)w4[(size_t)k * 4 + t];
    }
  }
}

int common_checks(const char* who, int F, int C, const uint16_t* masks, int K, int64_t n_keep, int dtype) {
  if (F < 1 || C < 1 || F > 65535 || C > 65535) return set_error(PAT_ERR_SHAPE, "%s: F=%d C=%d outside 1..65535", who, F, C);
  if (int rc = check_library(masks, K)) return rc;
  if (dtype != PAT_F32 && dtype != PAT_F16) return set_error(PAT_ERR_DTYPE, "%s: dtype %d", who, dtype);
  if (n_keep < 0 || n_keep > (int64_t)F * C) return set_error(PAT_ERR_INVALID_ARG, "%s: n_keep=%lld outside 0..F*C", who, (long long)n_keep);
  return PAT_OK;
}

MaskTable make_table(const uint16_t* masks, int K) {
  MaskTable lib;
  for (int j = 0; j <= kMaxK; ++j) lib.m[j] = (j < K) ? masks[j] : (uint16_t)0;
  lib.K = K;
  return lib;
}

}  // namespace
}  // namespace pat

using namespace pat;

extern "C" int pat_pack(const float* w_masked, const uint8_t* pattern_id, int F, int C,
                        const uint16_t* masks, int K, int64_t n_keep, int dtype,
                        void* blob, size_t blob_bytes, void* stream) {
  if (!w_masked || !pattern_id || !blob) return set_error(PAT_ERR_INVALID_ARG, "pat_pack: null pointer");
  if (int rc = common_checks("pat_pack", F, C, masks, K, n_keep, dtype)) return rc;
  if (!aligned(blob, 256)) return set_error(PAT_ERR_ALIGN, "pat_pack: blob must be 256-byte aligned");
  const BlobLayout L = blob_layout(F, C, K, n_keep, dtype);
  if (blob_bytes < L.total) return set_error(PAT_ERR_WORKSPACE, "pat_pack: blob has %zu bytes, needs %zu", blob_bytes, L.total);
  int* status = status_word();
  if (!status) return set_error(PAT_ERR_CUDA, "pat_pack: cannot resolve the status word");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const MaskTable lib = make_table(masks, K);
  const BlobPtrs bp = blob_ptrs(blob, L, F, K);
  // every check that can refuse the call comes before the first launch
  const size_t table = sizeof(int) * (size_t)L.nct * K;
  const bool use_table = table <= 24 * 1024;
  const size_t smem = (use_table ? table : 0) + sizeof(int) * ((size_t)L.nct + 1) + (size_t)C;
  if (smem > 48 * 1024) return set_error(PAT_ERR_SHAPE, "pat_pack: C=%d too large for the packing kernel", C);
  cudaError_t le = cudaSuccess;                   // first launch error, if any
  auto note = [&](cudaError_t e) { if (le == cudaSuccess) le = e; };
  note(launch_dependent(k_pack_count, dim3(F), dim3(256), K * sizeof(int), st, pattern_id, C, K, bp, status));
  note(launch_dependent(k_pack_rank, dim3(F), dim3(128), 0, st, F, K, bp));
  note(launch_dependent(k_pack_ptrs, dim3(1), dim3(kPtrsThreads), 0, st, F, C, K, (long long)n_keep, dtype, lib, (unsigned long long)L.total, bp, status));
  if (dtype == PAT_F16) {
    if (use_table) note(launch_dependent(k_pack_scatter<__half, true>, dim3(F), dim3(256), smem, st, w_masked, pattern_id, C, K, L.nct, lib, bp));
    else note(launch_dependent(k_pack_scatter<__half, false>, dim3(F), dim3(256), smem, st, w_masked, pattern_id, C, K, L.nct, lib, bp));
  } else {
    if (use_table) note(launch_dependent(k_pack_scatter<float, true>, dim3(F), dim3(256), smem, st, w_masked, pattern_id, C, K, L.nct, lib, bp));
    else note(launch_dependent(k_pack_scatter<float, false>, dim3(F), dim3(256), smem, st, w_masked, pattern_id, C, K, L.nct, lib, bp));
  }
  count_launches(4);
  if (L.nblk > 0) {
    if (dtype == PAT_F16) note(launch_dependent(k_pack_blocks, dim3(L.nblk), dim3(32), 0, st, L.nct, L.nblk, lib, bp));
    else note(launch_dependent(k_pack_blocks_f32, dim3(L.nblk), dim3(32), 0, st, L.nct, L.nblk, lib, bp));
    count_launches(1);
  }
  if (le != cudaSuccess) return check_cuda(le, "pat_pack launch");
  return check_cuda(cudaGetLastError(), "pat_pack launch");
}

extern "C" int pat_unpack(const void* blob, int F, int C, const uint16_t* masks, int K, int64_t n_keep,
                          int dtype, float* w_dense_out, void* stream) {
  if (!blob || !w_dense_out) return set_error(PAT_ERR_INVALID_ARG, "pat_unpack: null pointer");
  if (int rc = common_checks("pat_unpack", F, C, masks, K, n_keep, dtype)) return rc;
  if (!aligned(blob, 256)) return set_error(PAT_ERR_ALIGN, "pat_unpack: blob must be 256-byte aligned");
  int* status = status_word();
  if (!status) return set_error(PAT_ERR_CUDA, "pat_unpack: cannot resolve the status word");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const BlobLayout L = blob_layout(F, C, K, n_keep, dtype);
  const BlobPtrs bp = blob_ptrs(const_cast<void*>(blob), L, F, K);
  const MaskTable lib = make_table(masks, K);
  if (int rc = check_cuda(cudaMemsetAsync(w_dense_out, 0, sizeof(float) * 9 * (size_t)F * C, st), "pat_unpack memset")) return rc;
  if (dtype == PAT_F16) k_unpack<__half><<<F, 128, 0, st>>>(bp, F, C, K, (long long)n_keep, dtype, lib, w_dense_out, status);
  else k_unpack<float><<<F, 128, 0, st>>>(bp, F, C, K, (long long)n_keep, dtype, lib, w_dense_out, status);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "pat_unpack launch");
}
