// pat_project: per-kernel pattern selection and per-layer connectivity pruning, exact and deterministic.
//
// Pattern pruning multiplies each 3x3 kernel by one mask of the library (Section 4.1); the mask kept is the
// one that retains the largest squared L2 norm, the one-shot form of the argmax binarisation of Section 5.1.
// Connectivity pruning ranks kernels by their L2 norm (Section 6.1) and keeps the n_keep strongest of the layer.
//
// Exactness: squares of fp32 values are exact in fp64 and are added in ascending bit order, so the energies
// are the same bits on any IEEE machine.  The n_keep-th largest energy is found with a radix select over the
// (monotone) bit pattern of the non-negative doubles: two 16-bit digits by histograms over the whole layer (the
// second one also lists the keys that share the first digit with the threshold), the remaining 32 bits and the
// index that separates kept from removed ties by one thread block over that list.  Three launches per layer: the
// steps that need all blocks' results are done by the block that finishes last.
#include "common.cuh"
#include "select.cuh"

namespace pat {
namespace {

constexpr int kSelBlock = 256;
constexpr int kBins = 65536;

struct SelectState {
  unsigned long long prefix;   // bits of the threshold key decided so far; in the end the threshold itself
  long long remaining;         // how many keys with this prefix (and below-decided digits) are still to be kept
  unsigned int cut;            // kernels whose key equals the threshold are kept up to this index
  unsigned int pad;
};

// workspace layout
constexpr int kCoarse = 256;                 // coarse histogram: the upper 8 bits of a 16-bit digit
constexpr int kPasses = 2;                   // digits found with histograms over the whole layer (16 bits each)
constexpr size_t kHistWords = (size_t)kPasses * (kBins + kCoarse) + 4;   // one fine + one coarse histogram per pass, then two control words
constexpr size_t kTicketWord = (size_t)kPasses * (kBins + kCoarse);     // hist[kTicketWord]: blocks of the running kernel that are done
constexpr size_t kListWord = kTicketWord + 1;                             // hist[kListWord]: length of the candidate list

struct ProjWs {
  unsigned long long* key;     // [FC] energy bit patterns
  unsigned char* pid;          // [FC] best pattern per kernel
  unsigned int* hist;          // [kPasses][65536 fine | 256 coarse]; zeroed by every call
  unsigned int* cand;          // [FC] indices of the keys that share the first digit with the threshold (any order)
  SelectState* st;
  size_t bytes;
};

constexpr size_t ws_align(size_t x) { return (x + 255) & ~size_t(255); }
constexpr size_t ws_bytes(int64_t FC) {
  return ws_align(8 * (size_t)FC) + ws_align((size_t)FC) + ws_align(4 * kHistWords) +
         ws_align(4 * (size_t)FC) + ws_align(sizeof(SelectState));
}

inline ProjWs carve(void* base, int64_t FC) {
  ProjWs w;
  char* p = static_cast<char*>(base);
  size_t o = 0;
  w.key = reinterpret_cast<unsigned long long*>(p + o); o += ws_align(8 * (size_t)FC);
  w.pid = reinterpret_cast<unsigned char*>(p + o);      o += ws_align((size_t)FC);
  w.hist = reinterpret_cast<unsigned int*>(p + o);      o += ws_align(4 * kHistWords);
  w.cand = reinterpret_cast<unsigned int*>(p + o);      o += ws_align(4 * (size_t)FC);
  w.st = reinterpret_cast<SelectState*>(p + o);         o += ws_align(sizeof(SelectState));
  w.bytes = o;
  return w;
}

// The selection kernels end with a step that needs the work of all their blocks (choosing the digit from the
// complete histogram, finishing the selection on the candidate list).  Instead of a launch of its own that step is done by
// whichever block finishes last: every block publishes its results, takes a ticket, and the block that draws the
// last ticket (which also puts the counter back to zero for the next kernel) goes on.  Returns true in every thread
// of that block; its reads of the other blocks' results must bypass L1 (__ldcg).
// One fence per block, not per thread: the block barrier orders every thread's writes and atomics before thread 0's
// fence, and a fence is cumulative - what thread 0 has observed is visible device-wide before its ticket is.  (A
// fence in every thread made each of them wait for its own atomics to return; with a quarter of a million threads
// that wait was most of the kernel.)
__device__ inline bool last_block_done(unsigned int* ticket) {
  __shared__ bool s_last;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    s_last = atomicInc(ticket, gridDim.x - 1) == gridDim.x - 1;
  }
  __syncthreads();
  if (s_last) __threadfence();
  return s_last;
}

// Histogram of one 16-bit digit (fine: all 16 bits, coarse: its upper 8 bits).  Identical digits inside a warp are
// merged into one atomic.  Called by all threads of a warp; `in` = this thread takes part.
__device__ inline void hist_add(unsigned int* fine, unsigned int* coarse, bool in, unsigned d) {
  const unsigned active = __ballot_sync(0xFFFFFFFFu, in);
  if (in) {
    const int lane = threadIdx.x & 31;
    const unsigned same = __match_any_sync(active, d);
    if ((int)(__ffs(same) - 1) == lane) atomicAdd(&fine[d], (unsigned)__popc(same));
    const unsigned same_c = __match_any_sync(active, d >> 8);
    if ((int)(__ffs(same_c) - 1) == lane) atomicAdd(&coarse[d >> 8], (unsigned)__popc(same_c));
  }
}

// Inclusive scan over the threads of a block (any size up to 1024; warp_tot: 32 words), thread 0 first.
__device__ inline unsigned long long block_scan_256(unsigned long long v, unsigned long long* warp_tot) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const unsigned long long u = __shfl_up_sync(0xFFFFFFFFu, v, off);
    if (lane >= off) v += u;
  }
  if (lane == 31) warp_tot[wid] = v;
  __syncthreads();
  unsigned long long add = 0;
  for (int q = 0; q < wid; ++q) add += warp_tot[q];
  __syncthreads();
  return v + add;
}

// One block of 256 threads or more: find the digit d with  count(digit > d) < remaining <= count(digit >= d), first in
// the coarse histogram, then among the 256 fine bins of the coarse bin found.  Thread 0 owns the highest bin.
__device__ inline void pick_digit(SelectState* st, const unsigned int* hist, int pass) {
  __shared__ unsigned long long warp_tot[32];
  __shared__ int s_coarse;
  __shared__ unsigned long long s_above;
  const unsigned int* fine = hist + (size_t)pass * (kBins + kCoarse);
  const unsigned int* coarse = fine + kBins;
  const int t = threadIdx.x;
  const bool owner = t < kCoarse;            // threads beyond the first 256 only take part in the scans
  const unsigned long long rem = (unsigned long long)__ldcg(&st->remaining);
  const unsigned long long prefix = __ldcg(&st->prefix);
  if (t == 0) { s_coarse = 0; s_above = 0ull; }   // defined values even if no bin qualifies (a histogram that misses keys)
  __syncthreads();
  {
    const int bin = kCoarse - 1 - t;
    const unsigned long long c = owner ? __ldcg(coarse + bin) : 0ull;
    const unsigned long long incl = block_scan_256(c, warp_tot);
    if (owner && rem > incl - c && rem <= incl) { s_coarse = bin; s_above = incl - c; }
  }
  __syncthreads();
  const int cb = s_coarse;
  const unsigned long long above = s_above;
  {
    const int bin = cb * 256 + (255 - t);
    const unsigned long long c = owner ? __ldcg(fine + bin) : 0ull;
    const unsigned long long incl = above + block_scan_256(c, warp_tot);
    if (owner && rem > incl - c && rem <= incl) {
      st->prefix = (prefix << 16) | (unsigned long long)bin;
      st->remaining = (long long)(rem - (incl - c));
    }
  }
}

// kSelPerThread kernels per thread: energies of all masks, argmax (lowest id on ties); histogram of the first digit
// of the energies' bit patterns; the last block picks that digit.  do_select = false (everything or nothing is
// kept): pattern ids only.
//
// The first digit (sign, exponent, four mantissa bits) takes only a few dozen values in a layer, so its histogram is
// collected per block in shared memory and flushed with one global atomic per distinct value and block: atomics
// from a quarter of a million threads on those few addresses took longer than the rest of the projection.
constexpr int kSelPerThread = 4;
constexpr int kSelSlots = 1024;              // shared-memory counters, indexed by the digit's low bits and tagged with the digit
__global__ void __launch_bounds__(256) k_select_pattern(const float* __restrict__ w, int64_t FC, MaskTable lib,
                                                        unsigned long long* __restrict__ key, unsigned char* __restrict__ pid,
                                                        SelectState* st, long long n_keep, unsigned int* hist, bool do_select) {
  pdl_wait();
  __shared__ unsigned int s_tag[kSelSlots], s_cnt[kSelSlots], s_coarse[kCoarse];
  if (do_select) {
    for (int q = threadIdx.x; q < kSelSlots; q += blockDim.x) { s_tag[q] = 0u; s_cnt[q] = 0u; }
    for (int q = threadIdx.x; q < kCoarse; q += blockDim.x) s_coarse[q] = 0u;
    __syncthreads();
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) { st->prefix = 0ull; st->remaining = n_keep; }
  for (int r = 0; r < kSelPerThread; ++r) {
    const int64_t i = ((int64_t)blockIdx.x * kSelPerThread + r) * blockDim.x + threadIdx.x;
    const bool in = i < FC;
    unsigned long long k = 0ull;
    if (in) {
      double best_e;
      const int best = best_mask(w + i * 9, lib, best_e);
      k = (unsigned long long)__double_as_longlong(best_e);   // e >= +0: bit pattern is monotone
      key[i] = k;
      pid[i] = (unsigned char)best;
    }
    if (!do_select) continue;
    // identical digits inside the warp are merged first; the lane that speaks for a digit adds to the block's counters
    const unsigned d = (unsigned)(k >> 48);
    const unsigned active = __ballot_sync(0xFFFFFFFFu, in);
    if (in) {
      const int lane = threadIdx.x & 31;
      const unsigned same = __match_any_sync(active, d);
      if ((int)(__ffs(same) - 1) == lane) {
        const unsigned n = (unsigned)__popc(same);
        const unsigned slot = d & (unsigned)(kSelSlots - 1);
        const unsigned old = atomicCAS(&s_tag[slot], 0u, d + 1u);
        if (old == 0u || old == d + 1u) atomicAdd(&s_cnt[slot], n);
        else atomicAdd(&hist[d], n);         // the slot belongs to another digit: straight to the global histogram
        atomicAdd(&s_coarse[d >> 8], n);
      }
    }
  }
  if (!do_select) return;
  __syncthreads();
  for (int q = threadIdx.x; q < kSelSlots; q += blockDim.x)
    if (s_cnt[q]) atomicAdd(&hist[s_tag[q] - 1u], s_cnt[q]);
  for (int q = threadIdx.x; q < kCoarse; q += blockDim.x)
    if (s_coarse[q]) atomicAdd(&hist[kBins + q], s_coarse[q]);
  if (last_block_done(hist + kTicketWord)) pick_digit(st, hist, 0);
}

// Among 256 counters (one per thread of the first 256; the others pass 0), the bin where the running count - taken
// from the highest bin down (DESCENDING) or from the lowest bin up - first reaches `rem`.  Returns the bin and sets
// `before` to the count of the bins passed on the way.  All threads of the block call it; `cnt` is this thread's bin
// (thread t owns bin 255 - t when descending, bin t otherwise).
template <bool DESCENDING>
__device__ inline int pick_bin_256(unsigned long long cnt, unsigned long long rem, unsigned long long* warp_tot,
                                   unsigned long long& before) {
  __shared__ int s_bin;
  __shared__ unsigned long long s_before;
  if (threadIdx.x == 0) { s_bin = 0; s_before = 0ull; }
  __syncthreads();
  const unsigned long long incl = block_scan_256(cnt, warp_tot);
  if (threadIdx.x < 256 && rem > incl - cnt && rem <= incl) { s_bin = DESCENDING ? 255 - (int)threadIdx.x : (int)threadIdx.x; s_before = incl - cnt; }
  __syncthreads();
  before = s_before;
  const int bin = s_bin;
  __syncthreads();                           // the shared results may be overwritten by the next call
  return bin;
}

// Second digit and everything after it.  All blocks: histogram of the second 16-bit digit over the keys whose first
// digit is the threshold's, and a list of those keys' indices (any order).  The last block picks the second digit
// and then works alone: it gathers from the list the keys that agree with the threshold in both digits - a handful
// for ordinary weights, which are ranked directly in shared memory.  If there are more than fit there (weights with
// few distinct values), it finds the remaining 32 bits of the threshold in four 8-bit passes over the list with a
// histogram in shared memory and then, among the keys equal to the threshold, the index below which `remaining` of
// them lie (four more passes, over the index bits).  Kernels whose key equals the threshold are kept in index order.
constexpr int kRestThreads = 256;
constexpr int kShortList = 2048;
static_assert(kRestThreads == kSelBlock, "launched with one block per kSelBlock kernels");
__global__ void __launch_bounds__(kRestThreads) k_select_rest(const unsigned long long* __restrict__ key, int64_t FC,
                                                              SelectState* st, unsigned int* hist, unsigned int* cand) {
  pdl_wait();
  __shared__ unsigned long long warp_tot[32];
  __shared__ unsigned int s_hist[256];
  __shared__ unsigned long long s_key[kShortList];
  __shared__ unsigned int s_idx[kShortList];
  __shared__ unsigned int s_n;
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  bool in = i < FC;
  unsigned d = 0;
  if (in) {
    const unsigned long long k = key[i];
    in = (k >> 48) == st->prefix;
    d = (unsigned)((k >> 32) & 0xFFFFull);
  }
  unsigned int* fine = hist + (size_t)(kBins + kCoarse);
  hist_add(fine, fine + kBins, in, d);
  {
    // a place in the list: one atomic per block (the warps' counts are added up in shared memory first)
    __shared__ unsigned int s_wcount[kRestThreads / 32], s_base;
    const unsigned active = __ballot_sync(0xFFFFFFFFu, in);
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    if (lane == 0) s_wcount[wid] = (unsigned)__popc(active);
    __syncthreads();
    if (threadIdx.x == 0) {
      unsigned tot = 0u;
      for (int q = 0; q < kRestThreads / 32; ++q) { const unsigned c = s_wcount[q]; s_wcount[q] = tot; tot += c; }
      s_base = tot ? atomicAdd(&hist[kListWord], tot) : 0u;
    }
    __syncthreads();
    if (in) cand[s_base + s_wcount[wid] + __popc(active & ((1u << lane) - 1u))] = (unsigned)i;
  }
  if (!last_block_done(hist + kTicketWord)) return;
  pick_digit(st, hist, 1);
  const int t = threadIdx.x;
  if (t == 0) s_n = 0u;
  __syncthreads();
  unsigned long long prefix = __ldcg(&st->prefix);             // 32 bits decided
  unsigned long long rem = (unsigned long long)__ldcg(&st->remaining);
  const unsigned n = __ldcg(&hist[kListWord]);
  for (unsigned j = t; j < n; j += kRestThreads) {
    const unsigned idx = __ldcg(cand + j);
    const unsigned long long k = key[idx];
    if ((k >> 32) == prefix) {
      const unsigned pos = atomicAdd(&s_n, 1u);
      if (pos < (unsigned)kShortList) { s_key[pos] = k; s_idx[pos] = idx; }
    }
  }
  __syncthreads();
  const bool fits = s_n <= (unsigned)kShortList;
  const unsigned m = fits ? s_n : n;
  if (fits) {
    // The kept kernels of the short list are its first `rem` in the order (key descending, index ascending): the
    // entry with rem - 1 others before it carries the threshold and the last kept index.  A handful of entries: every
    // thread ranks its own against all others.
    for (unsigned j = t; j < m; j += kRestThreads) {
      const unsigned long long kj = s_key[j];
      const unsigned ij = s_idx[j];
      unsigned long long before = 0ull;
      for (unsigned q = 0; q < m; ++q) {
        const unsigned long long kq = s_key[q];
        before += (kq > kj || (kq == kj && s_idx[q] < ij)) ? 1ull : 0ull;
      }
      if (before + 1ull == rem) { st->prefix = kj; st->cut = ij; }
    }
    return;
  }
  // more entries than the short list holds (weights with few distinct values): digit by digit over the list itself
  auto entry = [&](unsigned j, unsigned long long& k, unsigned& idx) {
    idx = __ldcg(cand + j);
    k = key[idx];
  };
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (t < 256) s_hist[t] = 0u;
    __syncthreads();
    for (unsigned j = t; j < m; j += kRestThreads) {
      unsigned long long k; unsigned idx;
      entry(j, k, idx);
      if ((k >> (shift + 8)) == prefix) atomicAdd(&s_hist[(unsigned)(k >> shift) & 255u], 1u);
    }
    __syncthreads();
    unsigned long long above;
    const int bin = pick_bin_256<true>(t < 256 ? s_hist[255 - t] : 0u, rem, warp_tot, above);
    prefix = (prefix << 8) | (unsigned long long)bin;
    rem -= above;
  }
  // prefix is the threshold now and rem (>= 1) the number of keys equal to it that are kept: the rem lowest indices
  unsigned long long ipre = 0ull;
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (t < 256) s_hist[t] = 0u;
    __syncthreads();
    for (unsigned j = t; j < m; j += kRestThreads) {
      unsigned long long k; unsigned idx;
      entry(j, k, idx);
      if (k == prefix && ((unsigned long long)idx >> (shift + 8)) == ipre) atomicAdd(&s_hist[(idx >> shift) & 255u], 1u);
    }
    __syncthreads();
    unsigned long long below;
    const int bin = pick_bin_256<false>(t < 256 ? s_hist[t] : 0u, rem, warp_tot, below);
    ipre = (ipre << 8) | (unsigned long long)bin;
    rem -= below;
  }
  if (t == 0) { st->prefix = prefix; st->cut = (unsigned int)ipre; }
}

// Decide keep / remove per kernel and write pattern ids and masked weights.  The decision is taken by one thread per
// kernel; the weights are then copied by the whole block in the order they lie in memory (a thread that walked its
// own nine values would touch a different 32-byte sector with every lane, on the way in and on the way out).
__global__ void __launch_bounds__(kSelBlock) k_finalize(const float* w, int64_t FC, MaskTable lib,
                                                        const unsigned long long* __restrict__ key,
                                                        const unsigned char* __restrict__ pid_in,
                                                        const SelectState* __restrict__ st,
                                                        unsigned char* __restrict__ pid_out, float* wm, int keep_all_or_none) {
  pdl_wait();
  __shared__ unsigned short s_mask[kSelBlock];      // the kept positions of every kernel of the block (0: removed)
  const int64_t i0 = (int64_t)blockIdx.x * kSelBlock;
  const int64_t i = i0 + threadIdx.x;
  const bool valid = i < FC;
  bool keep;
  if (keep_all_or_none >= 0) {            // n_keep == F*C (1) or n_keep == 0 (0): no threshold needed
    keep = keep_all_or_none == 1;
  } else {
    const unsigned long long thr = st->prefix;
    const unsigned long long k = valid ? key[i] : 0ull;
    keep = valid && (k > thr || (k == thr && (unsigned int)i <= st->cut));   // ties: lowest indices first
  }
  unsigned m = 0u;
  if (valid) {
    const unsigned char p = pid_in[i];
    m = keep ? lib.m[p] : 0u;
    pid_out[i] = keep ? p : (unsigned char)PAT_PRUNED;
  }
  s_mask[threadIdx.x] = (unsigned short)m;
  __syncthreads();
  const int64_t e0 = i0 * 9;
  const int n = (int)(((FC - i0) < (int64_t)kSelBlock ? (FC - i0) : (int64_t)kSelBlock) * 9);
  for (int e = threadIdx.x; e < n; e += kSelBlock) {
    const int kq = e / 9, b = e - kq * 9;
    const float v = w[e0 + e];
    wm[e0 + e] = ((s_mask[kq] >> b) & 1u) ? v : 0.0f;
  }
}

}  // namespace
}  // namespace pat

using namespace pat;

extern "C" size_t pat_project_workspace(int F, int C) {
  if (F < 1 || C < 1 || F > 65535 || C > 65535) return 0;
  return ws_bytes((int64_t)F * C);
}

extern "C" int pat_project(const float* w, int F, int C, const uint16_t* masks, int K, int64_t n_keep,
                           uint8_t* pattern_id, float* w_masked, void* workspace, size_t workspace_bytes,
                           void* stream) {
  if (!w || !pattern_id || !w_masked || !workspace) return set_error(PAT_ERR_INVALID_ARG, "pat_project: null pointer");
  if (F < 1 || C < 1 || F > 65535 || C > 65535) return set_error(PAT_ERR_SHAPE, "pat_project: F=%d C=%d outside 1..65535", F, C);
  if (int rc = check_library(masks, K)) return rc;
  const int64_t FC = (int64_t)F * C;
  if (n_keep < 0 || n_keep > FC) return set_error(PAT_ERR_INVALID_ARG, "pat_project: n_keep=%lld outside 0..%lld", (long long)n_keep, (long long)FC);
  if (!aligned(w, 4) || !aligned(w_masked, 4)) return set_error(PAT_ERR_ALIGN, "pat_project: weights must be 4-byte aligned");
  if (!aligned(workspace, 256)) return set_error(PAT_ERR_ALIGN, "pat_project: workspace must be 256-byte aligned");
  const ProjWs ws = carve(workspace, FC);
  if (workspace_bytes < ws.bytes) return set_error(PAT_ERR_WORKSPACE, "pat_project: workspace has %zu bytes, needs %zu", workspace_bytes, ws.bytes);

  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  MaskTable lib;
  for (int j = 0; j <= kMaxK; ++j) lib.m[j] = (j < K) ? masks[j] : (uint16_t)0;
  lib.K = K;
  const int nb_sel = (int)((FC + 256 * kSelPerThread - 1) / (256 * kSelPerThread));
  const int nblk = (int)((FC + kSelBlock - 1) / kSelBlock);
  int mode = -1;
  if (n_keep == FC) mode = 1;
  else if (n_keep == 0) mode = 0;
  if (mode < 0) {
    if (int rc = check_cuda(cudaMemsetAsync(ws.hist, 0, 4 * kHistWords, st), "pat_project memset")) return rc;
  }
  cudaError_t le = cudaSuccess;                   // first launch error, if any
  auto note = [&](cudaError_t e) { if (le == cudaSuccess) le = e; };
  note(launch_dependent(k_select_pattern, dim3(nb_sel), dim3(256), 0, st, w, FC, lib, ws.key, ws.pid, ws.st, (long long)n_keep, ws.hist, mode < 0));
  if (mode < 0) {
    note(launch_dependent(k_select_rest, dim3(nblk), dim3(kRestThreads), 0, st, ws.key, FC, ws.st, ws.hist, ws.cand));
  }
  note(launch_dependent(k_finalize, dim3(nblk), dim3(kSelBlock), 0, st, w, FC, lib, ws.key, ws.pid, ws.st, pattern_id, w_masked, mode));
  count_launches(mode < 0 ? 3 : 2);
  if (le != cudaSuccess) return check_cuda(le, "pat_project launch");
  return check_cuda(cudaGetLastError(), "pat_project launch");
}

// ------------------------------------------------------------------------------------------------------------
// pat_project_static: the same projection for callers that cannot hand over a workspace.
//
// Some hosts of this library may not allocate device memory at the point where they project a layer: a serving
// process whose whole device budget was reserved up front by another component, a plug-in that runs inside
// somebody else's memory pool, or a latency-critical loop that must not risk the implicit device-wide
// synchronisation of an allocation.  For them the scratch space lives in the library image itself.
namespace pat {
namespace {

constexpr int64_t kStaticMaxKernels = 262144;   // F * C limit of pat_project_static (a 512 x 512 layer)
constexpr size_t kStaticScratchBytes = ws_bytes(kStaticMaxKernels);   // about 3.9 MB

// Every GPU that loads the library holds this array until the process ends.
static __device__ __align__(256) unsigned char g_project_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {};          // device address of the array, per device (host-side cache)

// The array's name is only a host-side handle in host code; the device address has to be asked for, once per
// device and with that device current.
int static_scratch(void** out) {
  int dev = -1;
  if (int rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice")) return rc;
  if (dev < 0 || dev >= kMaxDevices) return set_error(PAT_ERR_CUDA, "pat_project_static: device index %d not supported", dev);
  void* p = __atomic_load_n(&g_scratch_addr[dev], __ATOMIC_ACQUIRE);
  if (!p) {
    if (int rc = check_cuda(cudaGetSymbolAddress(&p, g_project_scratch), "cudaGetSymbolAddress(scratch)")) return rc;
    __atomic_store_n(&g_scratch_addr[dev], p, __ATOMIC_RELEASE);
  }
  *out = p;
  return PAT_OK;
}

}  // namespace
}  // namespace pat

extern "C" int64_t pat_project_static_max_kernels(void) { return kStaticMaxKernels; }

extern "C" int pat_project_static(const float* w, int F, int C, const uint16_t* masks, int K, int64_t n_keep,
                                  uint8_t* pattern_id, float* w_masked, void* stream) {
  if (F < 1 || C < 1 || F > 65535 || C > 65535)
    return set_error(PAT_ERR_SHAPE, "pat_project_static: F=%d C=%d outside 1..65535", F, C);
  if ((int64_t)F * C > kStaticMaxKernels)
    return set_error(PAT_ERR_WORKSPACE, "pat_project_static: F*C = %lld exceeds the built-in scratch (%lld kernels); use pat_project with a workspace",
                     (long long)F * C, (long long)kStaticMaxKernels);
  static_assert(kStaticScratchBytes >= 8 * (size_t)kStaticMaxKernels, "scratch holds at least the keys");
  if (carve(nullptr, (int64_t)F * C).bytes > kStaticScratchBytes)
    return set_error(PAT_ERR_WORKSPACE, "pat_project_static: internal scratch too small for F=%d C=%d", F, C);
  void* scratch = nullptr;
  if (int rc = static_scratch(&scratch)) return rc;
  return pat_project(w, F, C, masks, K, n_keep, pattern_id, w_masked, scratch, kStaticScratchBytes, stream);
}
