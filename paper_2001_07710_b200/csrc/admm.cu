// Primitives of the pattern-selection ADMM (Section 5.1) and of the library extraction (Algorithm 1, Section 5.2),
// batched over all kernels of a layer (or of a network): the training loop around them is not part of this library.
//
//   pat_simplex_project   u = [d - nu 1]_+ with nu the root of 1^T [d - nu 1]_+ = 1 (the proximal step's closed form)
//   pat_argmax_binarize   the one-hot vector closest to z: 1 at argmax_j z_j
//   pat_extract_library   "calculate the pattern distribution, remove the patterns with fewest occurrences"
//
// The first two stream n x K floats in and out once (8 and 4 - 8 bytes per element): a vector is shared by the lanes
// of a warp (or of a group of lanes), strided over its entries so that loads and stores cover whole sectors.
#include "common.cuh"
#include "select.cuh"

namespace pat {
namespace {

constexpr int kVecMaxK = 256;              // entries per vector
constexpr int kVecWarps = 8;               // warps per block

// Sums over the L lanes that share a vector (L a power of two, groups aligned): the same bits in every lane of a group.
template <int L, typename T>
__device__ __forceinline__ T group_sum(T v) {
#pragma unroll
  for (int off = L / 2; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
  return v;
}

// The root is found without sorting.  g(nu) = sum_j max(d_j - nu, 0) is convex, piecewise linear and decreasing, and
// Newton's step for g(nu) = 1 from a point nu is nu' = (sum of the entries above nu - 1) / (their number): from any
// start with at least one entry above it the steps reach the root in finitely many rounds (after the first step they
// approach it from below and never pass it).  The sets {entries above nu} are nested whatever nu is, so two rounds
// with the same number of entries above nu have the same set, and then nu is the root of that piece: no set has
// to be stored, a round is one pass "compare, add, count" over the entries.  The rounds run in fp32 from a lower
// bound of the root (see the kernel) until the count repeats, then in fp64 from the fp32 result until the count repeats again - usually
// two or three rounds - so the final piece and its root are exact: the sums are exact to about 1e-16 relative (the
// inputs are fp32), and there is one rounding to fp32 at the end.
//
// L lanes share a vector, sixteen entries each (K <= 16 L), so a warp works on 32 / L vectors at once: a round is a
// chain of dependent steps (a sum over the group, a division, a comparison), and what the kernel needs is many such
// chains in flight, not many lanes per chain.  Entry j of a vector sits in lane j % L, slot j / L.  u may be d.
constexpr int kVecQ = 16;
template <int L>
__global__ void __launch_bounds__(32 * kVecWarps, 5) k_simplex_project(const float* d, long long n, int K, float* u) {
  constexpr int G = 32 / L;                // vectors per warp
  const int lane = threadIdx.x & 31, sl = lane & (L - 1), g = lane / L;
  const long long stride = (long long)gridDim.x * kVecWarps * G;
  const long long first = ((long long)blockIdx.x * kVecWarps + (threadIdx.x >> 5)) * G;
  if (first >= n) return;                  // whole warps leave together
  for (long long base = first; base < n; base += stride) {
    const bool valid = base + g < n;
    const long long i = valid ? base + g : n - 1;       // a group without a vector repeats the last one and stores nothing
    float x[kVecQ];                        // slots beyond K hold the lowest float: never above any nu
    const float* di = d + i * K + sl;
    const int nq = (K - sl + L - 1) / L;   // this lane's entries: slots 0 .. nq - 1
#pragma unroll
    for (int q = 0; q < kVecQ; ++q) x[q] = (q < nq) ? __ldcs(di + L * q) : -3.402823466e38f;
    // Start: for any set S of entries (sum of S - 1) / |S| is at most the root (the root is the largest such value,
    // taken over the sets of the k largest entries), so the largest entry of every lane gives a lower bound that lies
    // close below the root when few entries are active, and at least one entry is above it (the root is below the largest
    // entry).  Rounding may lift it past the root: the first Newton step from there lands below the root again.
    float top = x[0];
#pragma unroll
    for (int q = 1; q < kVecQ; ++q) top = fmaxf(top, x[q]);
    float nu32 = (group_sum<L>(top) - 1.0f) / (float)L;
    if (!(nu32 > -3.402823466e38f)) nu32 = -3.402823466e38f;   // overflow of the sum (or a NaN): start below every entry
    // Counts are kept as floats (exact up to 2^24): a pass is then one comparison and two predicated additions per entry.
    float before = -1.0f;
    bool done = false;
    for (int round = 0; round < K + 2; ++round) {       // fp32 rounds
      float s = 0.0f, c = 0.0f;
#pragma unroll
      for (int q = 0; q < kVecQ; ++q)
        if (x[q] > nu32) { s += x[q]; c += 1.0f; }
      s = group_sum<L>(s);
      c = group_sum<L>(c);
      if (!done) {
        if (c == before || c == 0.0f) { done = true; before = c; }   // the set repeats (or rounding has pushed nu past the largest entry)
        else { nu32 = (s - 1.0f) / c; before = c; }
      }
      if (__all_sync(0xFFFFFFFFu, done)) break;          // every vector of the warp is through
    }
    // `before` is now the number of entries above nu32 (when the rounds ended because the count repeated); if that holds
    // for every vector of the warp the first exact round needs no counting pass
    const float known = done ? before : 0.0f;
    const bool skip_first_count = __all_sync(0xFFFFFFFFu, known > 0.0f);
    // Exact rounds.  A float x is above a double nu exactly when it is above nu rounded down to a float, so the sets are
    // formed by fp32 comparisons; only the sum of a set is taken in fp64.  A round: count the entries above the
    // current threshold; the same count as before means the same set, whose root nu already is; otherwise its exact
    // sum gives the next nu.  After the fp32 rounds the first set is usually the final one: one fp64 sum, two counts.
    double nu = (double)nu32;
    float thr = nu32;
    before = -1.0f;
    done = false;
    for (int round = 0; round < K + 4; ++round) {
      float c = known;
      if (round > 0 || !skip_first_count) {
        c = 0.0f;
#pragma unroll
        for (int q = 0; q < kVecQ; ++q)
          if (x[q] > thr) c += 1.0f;
        c = group_sum<L>(c);
      }
      if (!done && c == before) done = true;
      if (__all_sync(0xFFFFFFFFu, done)) break;
      double s = 0.0;
#pragma unroll
      for (int q = 0; q < kVecQ; ++q)
        if (x[q] > thr) s += (double)x[q];
      s = group_sum<L>(s);
      if (!done) {
        if (c == 0.0f) { thr = -3.402823466e38f; before = -1.0f; }   // past the largest entry: start again from all entries (not the padding)
        else { nu = (s - 1.0) / (double)c; thr = __double2float_rd(nu); before = c; }
      }
    }
    if (valid) {
      float* ui = u + i * K + sl;
      // x - nu in fp64 is exact up to one rounding; an entry at or below the threshold is not above nu
#pragma unroll
      for (int q = 0; q < kVecQ; ++q)
        if (q < nq) __stcs(ui + L * q, x[q] > thr ? (float)((double)x[q] - nu) : 0.0f);
    }
  }
}

// Largest entry of every vector, the lowest index among equal ones; optionally the one-hot vector itself.  As in the
// projection kernel L lanes share a vector (sixteen entries each, entry j in lane j % L, slot j / L), so a warp has
// 32 / L vectors in flight and the maximum over a vector takes log2(L) shuffle steps.
template <int L>
__global__ void __launch_bounds__(32 * kVecWarps) k_argmax_binarize(const float* __restrict__ z, long long n, int K,
                                                                     unsigned char* __restrict__ index_out,
                                                                     float* __restrict__ onehot_out) {
  constexpr int G = 32 / L;
  const int lane = threadIdx.x & 31, sl = lane & (L - 1), g = lane / L;
  const long long stride = (long long)gridDim.x * kVecWarps * G;
  const long long first = ((long long)blockIdx.x * kVecWarps + (threadIdx.x >> 5)) * G;
  if (first >= n) return;                  // whole warps leave together
  for (long long base = first; base < n; base += stride) {
    const bool valid = base + g < n;
    const long long i = valid ? base + g : n - 1;       // a group without a vector repeats the last one and stores nothing
    float x[kVecQ];
#pragma unroll
    for (int q = 0; q < kVecQ; ++q) x[q] = (sl + L * q < K) ? __ldcs(z + i * K + sl + L * q) : 0.0f;
    float best = x[0];                     // entry sl exists: K > 16 (L / 2) >= L > sl for L >= 2, and sl = 0 for L = 1
    int bj = sl;
#pragma unroll
    for (int q = 1; q < kVecQ; ++q) {
      const int j = sl + L * q;
      if (j < K && x[q] > best) { best = x[q]; bj = j; }   // ascending j inside a lane: the first maximum stays
    }
#pragma unroll
    for (int off = L / 2; off > 0; off >>= 1) {
      const float ob = __shfl_xor_sync(0xFFFFFFFFu, best, off);
      const int oj = __shfl_xor_sync(0xFFFFFFFFu, bj, off);
      if (ob > best || (ob == best && oj < bj)) { best = ob; bj = oj; }
    }
    if (valid) {
      if (sl == 0) index_out[i] = (unsigned char)bj;
      if (onehot_out) {
        float* oi = onehot_out + i * K;
#pragma unroll
        for (int q = 0; q < kVecQ; ++q) {
          const int j = sl + L * q;
          if (j < K) __stcs(oi + j, (j == bj) ? 1.0f : 0.0f);
        }
      }
    }
  }
}

// Pattern distribution: every kernel is given the mask that keeps most of its energy (as in pat_project) and the
// kernels per mask are counted, per block in shared memory first.
constexpr int kAssignPerThread = 4;
__global__ void __launch_bounds__(256) k_assign_count(const float* __restrict__ w, long long n, MaskTable lib,
                                                      unsigned long long* __restrict__ counts) {
  __shared__ unsigned int s_cnt[kMaxK + 1];
  for (int q = threadIdx.x; q <= kMaxK; q += blockDim.x) s_cnt[q] = 0u;
  __syncthreads();
  for (int r = 0; r < kAssignPerThread; ++r) {
    const long long i = ((long long)blockIdx.x * kAssignPerThread + r) * blockDim.x + threadIdx.x;
    if (i < n) {
      double e;
      atomicAdd(&s_cnt[best_mask(w + i * 9, lib, e)], 1u);
    }
  }
  __syncthreads();
  for (int q = threadIdx.x; q < lib.K; q += blockDim.x)
    if (s_cnt[q]) atomicAdd(&counts[q], (unsigned long long)s_cnt[q]);
}

// The K_out most frequent masks stay (equal counts: the lower id), in the order they have in the library.  One block:
// thread j ranks mask j among all masks, the survivors are written in id order.
__global__ void __launch_bounds__(256) k_pick_survivors(MaskTable lib, const unsigned long long* __restrict__ counts,
                                                        int K_out, unsigned short* __restrict__ masks_out) {
  pdl_wait();
  __shared__ unsigned long long s_c[kMaxK + 1];
  __shared__ int s_warp[8];
  const int j = threadIdx.x;
  s_c[j] = (j < lib.K) ? counts[j] : 0ull;
  __syncthreads();
  bool stays = false;
  if (j < lib.K) {
    int before = 0;
    const unsigned long long cj = s_c[j];
    for (int q = 0; q < lib.K; ++q) before += (s_c[q] > cj || (s_c[q] == cj && q < j)) ? 1 : 0;
    stays = before < K_out;
  }
  const unsigned ballot = __ballot_sync(0xFFFFFFFFu, stays);
  const int lane = j & 31, wid = j >> 5;
  if (lane == 0) s_warp[wid] = __popc(ballot);
  __syncthreads();
  int pos = __popc(ballot & ((1u << lane) - 1u));
  for (int q = 0; q < wid; ++q) pos += s_warp[q];
  if (stays) masks_out[pos] = lib.m[j];
}

// Blocks of the vector kernels: enough for eight resident blocks per SM, each warp then walks over its vectors.
unsigned vec_grid(int64_t n, int per_warp = 1) {
  static thread_local DeviceSlot slots[kMaxDevices];
  DeviceSlot* dv = device_slot(slots);
  const long long want = (long long)(dv ? dv->sms : 148) * 8;
  const long long need = (n + (long long)kVecWarps * per_warp - 1) / ((long long)kVecWarps * per_warp);
  return (unsigned)(need < want ? need : want);
}

}  // namespace
}  // namespace pat

using namespace pat;

extern "C" int pat_simplex_project(const float* d, int64_t n, int K, float* u, void* stream) {
  if (n == 0 && K >= 1 && K <= kVecMaxK) return PAT_OK;      // nothing to do (an empty batch may come with null pointers)
  if (!d || !u) return set_error(PAT_ERR_INVALID_ARG, "pat_simplex_project: null pointer");
  if (K < 1 || K > kVecMaxK) return set_error(PAT_ERR_SHAPE, "pat_simplex_project: K=%d outside 1..%d", K, kVecMaxK);
  if (n < 0 || n > 0x7FFFFFFFll * kVecWarps) return set_error(PAT_ERR_SHAPE, "pat_simplex_project: n=%lld out of range", (long long)n);
  if (!aligned(d, 4) || !aligned(u, 4)) return set_error(PAT_ERR_ALIGN, "pat_simplex_project: buffers must be 4-byte aligned");
  if (n == 0) return PAT_OK;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (K <= 16) k_simplex_project<1><<<vec_grid(n, 32), 32 * kVecWarps, 0, st>>>(d, (long long)n, K, u);
  else if (K <= 32) k_simplex_project<2><<<vec_grid(n, 16), 32 * kVecWarps, 0, st>>>(d, (long long)n, K, u);
  else if (K <= 64) k_simplex_project<4><<<vec_grid(n, 8), 32 * kVecWarps, 0, st>>>(d, (long long)n, K, u);
  else if (K <= 128) k_simplex_project<8><<<vec_grid(n, 4), 32 * kVecWarps, 0, st>>>(d, (long long)n, K, u);
  else k_simplex_project<16><<<vec_grid(n, 2), 32 * kVecWarps, 0, st>>>(d, (long long)n, K, u);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "pat_simplex_project launch");
}

extern "C" int pat_argmax_binarize(const float* z, int64_t n, int K, uint8_t* index_out, float* onehot_out, void* stream) {
  if (n == 0 && K >= 1 && K <= kVecMaxK) return PAT_OK;
  if (!z || !index_out) return set_error(PAT_ERR_INVALID_ARG, "pat_argmax_binarize: null pointer");
  if (K < 1 || K > kVecMaxK) return set_error(PAT_ERR_SHAPE, "pat_argmax_binarize: K=%d outside 1..%d", K, kVecMaxK);
  if (n < 0 || n > 0x7FFFFFFFll * kVecWarps) return set_error(PAT_ERR_SHAPE, "pat_argmax_binarize: n=%lld out of range", (long long)n);
  if (!aligned(z, 4) || (onehot_out && !aligned(onehot_out, 4))) return set_error(PAT_ERR_ALIGN, "pat_argmax_binarize: buffers must be 4-byte aligned");
  if (n == 0) return PAT_OK;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  // the smallest group of lanes that holds the vector (sixteen entries per lane), but never more lanes than entries
  if (K <= 16) k_argmax_binarize<1><<<vec_grid(n, 32), 32 * kVecWarps, 0, st>>>(z, (long long)n, K, index_out, onehot_out);
  else if (K <= 32) k_argmax_binarize<2><<<vec_grid(n, 16), 32 * kVecWarps, 0, st>>>(z, (long long)n, K, index_out, onehot_out);
  else if (K <= 64) k_argmax_binarize<4><<<vec_grid(n, 8), 32 * kVecWarps, 0, st>>>(z, (long long)n, K, index_out, onehot_out);
  else if (K <= 128) k_argmax_binarize<8><<<vec_grid(n, 4), 32 * kVecWarps, 0, st>>>(z, (long long)n, K, index_out, onehot_out);
  else k_argmax_binarize<16><<<vec_grid(n, 2), 32 * kVecWarps, 0, st>>>(z, (long long)n, K, index_out, onehot_out);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "pat_argmax_binarize launch");
}

extern "C" int pat_extract_library(const float* w, int64_t n, const uint16_t* masks_in, int K_in, int K_out,
                                   uint16_t* masks_out, uint64_t* counts_out, void* stream) {
  if (!w || !masks_out || !counts_out) return set_error(PAT_ERR_INVALID_ARG, "pat_extract_library: null pointer");
  if (int rc = check_library(masks_in, K_in)) return rc;
  if (K_out < 1 || K_out > K_in) return set_error(PAT_ERR_INVALID_ARG, "pat_extract_library: K_out=%d outside 1..%d", K_out, K_in);
  if (n < 0 || n > 0x7FFFFFFFll * 256) return set_error(PAT_ERR_SHAPE, "pat_extract_library: n=%lld out of range", (long long)n);
  if (!aligned(w, 4) || !aligned(counts_out, 8) || !aligned(masks_out, 2)) return set_error(PAT_ERR_ALIGN, "pat_extract_library: misaligned buffer");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  MaskTable lib;
  for (int j = 0; j <= kMaxK; ++j) lib.m[j] = (j < K_in) ? masks_in[j] : (uint16_t)0;
  lib.K = K_in;
  if (int rc = check_cuda(cudaMemsetAsync(counts_out, 0, sizeof(uint64_t) * (size_t)K_in, st), "pat_extract_library memset")) return rc;
  if (n > 0) {
    const unsigned grid = (unsigned)((n + 256 * kAssignPerThread - 1) / (256 * kAssignPerThread));
    k_assign_count<<<grid, 256, 0, st>>>(w, (long long)n, lib, reinterpret_cast<unsigned long long*>(counts_out));
    count_launches(1);
  }
  cudaError_t le = launch_dependent(k_pick_survivors, dim3(1), dim3(256), 0, st, lib,
                                    reinterpret_cast<const unsigned long long*>(counts_out), K_out,
                                    reinterpret_cast<unsigned short*>(masks_out));
  count_launches(1);
  if (le != cudaSuccess) return check_cuda(le, "pat_extract_library launch");
  return check_cuda(cudaGetLastError(), "pat_extract_library launch");
}
