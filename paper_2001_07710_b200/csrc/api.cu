// Host-side plumbing of the C ABI: error strings, built-in libraries, argument checks, blob layout.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <atomic>
#include "common.cuh"

namespace pat {

__device__ int g_status = 0;

int* status_word() {
  // one address per device; looked up on first use with that device current
  static thread_local int cached_dev = -1;
  static thread_local int* cached_ptr = nullptr;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
  if (dev != cached_dev) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_status) != cudaSuccess) return nullptr;
    cached_ptr = static_cast<int*>(p);
    cached_dev = dev;
  }
  return cached_ptr;
}

static thread_local char t_last_error[512] = "";
static std::atomic<uint64_t> g_launches{0};

void count_launches(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }
uint64_t launches() { return g_launches.load(std::memory_order_relaxed); }

int set_error(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(t_last_error, sizeof(t_last_error), fmt, ap);
  va_end(ap);
  return code;
}

int check_cuda(cudaError_t e, const char* what) {
  if (e == cudaSuccess) return PAT_OK;
  return set_error(PAT_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

int check_library(const uint16_t* masks, int K) {
  if (!masks) return set_error(PAT_ERR_INVALID_ARG, "masks is null");
  if (K < 1 || K > kMaxK) return set_error(PAT_ERR_LIBRARY, "library size %d outside 1..%d", K, kMaxK);
  for (int j = 0; j < K; ++j) {
    const unsigned m = masks[j];
    if (m >= 512u || __builtin_popcount(m) != 4)
      return set_error(PAT_ERR_LIBRARY, "mask %d (0x%x) does not have exactly four of nine bits", j, m);
    for (int i = 0; i < j; ++i)
      if (masks[i] == masks[j]) return set_error(PAT_ERR_LIBRARY, "masks %d and %d are identical", i, j);
  }
  return PAT_OK;
}

}  // namespace pat

using namespace pat;

extern "C" {

const char* pat_strerror(int code) {
  switch (code) {
    case PAT_OK: return "ok";
    case PAT_ERR_INVALID_ARG: return "invalid argument";
    case PAT_ERR_SHAPE: return "unsupported shape";
    case PAT_ERR_LIBRARY: return "invalid pattern library";
    case PAT_ERR_DTYPE: return "invalid dtype";
    case PAT_ERR_ALIGN: return "misaligned pointer";
    case PAT_ERR_BLOB: return "blob does not match arguments";
    case PAT_ERR_CUDA: return "CUDA error";
    case PAT_ERR_WORKSPACE: return "buffer too small";
    case PAT_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown error";
  }
}

const char* pat_last_error(void) { return t_last_error; }

uint64_t pat_launch_count(void) { return pat::launches(); }

int pat_library_builtin(int K, uint16_t* masks_out) {
  // bit b = 3*r + s.  cross family | 2x2 blocks holding the centre | centre + opposite arms + corner
  static const uint16_t kBuiltin[12] = {
      0x03A, 0x0B8, 0x0B2, 0x09A,
      0x01B, 0x036, 0x0D8, 0x1B0,
      0x093, 0x03C, 0x192, 0x078};
  if (!masks_out) return set_error(PAT_ERR_INVALID_ARG, "masks_out is null");
  if (K != 4 && K != 8 && K != 12) return set_error(PAT_ERR_LIBRARY, "built-in libraries have 4, 8 or 12 patterns, not %d", K);
  for (int j = 0; j < K; ++j) masks_out[j] = kBuiltin[j];
  return PAT_OK;
}

int pat_blob_layout(int F, int C, int K, int64_t n_keep, int dtype, size_t offsets[5]) {
  if (!offsets) return set_error(PAT_ERR_INVALID_ARG, "offsets is null");
  if (pat_pack_size(F, C, K, n_keep, dtype) == 0) return set_error(PAT_ERR_INVALID_ARG, "invalid blob parameters");
  const BlobLayout L = blob_layout(F, C, K, n_keep, dtype);
  offsets[0] = L.perm; offsets[1] = L.fptr; offsets[2] = L.pptr; offsets[3] = L.chan; offsets[4] = L.w4;
  return PAT_OK;
}

size_t pat_pack_size(int F, int C, int K, int64_t n_keep, int dtype) {
  if (F < 1 || C < 1 || C > 65535 || F > 65535 || K < 1 || K > kMaxK) return 0;
  if (n_keep < 0 || n_keep > (int64_t)F * C) return 0;
  if (dtype != PAT_F32 && dtype != PAT_F16) return 0;
  return blob_layout(F, C, K, n_keep, dtype).total;
}

int pat_query_status(void* stream) {
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  int h = 0;
  int rc = check_cuda(cudaMemcpyFromSymbolAsync(&h, g_status, sizeof(int), 0, cudaMemcpyDeviceToHost, st), "read status");
  if (rc) return rc;
  rc = check_cuda(cudaStreamSynchronize(st), "synchronize");
  if (rc) return rc;
  if (h != 0) {
    const int zero = 0;
    rc = check_cuda(cudaMemcpyToSymbolAsync(g_status, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, st), "clear status");
    if (rc) return rc;
    rc = check_cuda(cudaStreamSynchronize(st), "synchronize");
    if (rc) return rc;
    return set_error(h, "a kernel reported: %s", pat_strerror(h));
  }
  return PAT_OK;
}

}  // extern "C"
