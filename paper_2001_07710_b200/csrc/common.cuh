// Shared host/device definitions of the patconv library: error reporting, blob layout, launch helpers.
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stddef.h>
#include "../../include/patconv.h"

namespace pat {

constexpr uint32_t kBlobMagic = 0x50415443u;  // "PATC"
constexpr uint32_t kBlobVersion = 4u;
constexpr int kChanTile = 16;                 // granularity (input channels) of the execution section
constexpr int kExecGroup = 32;                // filters per execution group (aligned groups of original filters)
constexpr int kMaxK = 255;
constexpr int kBlockHeaderBytes = 4 * kExecGroup;   // header of a descriptor block: 32 words, one per consumer warp in use
constexpr int kBlockWarps = kExecGroup / 2;         // consumer warps that share a descriptor block (two filters each)
// Geometry of the stage images the descriptor blocks are written for (the last word of a descriptor is the byte
// offset of the kernel's window inside a stage image): bytes of a pixel row and of a channel plane.
constexpr int kImgRowBytes = 128;
constexpr int kImgPlaneBytes = 36 * kImgRowBytes;
// fp32 blobs: stages of 8 channels (the same bytes per stage), rows and planes twice as large, 32-byte operations
constexpr int kChanStageF32 = 8;
constexpr int kImgRowBytesF32 = 256;
constexpr int kImgPlaneBytesF32 = 36 * kImgRowBytesF32;
// Descriptor word (see pattern_word below): bits 18 / 19 / 20 = "swap the accumulator tiles before this kernel" /
// "last operation of this warp in this stage" / "no kernel: the warp has nothing to do in this stage",
// bits 21-31 = where the warp's list starts in the next stage's block.
constexpr uint32_t kOpSwap = 1u << 18, kOpEnd = 1u << 19, kOpNop = 1u << 20;
constexpr int kOpNextShift = 21;

// First 256 bytes of every blob.
struct BlobHeader {
  uint32_t magic, version;
  int32_t F, C, K, dtype;
  int64_t n_keep;
  uint64_t total_bytes;
  uint16_t masks[kMaxK + 1];  // library the blob was packed with (entries >= K are 0)
  int32_t max_block_entries;  // largest number of kernels in one descriptor block (0 when the blob has none)
};
static_assert(sizeof(BlobHeader) <= 768, "header must fit its slot");
constexpr size_t kHeaderBytes = 768;

// Byte offsets of every array in a blob; a pure function of (F, C, K, n_keep, dtype).
struct BlobLayout {
  size_t perm, fptr, pptr, chan, w4;   // canonical section
  size_t xfilt, tptr, tmeta, tw4;      // execution section (its own filter order, see pack.cu)
  size_t dboff, dblk;                  // descriptor blocks (blobs with F % 32 == 0 and C % 16 == 0; else empty)
  int nblk;                            // number of descriptor blocks = (F / 32) * (C / 16) for fp16, (F / 32) * (C / 8) for fp32, or 0
  size_t scratch;                      // pack-time temporaries: hist[F][K], count[F], inv[F], xinv[F], xbase[F]
  size_t total;
  int nct;                             // number of 16-channel tiles = ceil(C / 16)
};

__host__ __device__ inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }
__host__ __device__ inline int elem_bytes(int dtype) { return dtype == PAT_F16 ? 2 : 4; }

__host__ __device__ inline BlobLayout blob_layout(int F, int C, int K, int64_t n_keep, int dtype) {
  BlobLayout L;
  const size_t e = (size_t)elem_bytes(dtype);
  const size_t nk = (size_t)n_keep;
  L.nct = (C + kChanTile - 1) / kChanTile;
  size_t o = kHeaderBytes;
  L.perm = o;  o = align256(o + sizeof(int32_t) * (size_t)F);
  L.fptr = o;  o = align256(o + sizeof(int32_t) * ((size_t)F + 1));
  L.pptr = o;  o = align256(o + sizeof(int32_t) * (size_t)F * ((size_t)K + 1));
  L.chan = o;  o = align256(o + sizeof(uint16_t) * nk);
  L.w4 = o;    o = align256(o + 4 * e * nk);
  L.xfilt = o; o = align256(o + sizeof(int32_t) * (size_t)F);
  L.tptr = o;  o = align256(o + sizeof(int32_t) * (size_t)F * ((size_t)L.nct + 1));
  L.tmeta = o; o = align256(o + sizeof(uint32_t) * nk);
  L.tw4 = o;   o = align256(o + 4 * e * nk);
  const bool has_blocks = F % kExecGroup == 0 && C % kChanTile == 0;
  const size_t op_bytes = dtype == PAT_F16 ? 16 : 32;          // one operation of a descriptor block
  L.nblk = !has_blocks ? 0 : (dtype == PAT_F16 ? (F / kExecGroup) * L.nct : (F / kExecGroup) * (C / kChanStageF32));
  L.dboff = o; o = align256(o + (L.nblk ? sizeof(uint32_t) * ((size_t)L.nblk + 1) : 0));
  L.dblk = o;  o = align256(o + (L.nblk ? (size_t)L.nblk * (kBlockHeaderBytes + op_bytes * kBlockWarps) + op_bytes * nk : 0));
  L.scratch = o; o = align256(o + sizeof(int32_t) * (size_t)F * ((size_t)K + 4));
  L.total = o;
  return L;
}

// Library passed by value to kernels.
struct MaskTable {
  uint16_t m[kMaxK + 1];
  int K;
};

// Device address of the status word shared by all kernels of the library (nullptr on failure).
int* status_word();

// Host-side count of kernel launches (see pat_launch_count).
void count_launches(int n);

// Launch of a kernel that follows another kernel of this library in the same stream and begins with pdl_wait():
// as a programmatic dependent its launch overlaps the predecessor's tail (the small projection and packing kernels
// are launch-latency bound), and pdl_wait() holds it until the predecessor has completed and its writes are visible.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cfg.attrs = &attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

// Division of 0 <= n < 2^32 by a number known on the host (Granlund and Montgomery's multiply-and-shift): three
// instructions instead of the twenty-odd of a division by a run-time value.
struct FastDiv {
  uint32_t d, m, sh1, sh2;
  void set(int div) {
    d = (uint32_t)div;
    uint32_t l = 0;
    while ((1ull << l) < (unsigned long long)d) ++l;                       // ceil(log2 d)
    m = (uint32_t)(((1ull << 32) * ((1ull << l) - d)) / d + 1);
    sh1 = l < 1 ? l : 1;
    sh2 = l > 0 ? l - 1 : 0;
  }
#ifdef __CUDACC__
  __device__ __forceinline__ int div(int n) const {
    const uint32_t t = __umulhi(m, (uint32_t)n);
    return (int)((t + (((uint32_t)n - t) >> sh1)) >> sh2);
  }
  __device__ __forceinline__ int mod(int n) const { return n - div(n) * (int)d; }
#endif
};

int set_error(int code, const char* fmt, ...);

// Per-device facts and one-time set-up of a kernel family (function attributes and SM counts belong to a device, and
// a thread may switch devices between calls): each family keeps a thread-local table and asks for the current device's
// entry.  Returns nullptr when the device cannot be queried.
constexpr int kMaxDevices = 64;
struct DeviceSlot { int sms = 0; bool ready = false; };
inline DeviceSlot* device_slot(DeviceSlot (&table)[kMaxDevices]) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  DeviceSlot& d = table[dev];
  if (d.sms == 0 && cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return nullptr;
  return &d;
}
int check_library(const uint16_t* masks, int K);
int check_cuda(cudaError_t e, const char* what);
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// Tap positions of a mask: bits in ascending order.
__host__ __device__ inline void mask_bits(uint32_t m, int bits[4]) {
  int t = 0;
  for (int b = 0; b < 9 && t < 4; ++b)
    if (m & (1u << b)) bits[t++] = b;
  for (; t < 4; ++t) bits[t] = 4;
}

// ---- execution codes of the fp16 convolution kernels (written into the blob's descriptor blocks by pat_pack)
// Compiled pattern codes.  A pattern whose top row is empty is the same shape one row lower, so it runs the
// code of the shifted-up pattern on a window that starts one row lower: the twelve built-in patterns need ten
// codes (the eight patterns of Section 4.2 need six).  Any other pattern takes the generic code (kGenericCode).
constexpr int kNumCodes = 10;
constexpr int kGenericCode = 15;
__host__ __device__ constexpr uint32_t code_mask(int i) {
  constexpr uint32_t m[kNumCodes] = {0x03A, 0x017, 0x0B2, 0x09A, 0x01B, 0x036, 0x093, 0x03C, 0x192, 0x00F};
  return m[i];
}
__host__ __device__ constexpr int nth_bit(uint32_t mask, int t) {
  int seen = 0;
  for (int b = 0; b < 9; ++b)
    if (mask & (1u << b)) { if (seen == t) return b; ++seen; }
  return 4;
}

// descriptor word: bits 0-3 channel inside the block, 4-12 pattern mask, 13-16 code, 17 window row shift
__host__ __device__ inline uint32_t pattern_word(uint32_t mask) {
  const uint32_t shift = (mask & 7u) == 0u ? 1u : 0u;
  const uint32_t norm = mask >> (3u * shift);
  uint32_t code = kGenericCode;
  for (int i = 0; i < kNumCodes; ++i)
    if (code_mask(i) == norm) code = (uint32_t)i;
  if (code == (uint32_t)kGenericCode) return (mask << 4) | (code << 13);
  return (mask << 4) | (code << 13) | (shift << 17);
}

}  // namespace pat
