// Generic sparse / dense 3x3 convolution kernels: any shape, stride 1 or 2, fp32 or fp16 storage.
//
// These are the shape-agnostic kernels of the library (used for stride 2, odd sizes, batch 1 and the dense
// first layer); the tuned stride-1 kernels live in their own files.  Mapping: a thread block owns an 8 x 32
// tile of output pixels and 32 re-ordered filters; lanes run along x so every weight is warp-uniform; each
// thread keeps an 8-row column of outputs for 4 filters in registers.  Activations are staged 16 input
// channels at a time from NHWC global memory into a channel-planar fp32 shared-memory tile with its halo
// (zero outside the image), so each activation is read from global memory once per block.  Only the four
// stored taps of every kept kernel are visited (Section 6.2: per-pattern access, pattern-grouped kernels).
#include "common.cuh"

namespace pat {
namespace {

constexpr int TH = 8, TW = 32, NWARP = 8, RF = 4, FG = NWARP * RF, CB = kChanTile;

template <typename T> __device__ inline float to_f32(T v);
template <> __device__ inline float to_f32<float>(float v) { return v; }
template <> __device__ inline float to_f32<__half>(__half v) { return __half2float(v); }
template <typename T> __device__ inline T from_f32(float v);
template <> __device__ inline float from_f32<float>(float v) { return v; }
template <> __device__ inline __half from_f32<__half>(float v) { return __float2half_rn(v); }

struct ConvArgs {
  const void* x;
  void* y;
  const int32_t* perm;
  const int32_t* tptr;
  const uint32_t* tmeta;
  const void* tw4;
  const BlobHeader* hdr;
  int* status;
  int N, H, W, C, F, Ho, Wo, K, nct, dtype;
  long long n_keep;
  int tiles_x, tiles_y;
};

template <int STRIDE> struct Geo {
  static constexpr int IH = (TH - 1) * STRIDE + 3;
  static constexpr int IW = (TW - 1) * STRIDE + 3;
  static constexpr int IWP = IW | 1;                 // odd row pitch
  static constexpr int PLANE = IH * IWP + ((IH * IWP) % 2 == 0 ? 1 : 0);   // odd plane pitch
};

// Stage channels [c0, c0+CB) of the input tile into shared memory as fp32, channel-planar.
template <typename T, int STRIDE>
__device__ inline void stage_tile(float* tile, const T* __restrict__ x, int n, int iy0, int ix0, int c0,
                                  int H, int W, int C) {
  using G = Geo<STRIDE>;
  for (int idx = threadIdx.x; idx < G::IH * G::IW * CB; idx += blockDim.x) {
    const int c = idx % CB;
    const int pos = idx / CB;
    const int ty = pos / G::IW, tx = pos % G::IW;
    const int yi = iy0 + ty, xi = ix0 + tx, ci = c0 + c;
    float v = 0.0f;
    if (yi >= 0 && yi < H && xi >= 0 && xi < W && ci < C)
      v = to_f32<T>(x[(((size_t)n * H + yi) * W + xi) * C + ci]);
    tile[c * G::PLANE + ty * G::IWP + tx] = v;
  }
}

template <typename T, int STRIDE>
__global__ void __launch_bounds__(NWARP * 32) k_conv_sparse_generic(ConvArgs a, MaskTable lib) {
  using G = Geo<STRIDE>;
  extern __shared__ __align__(16) float smem[];
  float* tile = smem;                                        // [CB][PLANE]
  int* tapoff = reinterpret_cast<int*>(smem + CB * G::PLANE); // [K][4] offsets of the stored taps inside a plane

  // refuse a blob that was packed with other parameters
  {
    const BlobHeader* h = a.hdr;
    bool ok = h->magic == kBlobMagic && h->version == kBlobVersion && h->F == a.F && h->C == a.C && h->K == a.K &&
              h->dtype == a.dtype && h->n_keep == a.n_keep;
    if (ok) for (int j = 0; j < a.K; ++j) ok = ok && (h->masks[j] == lib.m[j]);
    if (!ok) {
      if (threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.y == 0) atomicExch(a.status, PAT_ERR_BLOB);
      return;
    }
  }
  for (int i = threadIdx.x; i < a.K * 4; i += blockDim.x) {
    int bits[4];
    mask_bits(lib.m[i >> 2], bits);
    const int b = bits[i & 3];
    tapoff[i] = (b / 3) * G::IWP + (b % 3);
  }

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int t = blockIdx.x;
  const int tx = t % a.tiles_x; t /= a.tiles_x;
  const int ty = t % a.tiles_y;
  const int n = t / a.tiles_y;
  const int oy0 = ty * TH, ox0 = tx * TW;
  const int iy0 = oy0 * STRIDE - 1, ix0 = ox0 * STRIDE - 1;
  const int q0 = blockIdx.y * FG + warp * RF;

  float acc[RF][TH];
#pragma unroll
  for (int r = 0; r < RF; ++r)
#pragma unroll
    for (int p = 0; p < TH; ++p) acc[r][p] = 0.0f;

  const T* x = static_cast<const T*>(a.x);
  const T* tw4 = static_cast<const T*>(a.tw4);
  const int lane_off = lane * STRIDE;

  for (int cb = 0; cb < a.nct; ++cb) {
    __syncthreads();
    stage_tile<T, STRIDE>(tile, x, n, iy0, ix0, cb * CB, a.H, a.W, a.C);
    __syncthreads();
#pragma unroll
    for (int r = 0; r < RF; ++r) {
      const int q = q0 + r;
      if (q >= a.F) continue;
      const int kb = a.tptr[(size_t)q * (a.nct + 1) + cb], ke = a.tptr[(size_t)q * (a.nct + 1) + cb + 1];
      for (int k = kb; k < ke; ++k) {
        const uint32_t meta = a.tmeta[k];
        const int c = (int)(meta & 0xFFFFu) - cb * CB;
        const int j = (int)(meta >> 16);
        const float* plane = tile + c * G::PLANE + lane_off;
#pragma unroll
        for (int tp = 0; tp < 4; ++tp) {
          const float w = to_f32<T>(tw4[(size_t)k * 4 + tp]);
          const float* src = plane + tapoff[j * 4 + tp];
#pragma unroll
          for (int p = 0; p < TH; ++p) acc[r][p] = fmaf(w, src[p * STRIDE * G::IWP], acc[r][p]);
        }
      }
    }
  }

  T* y = static_cast<T*>(a.y);
  const int ox = ox0 + lane;
  if (ox < a.Wo) {
#pragma unroll
    for (int r = 0; r < RF; ++r) {
      const int q = q0 + r;
      if (q >= a.F) continue;
      const int f = a.perm[q];
#pragma unroll
      for (int p = 0; p < TH; ++p) {
        const int oy = oy0 + p;
        if (oy < a.Ho) y[(((size_t)n * a.Ho + oy) * a.Wo + ox) * a.F + f] = from_f32<T>(acc[r][p]);
      }
    }
  }
}

// Dense layer with few input channels (C <= 16): all nine taps of every kernel.
struct DenseArgs {
  const void* x;
  void* y;
  const float* w;
  int N, H, W, C, F, Ho, Wo, tiles_x, tiles_y;
};

template <typename T, int STRIDE>
__global__ void __launch_bounds__(NWARP * 32) k_conv_dense_small_c(DenseArgs a) {
  using G = Geo<STRIDE>;
  extern __shared__ __align__(16) float smem[];
  float* tile = smem;                       // [CB][PLANE]
  float* wsm = smem + CB * G::PLANE;        // [FG][C][9], rounded to the storage type
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int t = blockIdx.x;
  const int tx = t % a.tiles_x; t /= a.tiles_x;
  const int ty = t % a.tiles_y;
  const int n = t / a.tiles_y;
  const int oy0 = ty * TH, ox0 = tx * TW;
  const int f0 = blockIdx.y * FG;
  for (int i = threadIdx.x; i < FG * a.C * 9; i += blockDim.x) {
    const int f = f0 + i / (a.C * 9);
    wsm[i] = (f < a.F) ? to_f32<T>(from_f32<T>(a.w[(size_t)f * a.C * 9 + i % (a.C * 9)])) : 0.0f;
  }
  stage_tile<T, STRIDE>(tile, static_cast<const T*>(a.x), n, oy0 * STRIDE - 1, ox0 * STRIDE - 1, 0, a.H, a.W, a.C);
  __syncthreads();
  float acc[RF][TH];
#pragma unroll
  for (int r = 0; r < RF; ++r)
#pragma unroll
    for (int p = 0; p < TH; ++p) acc[r][p] = 0.0f;
  for (int c = 0; c < a.C; ++c) {
#pragma unroll
    for (int b = 0; b < 9; ++b) {
      const float* src = tile + c * G::PLANE + (b / 3) * G::IWP + (b % 3) + lane * STRIDE;
      float v[TH];
#pragma unroll
      for (int p = 0; p < TH; ++p) v[p] = src[p * STRIDE * G::IWP];
#pragma unroll
      for (int r = 0; r < RF; ++r) {
        const float w = wsm[((warp * RF + r) * a.C + c) * 9 + b];
#pragma unroll
        for (int p = 0; p < TH; ++p) acc[r][p] = fmaf(w, v[p], acc[r][p]);
      }
    }
  }
  T* y = static_cast<T*>(a.y);
  const int ox = ox0 + lane;
  if (ox < a.Wo) {
#pragma unroll
    for (int r = 0; r < RF; ++r) {
      const int f = f0 + warp * RF + r;
      if (f >= a.F) continue;
#pragma unroll
      for (int p = 0; p < TH; ++p) {
        const int oy = oy0 + p;
        if (oy < a.Ho) y[(((size_t)n * a.Ho + oy) * a.Wo + ox) * a.F + f] = from_f32<T>(acc[r][p]);
      }
    }
  }
}

// Dense first layer of an RGB network (C = 3, stride 1): one output pixel per thread.  The 27 inputs of the
// pixel sit in registers; filters are taken 8 at a time: for each of the 27 kernel entries one warp-uniform
// 16-byte (fp16) or 2 x 16-byte (fp32) shared-memory load brings the entry of 8 filters, followed by 8
// multiply-adds on the same input register; the 8 results leave as one 16-byte (32-byte) store.
template <typename T> struct DenseC3;
template <> struct DenseC3<__half> {
  static __device__ __forceinline__ void mac8(float (&acc)[8], unsigned short in, const void* wrow) {
    const uint4 w = *static_cast<const uint4*>(wrow);
    const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      unsigned short lo, hi;
      asm("mov.b32 {%0,%1}, %2;" : "=h"(lo), "=h"(hi) : "r"(ws[j]));
      asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc[2 * j]) : "h"(in), "h"(lo));
      asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc[2 * j + 1]) : "h"(in), "h"(hi));
    }
  }
  static __device__ __forceinline__ unsigned short load(const __half* p) { return __half_as_ushort(*p); }
  static __device__ __forceinline__ unsigned short zero() { return 0; }
  using In = unsigned short;
  static __device__ __forceinline__ void store8(__half* dst, const float (&acc)[8]) {
    uint4 v;
    v.x = (uint32_t)__half_as_ushort(__float2half_rn(acc[0])) | ((uint32_t)__half_as_ushort(__float2half_rn(acc[1])) << 16);
    v.y = (uint32_t)__half_as_ushort(__float2half_rn(acc[2])) | ((uint32_t)__half_as_ushort(__float2half_rn(acc[3])) << 16);
    v.z = (uint32_t)__half_as_ushort(__float2half_rn(acc[4])) | ((uint32_t)__half_as_ushort(__float2half_rn(acc[5])) << 16);
    v.w = (uint32_t)__half_as_ushort(__float2half_rn(acc[6])) | ((uint32_t)__half_as_ushort(__float2half_rn(acc[7])) << 16);
    *reinterpret_cast<uint4*>(dst) = v;
  }
};
template <> struct DenseC3<float> {
  static __device__ __forceinline__ void mac8(float (&acc)[8], float in, const void* wrow) {
    const float4 a = static_cast<const float4*>(wrow)[0], b = static_cast<const float4*>(wrow)[1];
    acc[0] = fmaf(in, a.x, acc[0]); acc[1] = fmaf(in, a.y, acc[1]); acc[2] = fmaf(in, a.z, acc[2]); acc[3] = fmaf(in, a.w, acc[3]);
    acc[4] = fmaf(in, b.x, acc[4]); acc[5] = fmaf(in, b.y, acc[5]); acc[6] = fmaf(in, b.z, acc[6]); acc[7] = fmaf(in, b.w, acc[7]);
  }
  static __device__ __forceinline__ float load(const float* p) { return *p; }
  static __device__ __forceinline__ float zero() { return 0.0f; }
  using In = float;
  static __device__ __forceinline__ void store8(float* dst, const float (&acc)[8]) {
    reinterpret_cast<float4*>(dst)[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
    reinterpret_cast<float4*>(dst)[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
  }
};

template <typename T>
__global__ void __launch_bounds__(256) k_conv_dense_c3(DenseArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  T* wsm = reinterpret_cast<T*>(smem_raw);            // [F / 8][27][8]: entry k of 8 consecutive filters
  using D = DenseC3<T>;
  for (int i = threadIdx.x; i < a.F * 27; i += blockDim.x) {
    const int f = i / 27, k = i % 27;                 // k = 9 * c + 3 * r + s  (weights are [F][3][3][3])
    wsm[((f >> 3) * 27 + k) * 8 + (f & 7)] = from_f32<T>(a.w[i]);
  }
  __syncthreads();
  const long long pix = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long npix = (long long)a.N * a.H * a.W;
  if (pix >= npix) return;
  const int x = (int)(pix % a.W);
  const int y = (int)((pix / a.W) % a.H);
  const int n = (int)(pix / ((long long)a.W * a.H));
  const T* xin = static_cast<const T*>(a.x);
  typename D::In in[27];
#pragma unroll
  for (int r = 0; r < 3; ++r)
#pragma unroll
    for (int s2 = 0; s2 < 3; ++s2) {
      const int yi = y + r - 1, xi = x + s2 - 1;
      const bool ok = yi >= 0 && yi < a.H && xi >= 0 && xi < a.W;
      const T* src = xin + (((size_t)n * a.H + (ok ? yi : 0)) * a.W + (ok ? xi : 0)) * 3;
#pragma unroll
      for (int c = 0; c < 3; ++c) in[9 * c + 3 * r + s2] = ok ? D::load(src + c) : D::zero();
    }
  T* yout = static_cast<T*>(a.y) + (size_t)pix * a.F;
  for (int fb = 0; fb < a.F / 8; ++fb) {
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    const T* wrow = wsm + (size_t)fb * 27 * 8;
#pragma unroll
    for (int k = 0; k < 27; ++k) D::mac8(acc, in[k], wrow + k * 8);
    D::store8(yout + fb * 8, acc);
  }
}

template <typename KernelT>
int prepare(KernelT kernel, size_t smem) {
  if (smem > 48 * 1024)
    return check_cuda(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem), "set shared memory size");
  return PAT_OK;
}

template <typename T, int STRIDE>
int launch_sparse(const ConvArgs& a, const MaskTable& lib, cudaStream_t st) {
  using G = Geo<STRIDE>;
  const size_t smem = sizeof(float) * CB * G::PLANE + sizeof(int) * 4 * (size_t)a.K;
  if (int rc = prepare(k_conv_sparse_generic<T, STRIDE>, smem)) return rc;
  const dim3 grid((unsigned)((size_t)a.N * a.tiles_x * a.tiles_y), (unsigned)((a.F + FG - 1) / FG));
  k_conv_sparse_generic<T, STRIDE><<<grid, NWARP * 32, smem, st>>>(a, lib);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "pat_conv3x3 launch");
}

template <typename T, int STRIDE>
int launch_dense(const DenseArgs& a, cudaStream_t st) {
  using G = Geo<STRIDE>;
  const size_t smem = sizeof(float) * (CB * G::PLANE + (size_t)FG * a.C * 9);
  if (int rc = prepare(k_conv_dense_small_c<T, STRIDE>, smem)) return rc;
  const dim3 grid((unsigned)((size_t)a.N * a.tiles_x * a.tiles_y), (unsigned)((a.F + FG - 1) / FG));
  k_conv_dense_small_c<T, STRIDE><<<grid, NWARP * 32, smem, st>>>(a);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "pat_conv3x3_dense launch");
}

}  // namespace

int conv_generic(const void* blob, int F, int C, const uint16_t* masks, int K, int64_t n_keep, int dtype,
                 const void* x, void* y, int N, int H, int W, int stride, cudaStream_t st) {
  const BlobLayout L = blob_layout(F, C, K, n_keep, dtype);
  const char* b = static_cast<const char*>(blob);
  ConvArgs a;
  a.x = x; a.y = y;
  a.hdr = reinterpret_cast<const BlobHeader*>(b);
  a.perm = reinterpret_cast<const int32_t*>(b + L.xfilt);   // execution order of the filters
  a.tptr = reinterpret_cast<const int32_t*>(b + L.tptr);
  a.tmeta = reinterpret_cast<const uint32_t*>(b + L.tmeta);
  a.tw4 = b + L.tw4;
  a.status = status_word();
  if (!a.status) return set_error(PAT_ERR_CUDA, "pat_conv3x3: cannot resolve the status word");
  a.N = N; a.H = H; a.W = W; a.C = C; a.F = F; a.K = K; a.nct = L.nct; a.dtype = dtype; a.n_keep = n_keep;
  a.Ho = (H - 1) / stride + 1; a.Wo = (W - 1) / stride + 1;
  a.tiles_x = (a.Wo + TW - 1) / TW; a.tiles_y = (a.Ho + TH - 1) / TH;
  MaskTable lib;
  for (int j = 0; j <= kMaxK; ++j) lib.m[j] = (j < K) ? masks[j] : (uint16_t)0;
  lib.K = K;
  if (dtype == PAT_F16) return stride == 1 ? launch_sparse<__half, 1>(a, lib, st) : launch_sparse<__half, 2>(a, lib, st);
  return stride == 1 ? launch_sparse<float, 1>(a, lib, st) : launch_sparse<float, 2>(a, lib, st);
}

}  // namespace pat

namespace pat {
bool conv_dense_c3_mma_supported(int F, int C, int dtype, int stride);
int conv_dense_c3_mma(const float* w, const void* x, void* y, int N, int H, int W, cudaStream_t st);
}

using namespace pat;

extern "C" int pat_conv3x3_dense(const float* w, int F, int C, int dtype, const void* x, void* y,
                                 int N, int H, int W, int stride, void* stream) {
  if (!w || !x || !y) return set_error(PAT_ERR_INVALID_ARG, "pat_conv3x3_dense: null pointer");
  if (dtype != PAT_F32 && dtype != PAT_F16) return set_error(PAT_ERR_DTYPE, "pat_conv3x3_dense: dtype %d", dtype);
  if (F < 1 || F > 65535 || C < 1 || C > 16) return set_error(PAT_ERR_SHAPE, "pat_conv3x3_dense: needs 1 <= C <= 16 and 1 <= F <= 65535 (F=%d C=%d)", F, C);
  if (N < 1 || H < 1 || W < 1) return set_error(PAT_ERR_SHAPE, "pat_conv3x3_dense: N, H, W must be positive");
  if (stride != 1 && stride != 2) return set_error(PAT_ERR_INVALID_ARG, "pat_conv3x3_dense: stride %d", stride);
  if (!aligned(x, 16) || !aligned(y, 16) || !aligned(w, 4)) return set_error(PAT_ERR_ALIGN, "pat_conv3x3_dense: x and y must be 16-byte aligned");
  DenseArgs a;
  a.x = x; a.y = y; a.w = w; a.N = N; a.H = H; a.W = W; a.C = C; a.F = F;
  a.Ho = (H - 1) / stride + 1; a.Wo = (W - 1) / stride + 1;
  a.tiles_x = (a.Wo + TW - 1) / TW; a.tiles_y = (a.Ho + TH - 1) / TH;
  if ((size_t)N * a.tiles_x * a.tiles_y > 0x7FFFFFFFull) return set_error(PAT_ERR_SHAPE, "pat_conv3x3_dense: too many tiles");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (conv_dense_c3_mma_supported(F, C, dtype, stride)) return conv_dense_c3_mma(w, x, y, N, H, W, st);
  if (C == 3 && stride == 1 && F % 8 == 0 && (size_t)F * 27 * 4 <= 48 * 1024) {
    const long long npix = (long long)N * H * W;
    const unsigned blocks = (unsigned)((npix + 255) / 256);
    if (dtype == PAT_F16) k_conv_dense_c3<__half><<<blocks, 256, (size_t)F * 27 * 2, st>>>(a);
    else k_conv_dense_c3<float><<<blocks, 256, (size_t)F * 27 * 4, st>>>(a);
    count_launches(1);
    return check_cuda(cudaGetLastError(), "pat_conv3x3_dense launch");
  }
  if (dtype == PAT_F16) return stride == 1 ? launch_dense<__half, 1>(a, st) : launch_dense<__half, 2>(a, st);
  return stride == 1 ? launch_dense<float, 1>(a, st) : launch_dense<float, 2>(a, st);
}
