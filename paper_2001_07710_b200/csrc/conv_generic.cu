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
  if (dtype == PAT_F16) return stride == 1 ? launch_dense<__half, 1>(a, st) : launch_dense<__half, 2>(a, st);
  return stride == 1 ? launch_dense<float, 1>(a, st) : launch_dense<float, 2>(a, st);
}
