// What stands between two convolution layers of the models of Section 7 (VGG-16, ResNet-50): the rectifier
// max(x, 0) and, after some layers, 2x2 max pooling with stride 2.  NHWC, fp16 or fp32, one pass: every thread takes
// 16 bytes of channels of one output pixel (eight fp16 or four fp32 values), reads the one or four input pixels it
// depends on and writes the result.  Plain streaming work: the bytes are read once and written once.
#include <cuda_fp16.h>
#include "common.cuh"

namespace pat {
namespace {

__device__ __forceinline__ uint4 relu_max(uint4 a, uint4 b, bool f16) {
  uint4 r;
  if (f16) {
    const __half2 z = __float2half2_rn(0.0f);
    const __half2* pa = reinterpret_cast<const __half2*>(&a);
    const __half2* pb = reinterpret_cast<const __half2*>(&b);
    __half2* pr = reinterpret_cast<__half2*>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) pr[i] = __hmax2(__hmax2(pa[i], pb[i]), z);
  } else {
    const float* pa = reinterpret_cast<const float*>(&a);
    const float* pb = reinterpret_cast<const float*>(&b);
    float* pr = reinterpret_cast<float*>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) pr[i] = fmaxf(fmaxf(pa[i], pb[i]), 0.0f);
  }
  return r;
}

// chunks: 16-byte chunks per pixel (C * element size / 16).  One thread per (output pixel, chunk), chunks fastest.
template <bool POOL>
__global__ void __launch_bounds__(256) k_relu_maxpool(const uint4* __restrict__ x, uint4* __restrict__ y, long long n_out,
                                                      int Ho, int Wo, int W, int chunks, bool f16) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < n_out; t += stride) {
    const int ck = (int)(t % chunks);
    const long long px = t / chunks;                         // (n, yo, xo) flattened
    if (!POOL) {
      const uint4 v = __ldcs(x + t);
      __stcs(y + t, relu_max(v, v, f16));
    } else {
      const int xo = (int)(px % Wo);
      const long long row = px / Wo;                         // n * Ho + yo  ->  input row 2 * row (H = 2 Ho)
      const long long i00 = ((2 * row) * W + 2 * xo) * chunks + ck;
      const uint4 a = __ldcs(x + i00), b = __ldcs(x + i00 + chunks);
      const uint4 c = __ldcs(x + i00 + (long long)W * chunks), d = __ldcs(x + i00 + (long long)W * chunks + chunks);
      __stcs(y + t, relu_max(relu_max(a, b, f16), relu_max(c, d, f16), f16));
    }
  }
}

// Any channel count (no 16-byte chunks): one thread per output element.
template <typename T>
__global__ void __launch_bounds__(256) k_relu_maxpool_scalar(const T* __restrict__ x, T* __restrict__ y, long long n_out,
                                                             int Ho, int Wo, int W, int C, int pool) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < n_out; t += stride) {
    const int c = (int)(t % C);
    const long long px = t / C;
    float m = 0.0f;
    if (!pool) m = fmaxf((float)x[t], 0.0f);
    else {
      const int xo = (int)(px % Wo);
      const long long row = px / Wo;
      const long long i00 = ((2 * row) * W + 2 * xo) * C + c;
      m = fmaxf(fmaxf(fmaxf((float)x[i00], (float)x[i00 + C]), fmaxf((float)x[i00 + (long long)W * C], (float)x[i00 + (long long)W * C + C])), 0.0f);
    }
    y[t] = (T)m;                                             // the maximum of representable values: exact
  }
}

}  // namespace
}  // namespace pat

using namespace pat;

extern "C" int pat_relu_maxpool(const void* x, int dtype, int N, int H, int W, int C, int pool, void* y, void* stream) {
  if (!x || !y) return set_error(PAT_ERR_INVALID_ARG, "pat_relu_maxpool: null pointer");
  if (dtype != PAT_F32 && dtype != PAT_F16) return set_error(PAT_ERR_DTYPE, "pat_relu_maxpool: dtype %d", dtype);
  if (N < 1 || H < 1 || W < 1 || C < 1) return set_error(PAT_ERR_SHAPE, "pat_relu_maxpool: N, H, W, C must be positive");
  if (pool != 0 && pool != 1) return set_error(PAT_ERR_INVALID_ARG, "pat_relu_maxpool: pool %d (0 or 1)", pool);
  if (pool && ((H & 1) || (W & 1))) return set_error(PAT_ERR_SHAPE, "pat_relu_maxpool: 2x2 pooling needs even H and W (%d x %d)", H, W);
  const int elem = dtype == PAT_F16 ? 2 : 4;
  if (!aligned(x, elem) || !aligned(y, elem)) return set_error(PAT_ERR_ALIGN, "pat_relu_maxpool: misaligned buffer");
  const int Ho = pool ? H / 2 : H, Wo = pool ? W / 2 : W;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const bool vec = ((size_t)C * elem) % 16 == 0 && aligned(x, 16) && aligned(y, 16);
  const long long n_out = (long long)N * Ho * Wo * (vec ? (C * elem / 16) : C);
  const long long blocks = (n_out + 255) / 256;
  const unsigned grid = (unsigned)(blocks < 148 * 64 ? blocks : 148 * 64);   // grid-stride beyond that
  if (vec) {
    const int chunks = C * elem / 16;
    if (pool) k_relu_maxpool<true><<<grid, 256, 0, st>>>(static_cast<const uint4*>(x), static_cast<uint4*>(y), n_out, Ho, Wo, W, chunks, dtype == PAT_F16);
    else k_relu_maxpool<false><<<grid, 256, 0, st>>>(static_cast<const uint4*>(x), static_cast<uint4*>(y), n_out, Ho, Wo, W, chunks, dtype == PAT_F16);
  } else if (dtype == PAT_F16) {
    k_relu_maxpool_scalar<__half><<<grid, 256, 0, st>>>(static_cast<const __half*>(x), static_cast<__half*>(y), n_out, Ho, Wo, W, C, pool);
  } else {
    k_relu_maxpool_scalar<float><<<grid, 256, 0, st>>>(static_cast<const float*>(x), static_cast<float*>(y), n_out, Ho, Wo, W, C, pool);
  }
  count_launches(1);
  return check_cuda(cudaGetLastError(), "pat_relu_maxpool launch");
}
