// pat_conv3x3: argument validation and choice of the kernel for a layer shape.
#include "common.cuh"

namespace pat {
int conv_generic(const void* blob, int F, int C, const uint16_t* masks, int K, int64_t n_keep, int dtype,
                 const void* x, void* y, int N, int H, int W, int stride, cudaStream_t st);
bool conv_f16_fast_supported(int F, int C, const uint16_t* masks, int K, int dtype, int N, int H, int W, int stride);
int conv_f16_fast(const void* blob, int F, int C, const uint16_t* masks, int K, int64_t n_keep,
                  const void* x, void* y, int N, int H, int W, cudaStream_t st);
bool conv_f16_img_supported(int F, int C, int dtype, int N, int H, int W, int stride);
size_t conv_f16_img_workspace(int F, int C, int dtype, int N, int H, int W, int stride);
int conv_f16_img(const void* blob, int F, int C, const uint16_t* masks, int K, int64_t n_keep,
                 const void* x, void* y, int N, int H, int W, int stride, int relu, void* workspace, cudaStream_t st);
int conv_f16_img_debug(int what, long long value);
size_t conv_f32_img_workspace(int F, int C, int dtype, int N, int H, int W, int stride);
int conv_f32_img(const void* blob, int F, int C, const uint16_t* masks, int K, int64_t n_keep,
                 const void* x, void* y, int N, int H, int W, int stride, int relu, void* workspace, cudaStream_t st);
}

using namespace pat;

extern "C" int pat_debug_set(int what, long long value) { return conv_f16_img_debug(what, value); }

static int check_conv_args(const void* blob, int F, int C, const uint16_t* masks, int K, int64_t n_keep, int dtype,
                           const void* x, const void* y, int N, int H, int W, int stride) {
  if (!blob || !x || !y) return set_error(PAT_ERR_INVALID_ARG, "pat_conv3x3: null pointer");
  if (F < 1 || C < 1 || F > 65535 || C > 65535) return set_error(PAT_ERR_SHAPE, "pat_conv3x3: F=%d C=%d outside 1..65535", F, C);
  if (int rc = check_library(masks, K)) return rc;
  if (dtype != PAT_F32 && dtype != PAT_F16) return set_error(PAT_ERR_DTYPE, "pat_conv3x3: dtype %d", dtype);
  if (n_keep < 0 || n_keep > (int64_t)F * C) return set_error(PAT_ERR_INVALID_ARG, "pat_conv3x3: n_keep outside 0..F*C");
  if (N < 1 || H < 1 || W < 1) return set_error(PAT_ERR_SHAPE, "pat_conv3x3: N, H, W must be positive");
  if (stride != 1 && stride != 2) return set_error(PAT_ERR_INVALID_ARG, "pat_conv3x3: stride %d (1 or 2)", stride);
  if (!aligned(blob, 256)) return set_error(PAT_ERR_ALIGN, "pat_conv3x3: blob must be 256-byte aligned");
  if (!aligned(x, 16) || !aligned(y, 16)) return set_error(PAT_ERR_ALIGN, "pat_conv3x3: x and y must be 16-byte aligned");
  const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
  if ((size_t)N * ((Ho + 7) / 8) * ((Wo + 31) / 32) > 0x7FFFFFFFull) return set_error(PAT_ERR_SHAPE, "pat_conv3x3: too many tiles");
  return PAT_OK;
}

extern "C" int pat_conv3x3(const void* blob, int F, int C, const uint16_t* masks, int K, int64_t n_keep,
                           int dtype, const void* x, void* y, int N, int H, int W, int stride, void* stream) {
  if (int rc = check_conv_args(blob, F, C, masks, K, n_keep, dtype, x, y, N, H, W, stride)) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (conv_f16_fast_supported(F, C, masks, K, dtype, N, H, W, stride))
    return conv_f16_fast(blob, F, C, masks, K, n_keep, x, y, N, H, W, st);
  return conv_generic(blob, F, C, masks, K, n_keep, dtype, x, y, N, H, W, stride, st);
}

extern "C" size_t pat_conv3x3_workspace(int F, int C, int dtype, int N, int H, int W, int stride) {
  if (F < 1 || C < 1 || N < 1 || H < 1 || W < 1) return 0;
  return dtype == PAT_F32 ? conv_f32_img_workspace(F, C, dtype, N, H, W, stride) : conv_f16_img_workspace(F, C, dtype, N, H, W, stride);
}

extern "C" int pat_relu_maxpool(const void* x, int dtype, int N, int H, int W, int C, int pool, void* y, void* stream);

extern "C" int pat_conv3x3_ws_act(const void* blob, int F, int C, const uint16_t* masks, int K, int64_t n_keep,
                                  int dtype, const void* x, void* y, int N, int H, int W, int stride, int act,
                                  void* workspace, size_t workspace_bytes, void* stream) {
  if (act < 0 || act > 2) return set_error(PAT_ERR_INVALID_ARG, "pat_conv3x3_ws_act: act %d (0: none, 1: rectifier, 2: rectifier and 2 x 2 max pooling)", act);
  if (int rc = check_conv_args(blob, F, C, masks, K, n_keep, dtype, x, y, N, H, W, stride)) return rc;
  const size_t need = pat_conv3x3_workspace(F, C, dtype, N, H, W, stride);
  // pooling happens inside a thread tile of the workspace kernels: no other kernel writes a pooled image (y is too
  // small for the full-size result, so there is no two-pass substitute without memory of the library's own)
  if (act == 2 && (need == 0 || stride != 1 || (H & 1) || (W & 1)))
    return set_error(PAT_ERR_SHAPE, "pat_conv3x3_ws_act: act 2 needs a layer the workspace kernels cover, stride 1, even H and W "
                                    "(otherwise: act 1, then pat_relu_maxpool)");
  if (need == 0) {
    // a layer the workspace kernels do not cover: the plain convolution, then the rectifier in place
    if (int rc = pat_conv3x3(blob, F, C, masks, K, n_keep, dtype, x, y, N, H, W, stride, stream)) return rc;
    if (!act) return PAT_OK;
    return pat_relu_maxpool(y, dtype, N, (H - 1) / stride + 1, (W - 1) / stride + 1, F, 0, y, stream);
  }
  if (!workspace || workspace_bytes < need)
    return set_error(PAT_ERR_WORKSPACE, "pat_conv3x3_ws: workspace has %zu bytes, needs %zu", workspace_bytes, need);
  if (!aligned(workspace, 256)) return set_error(PAT_ERR_ALIGN, "pat_conv3x3_ws: workspace must be 256-byte aligned");
  if (dtype == PAT_F32) return conv_f32_img(blob, F, C, masks, K, n_keep, x, y, N, H, W, stride, act, workspace, reinterpret_cast<cudaStream_t>(stream));
  return conv_f16_img(blob, F, C, masks, K, n_keep, x, y, N, H, W, stride, act, workspace, reinterpret_cast<cudaStream_t>(stream));
}

extern "C" int pat_conv3x3_ws(const void* blob, int F, int C, const uint16_t* masks, int K, int64_t n_keep,
                              int dtype, const void* x, void* y, int N, int H, int W, int stride,
                              void* workspace, size_t workspace_bytes, void* stream) {
  return pat_conv3x3_ws_act(blob, F, C, masks, K, n_keep, dtype, x, y, N, H, W, stride, 0, workspace, workspace_bytes, stream);
}
