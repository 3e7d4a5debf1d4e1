// pat_measure_fma_peak: the multiply-add rate of the device, measured with the instructions the convolution kernels
// use.  It is the denominator of their roofline (2 flop x 128 fp32 lanes x SMs x clock on paper); measuring it on
// the spot shows what that figure is worth at the clock the device actually runs at.
#include "common.cuh"

namespace pat {
namespace {

constexpr int kChains = 16;        // independent accumulators per thread (the FMA latency is 4 cycles)
constexpr int kInner = 64;         // multiply-adds per chain and loop trip

// kind 0: fma.rn.f32 (fp32 operands); kind 1: fma.rn.f32.f16 (fp16 operands, fp32 accumulator), the instruction of
// the fp16 convolution kernels.  Operands come from memory so that nothing folds at compile time.
template <int KIND>
__global__ void __launch_bounds__(256) k_fma_peak(const float* __restrict__ in, float* __restrict__ out, int trips) {
  float acc[kChains];
  const float a = in[threadIdx.x & 31], b = in[32 + (threadIdx.x & 31)];
  const unsigned short ha = __half_as_ushort(__float2half_rn(a)), hb = __half_as_ushort(__float2half_rn(b));
#pragma unroll
  for (int c = 0; c < kChains; ++c) acc[c] = a + (float)c;
  for (int t = 0; t < trips; ++t) {
#pragma unroll
    for (int i = 0; i < kInner; ++i)
#pragma unroll
      for (int c = 0; c < kChains; ++c) {
        if (KIND == 0) asm volatile("fma.rn.f32 %0, %1, %2, %0;" : "+f"(acc[c]) : "f"(a), "f"(b));
        else asm volatile("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc[c]) : "h"(ha), "h"(hb));
      }
  }
  float s = 0.0f;
#pragma unroll
  for (int c = 0; c < kChains; ++c) s += acc[c];
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

}  // namespace
}  // namespace pat

using namespace pat;

extern "C" int pat_measure_fma_peak(int kind, void* scratch, size_t scratch_bytes, double* tflops_out, void* stream) {
  if (!scratch || !tflops_out) return set_error(PAT_ERR_INVALID_ARG, "pat_measure_fma_peak: null pointer");
  if (kind != 0 && kind != 1) return set_error(PAT_ERR_INVALID_ARG, "pat_measure_fma_peak: kind %d (0 or 1)", kind);
  static thread_local DeviceSlot slots[kMaxDevices];
  DeviceSlot* dv = device_slot(slots);
  if (!dv) return set_error(PAT_ERR_CUDA, "pat_measure_fma_peak: cannot query the current device");
  const int blocks = dv->sms * 8, threads = 256, trips = 512;
  const size_t need = 256 + sizeof(float) * (size_t)blocks * threads;
  if (scratch_bytes < need) return set_error(PAT_ERR_WORKSPACE, "pat_measure_fma_peak: scratch has %zu bytes, needs %zu", scratch_bytes, need);
  if (!aligned(scratch, 256)) return set_error(PAT_ERR_ALIGN, "pat_measure_fma_peak: scratch must be 256-byte aligned");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  float* in = static_cast<float*>(scratch);
  float* out = in + 64;
  float host_in[64];
  for (int i = 0; i < 64; ++i) host_in[i] = 1.0f + 1e-3f * (float)i;
  if (int rc = check_cuda(cudaMemcpyAsync(in, host_in, sizeof(host_in), cudaMemcpyHostToDevice, st), "pat_measure_fma_peak copy")) return rc;
  cudaEvent_t e0, e1;
  if (int rc = check_cuda(cudaEventCreate(&e0), "cudaEventCreate")) return rc;
  if (int rc = check_cuda(cudaEventCreate(&e1), "cudaEventCreate")) { cudaEventDestroy(e0); return rc; }
  double best = 0.0;
  int rc = PAT_OK;
  for (int rep = 0; rep < 4 && rc == PAT_OK; ++rep) {        // first repetition warms up
    cudaEventRecord(e0, st);
    if (kind == 0) k_fma_peak<0><<<blocks, threads, 0, st>>>(in, out, trips);
    else k_fma_peak<1><<<blocks, threads, 0, st>>>(in, out, trips);
    cudaEventRecord(e1, st);
    count_launches(1);
    rc = check_cuda(cudaEventSynchronize(e1), "pat_measure_fma_peak");
    float ms = 0.0f;
    if (rc == PAT_OK) rc = check_cuda(cudaEventElapsedTime(&ms, e0, e1), "cudaEventElapsedTime");
    const double flop = 2.0 * kChains * kInner * (double)trips * blocks * threads;
    if (rc == PAT_OK && rep > 0 && ms > 0.0f) best = flop / (ms * 1e-3) / 1e12 > best ? flop / (ms * 1e-3) / 1e12 : best;
  }
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (rc == PAT_OK) *tflops_out = best;
  return rc;
}
