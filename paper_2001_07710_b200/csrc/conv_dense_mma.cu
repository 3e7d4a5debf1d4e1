// Dense 3x3 convolution of a 3-channel image with 64 filters, fp16 storage / fp32 accumulation, stride 1 (the first
// layer of VGG-16, which is not pruned).  This layer is a dense contraction - every output pixel is the product of
// its 27 input values with a 27 x 64 weight matrix - so it runs on the tensor cores (mma.sync m16n8k16, fp16
// inputs, fp32 accumulators) and is bound by writing the output (64 channels per pixel against 3 read).
//
// A block stages an (8 + 2) x (32 + 2) pixel window of the NHWC image in shared memory (zero outside the image:
// the padding).  For kernel row r the nine values (column s, channel c) that pixel x needs are nine consecutive
// halves of staged row y + r, starting at pixel x - 1: the A operand of one k-step is read straight from the
// staged rows, no im2col copy.  K is laid out as three k-steps of 16 (one per kernel row; slots 9-15 hold zero
// weights, and the A values of those slots are forced to zero as well, so nothing outside the 3x3 window can
// reach an output).  A warp owns 16 consecutive pixels of a row per step and all 64 filters (8 n-tiles); the
// weight fragments (48 registers) are loaded once per block.  The columns of the n-tiles are assigned to output
// channels so that a thread ends up with 2 x 8 adjacent channels of a pixel and the four threads of a pixel write
// two 64-byte runs.
#include "common.cuh"

namespace pat {
namespace densemma {

constexpr int TW = 32, TH = 8;             // output pixels of a block
constexpr int NTHREADS = 128;              // four warps: warp w owns tile rows 2w and 2w + 1
constexpr int ROWP = (TW + 2) * 3 + 2;     // halves per staged row (102 used)
constexpr int F = 64;

struct Args {
  const float* w;      // [64][3][3][3] fp32
  const __half* x;     // NHWC, C = 3
  __half* y;           // NHWC, F = 64
  int N, H, W;
  int tiles_x, tiles_y;
  long long n_tiles;
};

__device__ __forceinline__ uint32_t pack2(__half lo, __half hi) {
  return (uint32_t)__half_as_ushort(lo) | ((uint32_t)__half_as_ushort(hi) << 16);
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// Output channel computed by column `col` (0..7) of n-tile `jt` (0..7): thread t of a pixel (col = 2t, 2t + 1)
// gets channels 8t .. 8t + 7 from n-tiles 0-3 and 32 + 8t .. 32 + 8t + 7 from n-tiles 4-7.
__device__ __forceinline__ int channel_of(int jt, int col) {
  return (jt < 4 ? 0 : 32) + 8 * (col >> 1) + 2 * (jt & 3) + (col & 1);
}

// WORDS (W even): the window is moved as aligned 4-byte words.  The first half of a staged row is then the half in
// front of pixel x0 - 1 (that pixel starts at an odd half index of the image whenever W and x0 are even), pixel
// boundaries of the window's edges fall on word boundaries, and a row of the window is 52 consecutive words.
template <bool WORDS>
__global__ void __launch_bounds__(NTHREADS, 4) k_conv_dense_c3_mma(const Args a) {
  __shared__ __align__(16) __half tile[(TH + 2) * ROWP];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;

  // weight fragments: k-step r, n-tile jt: b0 = B[k = 2t, 2t + 1][n = g], b1 = B[k = 2t + 8, 2t + 9][n = g], with
  // B[k = 3 s + c][n] = w[channel_of(jt, n)][c][r][s] for k < 9 and zero above
  uint32_t bw[3][8][2];
#pragma unroll
  for (int r = 0; r < 3; ++r)
#pragma unroll
    for (int jt = 0; jt < 8; ++jt) {
      const float* wf = a.w + (size_t)channel_of(jt, g) * 27;
      auto wk = [&](int k) { return k < 9 ? __float2half_rn(__ldg(wf + 9 * (k % 3) + 3 * r + k / 3)) : __float2half_rn(0.0f); };
      bw[r][jt][0] = pack2(wk(2 * t), wk(2 * t + 1));
      bw[r][jt][1] = pack2(wk(2 * t + 8), wk(2 * t + 9));
    }

  // the input window of a tile travels through registers: the next tile's loads are in flight while this one is computed
  // (staged rows start one half early in both variants: half 0 of a row is unused, pixel x0 - 1 begins at half 1)
  constexpr int RW = ROWP / 2;             // words per staged row (52)
  constexpr int WIN = WORDS ? (TH + 2) * RW : (TH + 2) * (TW + 2) * 3, PER_THREAD = (WIN + NTHREADS - 1) / NTHREADS;
  static_assert(ROWP % 2 == 0 && ROWP >= (TW + 2) * 3 + 2, "a staged row holds the unused first half, 34 pixels and a last half");
  uint32_t win[PER_THREAD];                // WORDS: a word each; otherwise one half each
  auto load_window = [&](long long tl) {
    const int tx = (int)(tl % a.tiles_x), ty = (int)((tl / a.tiles_x) % a.tiles_y), n = (int)(tl / ((long long)a.tiles_x * a.tiles_y));
#pragma unroll
    for (int q = 0; q < PER_THREAD; ++q) {
      const int i = (int)threadIdx.x + q * NTHREADS;
      win[q] = 0u;
      if constexpr (WORDS) {
        // word j of a row = halves 2 j - 1, 2 j of the window row; both belong to pixels on the same side of the
        // image's edge (or one of them is an unused half), so the pixel of half 2 j decides (half 101 for the last word)
        const int row = i / RW, j = i % RW;
        const int yy = ty * TH - 1 + row, xx = tx * TW - 1 + (j == RW - 1 ? TW + 1 : (2 * j) / 3);
        if (i < WIN && yy >= 0 && yy < a.H && xx >= 0 && xx < a.W) {
          const long long h0 = (((long long)n * a.H + yy) * a.W + tx * TW - 1) * 3 - 1;   // even: the row's first word
          win[q] = __ldg(reinterpret_cast<const uint32_t*>(a.x + h0) + j);
        }
      } else {
        const int row = i / ((TW + 2) * 3), rem = i % ((TW + 2) * 3);
        const int yy = ty * TH - 1 + row, xx = tx * TW - 1 + rem / 3;
        if (i < WIN && yy >= 0 && yy < a.H && xx >= 0 && xx < a.W)
          win[q] = __half_as_ushort(a.x[(((size_t)n * a.H + yy) * a.W + xx) * 3 + rem % 3]);
      }
    }
  };
  if ((long long)blockIdx.x < a.n_tiles) load_window(blockIdx.x);
  for (long long tl = blockIdx.x; tl < a.n_tiles; tl += gridDim.x) {
    const int tx = (int)(tl % a.tiles_x), ty = (int)((tl / a.tiles_x) % a.tiles_y), n = (int)(tl / ((long long)a.tiles_x * a.tiles_y));
    const int x0 = tx * TW, y0 = ty * TH;
    __syncthreads();                       // the previous tile has been read
#pragma unroll
    for (int q = 0; q < PER_THREAD; ++q) {
      const int i = (int)threadIdx.x + q * NTHREADS;
      if constexpr (WORDS) {
        if (i < WIN) reinterpret_cast<uint32_t*>(tile)[i] = win[q];
      } else {
        if (i < WIN) tile[(i / ((TW + 2) * 3)) * ROWP + 1 + i % ((TW + 2) * 3)] = __ushort_as_half((unsigned short)win[q]);
      }
    }
    __syncthreads();
    if (tl + gridDim.x < a.n_tiles) load_window(tl + gridDim.x);

#pragma unroll 1
    for (int sub = 0; sub < 4; ++sub) {    // the warp's four groups of 16 pixels
      const int ry = 2 * warp + (sub >> 1), px0 = (sub & 1) * 16;
      float acc[8][4];
#pragma unroll
      for (int jt = 0; jt < 8; ++jt) { acc[jt][0] = 0.f; acc[jt][1] = 0.f; acc[jt][2] = 0.f; acc[jt][3] = 0.f; }
#pragma unroll
      for (int r = 0; r < 3; ++r) {
        // A[m][k] = tile[ry + r][(px0 + m) * 3 + k] for k < 9, zero above
        const __half* rowp = tile + (ry + r) * ROWP + 1 + px0 * 3;
        const __half z = __float2half_rn(0.0f);
        uint32_t af[4];
        af[0] = pack2(rowp[g * 3 + 2 * t], rowp[g * 3 + 2 * t + 1]);
        af[1] = pack2(rowp[(g + 8) * 3 + 2 * t], rowp[(g + 8) * 3 + 2 * t + 1]);
        af[2] = t == 0 ? pack2(rowp[g * 3 + 8], z) : 0u;
        af[3] = t == 0 ? pack2(rowp[(g + 8) * 3 + 8], z) : 0u;
#pragma unroll
        for (int jt = 0; jt < 8; ++jt) mma16816(acc[jt], af, bw[r][jt][0], bw[r][jt][1]);
      }
      // c0, c1 = D[g][2t, 2t + 1], c2, c3 = D[g + 8][2t, 2t + 1]
      const int yy = y0 + ry;
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int xx = x0 + px0 + g + 8 * hh;
        if (yy < a.H && xx < a.W) {
          __half* dst = a.y + (((size_t)n * a.H + yy) * a.W + xx) * F + 8 * t;
#pragma unroll
          for (int part = 0; part < 2; ++part) {
            uint32_t v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
              v[j] = pack2(__float2half_rn(acc[4 * part + j][2 * hh]), __float2half_rn(acc[4 * part + j][2 * hh + 1]));
            *reinterpret_cast<uint4*>(dst + 32 * part) = make_uint4(v[0], v[1], v[2], v[3]);
          }
        }
      }
    }
  }
}

}  // namespace densemma

bool conv_dense_c3_mma_supported(int F, int C, int dtype, int stride) {
  return F == densemma::F && C == 3 && dtype == PAT_F16 && stride == 1;
}

int conv_dense_c3_mma(const float* w, const void* x, void* y, int N, int H, int W, cudaStream_t st) {
  using namespace densemma;
  Args a;
  a.w = w; a.x = static_cast<const __half*>(x); a.y = static_cast<__half*>(y);
  a.N = N; a.H = H; a.W = W;
  a.tiles_x = (W + TW - 1) / TW; a.tiles_y = (H + TH - 1) / TH;
  a.n_tiles = (long long)N * a.tiles_x * a.tiles_y;
  static thread_local DeviceSlot slots[kMaxDevices];
  DeviceSlot* dv = device_slot(slots);
  if (!dv) return set_error(PAT_ERR_CUDA, "pat_conv3x3_dense: cannot query the current device");
  const int sm_count = dv->sms;
  const long long want = (long long)sm_count * 8;         // eight resident blocks of four warps per SM
  const unsigned grid = (unsigned)(a.n_tiles < want ? a.n_tiles : want);
  if (W % 2 == 0) k_conv_dense_c3_mma<true><<<grid, NTHREADS, 0, st>>>(a);
  else k_conv_dense_c3_mma<false><<<grid, NTHREADS, 0, st>>>(a);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "pat_conv3x3_dense launch");
}

}  // namespace pat
