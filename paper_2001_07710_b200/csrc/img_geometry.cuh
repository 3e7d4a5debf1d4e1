// Geometry and work planning shared by the two workspace convolution paths (conv_f16_img.cu, conv_f32_img.cu): how a
// batch of images is cut into regions of 8 x 4 thread tiles, how regions and filter groups make work items, and how
// the items of a last, mostly idle round are cut along the input channels.  The two paths differ in what a ring
// stage holds (16 fp16 or 8 fp32 channels) and in their kernels, not in any of this.
#pragma once
#include <algorithm>
#include "f16_tile.cuh"

namespace pat {
namespace imggeo {
using namespace fast16;

constexpr int MAXROWS = LY * TR4 + 4;      // image rows of a region: two bands, each with a top and a bottom halo row (36)
constexpr int MAX_PIECES = 256;            // pieces of cut items in flight (the workspace holds that many partial tiles)
constexpr int MAX_PARTS = 8;               // pieces per cut item
constexpr size_t PIECE_FLOATS = (size_t)FG * TR4 * TC * 32;   // fp32 partial sums of one piece: [32 filters][56 values][32 lanes]

// The first members of both kernels' parameter blocks.
struct ImgGeometry {
  int N, H, W, C, F;
  int nct;                 // ring stages per work item: C / (channels of a stage)
  int Ho, Wo, sub;         // output size; sub = stride - 1: with stride 2 only the results at even rows and columns are written
  int relu;                // 1: results below zero are written as zero (the rectifier that follows the layer, fused);
                           // 2: that, then 2 x 2 max pooling (Ho, Wo are then the pooled sizes H / 2, W / 2)
  int TY;                  // tile rows per image (ceil(H / 4), at least four)
  int TXe, NI;             // tile columns per region, images side by side
  int CG, NIG;             // column groups per image, image groups
  int NG;                  // filter groups (F / 32)
  int n_regions, n_items;  // n_items = n_regions * NG
  // Tail balancing: items [0, n_whole) are processed whole, one per block and round.  Each of the n_split items
  // that would start another, mostly idle round is cut along the input channels into `parts` pieces that run on
  // different blocks and write fp32 partial sums (`partials`: [piece][32 filters][56 values][32 lanes]); a reduce
  // kernel adds them up in a fixed order.  parts == 1: no cutting.
  int n_whole, n_split, parts;
  float* partials;
  FastDiv d_CG, d_TY, d_NG;     // divisions by CG, TY, NG
};

// A region = LY consecutive tile rows (of four pixel rows) x LX column slots.  Tile rows are numbered through all
// image groups (group g, tile row t -> g * TY + t), so a region may straddle two image groups: it then has two
// bands, each with its own halo rows.
struct Region {
  int cg;           // column group
  int ig0, ta0, n0; // band 0: image group, first tile row, number of tile rows
  bool band1;       // band 1 exists (image group ig0 + 1, tile rows 0 .. LY - n0)
  int nrows;        // image rows in use
};

__device__ __forceinline__ Region decode_region(const ImgGeometry& p, int reg) {
  Region r;
  const int rb = p.d_CG.div(reg);
  r.cg = reg - rb * p.CG;
  const int gt0 = rb * LY;
  r.ig0 = p.d_TY.div(gt0);
  r.ta0 = gt0 - r.ig0 * p.TY;
  r.n0 = min(LY, p.TY - r.ta0);
  r.band1 = (r.n0 < LY) && (r.ig0 + 1 < p.NIG);
  r.nrows = r.band1 ? MAXROWS : TR4 * r.n0 + 2;
  return r;
}

// stage_channels: input channels per ring stage.  False when the layer has more regions or items than an int holds.
inline bool fill_geometry(ImgGeometry& p, int F, int C, int N, int H, int W, int stage_channels) {
  p.N = N; p.H = H; p.W = W; p.C = C; p.F = F;
  p.nct = C / stage_channels;
  p.TY = std::max((H + TR4 - 1) / TR4, LY / 2);   // a last, partly empty tile row when H is not a multiple of 4; small images take four tile rows
  const int TX = W < TC ? 1 : W / TC;                // an image narrower than a thread tile takes one tile column
  p.TXe = TX >= LX ? LX : TX;
  p.NI = LX / p.TXe;
  p.CG = TX / p.TXe;
  p.NIG = (N + p.NI - 1) / p.NI;
  p.NG = F / FG;
  const long long row_blocks = ((long long)p.NIG * p.TY + LY - 1) / LY;
  const long long regions = row_blocks * p.CG;
  const long long items = regions * p.NG;
  if (items > 0x7FFFFFFFll || regions * p.nct > 0x7FFFFFFFll) return false;
  p.n_regions = (int)regions;
  p.n_items = (int)items;
  p.n_whole = p.n_items; p.n_split = 0; p.parts = 1; p.partials = nullptr;
  p.d_CG.set(p.CG); p.d_TY.set(p.TY); p.d_NG.set(p.NG);
  return true;
}

// Shapes the stage-image kernels cover (both precisions): W a multiple of 14 (or narrower than 14), one, two or a
// multiple of four tile columns, a region spanning at most two image groups, whole stages and filter groups.
inline bool shape_supported(int F, int C, int N, int H, int W, int stride, int channel_multiple, int stage_channels) {
  if (stride != 1 && stride != 2) return false;       // stride 2: computed like stride 1, one result in four written
  const int TY = std::max((H + TR4 - 1) / TR4, LY / 2);
  if ((W % TC != 0 && W > TC) || !(TY >= LY - 1 || 2 * TY == LY)) return false;
  const int TX = W < TC ? 1 : W / TC;
  if (!(TX == 1 || TX == 2 || TX % 4 == 0)) return false;
  if (C % channel_multiple != 0 || F % FG != 0) return false;   // the blob's execution section is cut in tiles of 16 channels
  ImgGeometry g;
  return N >= 1 && fill_geometry(g, F, C, N, H, W, stage_channels);
}

// Decides which items are cut and returns the grid of the convolution kernel.  partials: where the partial sums go.
inline int plan_items(ImgGeometry& p, int sm_count, int stage_channels, float* partials) {
  int grid = std::min(p.n_items, sm_count);
  // fewer work items than half the SMs (small batches): every item is cut along the input channels, so that up to
  // eight blocks share an item; their partial sums are added by the reduce kernel
  if (2 * p.n_items <= sm_count) {
    // a piece keeps at least 32 input channels - below that its partial sums cost more than the idle SMs - unless
    // the items are so few (a single small image) that the partial sums are a few megabytes in all
    const int min_channels = p.n_items <= 8 ? stage_channels : 32;
    const int parts = std::min(std::min(MAX_PARTS, p.C / min_channels), std::min(sm_count, MAX_PIECES) / p.n_items);
    if (parts >= 3) {
      p.n_whole = 0; p.n_split = p.n_items; p.parts = parts;
      p.partials = partials;
      grid = p.n_items * parts;
    }
  }
  // the items of a last, mostly idle round are cut into up to eight pieces
  const int left = p.parts > 1 ? 0 : p.n_items % grid;
  if (left > 0) {
    const int parts = std::min(std::min(MAX_PARTS, p.nct), std::min(grid, MAX_PIECES) / left);
    if (parts >= 2) {
      p.n_whole = p.n_items - left; p.n_split = left; p.parts = parts;
      p.partials = partials;
    }
  }
  return grid;
}

}  // namespace imggeo
}  // namespace pat
