"""How dense are pattern-grouped weight tiles as matrix contractions?

The convolution kernels use the fp32 multiply-add pipe because a pruned layer is not a dense contraction.  This
script measures that on the workloads: every sparse layer of the five configurations is projected (pat_project on
the GPU), cut into tiles of 32 filters x 16 input channels (the unit the kernels work on), and two matrix
formulations of a tile are compared with the useful work, 4 multiply-adds per kept kernel and output pixel:

* dense tile:        all 32 x 16 kernels with all 9 taps (what an im2col contraction of the tile would execute);
* pattern segments:  per pattern present in the tile, the filters and channels that have a kernel of that pattern
                     form a (filters x channels x 4 taps) contraction - the re-ordering of Section 6.2 carried to
                     its limit; rows and columns that hold no kernel of the pattern are dropped.

* padded segments:   the same with every segment padded to the smallest tensor-core tile (64 rows, 16 deep), which
                     is what a tcgen05 instruction would really execute.

density = useful multiply-adds / multiply-adds of the formulation.  With the tensor cores about 22 times faster than
the fp32 pipe (dense fp16 against 2 x 128 lanes per SM), a formulation pays above a density of about 1/22 = 4.6 % at
perfect tensor-core efficiency and without padding to the instruction's minimum tile (64 x 8 x 16); in practice
several times that.  Prints a markdown table.

    python -m paper_2001_07710_b200.density
"""
from __future__ import annotations

import numpy as np
import torch

import paper_2001_07710_b200 as pc
from paper_2001_07710_b200 import workloads

TILE_F, TILE_C = 32, 16
BREAK_EVEN = 1.0 / 21.9


def tile_densities(pid: np.ndarray, K: int):
    """pid: [F][C] pattern ids (255 = pruned).  Returns per tile (dense-tile, pattern-segment, padded-segment density)."""
    F, C = pid.shape
    out = []
    for f0 in range(0, F - F % TILE_F, TILE_F):
        for c0 in range(0, C - C % TILE_C, TILE_C):
            t = pid[f0:f0 + TILE_F, c0:c0 + TILE_C]
            kept = int((t != 255).sum())
            if kept == 0:
                out.append((0.0, 0.0, 0))
                continue
            seg = pad = 0
            for p in range(K):
                m = t == p
                if m.any():
                    rows, cols = int(m.any(axis=1).sum()), int(m.any(axis=0).sum())
                    seg += rows * cols
                    pad += 64 * ((4 * cols + 15) // 16) * 16          # multiply-adds per pixel of a 64 x (4 cols -> 16) tile
            out.append((4.0 * kept / (9.0 * TILE_F * TILE_C), kept / float(seg), 4.0 * kept / float(pad)))
    return np.array(out)


def main():
    rows = []
    for cfg in workloads.configs():
        seen = set()
        for L in cfg.layers:
            key = (L.F, L.C, L.K, L.keep)
            if L.dense or key in seen or L.F % TILE_F or L.C % TILE_C:
                continue
            seen.add(key)
            w, _ = workloads.make_layer_tensors(cfg.number, L, 1, n_limit=1)
            masks = pc.pat_library_builtin(L.K)
            pid, _ = pc.pat_project(torch.from_numpy(w).cuda(), masks, L.n_keep)
            d = tile_densities(pid.cpu().numpy(), L.K)
            q = lambda a: "%.3f / %.3f / %.3f" % (np.quantile(a, 0.05), np.median(a), a.max())
            rows.append((cfg.number, f"{L.F}x{L.C}", L.K, f"{L.keep.numerator}/{L.keep.denominator}", len(d),
                         q(d[:, 0]), q(d[:, 1]), q(d[:, 2]), "%.1f %%" % (100.0 * float((d[:, 2] > BREAK_EVEN).mean()))))
    print("| config | F x C | K | keep | tiles | dense tile (5 % / median / max) | pattern segments | padded segments | tiles whose padded segments beat break-even |")
    print("|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        print("| " + " | ".join(str(v) for v in r) + " |")
    print(f"\nbreak-even density at perfect tensor-core efficiency: {BREAK_EVEN:.3f}")


if __name__ == "__main__":
    main()
