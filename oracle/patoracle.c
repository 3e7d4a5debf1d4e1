/*
 * CPU oracle for pattern-based sparse 3x3 convolution.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, float64 restatement of what the GPU library computes, written from the
 * paper's definitions and sharing no code with the CUDA path.  Only the test-suite, the
 * smoke check and the CPU-baseline leg of the benchmark may call it.
 *
 * Conventions (the paper leaves them open; they are fixed here and in the C-ABI header):
 *   - a 3x3 kernel position is (r,s), r = row 0..2 top to bottom, s = column 0..2 left to right;
 *     mask bit b = 3*r + s; a pattern is a 9-bit integer with exactly four bits set.
 *   - weights are [F][C][3][3] (filter, input channel, r, s); activations are NHWC.
 *   - convolution is cross-correlation (no kernel flip), zero padding 1, no bias.
 *
 * Parity status of each function (what it is pinned to by the CPU tests):
 *   orc_library          pinned: family sums of Section 4.2, popcount 4, rotation closure;
 *                        the identity of patterns 8..11 is a convention: "parity unpinned".
 *   orc_project          pinned: brute force over all C(9,4) masks vs "keep the 4 largest |w|",
 *                        hand cases, energy/ordering invariants.
 *   orc_pack             the canonical ordering key is a convention of this build:
 *                        "parity unpinned" against the paper; pinned by round trip and invariants.
 *   orc_conv3x3          pinned: library float64 conv2d, delta / identity / all-ones closed forms,
 *                        an independent sparse-gather evaluation, stride-2 subsampling, linearity.
 *   orc_f32_to_f16       pinned: library round-to-nearest-even conversion, exhaustive round trip.
 *   orc_simplex_project  pinned: bisection on the defining equation, optimality conditions, closed forms
 *                        (vector already on the simplex, constant vector, one dominant entry, K = 1, 2).
 *   orc_argmax_binarize  pinned: library argmax, distance to every one-hot vector; the tie rule is a
 *                        convention: "parity unpinned".
 *   orc_extract_library  pinned: for the full 126-mask library the assignment is "the four largest |w|"
 *                        (independent numpy), planted pattern frequencies are recovered; the tie rule and
 *                        the order of the survivors are conventions: "parity unpinned".
 *   orc_relu_maxpool     pinned: library relu + max_pool2d (float64), hand case.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------------
 * Pattern library (Section 4.2 for the two derived families; Section 7.1 for the library sizes).
 * Built from the verbal description, not from a table:
 *   ids 0..3   centre + three of the four arms {up,left,right,down}; the missing arm is
 *              down, up, left, right in that order.
 *   ids 4..7   centre + two adjacent arms + the corner between them = the 2x2 blocks that hold
 *              the centre, in the order top-left, top-right, bottom-left, bottom-right.
 *   ids 8..11  centre + two opposite arms + one corner: {up,down,top-left} and its three
 *              successive quarter-turn rotations (clockwise).
 * K = 4 is ids 0..3, K = 8 is ids 0..7, K = 12 is all of them.
 * ---------------------------------------------------------------------------------------- */
static int bit_of(int r, int s) { return 3 * r + s; }

/* quarter turn clockwise of a position: (r,s) -> (s, 2-r) */
static int rot_bit(int b) { int r = b / 3, s = b % 3; return bit_of(s, 2 - r); }

static int rot_mask(int m) {
    int out = 0;
    for (int b = 0; b < 9; ++b) if (m & (1 << b)) out |= 1 << rot_bit(b);
    return out;
}

int orc_library(int K, uint16_t *masks_out) {
    if (K != 4 && K != 8 && K != 12) return 1;
    const int centre = bit_of(1, 1), up = bit_of(0, 1), left = bit_of(1, 0), right = bit_of(1, 2), down = bit_of(2, 1);
    const int arms[4] = { up, left, right, down };
    const int missing[4] = { down, up, left, right };
    int n = 0;
    for (int i = 0; i < 4; ++i) {
        int m = 1 << centre;
        for (int a = 0; a < 4; ++a) if (arms[a] != missing[i]) m |= 1 << arms[a];
        masks_out[n++] = (uint16_t)m;
    }
    if (K >= 8) {
        for (int br = 0; br < 2; ++br)          /* block's top row   */
            for (int bs = 0; bs < 2; ++bs) {    /* block's left col  */
                int m = 0;
                for (int r = br; r < br + 2; ++r) for (int s = bs; s < bs + 2; ++s) m |= 1 << bit_of(r, s);
                masks_out[n++] = (uint16_t)m;
            }
    }
    if (K >= 12) {
        int m = (1 << centre) | (1 << up) | (1 << down) | (1 << bit_of(0, 0));
        for (int i = 0; i < 4; ++i) { masks_out[n++] = (uint16_t)m; m = rot_mask(m); }
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Projection: pattern selection (Section 4.1: pruning = kernel o mask; Section 5.1: one mask of the
 * library per kernel, the binarisation being an argmax) and connectivity pruning (Section 6.1:
 * score gamma = L2 norm of the kernel).
 *
 * For each kernel every mask is tried; the energy of a mask is the sum of squares of the weights
 * it keeps, accumulated in float64 in ascending bit order.  The mask of largest energy wins
 * (lowest id on ties).  Then the n_keep kernels of largest winning energy (gamma^2 after pattern
 * pruning) are kept, the lower linear index f*C+c winning ties; all others are removed.
 * Outputs: pid[F*C] (0xFF = removed), wm = masked weights (+0.0 elsewhere), gamma2[F*C].
 * ---------------------------------------------------------------------------------------- */
typedef struct { double e; int64_t idx; } rank_t;

static int rank_cmp(const void *a, const void *b) {
    const rank_t *x = (const rank_t *)a, *y = (const rank_t *)b;
    if (x->e > y->e) return -1;
    if (x->e < y->e) return 1;
    return (x->idx < y->idx) ? -1 : (x->idx > y->idx);
}

int orc_project(const float *w, int F, int C, const uint16_t *masks, int K, int64_t n_keep,
                uint8_t *pid, float *wm, double *gamma2) {
    const int64_t FC = (int64_t)F * C;
    if (K < 1 || K > 255 || n_keep < 0 || n_keep > FC) return 1;
    rank_t *rk = (rank_t *)malloc(sizeof(rank_t) * (size_t)(FC > 0 ? FC : 1));
    if (!rk) return 2;
    for (int64_t i = 0; i < FC; ++i) {
        const float *k = w + 9 * i;
        int best = 0; double best_e = -1.0;
        for (int j = 0; j < K; ++j) {
            double e = 0.0;
            for (int b = 0; b < 9; ++b)
                if (masks[j] & (1 << b)) e += (double)k[b] * (double)k[b];
            if (e > best_e) { best_e = e; best = j; }
        }
        pid[i] = (uint8_t)best;
        gamma2[i] = best_e;
        rk[i].e = best_e; rk[i].idx = i;
    }
    qsort(rk, (size_t)FC, sizeof(rank_t), rank_cmp);
    for (int64_t q = n_keep; q < FC; ++q) pid[rk[q].idx] = 0xFF;
    free(rk);
    for (int64_t i = 0; i < FC; ++i)
        for (int b = 0; b < 9; ++b) {
            int kept = pid[i] != 0xFF && (masks[pid[i]] & (1 << b));
            wm[9 * i + b] = kept ? w[9 * i + b] : 0.0f;
        }
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * fp32 -> fp16, round to nearest, ties to even (IEEE 754 binary16), written out on the bits.
 * ---------------------------------------------------------------------------------------- */
uint16_t orc_f32_to_f16(float f) {
    uint32_t u; memcpy(&u, &f, 4);
    const uint32_t sign = (u >> 16) & 0x8000u;
    const uint32_t absu = u & 0x7FFFFFFFu;
    if (absu >= 0x7F800000u) return (uint16_t)(sign | 0x7C00u | ((absu > 0x7F800000u) ? 0x0200u : 0u));
    if (absu == 0) return (uint16_t)sign;
    /* exact value = mant * 2^(e-23) with mant in [2^23, 2^24) for normal floats */
    int e = (int)(absu >> 23);
    uint64_t mant = absu & 0x7FFFFFu;
    if (e == 0) e = 1; else mant |= 0x800000u;
    /* target: q = value / 2^-24 (half subnormal unit) for small values, else normal rounding */
    int unbiased = e - 127;                 /* value = mant * 2^(unbiased-23) */
    int shift;                              /* bits to drop from mant */
    int he;                                 /* biased half exponent of the result before carry */
    if (unbiased < -14) { shift = 13 + (-14 - unbiased); he = 0; }
    else { shift = 13; he = unbiased + 15; }
    if (shift > 40) return (uint16_t)sign;
    uint64_t q = mant >> shift;
    uint64_t rem = mant & (((uint64_t)1 << shift) - 1);
    uint64_t half = (uint64_t)1 << (shift - 1);
    if (rem > half || (rem == half && (q & 1))) q += 1;
    uint32_t h;
    if (he == 0) h = (uint32_t)q;                       /* subnormal; q may reach 0x400 = smallest normal */
    else h = (uint32_t)(((uint32_t)(he - 1) << 10) + q); /* q holds the hidden bit: adds 1 to the exponent */
    if (h >= 0x7C00u) h = 0x7C00u;
    return (uint16_t)(sign | h);
}

double orc_f16_to_f64(uint16_t h) {
    int s = (h >> 15) & 1, e = (h >> 10) & 0x1F, m = h & 0x3FF;
    double v;
    if (e == 0) v = ldexp((double)m, -24);
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp((double)(m | 0x400), e - 25);
    return s ? -v : v;
}

/* ------------------------------------------------------------------------------------------
 * Canonical pack (Section 6.2: filters with similar kernels are put together, and inside a filter
 * the kernels of identical pattern are grouped).  The paper gives no format; this build's is:
 *   perm[F]      new position -> original filter.  Order: kept-kernel count descending, then the
 *                per-pattern count vector (h[0],..,h[K-1]) lexicographically descending, then
 *                original index ascending.
 *   fptr[F+1]    start of each (reordered) filter's kernels; fptr[F] = n_keep.
 *   pptr[F][K+1] start of each pattern segment inside the filter (absolute positions).
 *   chan[n_keep] input channel of each kernel; kernels ordered by (pattern id, channel).
 *   w4[n_keep][4] the four kept taps in ascending bit order, as fp32 bit patterns (dtype 0) or
 *                fp16 bit patterns after round-to-nearest-even (dtype 1; stored in the low 16 bits).
 * ---------------------------------------------------------------------------------------- */
typedef struct { int f; int n; const int32_t *h; int K; } fkey_t;

static int fkey_cmp(const void *a, const void *b) {
    const fkey_t *x = (const fkey_t *)a, *y = (const fkey_t *)b;
    if (x->n != y->n) return (x->n > y->n) ? -1 : 1;
    for (int j = 0; j < x->K; ++j)
        if (x->h[j] != y->h[j]) return (x->h[j] > y->h[j]) ? -1 : 1;
    return (x->f < y->f) ? -1 : (x->f > y->f);
}

int orc_pack(const float *wm, const uint8_t *pid, int F, int C, const uint16_t *masks, int K,
             int dtype, int32_t *perm, int32_t *fptr, int32_t *pptr, uint16_t *chan, uint32_t *w4) {
    int32_t *hist = (int32_t *)calloc((size_t)F * K + 1, sizeof(int32_t));
    fkey_t *keys = (fkey_t *)malloc(sizeof(fkey_t) * (size_t)(F > 0 ? F : 1));
    if (!hist || !keys) { free(hist); free(keys); return 2; }
    for (int f = 0; f < F; ++f) {
        int n = 0;
        for (int c = 0; c < C; ++c) {
            uint8_t p = pid[(int64_t)f * C + c];
            if (p != 0xFF) { if (p >= K) { free(hist); free(keys); return 1; } hist[(int64_t)f * K + p]++; n++; }
        }
        keys[f].f = f; keys[f].n = n; keys[f].h = hist + (int64_t)f * K; keys[f].K = K;
    }
    qsort(keys, (size_t)F, sizeof(fkey_t), fkey_cmp);
    int32_t pos = 0;
    for (int q = 0; q < F; ++q) {
        const int f = keys[q].f;
        perm[q] = f;
        fptr[q] = pos;
        for (int j = 0; j < K; ++j) {
            pptr[(int64_t)q * (K + 1) + j] = pos;
            for (int c = 0; c < C; ++c) {
                if (pid[(int64_t)f * C + c] != j) continue;
                chan[pos] = (uint16_t)c;
                int t = 0;
                for (int b = 0; b < 9; ++b) {
                    if (!(masks[j] & (1 << b))) continue;
                    float v = wm[((int64_t)f * C + c) * 9 + b];
                    uint32_t bits;
                    if (dtype == 0) memcpy(&bits, &v, 4); else bits = orc_f32_to_f16(v);
                    w4[(int64_t)pos * 4 + t] = bits;
                    ++t;
                }
                ++pos;
            }
        }
        pptr[(int64_t)q * (K + 1) + K] = pos;
    }
    fptr[F] = pos;
    free(hist); free(keys);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Convolution: the plain definition.  A pattern-pruned layer is the dense layer whose kernels are
 * multiplied element-wise by their masks (Section 4.1) and whose removed kernels are zero
 * (Section 3), so the reference result is the direct dense cross-correlation of the masked
 * weights, every tap of every channel visited, accumulated in float64:
 *   Y[n][y][x][f] = sum_c sum_r sum_s Wm[f][c][r][s] * X[n][y*st + r - 1][x*st + s - 1][c]
 * with X = 0 outside the image.  Ho = (H - 1) / st + 1.
 * ---------------------------------------------------------------------------------------- */
/* activations may be handed over as float64 (0), float32 (1) or binary16 bit patterns (2); every
 * stored value is converted to float64 exactly before use */
static double act(const void *x, int xdt, int64_t i) {
    if (xdt == 0) return ((const double *)x)[i];
    if (xdt == 1) return (double)((const float *)x)[i];
    return orc_f16_to_f64(((const uint16_t *)x)[i]);
}

static double conv_point(const double *wm, const void *x, int xdt, int H, int W, int C,
                         int n, int yo, int xo, int f, int st) {
    double acc = 0.0;
    for (int c = 0; c < C; ++c)
        for (int r = 0; r < 3; ++r)
            for (int s = 0; s < 3; ++s) {
                const int yi = yo * st + r - 1, xi = xo * st + s - 1;
                if (yi < 0 || yi >= H || xi < 0 || xi >= W) continue;
                acc += wm[((int64_t)f * C + c) * 9 + 3 * r + s] * act(x, xdt, (((int64_t)n * H + yi) * W + xi) * C + c);
            }
    return acc;
}

int orc_conv3x3(const double *wm, int F, int C, const void *x, int xdt, int N, int H, int W, int stride, double *y) {
    if ((stride != 1 && stride != 2) || xdt < 0 || xdt > 2) return 1;
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    const int64_t rows = (int64_t)N * Ho;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t row = 0; row < rows; ++row) {
        const int n = (int)(row / Ho), yo = (int)(row % Ho);
        for (int xo = 0; xo < Wo; ++xo)
            for (int f = 0; f < F; ++f)
                y[(((int64_t)n * Ho + yo) * Wo + xo) * F + f] = conv_point(wm, x, xdt, H, W, C, n, yo, xo, f, stride);
    }
    return 0;
}

/* The same definition evaluated only at listed output coordinates (n, yo, xo, f), for checks on
 * tensors too large to convolve whole. */
int orc_conv3x3_at(const double *wm, int F, int C, const void *x, int xdt, int N, int H, int W, int stride,
                   const int32_t *coords, int64_t n_points, double *out) {
    if ((stride != 1 && stride != 2) || xdt < 0 || xdt > 2) return 1;
    (void)N; (void)F;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n_points; ++i)
        out[i] = conv_point(wm, x, xdt, H, W, C, coords[4 * i], coords[4 * i + 1], coords[4 * i + 2], coords[4 * i + 3], stride);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Proximal step of the pattern-selection ADMM (Section 5.1): for a vector d of K reals,
 *     u = [d - nu 1]_+   with nu the root of   1^T [d - nu 1]_+ = 1,
 * the Euclidean projection of d onto the probability simplex.  g(nu) = sum_j max(d_j - nu, 0) is
 * continuous, piecewise linear and strictly decreasing wherever it is positive, so the root is
 * unique; between two consecutive sorted entries g is linear, so the root is found exactly: with
 * d sorted descending, d_(1) >= d_(2) >= ..., the root lies in the piece where the first r entries
 * are above nu, nu = (d_(1) + ... + d_(r) - 1) / r, and r is the largest count for which the
 * r-th entry is still above that value.  Inputs are fp32, all arithmetic is float64, the result
 * is rounded once to fp32.  n vectors, row-major [n][K].
 * ---------------------------------------------------------------------------------------- */
static int cmp_desc_double(const void *a, const void *b) {
    const double x = *(const double *)a, y = *(const double *)b;
    return (x < y) - (x > y);
}

int orc_simplex_project(const float *d, int64_t n, int K, float *u, double *nu_out) {
    if (K < 1 || n < 0) return 1;
    double *s = (double *)malloc(sizeof(double) * (size_t)K);
    if (!s) return 2;
    for (int64_t i = 0; i < n; ++i) {
        const float *di = d + i * K;
        for (int j = 0; j < K; ++j) s[j] = (double)di[j];
        qsort(s, (size_t)K, sizeof(double), cmp_desc_double);
        double run = 0.0, nu = 0.0;
        for (int r = 1; r <= K; ++r) {
            run += s[r - 1];
            const double cand = (run - 1.0) / (double)r;
            if (s[r - 1] > cand) nu = cand;      /* the r largest entries are all above cand */
            else break;                          /* and once one is not, no longer prefix is */
        }
        for (int j = 0; j < K; ++j) {
            const double v = (double)di[j] - nu;
            u[i * K + j] = (float)(v > 0.0 ? v : 0.0);
        }
        if (nu_out) nu_out[i] = nu;
    }
    free(s);
    return 0;
}

/* Binarisation (Section 5.1): the closest one-hot vector to z is the one with its 1 at
 * argmax_j z_j.  The paper does not say which of several equal maxima wins: the lowest index. */
int orc_argmax_binarize(const float *z, int64_t n, int K, uint8_t *index_out, float *onehot_out) {
    if (K < 1 || K > 256 || n < 0) return 1;
    for (int64_t i = 0; i < n; ++i) {
        int best = 0;
        for (int j = 1; j < K; ++j)
            if (z[i * K + j] > z[i * K + best]) best = j;
        index_out[i] = (uint8_t)best;
        if (onehot_out)
            for (int j = 0; j < K; ++j) onehot_out[i * K + j] = (j == best) ? 1.0f : 0.0f;
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * One reduction step of the library extraction (Algorithm 1, Section 5.2), without the training
 * loop around it: "calculate the pattern distribution of the current library" = every kernel is
 * given the mask of the library that keeps most of its energy (the argmax of Section 5.1, as in
 * orc_project: float64 sums in ascending bit order, lowest id on ties) and the kernels per mask
 * are counted; "remove the patterns with fewest occurrences" = the K_out most frequent masks
 * stay.  Readings where the paper is silent: among masks of equal count the lower id stays; the
 * surviving masks keep their order in the library.  w: n kernels [n][3][3] (the kernels of all
 * layers that share a library, one after another).  counts_out[K_in]; masks_out[K_out].
 * The paper's schedule is 126 -> 12 -> 8 / 4 (Section 5.2, Section 7.1): call it once per step.
 * ---------------------------------------------------------------------------------------- */
int orc_extract_library(const float *w, int64_t n, const uint16_t *masks_in, int K_in, int K_out,
                        uint16_t *masks_out, int64_t *counts_out) {
    if (K_in < 1 || K_out < 1 || K_out > K_in || n < 0) return 1;
    for (int j = 0; j < K_in; ++j) counts_out[j] = 0;
    for (int64_t i = 0; i < n; ++i) {
        int best = 0;
        double best_e = -1.0;
        for (int j = 0; j < K_in; ++j) {
            double e = 0.0;
            for (int b = 0; b < 9; ++b)
                if (masks_in[j] & (1 << b)) e += (double)w[i * 9 + b] * (double)w[i * 9 + b];
            if (e > best_e) { best_e = e; best = j; }
        }
        counts_out[best] += 1;
    }
    /* a mask stays if fewer than K_out masks come before it in (count descending, id ascending) */
    int m = 0;
    for (int j = 0; j < K_in; ++j) {
        int before = 0;
        for (int q = 0; q < K_in; ++q)
            if (counts_out[q] > counts_out[j] || (counts_out[q] == counts_out[j] && q < j)) ++before;
        if (before < K_out) masks_out[m++] = masks_in[j];
    }
    return m == K_out ? 0 : 2;
}

/* ------------------------------------------------------------------------------------------
 * What stands between two convolution layers of the VGG-16 / ResNet models of Section 7: the
 * rectifier max(x, 0) and, after some layers, 2x2 max pooling with stride 2 (the models' own
 * definition, not the paper's).  NHWC, values given as float64; pool = 0: rectifier only,
 * pool = 1: rectifier, then the maximum over each 2x2 block (H and W even).
 * ---------------------------------------------------------------------------------------- */
int orc_relu_maxpool(const double *x, int N, int H, int W, int C, int pool, double *y) {
    if (pool != 0 && pool != 1) return 1;
    if (pool && ((H & 1) || (W & 1))) return 1;
    const int Ho = pool ? H / 2 : H, Wo = pool ? W / 2 : W;
    for (int n = 0; n < N; ++n)
        for (int yo = 0; yo < Ho; ++yo)
            for (int xo = 0; xo < Wo; ++xo)
                for (int c = 0; c < C; ++c) {
                    double m = 0.0;                       /* the rectifier's floor */
                    const int k = pool ? 2 : 1;
                    for (int dy = 0; dy < k; ++dy)
                        for (int dx = 0; dx < k; ++dx) {
                            const double v = x[(((int64_t)n * H + yo * k + dy) * W + xo * k + dx) * C + c];
                            if (v > m) m = v;
                        }
                    y[(((int64_t)n * Ho + yo) * Wo + xo) * C + c] = m;
                }
    return 0;
}
