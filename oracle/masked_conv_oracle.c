/*
 * CPU oracle for the masked convolution (test infrastructure only).
 *
 * This file is the slow, plain definition of what the GPU library must compute.  It is
 * used by the tests, by the smoke check and by the benchmark's CPU-baseline leg, and by
 * nothing else; it shares no code with the CUDA path.
 *
 * What it computes (paper, Section 3 and Section 3.2; Appendix A, Algorithm 2):
 * a convolution is a product of the filter matrix with the lowered activation matrix that
 * has one entry per sliding window (Section 3).  A binary mask with one entry per output
 * spatial position selects the windows that are computed (mask == 1); for mask == 0 the
 * whole output pixel, in every channel, is zero (Algorithm 2, post-processing: zeros are
 * inserted where the mask is 0, computed rows are copied where it is 1).  The product on
 * the kept windows is the ordinary one ("the GEMM remains unaltered", Appendix A), so the
 * result equals   y = mask (.) act(conv(x, w) + b)   with the mask broadcast over channels.
 * Because that result has a plain definition, the oracle is the definition itself: a
 * direct convolution in raster order, with no lowering, no index list and no blocking.
 *
 * Readings where the paper is silent:
 *  - dropped positions are exactly 0: neither bias nor activation is applied there;
 *  - mask index is row-major, p = oy*Wo + ox (the loops of Algorithm 2 run out_y outer,
 *    out_x inner); a mask of Ho*Wo entries is shared by all images of the batch, a mask of
 *    Nb*Ho*Wo entries gives one bit per lowered row;
 *  - cross-correlation (no kernel flip), symmetric zero padding, dilation 1, groups 1;
 *  - the activation `act` is a code: 0 identity, 1 ReLU max(z, 0), 2 SiLU z / (1 + exp(-z))
 *    (the activation of YOLOv5, one of the networks of Section 4); both map 0 to 0, so a
 *    dropped position equals the activation of a zero pre-activation without bias;
 *  - adding 16 to the activation code selects fp32 storage (the paper's, Appendix A: sizeof(float)):
 *    inputs and weights are then taken as given instead of being rounded to bfloat16;
 *  - inputs and weights are rounded to bfloat16 (round to nearest, ties to even) first,
 *    then every product and sum is taken in double precision; the bias is an fp32 vector
 *    added before the activation; the result is NOT rounded.
 *
 * Pins (tests/test_oracle_pins.py): a library fp64 convolution at sparsity 0, an explicit
 * lowered-matrix product on the kept rows with zero rows re-inserted, closed forms for
 * all-ones inputs, unit impulses, hand-computed tiny integer cases, and the invariants of
 * the kept-row list.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* Activation by code, in double precision. */
static double activate(double z, int act)
{
    if (act == 1) return z < 0.0 ? 0.0 : z;
    if (act == 2) return z / (1.0 + exp(-z));
    return z;
}

/* bfloat16 rounding, round-to-nearest-even, written out on the bit pattern. */
static float bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7f800000u) == 0x7f800000u) {          /* inf or nan */
        if (u & 0x007fffffu) u |= 0x00400000u;       /* keep a nan a nan */
        u &= 0xffff0000u;
    } else {
        uint32_t lsb = (u >> 16) & 1u;
        u += 0x7fffu + lsb;
        u &= 0xffff0000u;
    }
    memcpy(&f, &u, 4);
    return f;
}

void asxo_bf16_round(const float *in, float *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = bf16_rne(in[i]);
}

/* Kept-row list: ascending positions whose mask entry is 1 (Algorithm 2, the running
 * index of the indirection-initialisation loop).  Returns the count. */
int64_t asxo_kept_list(const uint8_t *mask, int64_t rows, int32_t *kept)
{
    int64_t c = 0;
    for (int64_t r = 0; r < rows; ++r)
        if (mask[r]) kept[c++] = (int32_t)r;
    return c;
}

typedef struct {
    int Nb, H, W, C_in, C_out, kh, kw, stride, pad, Ho, Wo;
} geom_t;

/* One output pixel (all channels) by the definition. */
static void one_position(const geom_t *g, const float *xr, const float *wr, const float *bias,
                         int act, int n, int oy, int ox, double *y)
{
    for (int co = 0; co < g->C_out; ++co) {
        double s = bias ? (double)bias[co] : 0.0;
        for (int ky = 0; ky < g->kh; ++ky) {
            int iy = oy * g->stride - g->pad + ky;
            if (iy < 0 || iy >= g->H) continue;
            for (int kx = 0; kx < g->kw; ++kx) {
                int ix = ox * g->stride - g->pad + kx;
                if (ix < 0 || ix >= g->W) continue;
                const float *xp = xr + (((int64_t)n * g->H + iy) * g->W + ix) * g->C_in;
                const float *wp = wr + (((int64_t)co * g->kh + ky) * g->kw + kx) * g->C_in;
                for (int ci = 0; ci < g->C_in; ++ci)
                    s += (double)xp[ci] * (double)wp[ci];
            }
        }
        y[co] = activate(s, act);
    }
}

static int fill_geom(geom_t *g, int Nb, int H, int W, int C_in, int C_out, int kh, int kw,
                     int stride, int pad)
{
    if (Nb < 1 || H < 1 || W < 1 || C_in < 1 || C_out < 1 || kh < 1 || kw < 1 || stride < 1 || pad < 0)
        return 1;
    if (H + 2 * pad < kh || W + 2 * pad < kw) return 1;
    g->Nb = Nb; g->H = H; g->W = W; g->C_in = C_in; g->C_out = C_out;
    g->kh = kh; g->kw = kw; g->stride = stride; g->pad = pad;
    g->Ho = (H + 2 * pad - kh) / stride + 1;
    g->Wo = (W + 2 * pad - kw) / stride + 1;
    return 0;
}

/* Full output y[Nb][Ho][Wo][C_out] in double.  x, w are fp32 and are rounded to bf16 here.
 * rows == Ho*Wo: mask shared by the batch; rows == Nb*Ho*Wo: one entry per lowered row.
 * Returns 0, or 1 on bad arguments, 2 on allocation failure. */
int asxo_masked_conv(const float *x, int Nb, int H, int W, int C_in,
                     const float *w, int C_out, int kh, int kw, int stride, int pad,
                     const float *bias, const uint8_t *mask, int64_t rows, int act, double *y)
{
    geom_t g;
    if (fill_geom(&g, Nb, H, W, C_in, C_out, kh, kw, stride, pad)) return 1;
    const int64_t P = (int64_t)g.Ho * g.Wo;
    if (rows != P && rows != P * Nb) return 1;
    const int64_t nx = (int64_t)Nb * H * W * C_in, nw = (int64_t)C_out * kh * kw * C_in;
    float *xr = (float *)malloc(sizeof(float) * (size_t)nx);
    float *wr = (float *)malloc(sizeof(float) * (size_t)nw);
    if (!xr || !wr) { free(xr); free(wr); return 2; }
    if (act & 16) {                       /* fp32 storage: the values as given */
        memcpy(xr, x, sizeof(float) * (size_t)nx);
        memcpy(wr, w, sizeof(float) * (size_t)nw);
    } else {
        asxo_bf16_round(x, xr, nx);
        asxo_bf16_round(w, wr, nw);
    }
    act &= 15;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int n = 0; n < Nb; ++n)
        for (int oy = 0; oy < g.Ho; ++oy)
            for (int ox = 0; ox < g.Wo; ++ox) {
                int64_t p = (int64_t)oy * g.Wo + ox;
                int keep = (rows == P) ? mask[p] : mask[(int64_t)n * P + p];
                double *yo = y + ((int64_t)n * P + p) * C_out;
                if (!keep) {
                    for (int co = 0; co < C_out; ++co) yo[co] = 0.0;
                } else {
                    one_position(&g, xr, wr, bias, act, n, oy, ox, yo);
                }
            }
    free(xr); free(wr);
    return 0;
}

/* The same definition evaluated only at selected lowered rows sel[i] in [0, Nb*Ho*Wo):
 * y[i][0..C_out).  For checking samples of problems too large to evaluate in full.
 * x and w must already hold bf16-representable values when pre_rounded != 0. */
int asxo_masked_conv_rows(const float *x, int Nb, int H, int W, int C_in,
                          const float *w, int C_out, int kh, int kw, int stride, int pad,
                          const float *bias, const uint8_t *mask, int64_t rows, int act,
                          const int64_t *sel, int64_t nsel, double *y)
{
    geom_t g;
    if (fill_geom(&g, Nb, H, W, C_in, C_out, kh, kw, stride, pad)) return 1;
    const int64_t P = (int64_t)g.Ho * g.Wo;
    if (rows != P && rows != P * Nb) return 1;
    const int64_t nw = (int64_t)C_out * kh * kw * C_in;
    float *wr = (float *)malloc(sizeof(float) * (size_t)nw);
    if (!wr) return 2;
    const int exact = (act & 16) != 0;    /* fp32 storage: the values as given */
    act &= 15;
    if (exact) memcpy(wr, w, sizeof(float) * (size_t)nw);
    else asxo_bf16_round(w, wr, nw);
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t i = 0; i < nsel; ++i) {
        int64_t r = sel[i];
        if (r < 0 || r >= P * Nb) { bad = 1; continue; }
        int n = (int)(r / P);
        int64_t p = r % P;
        int oy = (int)(p / g.Wo), ox = (int)(p % g.Wo);
        int keep = (rows == P) ? mask[p] : mask[r];
        double *yo = y + i * C_out;
        if (!keep) {
            for (int co = 0; co < C_out; ++co) yo[co] = 0.0;
            continue;
        }
        /* round only the window this row reads */
        for (int co = 0; co < C_out; ++co) {
            double s = bias ? (double)bias[co] : 0.0;
            for (int ky = 0; ky < kh; ++ky) {
                int iy = oy * stride - pad + ky;
                if (iy < 0 || iy >= H) continue;
                for (int kx = 0; kx < kw; ++kx) {
                    int ix = ox * stride - pad + kx;
                    if (ix < 0 || ix >= W) continue;
                    const float *xp = x + (((int64_t)n * H + iy) * W + ix) * C_in;
                    const float *wp = wr + (((int64_t)co * kh + ky) * kw + kx) * C_in;
                    for (int ci = 0; ci < C_in; ++ci)
                        s += (double)(exact ? xp[ci] : bf16_rne(xp[ci])) * (double)wp[ci];
                }
            }
            yo[co] = activate(s, act);
        }
    }
    free(wr);
    return bad;
}
