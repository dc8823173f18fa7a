/*
 * The paper's inference procedure on a CPU, stage by stage, in fp32 (test infrastructure and a
 * second, closer-to-the-paper CPU baseline; not part of the product, shares nothing with the CUDA
 * path).
 *
 * Appendix A, Algorithm 2 and Section 3.2 describe three stages for one image:
 *   (i)   an indirection table that holds, for every output position whose mask entry is 1 and in
 *         raster order, where the input pixels under the filter window are (the paper keeps
 *         pointers, this file element offsets); positions with mask 0 get no entry, so the table
 *         has P' = sum(mask) rows of kh*kw entries;
 *   (ii)  the unmodified dense GEMM over that reduced range: row r of the compact output is the
 *         product of the gathered window of kept position r with the filter matrix, plus the bias
 *         (the engine's fp32 arithmetic; the activation is applied here, on computed rows only);
 *   (iii) the post-processing pass that makes the output dense again IN PLACE: the compact rows sit
 *         at the start of the output buffer; positions are visited from the last to the first; a
 *         position with mask 0 is cleared, a position with mask 1 receives compact row id and id is
 *         decremented, so no row is overwritten before it has been moved.
 *
 * Readings: the printed index out_y * output_height + out_x is taken as the row-major position
 * out_y * output_width + out_x; padding taps are marked and contribute zeros; the mask is shared by the
 * images of a batch; the GEMM is a plain triple loop (the paper uses the engine's micro-kernels,
 * whose blocking is not part of the method).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* Stage (i): the window table of one image.  Entry (r, t) is the element offset, within the image,
 * of the input pixel under filter tap t of the r-th kept position (kept positions in ascending flat
 * order), or -1 where the tap falls into the padding.  Returns the number of kept positions. */
static int64_t build_window_table(int H, int W, int C_in, int kh, int kw, int stride, int pad, int Wo, int64_t P,
                                  const uint8_t *mask, int64_t *table)
{
    const int taps = kh * kw;
    int64_t n_kept = 0;
    for (int64_t p = 0; p < P; ++p) {
        if (!mask[p]) continue;                       /* a dropped position gets no entry */
        const int top = (int)(p / Wo) * stride - pad, left = (int)(p % Wo) * stride - pad;
        int64_t *entry = table + n_kept * taps;
        for (int t = 0; t < taps; ++t) {
            const int iy = top + t / kw, ix = left + t % kw;
            entry[t] = (iy >= 0 && iy < H && ix >= 0 && ix < W) ? ((int64_t)iy * W + ix) * C_in : -1;
        }
        ++n_kept;
    }
    return n_kept;
}

/* Stage (ii): the dense product restricted to the kept rows; compact row r goes to rows[r]. */
static void product_on_kept_rows(const float *x_img, const int64_t *table, int64_t n_kept, int taps, int C_in,
                                 const float *w, const float *bias, int C_out, int relu, float *rows)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < n_kept; ++r)
        for (int co = 0; co < C_out; ++co) {
            float acc = bias ? bias[co] : 0.0f;
            for (int t = 0; t < taps; ++t) {
                const int64_t off = table[r * taps + t];
                if (off < 0) continue;                /* padding contributes zeros */
                const float *px = x_img + off;
                const float *wt = w + ((int64_t)co * taps + t) * C_in;
                for (int ci = 0; ci < C_in; ++ci) acc += px[ci] * wt[ci];
            }
            rows[r * C_out + co] = (relu && acc < 0.0f) ? 0.0f : acc;
        }
}

/* Stage (iii): the compact rows occupy the first n_kept rows of the image's output; spread them to
 * their positions in place.  Going from the last position down, the row still to be placed (`src`)
 * never lies above its destination, so a row is moved before anything can overwrite it; dropped
 * positions are cleared on the way. */
static void expand_in_place(float *out, int64_t P, int C_out, const uint8_t *mask, int64_t n_kept)
{
    const size_t row_bytes = (size_t)C_out * sizeof(float);
    int64_t src = n_kept;                             /* rows [0, src) are still compact */
    for (int64_t p = P; p-- > 0;) {
        float *dst = out + p * C_out;
        if (mask[p]) {
            --src;
            if (src != p) memmove(dst, out + src * C_out, row_bytes);
        } else {
            memset(dst, 0, row_bytes);
        }
    }
}

/*
 * x [Nb][H][W][C_in], w [C_out][kh][kw][C_in], bias [C_out] or NULL, mask [Ho*Wo], y [Nb][Ho][Wo][C_out],
 * all fp32.  Returns 0, or 1 on a bad geometry or allocation failure.
 */
int asxo_alg2_fp32(const float *x, int Nb, int H, int W, int C_in, const float *w, int C_out, int kh, int kw,
                   int stride, int pad, const float *bias, const uint8_t *mask, int relu, float *y)
{
    if (Nb < 1 || H < 1 || W < 1 || C_in < 1 || C_out < 1 || kh < 1 || kw < 1 || stride < 1 || pad < 0) return 1;
    if (H + 2 * pad < kh || W + 2 * pad < kw) return 1;
    const int Ho = (H + 2 * pad - kh) / stride + 1, Wo = (W + 2 * pad - kw) / stride + 1;
    const int taps = kh * kw;
    const int64_t P = (int64_t)Ho * Wo;
    int64_t *table = (int64_t *)malloc((size_t)P * taps * sizeof(int64_t));
    if (!table) return 1;
    for (int n = 0; n < Nb; ++n) {
        const float *x_img = x + (int64_t)n * H * W * C_in;
        float *y_img = y + (int64_t)n * P * C_out;
        const int64_t n_kept = build_window_table(H, W, C_in, kh, kw, stride, pad, Wo, P, mask, table);
        product_on_kept_rows(x_img, table, n_kept, taps, C_in, w, bias, C_out, relu, y_img);
        expand_in_place(y_img, P, C_out, mask, n_kept);
    }
    free(table);
    return 0;
}
