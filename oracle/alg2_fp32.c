/*
 * The paper's inference procedure on a CPU, stage by stage, in fp32 (test infrastructure and a
 * second, closer-to-the-paper CPU baseline; not part of the product, shares nothing with the CUDA
 * path).
 *
 * Appendix A, Algorithm 2 and Section 3.2 describe three stages for one image:
 *   (i)   an indirection buffer that holds, for every output position whose mask entry is 1 and in
 *         raster order, the pointers to the input pixels under the filter window; positions with
 *         mask 0 get no entry, so the buffer has P' = sum(mask) rows of kh*kw pointers;
 *   (ii)  the unmodified dense GEMM over that reduced range: row r of the compact output is the
 *         product of the gathered window of kept position r with the filter matrix, plus the bias
 *         (the engine's fp32 arithmetic; the activation is applied here, on computed rows only);
 *   (iii) the post-processing pass that makes the output dense again IN PLACE: the compact rows sit
 *         at the start of the output buffer; positions are visited from the last to the first; a
 *         position with mask 0 is cleared, a position with mask 1 receives compact row id and id is
 *         decremented, so no row is overwritten before it has been moved.
 *
 * Readings: the printed index out_y * output_height + out_x is taken as the row-major position
 * out_y * output_width + out_x; padding taps point at a row of zeros; the mask is shared by the
 * images of a batch; the GEMM is a plain triple loop (the paper uses the engine's micro-kernels,
 * whose blocking is not part of the method).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* Stage (i): pointers of the kept windows of one image.  Returns P'. */
static int64_t indirection_init(const float *x_img, int H, int W, int C_in, int kh, int kw, int stride, int pad,
                                int Ho, int Wo, const uint8_t *mask, const float *zero_row, const float **ind)
{
    int64_t index = 0;
    for (int out_y = 0; out_y < Ho; ++out_y)
        for (int out_x = 0; out_x < Wo; ++out_x) {
            if (mask[(int64_t)out_y * Wo + out_x] == 0) continue;
            for (int ky = 0; ky < kh; ++ky)
                for (int kx = 0; kx < kw; ++kx) {
                    const int iy = out_y * stride - pad + ky, ix = out_x * stride - pad + kx;
                    const int inside = iy >= 0 && iy < H && ix >= 0 && ix < W;
                    ind[index * kh * kw + ky * kw + kx] = inside ? x_img + ((int64_t)iy * W + ix) * C_in : zero_row;
                }
            ++index;
        }
    return index;
}

/* Stage (ii): dense product over the kept rows, written compactly at the start of `out`. */
static void gemm_reduced(const float **ind, int64_t kept, int taps, int C_in, const float *w, const float *bias,
                         int C_out, int relu, float *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < kept; ++r)
        for (int co = 0; co < C_out; ++co) {
            float acc = bias ? bias[co] : 0.0f;
            for (int t = 0; t < taps; ++t) {
                const float *px = ind[r * taps + t];
                const float *wt = w + ((int64_t)co * taps + t) * C_in;
                for (int ci = 0; ci < C_in; ++ci) acc += px[ci] * wt[ci];
            }
            out[r * C_out + co] = (relu && acc < 0.0f) ? 0.0f : acc;
        }
}

/* Stage (iii): reverse in-place expansion of the compact rows to the dense output of one image. */
static void post_process(float *out, int Ho, int Wo, int C_out, const uint8_t *mask, int64_t kept)
{
    const size_t outch_size = (size_t)C_out * sizeof(float);
    int64_t id = kept - 1;
    for (int out_y = Ho - 1; out_y >= 0; --out_y)
        for (int out_x = Wo - 1; out_x >= 0; --out_x) {
            const int64_t pos = (int64_t)out_y * Wo + out_x;
            if (mask[pos] == 0) {
                memset(out + pos * C_out, 0, outch_size);
            } else {
                if (pos != id) memmove(out + pos * C_out, out + id * C_out, outch_size);
                --id;
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
    float *zero_row = (float *)calloc((size_t)C_in, sizeof(float));
    const float **ind = (const float **)malloc((size_t)P * taps * sizeof(const float *));
    if (!zero_row || !ind) { free(zero_row); free((void *)ind); return 1; }
    for (int n = 0; n < Nb; ++n) {
        const float *x_img = x + (int64_t)n * H * W * C_in;
        float *y_img = y + (int64_t)n * P * C_out;
        const int64_t kept = indirection_init(x_img, H, W, C_in, kh, kw, stride, pad, Ho, Wo, mask, zero_row, ind);
        gemm_reduced(ind, kept, taps, C_in, w, bias, C_out, relu, y_img);
        post_process(y_img, Ho, Wo, C_out, mask, kept);
    }
    free(zero_row);
    free((void *)ind);
    return 0;
}
