/*
 * AMS-KV oracle: plain, slow, fp64 CPU definitions of what the hot path computes.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may include, link or call
 * this file; it shares no code with the CUDA library.  It exists so that the CUDA
 * kernels can be checked, element by element, against the textbook definitions.
 *
 * Layout used everywhere here: a tensor is [item][token][channel], contiguous, fp64,
 * where an item is one (row, head) pair.  Tokens of a scale with side s are the
 * s*s positions of its square token map in row-major raster order (token = y*s + x)
 * (square maps: Preliminaries, Eq. 1 and its footnote).
 *
 * Nothing is tiled, fused or reordered: softmax is the two-pass max / sum form.
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int amskv_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Exact attention of every query over one gathered key set (Eq. 2 conditions a whole
 * scale on whole earlier scales, so there is no mask inside the set):
 *   z_j = scale * <q, k_j>,  p = softmax(z),  out = sum_j p_j v_j.
 * Q,out: [n_items][T][D]; K,V: [n_items][L][D].  L >= 1.
 */
void amskv_oracle_attention(const double* Q, const double* K, const double* V, double* out,
                            long n_items, long T, long L, long D, double scale)
{
#pragma omp parallel
    {
        double* z = (double*)malloc(sizeof(double) * (size_t)L);
#pragma omp for collapse(2) schedule(static)
        for (long it = 0; it < n_items; ++it) {
            for (long q = 0; q < T; ++q) {
                const double* qv = Q + ((size_t)it * T + q) * D;
                const double* Kb = K + (size_t)it * L * D;
                const double* Vb = V + (size_t)it * L * D;
                double* o = out + ((size_t)it * T + q) * D;
                double zmax = -INFINITY;
                for (long j = 0; j < L; ++j) {
                    double acc = 0.0;
                    for (long d = 0; d < D; ++d) acc += qv[d] * Kb[j * D + d];
                    z[j] = scale * acc;
                    if (z[j] > zmax) zmax = z[j];
                }
                double denom = 0.0;
                for (long j = 0; j < L; ++j) {
                    z[j] = exp(z[j] - zmax);
                    denom += z[j];
                }
                for (long d = 0; d < D; ++d) o[d] = 0.0;
                for (long j = 0; j < L; ++j) {
                    double p = z[j] / denom;
                    for (long d = 0; d < D; ++d) o[d] += p * Vb[j * D + d];
                }
            }
        }
        free(z);
    }
}

/*
 * Vanilla next-scale attention in one shot: all tokens of all scales concatenated,
 * query token q sees key token j iff scale_of[j] <= scale_of[q] (Eq. 2: scale k is
 * conditioned on scales <= k, its own tokens included).  This is the "no removal"
 * baseline of Table 1.  Q,K,V,out: [n_items][N][D]; scale_of: [N].
 */
void amskv_oracle_block_causal_attention(const double* Q, const double* K, const double* V,
                                         double* out, const int* scale_of, long n_items, long N,
                                         long D, double scale)
{
#pragma omp parallel
    {
        double* z = (double*)malloc(sizeof(double) * (size_t)N);
#pragma omp for collapse(2) schedule(static)
        for (long it = 0; it < n_items; ++it) {
            for (long q = 0; q < N; ++q) {
                const double* qv = Q + ((size_t)it * N + q) * D;
                const double* Kb = K + (size_t)it * N * D;
                const double* Vb = V + (size_t)it * N * D;
                double* o = out + ((size_t)it * N + q) * D;
                double zmax = -INFINITY;
                for (long j = 0; j < N; ++j) {
                    if (scale_of[j] > scale_of[q]) continue;
                    double acc = 0.0;
                    for (long d = 0; d < D; ++d) acc += qv[d] * Kb[j * D + d];
                    z[j] = scale * acc;
                    if (z[j] > zmax) zmax = z[j];
                }
                double denom = 0.0;
                for (long j = 0; j < N; ++j) {
                    if (scale_of[j] > scale_of[q]) continue;
                    z[j] = exp(z[j] - zmax);
                    denom += z[j];
                }
                for (long d = 0; d < D; ++d) o[d] = 0.0;
                for (long j = 0; j < N; ++j) {
                    if (scale_of[j] > scale_of[q]) continue;
                    double p = z[j] / denom;
                    for (long d = 0; d < D; ++d) o[d] += p * Vb[j * D + d];
                }
            }
        }
        free(z);
    }
}

/*
 * 2-D bilinear resize of a square token map, per item and channel (the "2D
 * interpolation" that produces k-hat in Eq. 4; the paper does not name the mode, so
 * the reading taken is bilinear with half-pixel centres and edge clamping):
 *   src coordinate of output pixel i is (i + 0.5) * s_in / s_out - 0.5, clamped to
 *   [0, s_in - 1]; the two neighbours are floor and floor+1 (clamped).
 * src: [n_items][s_in*s_in][D] -> dst: [n_items][s_out*s_out][D].
 */
void amskv_oracle_bilinear_resize(const double* src, long s_in, double* dst, long s_out,
                                  long n_items, long D)
{
    const double ratio = (double)s_in / (double)s_out;
#pragma omp parallel for schedule(static)
    for (long it = 0; it < n_items; ++it) {
        const double* S = src + (size_t)it * s_in * s_in * D;
        double* O = dst + (size_t)it * s_out * s_out * D;
        for (long y = 0; y < s_out; ++y) {
            double fy = ((double)y + 0.5) * ratio - 0.5;
            if (fy < 0.0) fy = 0.0;
            if (fy > (double)(s_in - 1)) fy = (double)(s_in - 1);
            long y0 = (long)floor(fy);
            long y1 = y0 + 1 < s_in ? y0 + 1 : s_in - 1;
            double wy = fy - (double)y0;
            for (long x = 0; x < s_out; ++x) {
                double fx = ((double)x + 0.5) * ratio - 0.5;
                if (fx < 0.0) fx = 0.0;
                if (fx > (double)(s_in - 1)) fx = (double)(s_in - 1);
                long x0 = (long)floor(fx);
                long x1 = x0 + 1 < s_in ? x0 + 1 : s_in - 1;
                double wx = fx - (double)x0;
                for (long d = 0; d < D; ++d) {
                    double v00 = S[(y0 * s_in + x0) * D + d];
                    double v01 = S[(y0 * s_in + x1) * D + d];
                    double v10 = S[(y1 * s_in + x0) * D + d];
                    double v11 = S[(y1 * s_in + x1) * D + d];
                    double top = v00 + wx * (v01 - v00);
                    double bot = v10 + wx * (v11 - v10);
                    O[(y * s_out + x) * D + d] = top + wy * (bot - top);
                }
            }
        }
    }
}

/*
 * Sum of squared differences between the keys of scale i and the resized keys of
 * scale i-1, over every item, token and channel: the square of the norm in Eq. 4,
 * so that S = -sqrt(ss).  K_prev: [n_items][s_prev^2][D]; K_cur: [n_items][s_cur^2][D].
 */
double amskv_oracle_similarity_ss(const double* K_prev, long s_prev, const double* K_cur,
                                  long s_cur, long n_items, long D)
{
    size_t n = (size_t)n_items * s_cur * s_cur * D;
    double* khat = (double*)malloc(sizeof(double) * n);
    amskv_oracle_bilinear_resize(K_prev, s_prev, khat, s_cur, n_items, D);
    double ss = 0.0;
    for (size_t i = 0; i < n; ++i) {
        double diff = K_cur[i] - khat[i];
        ss += diff * diff;
    }
    free(khat);
    return ss;
}
