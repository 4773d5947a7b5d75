/*
 * CPU oracle for forward 2-D convolution -- TEST INFRASTRUCTURE ONLY.
 *
 * Only the tests, the smoke check and the benchmark's cpu-baseline leg may
 * build, load or call this file.  It shares no code, header, table or helper
 * with the CUDA library and must never be reachable from the product path.
 *
 * What it computes (the paper's problem statement: Fig. 3a -- one C-channel
 * image, F filters of size K x K x C, F output maps; Section 3.1 -- a block
 * needs extra pixels only beyond its right and bottom edges, i.e. outputs are
 * anchored top-left: "valid" extent, stride 1; Section 4 -- one output is
 * K x K fused multiply-adds per channel, accumulated over all channels;
 * Algorithm 2's update reads the image at an offset that grows with the tap
 * index, i.e. the filter is applied un-flipped):
 *
 *   y[n,k,p,q]    = sum_{c,r,s}  x[n,c,p+r,q+s] * w[k,c,r,s]
 *   yabs[n,k,p,q] = sum_{c,r,s} |x[n,c,p+r,q+s] * w[k,c,r,s]|
 *
 * with P = H-R+1, Q = W-S+1.  Symbols here are the library's (N batch, C
 * channels, H x W image, K filters, R x S taps); the paper writes F for the
 * filter count and K for the square filter size and has no batch.
 *
 * The definition is written out as seven literal nested loops in the order
 * n,k,p,q,c,r,s.  Each product is formed in double (exact: two 24-bit
 * significands) and summed in double in that order.  OpenMP only distributes
 * whole output rows over threads, so every output is summed sequentially by
 * one thread and the result does not depend on the thread count.
 *
 * Operand modes (diagnostics for the tensor-core path; the parity reference
 * is always mode 0):
 *   0  operands used as given (fp32 values, exact products)
 *   1  both operands first rounded to TF32 (10 explicit mantissa bits),
 *      round-to-nearest with ties away from zero
 *   2  both operands first truncated to TF32 (low 13 mantissa bits cleared)
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static float to_tf32(float v, int mode)
{
    uint32_t u;
    memcpy(&u, &v, sizeof u);
    if (mode == 1) {
        /* nearest, ties away: add half an ulp of the 10-bit mantissa, then clear.
           Finite inputs of the tests never overflow the exponent here. */
        if ((u & 0x7f800000u) != 0x7f800000u) u += 0x00001000u;
    }
    if (mode != 0) u &= 0xffffe000u;
    memcpy(&v, &u, sizeof u);
    return v;
}

int conv2d_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Computes output rows p in [p_begin, p_end) of maps k in [k_begin, k_end) of
 * images n in [n_begin, n_end) into dense arrays
 * [n_end-n_begin][k_end-k_begin][p_end-p_begin][Q]; the whole problem is the
 * range [0,N) x [0,K) x [0,P).  y64 and yabs may each be NULL.
 * Returns 0, or 1 on a bad argument.
 */
int conv2d_oracle_range(const float *x, const float *w,
                        double *y64, double *yabs,
                        int N, int C, int H, int W, int K, int R, int S,
                        int n_begin, int n_end, int k_begin, int k_end,
                        int p_begin, int p_end, int mode)
{
    if (!x || !w) return 1;
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0 || K <= 0 || R <= 0 || S <= 0) return 1;
    if (R > H || S > W) return 1;
    const int P = H - R + 1, Q = W - S + 1;
    if (n_begin < 0 || n_end > N || k_begin < 0 || k_end > K || p_begin < 0 || p_end > P) return 1;
    if (n_begin > n_end || k_begin > k_end || p_begin > p_end) return 1;
    if (mode < 0 || mode > 2) return 1;

    const int nn = n_end - n_begin, nk = k_end - k_begin, np = p_end - p_begin;
    const long long rows = (long long)nn * nk * np;

#pragma omp parallel for schedule(static)
    for (long long row = 0; row < rows; ++row) {
        const int n = n_begin + (int)(row / ((long long)nk * np));
        const int k = k_begin + (int)((row / np) % nk);
        const int p = p_begin + (int)(row % np);
        for (int q = 0; q < Q; ++q) {
            double acc = 0.0, mag = 0.0;
            for (int c = 0; c < C; ++c) {
                for (int r = 0; r < R; ++r) {
                    for (int s = 0; s < S; ++s) {
                        const size_t xi = (((size_t)n * C + c) * H + (size_t)(p + r)) * W + (size_t)(q + s);
                        const size_t wi = (((size_t)k * C + c) * R + (size_t)r) * S + (size_t)s;
                        const double prod = (double)to_tf32(x[xi], mode) * (double)to_tf32(w[wi], mode);
                        acc += prod;
                        mag += fabs(prod);
                    }
                }
            }
            const size_t yi = (((size_t)(n - n_begin) * nk + (size_t)(k - k_begin)) * np + (size_t)(p - p_begin)) * Q + (size_t)q;
            if (y64) y64[yi] = acc;
            if (yabs) yabs[yi] = mag;
        }
    }
    return 0;
}
