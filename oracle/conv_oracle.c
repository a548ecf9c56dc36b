/*
 * CPU oracle for the pattern-pruned 3x3 convolution.  TEST INFRASTRUCTURE ONLY: it is called by the tests,
 * by the smoke check and by the benchmark's CPU-baseline leg, never by the library.  It shares no code, header,
 * table or data structure with the CUDA path and never sees the FKW arrays.
 *
 * What it computes is the plain definition of the layer (Section 2.1 of the paper: a CONV layer followed by
 * ReLU) restricted to 3x3 / stride 1 / pad 1 and applied to weights that satisfy the two constraint sets of
 * Section 4.2 (Eq. 1), i.e. to Wm = weights * mask:
 *
 *   out[n,f,y,x] = act( bias[f] + sum_c sum_r sum_s Wm[f,c,r,s] * in[n,c,y+r-1,x+s-1] ),
 *
 * with the input read as 0 outside the image (cross-correlation, no kernel flip) and act = max(0,.) when relu.
 * Seven nested loops, accumulation and bias add in double, one rounding to float at the end.  The only liberty
 * taken is skipping a (f,c,r,s) whose masked weight is exactly zero, which cannot change a sum.
 */
#include <stddef.h>
#include <stdlib.h>

int oracle_conv3x3(const float *in,            /* [N][C][H][W] */
                   const float *weights,       /* [F][C][3][3] */
                   const unsigned char *mask,  /* [F][C][3][3], 0/1 */
                   const float *bias,          /* [F] or NULL  */
                   int N, int C, int H, int W, int F, int relu,
                   float *out)                 /* [N][F][H][W] */
{
    if (!in || !weights || !mask || !out || N < 0 || C < 1 || H < 1 || W < 1 || F < 1) return 1;
    const size_t plane = (size_t)H * (size_t)W;
    int failed = 0;
#ifdef _OPENMP
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
#endif
    for (int n = 0; n < N; ++n) {
        for (int f = 0; f < F; ++f) {
            double *acc = (double *)malloc(plane * sizeof(double));
            if (!acc) { failed = 1; continue; }
            const double b = bias ? (double)bias[f] : 0.0;
            for (size_t i = 0; i < plane; ++i) acc[i] = 0.0;
            for (int c = 0; c < C; ++c) {
                const float *ip = in + ((size_t)n * C + c) * plane;
                for (int r = 0; r < 3; ++r) {
                    for (int s = 0; s < 3; ++s) {
                        const size_t wi = (((size_t)f * C + c) * 3 + r) * 3 + s;
                        if (!mask[wi]) continue;
                        const double w = (double)weights[wi];
                        if (w == 0.0) continue;
                        for (int y = 0; y < H; ++y) {
                            const int yy = y + r - 1;
                            if (yy < 0 || yy >= H) continue;
                            for (int x = 0; x < W; ++x) {
                                const int xx = x + s - 1;
                                if (xx < 0 || xx >= W) continue;
                                acc[(size_t)y * W + x] += w * (double)ip[(size_t)yy * W + xx];
                            }
                        }
                    }
                }
            }
            float *op = out + ((size_t)n * F + f) * plane;
            for (size_t i = 0; i < plane; ++i) {
                double v = acc[i] + b;
                if (relu && v < 0.0) v = 0.0;
                op[i] = (float)v;
            }
            free(acc);
        }
    }
    return failed ? 2 : 0;
}

/* One output element by the same definition (for spot checks at sizes where the whole tensor is too slow). */
double oracle_conv3x3_point(const float *in, const float *weights, const unsigned char *mask, const float *bias,
                            int C, int H, int W, int relu, int n, int f, int y, int x)
{
    double acc = 0.0;
    const size_t plane = (size_t)H * (size_t)W;
    for (int c = 0; c < C; ++c)
        for (int r = 0; r < 3; ++r)
            for (int s = 0; s < 3; ++s) {
                const size_t wi = (((size_t)f * C + c) * 3 + r) * 3 + s;
                const int yy = y + r - 1, xx = x + s - 1;
                if (!mask[wi] || yy < 0 || yy >= H || xx < 0 || xx >= W) continue;
                acc += (double)weights[wi] * (double)in[((size_t)n * C + c) * plane + (size_t)yy * W + xx];
            }
    acc += bias ? (double)bias[f] : 0.0;
    if (relu && acc < 0.0) acc = 0.0;
    return acc;
}

/* 2x2 / stride 2 max-pool (floor), used only to chain the VGG-shaped stack on the oracle side. */
int oracle_maxpool2x2(const float *in, int N, int C, int H, int W, float *out)
{
    if (!in || !out) return 1;
    const int Ho = H / 2, Wo = W / 2;
    for (size_t nc = 0; nc < (size_t)N * C; ++nc)
        for (int y = 0; y < Ho; ++y)
            for (int x = 0; x < Wo; ++x) {
                const float *p = in + nc * (size_t)H * W + (size_t)(2 * y) * W + 2 * x;
                float m = p[0];
                if (p[1] > m) m = p[1];
                if (p[W] > m) m = p[W];
                if (p[W + 1] > m) m = p[W + 1];
                out[nc * (size_t)Ho * Wo + (size_t)y * Wo + x] = m;
            }
    return 0;
}

#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}
