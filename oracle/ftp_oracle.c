/*
 * CPU oracle for the tiled/fused CNN training step -- TEST INFRASTRUCTURE ONLY.
 *
 * The method (grid tiling of feature and delta maps, fusing, grouping; paper
 * Sections 3 and 4) reaches exactly the result of ordinary, untiled training:
 * the paper states the partition costs no accuracy (abstract) and that the
 * per-tile filter-gradient sets simply add up to the full gradient
 * (Section 4.1).  The oracle is therefore the plain definition of the layer
 * math written out with naive loops in fp64: no tiling, no im2col, no
 * blocking, no reordering.  It shares no code with the CUDA library and must
 * never be used by it; only the tests, the smoke check and the CPU-baseline
 * timing of the benchmark call it.
 *
 * All tensors are dense row-major NCHW doubles.  OpenMP splits only over
 * independent outputs (image, channel), so the summation order of every single
 * output value is fixed and the result is independent of the thread count.
 *
 * Parity pins (tests marked "not gpu"): central finite differences of the
 * loss, agreement with a library conv/pool + autograd in fp64, closed forms
 * for constant inputs, and hand-evaluated tiny cases.  No function here is
 * "parity unpinned".
 */
#include <stddef.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Convolution layer forward (Section 4.1, forward pass of layer l):
 *   Z[n,co,y,x] = b[co] + sum_{ci,ky,kx} F[co,ci,ky,kx] * X[n,ci,y+ky-P,x+kx-P]
 * with X = 0 outside the map (zero padding), stride 1, output size = input
 * size (P = floor(K/2), K odd).  The filter is applied un-rotated; the rotated
 * filter appears only in the delta back-propagation.  Activation:
 *   Y = Z          if Z > 0
 *   Y = slope * Z  otherwise (leaky ReLU; slope 0.1 in every workload).
 * Both Z and Y are returned; the backward pass takes its mask from Z.
 */
void orc_conv_forward(const double *X, const double *F, const double *b,
                      int N, int Cin, int H, int W, int Cout, int K, int P,
                      double slope, double *Z, double *Y)
{
    #pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int co = 0; co < Cout; ++co)
            for (int y = 0; y < H; ++y)
                for (int x = 0; x < W; ++x) {
                    double acc = b[co];
                    for (int ci = 0; ci < Cin; ++ci)
                        for (int ky = 0; ky < K; ++ky) {
                            int iy = y + ky - P;
                            if (iy < 0 || iy >= H) continue;
                            for (int kx = 0; kx < K; ++kx) {
                                int ix = x + kx - P;
                                if (ix < 0 || ix >= W) continue;
                                acc += F[(((size_t)co * Cin + ci) * K + ky) * K + kx] *
                                       X[(((size_t)n * Cin + ci) * H + iy) * W + ix];
                            }
                        }
                    size_t o = (((size_t)n * Cout + co) * H + y) * W + x;
                    Z[o] = acc;
                    Y[o] = acc > 0.0 ? acc : slope * acc;
                }
}

/*
 * Convolution layer backward (Section 4.1, back-propagation of layer l).
 * dY is dLoss/dX_{l+1}.  With dZ = dY * (Z > 0 ? 1 : slope):
 *   db[co]          = sum_{n,y,x} dZ[n,co,y,x]
 *   dF[co,ci,ky,kx] = sum_{n,y,x} dZ[n,co,y,x] * X[n,ci,y+ky-P,x+kx-P]
 *        (feature map convolved with the delta map: the filter gradient)
 *   dX[n,ci,u,v]    = sum_{co,ky,kx} F[co,ci,ky,kx] * dZ[n,co,u-ky+P,v-kx+P]
 *        (delta map correlated with the 180-degree rotated filter)
 * dZ out of range counts as 0.  dF and db are overwritten (not accumulated).
 */
void orc_conv_backward(const double *X, const double *F, const double *Z,
                       const double *dY, int N, int Cin, int H, int W,
                       int Cout, int K, int P, double slope,
                       double *dZ /* scratch N*Cout*H*W */, double *dX,
                       double *dF, double *db)
{
    #pragma omp parallel for schedule(static)
    for (long i = 0; i < (long)N * Cout * H * W; ++i)
        dZ[i] = dY[i] * (Z[i] > 0.0 ? 1.0 : slope);

    #pragma omp parallel for schedule(static)
    for (int co = 0; co < Cout; ++co) {
        double s = 0.0;
        for (int n = 0; n < N; ++n)
            for (int y = 0; y < H; ++y)
                for (int x = 0; x < W; ++x)
                    s += dZ[(((size_t)n * Cout + co) * H + y) * W + x];
        db[co] = s;
    }

    #pragma omp parallel for collapse(2) schedule(static)
    for (int co = 0; co < Cout; ++co)
        for (int ci = 0; ci < Cin; ++ci)
            for (int ky = 0; ky < K; ++ky)
                for (int kx = 0; kx < K; ++kx) {
                    double s = 0.0;
                    for (int n = 0; n < N; ++n)
                        for (int y = 0; y < H; ++y) {
                            int iy = y + ky - P;
                            if (iy < 0 || iy >= H) continue;
                            for (int x = 0; x < W; ++x) {
                                int ix = x + kx - P;
                                if (ix < 0 || ix >= W) continue;
                                s += dZ[(((size_t)n * Cout + co) * H + y) * W + x] *
                                     X[(((size_t)n * Cin + ci) * H + iy) * W + ix];
                            }
                        }
                    dF[(((size_t)co * Cin + ci) * K + ky) * K + kx] = s;
                }

    #pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int ci = 0; ci < Cin; ++ci)
            for (int u = 0; u < H; ++u)
                for (int v = 0; v < W; ++v) {
                    double s = 0.0;
                    for (int co = 0; co < Cout; ++co)
                        for (int ky = 0; ky < K; ++ky) {
                            int y = u - ky + P;
                            if (y < 0 || y >= H) continue;
                            for (int kx = 0; kx < K; ++kx) {
                                int x = v - kx + P;
                                if (x < 0 || x >= W) continue;
                                s += F[(((size_t)co * Cin + ci) * K + ky) * K + kx] *
                                     dZ[(((size_t)n * Cout + co) * H + y) * W + x];
                            }
                        }
                    dX[(((size_t)n * Cin + ci) * H + u) * W + v] = s;
                }
}

/*
 * Max pooling 2x2, stride 2, no padding ("simple pooling operations",
 * Section 3).  H and W must be even.  arg[n,c,y,x] in {0,1,2,3} is the
 * position dy*2+dx of the FIRST maximum in row-major window order (strict
 * '>' scan); the paper does not fix a tie rule, this is the reading both
 * sides use.
 */
void orc_maxpool_forward(const double *X, int N, int C, int H, int W,
                         double *Y, int *arg)
{
    int Ho = H / 2, Wo = W / 2;
    #pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c)
            for (int y = 0; y < Ho; ++y)
                for (int x = 0; x < Wo; ++x) {
                    const double *p = X + (((size_t)n * C + c) * H + 2 * y) * W + 2 * x;
                    double best = p[0];
                    int a = 0;
                    if (p[1] > best)     { best = p[1];     a = 1; }
                    if (p[W] > best)     { best = p[W];     a = 2; }
                    if (p[W + 1] > best) { best = p[W + 1]; a = 3; }
                    size_t o = (((size_t)n * C + c) * Ho + y) * Wo + x;
                    Y[o] = best;
                    arg[o] = a;
                }
}

/* Max pooling backward: the delta of each window goes to its arg-max
 * position, every other position of the window receives 0. */
void orc_maxpool_backward(const double *dY, const int *arg, int N, int C,
                          int H, int W, double *dX)
{
    int Ho = H / 2, Wo = W / 2;
    #pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c) {
            double *d = dX + ((size_t)n * C + c) * H * W;
            for (int i = 0; i < H * W; ++i) d[i] = 0.0;
            for (int y = 0; y < Ho; ++y)
                for (int x = 0; x < Wo; ++x) {
                    size_t o = (((size_t)n * C + c) * Ho + y) * Wo + x;
                    int a = arg[o];
                    d[(2 * y + a / 2) * W + 2 * x + a % 2] = dY[o];
                }
        }
}
