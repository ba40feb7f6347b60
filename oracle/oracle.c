/*
 * CPU oracle for the pruned-CNN task path.  TEST INFRASTRUCTURE ONLY: it is the slow,
 * plain definition that the CUDA library is checked against and timed beside.  The
 * product never calls it, and it shares no code with the CUDA sources.
 *
 * Everything is float64.  Tensors: activations [N][H][W][C], conv filters
 * [K][C/groups][R][S] (the paper's filter tensor c_{i+1} x c_i x k x k, Sec. 2.1 / Fig. 2),
 * fully-connected weights [out][in].
 *
 * A task is Conv2d + (folded) BatchNorm bias + activation (paper Sec. 3.4, Sec. 3.5);
 * the residual add of a ResNet shortcut (Sec. 3.5, last paragraph) comes before the
 * activation.  The convolution is a cross-correlation with zero padding, dilation 1,
 * output extent floor((H + 2 pad - R) / stride) + 1.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ACT_NONE 0
#define ACT_RELU 1
#define ACT_RELU6 2

static double apply_act(double v, int act) {
    if (act == ACT_RELU) return v > 0.0 ? v : 0.0;
    if (act == ACT_RELU6) return v < 0.0 ? 0.0 : (v > 6.0 ? 6.0 : v);
    return v;
}

/* One output element of the task, before the bias: sum over c, r, s of x * w.
 * *abs_sum receives the sum of |x| * |w| over the same terms. */
static double conv_point(const double *x, int H, int W, int C, const double *w, int K, int R, int S,
                         int groups, int stride, int pad, int n, int p, int q, int k, double *abs_sum) {
    int cg = C / groups;          /* input channels seen by one filter */
    int kg = K / groups;          /* filters per group */
    int c0 = (k / kg) * cg;       /* first input channel of filter k's group */
    double acc = 0.0, aacc = 0.0;
    for (int c = 0; c < cg; ++c)
        for (int r = 0; r < R; ++r)
            for (int s = 0; s < S; ++s) {
                int h = p * stride - pad + r;
                int v = q * stride - pad + s;
                if (h < 0 || h >= H || v < 0 || v >= W) continue; /* zero padding */
                double xv = x[(((size_t)n * H + h) * W + v) * C + c0 + c];
                double wv = w[(((size_t)k * cg + c) * R + r) * S + s];
                acc += xv * wv;
                aacc += fabs(xv) * fabs(wv);
            }
    *abs_sum = aacc;
    return acc;
}

/* y[n][p][q][k] = act(b[k] + conv + res[n][p][q][k]);  bound[...] = |b| + sum|x||w| + |res|.
 * b, res and bound may be NULL. */
void oracle_conv2d(const double *x, int N, int H, int W, int C, const double *w, int K, int R, int S,
                   int groups, const double *b, int stride, int pad, int act, const double *res,
                   double *y, double *bound) {
    int P = (H + 2 * pad - R) / stride + 1;
    int Q = (W + 2 * pad - S) / stride + 1;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int n = 0; n < N; ++n)
        for (int p = 0; p < P; ++p)
            for (int q = 0; q < Q; ++q)
                for (int k = 0; k < K; ++k) {
                    size_t o = (((size_t)n * P + p) * Q + q) * K + k;
                    double a;
                    double v = conv_point(x, H, W, C, w, K, R, S, groups, stride, pad, n, p, q, k, &a);
                    if (b) { v += b[k]; a += fabs(b[k]); }
                    if (res) { v += res[o]; a += fabs(res[o]); }
                    y[o] = apply_act(v, act);
                    if (bound) bound[o] = a;
                }
}

/* The same definition at a list of output coordinates pts[i] = {n, p, q, k}. */
void oracle_conv2d_points(const double *x, int N, int H, int W, int C, const double *w, int K, int R, int S,
                          int groups, const double *b, int stride, int pad, int act, const double *res,
                          const int32_t *pts, int npts, double *y, double *bound) {
    int P = (H + 2 * pad - R) / stride + 1;
    int Q = (W + 2 * pad - S) / stride + 1;
    (void)N;
#pragma omp parallel for schedule(dynamic, 64)
    for (int i = 0; i < npts; ++i) {
        int n = pts[4 * i], p = pts[4 * i + 1], q = pts[4 * i + 2], k = pts[4 * i + 3];
        size_t o = (((size_t)n * P + p) * Q + q) * K + k;
        double a;
        double v = conv_point(x, H, W, C, w, K, R, S, groups, stride, pad, n, p, q, k, &a);
        if (b) { v += b[k]; a += fabs(b[k]); }
        if (res) { v += res[o]; a += fabs(res[o]); }
        y[i] = apply_act(v, act);
        if (bound) bound[i] = a;
    }
}

/* Max-pool k x k; padded positions never win. */
void oracle_maxpool(const double *x, int N, int H, int W, int C, int k, int stride, int pad, double *y) {
    int P = (H + 2 * pad - k) / stride + 1;
    int Q = (W + 2 * pad - k) / stride + 1;
#pragma omp parallel for collapse(2)
    for (int n = 0; n < N; ++n)
        for (int p = 0; p < P; ++p)
            for (int q = 0; q < Q; ++q)
                for (int c = 0; c < C; ++c) {
                    double m = -INFINITY;
                    for (int r = 0; r < k; ++r)
                        for (int s = 0; s < k; ++s) {
                            int h = p * stride - pad + r, v = q * stride - pad + s;
                            if (h < 0 || h >= H || v < 0 || v >= W) continue;
                            double t = x[(((size_t)n * H + h) * W + v) * C + c];
                            if (t > m) m = t;
                        }
                    y[(((size_t)n * P + p) * Q + q) * C + c] = m;
                }
}

/* Global average pool: y[n][c] = mean over h, w. */
void oracle_gap(const double *x, int N, int H, int W, int C, double *y) {
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c) {
            double s = 0.0;
            for (int i = 0; i < H * W; ++i) s += x[((size_t)n * H * W + i) * C + c];
            y[(size_t)n * C + c] = s / (double)(H * W);
        }
}

/* y[n][o] = act(b[o] + sum_i x[n][i] w[o][i]);  bound = |b| + sum |x||w|. */
void oracle_fc(const double *x, int N, int in, const double *w, int out, const double *b, int act,
               double *y, double *bound) {
#pragma omp parallel for
    for (int n = 0; n < N; ++n)
        for (int o = 0; o < out; ++o) {
            double s = 0.0, a = 0.0;
            for (int i = 0; i < in; ++i) {
                double xv = x[(size_t)n * in + i], wv = w[(size_t)o * in + i];
                s += xv * wv;
                a += fabs(xv) * fabs(wv);
            }
            if (b) { s += b[o]; a += fabs(b[o]); }
            y[(size_t)n * out + o] = apply_act(s, act);
            if (bound) bound[(size_t)n * out + o] = a;
        }
}

/* Round to the nearest bfloat16 (8 exponent bits, 7 stored fraction bits), ties to even,
 * computed directly from the float64 value.  Finite inputs well inside the bfloat16 range. */
void oracle_round_bf16(const double *x, size_t n, double *y) {
    for (size_t i = 0; i < n; ++i) {
        double v = x[i];
        if (v == 0.0 || !isfinite(v)) { y[i] = v; continue; }
        int e;
        double m = frexp(fabs(v), &e);        /* |v| = m * 2^e, m in [0.5, 1) */
        if (e < -125) {                       /* below the bfloat16 normal range: fixed quantum 2^-133 */
            double qn = ldexp(1.0, -133);
            y[i] = copysign(nearbyint(fabs(v) / qn) * qn, v);
            continue;
        }
        double scaled = ldexp(m, 8);          /* 8 significant bits: [128, 256) */
        double r = nearbyint(scaled);         /* default rounding mode: nearest, ties to even */
        y[i] = copysign(ldexp(r, e - 8), v);
    }
}

/* L1 norm of each filter on a 2^-40 grid (paper Sec. 3.5: the sum of a filter's absolute
 * weights).  Each |w| is scaled by 2^40 (exact in float64), rounded once to the nearest
 * integer (ties to even), and the integers are added; integer addition has no order
 * dependence, which is what makes the ranking reproducible bit for bit. */
void oracle_l1_norms(const float *w, int K, size_t inner, int64_t *norms) {
    for (int k = 0; k < K; ++k) {
        int64_t s = 0;
        for (size_t i = 0; i < inner; ++i) s += llrint(fabs((double)w[(size_t)k * inner + i]) * 1099511627776.0);
        norms[k] = s;
    }
}

/* Keep the keep_k filters with the largest norm; among equal norms the lower index is
 * kept (stable order).  kept[] receives the surviving indices in ascending order. */
void oracle_select(const int64_t *norms, int K, int keep_k, int32_t *kept) {
    int32_t *order = (int32_t *)malloc(sizeof(int32_t) * (size_t)K);
    for (int i = 0; i < K; ++i) order[i] = i;
    /* stable insertion sort, norm descending */
    for (int i = 1; i < K; ++i) {
        int32_t t = order[i];
        int j = i - 1;
        while (j >= 0 && norms[order[j]] < norms[t]) { order[j + 1] = order[j]; --j; }
        order[j + 1] = t;
    }
    char *flag = (char *)calloc((size_t)K, 1);
    for (int i = 0; i < keep_k; ++i) flag[order[i]] = 1;
    int m = 0;
    for (int i = 0; i < K; ++i) if (flag[i]) kept[m++] = i;
    free(flag);
    free(order);
}
