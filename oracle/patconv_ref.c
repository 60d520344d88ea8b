/*
 * CPU oracle for the pattern-pruned 3x3 convolution layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code with that library and is
 * never called by it; only the tests, the smoke check and the benchmark's CPU
 * baseline may use it.
 *
 * What it computes (paper Sec. 2.1 "Pattern-Based Pruning": every surviving
 * 3x3 kernel keeps the 4 weights of one pre-defined pattern; "connectivity
 * pruning" removes whole kernels; Sec. 2.3 "Filter Kernel Reorder and Compact
 * FKW Storage" and "Load Redundancy Elimination" change the execution order and
 * the storage, not the function; Sec. 2.2 operator fusion: bias and ReLU fused
 * into the layer compute the same as separate operators):
 *
 *   pre[n,oy,ox,oc] = bias[oc]
 *        + sum_{ic} sum_{dy=0..2} sum_{dx=0..2} Wm[oc,ic,dy,dx] * X[n, oy*s+dy-1, ox*s+dx-1, ic]
 *   Wm[oc,ic,dy,dx] = W[oc,ic,dy,dx]  if pid[oc,ic] >= 0 and bit (3*dy+dx) of masks[pid[oc,ic]] is set
 *                   = 0               otherwise (pruned entries are zeroed explicitly)
 *   X = 0 outside the image (padding 1);  Y = relu ? max(pre, 0) : pre
 *   Ho = (H + 2 - 3)/s + 1, likewise Wo.  Cross-correlation (no kernel flip).
 *
 * It is a direct convolution over the DENSE 9-tap weight tensor: it never sees
 * a packed or reordered layout.  Floating point accumulates in double in the
 * fixed order (ic, dy, dx); integers accumulate in int64.  OpenMP splits only
 * (n, oy): each output element is summed by one thread in one order, so the
 * result does not depend on the number of cores.
 *
 * Parity status: pinned (hand-computed cases, impulse response, constant-input
 * closed forms, pruned-contributes-nothing, linearity, a library convolution on
 * the masked dense tensor, a scatter-form brute force; the error scale s_abs by a
 * hand-computed case, by S == y for non-negative terms, by S(x, W, b) ==
 * y(|x|, |W|, |b|) and by homogeneity) -- see the CPU tests.
 */
#include <stdint.h>
#include <stdlib.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int patconv_ref_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Dense tensor with pruned entries zeroed: wm[oc][ic][9] (row-major taps). */
static int mask_dense_f64(const double *w, const int16_t *pid, const uint16_t *masks, int P,
                          int c_in, int c_out, double *wm) {
    for (long k = 0; k < (long)c_out * c_in; ++k) {
        int p = pid[k];
        if (p >= P) return 1;
        for (int t = 0; t < 9; ++t) {
            int keep = (p >= 0) && ((masks[p] >> t) & 1);
            wm[k * 9 + t] = keep ? w[k * 9 + t] : 0.0;
        }
    }
    return 0;
}

/*
 * Floating-point layer.  All tensors are double; the caller converts fp32 or
 * fp16 data to double (exact) beforehand.
 *   x [n][h][w][c_in], wt [c_out][c_in][3][3], pid [c_out][c_in], masks [P],
 *   bias [c_out] or NULL, y [n][ho][wo][c_out],
 *   s_abs (optional, same shape as y): |bias| + sum |Wm * X|, the scale of the
 *   rounding error of any summation order.
 * Returns 0, or 1 for a pattern id outside the library, 2 for a bad shape.
 */
int patconv_ref_f64(const double *x, const double *wt, const int16_t *pid, const uint16_t *masks,
                    int P, const double *bias, int relu, int n, int h, int w, int c_in, int c_out,
                    int stride, double *y, double *s_abs) {
    if (n < 0 || h < 1 || w < 1 || c_in < 1 || c_out < 1 || (stride != 1 && stride != 2)) return 2;
    int ho = (h + 2 - 3) / stride + 1, wo = (w + 2 - 3) / stride + 1;
    double *wm = (double *)malloc(sizeof(double) * 9 * (size_t)c_in * c_out);
    if (!wm) return 3;
    if (mask_dense_f64(wt, pid, masks, P, c_in, c_out, wm)) { free(wm); return 1; }
    long rows = (long)n * ho;
#pragma omp parallel for schedule(dynamic, 1)
    for (long r = 0; r < rows; ++r) {
        int in = (int)(r / ho), oy = (int)(r % ho);
        for (int ox = 0; ox < wo; ++ox) {
            for (int oc = 0; oc < c_out; ++oc) {
                double acc = bias ? bias[oc] : 0.0;
                double sab = bias ? fabs(bias[oc]) : 0.0;
                for (int ic = 0; ic < c_in; ++ic) {
                    const double *k9 = wm + ((size_t)oc * c_in + ic) * 9;
                    for (int dy = 0; dy < 3; ++dy) {
                        int iy = oy * stride + dy - 1;
                        if (iy < 0 || iy >= h) continue;       /* padding contributes 0 */
                        for (int dx = 0; dx < 3; ++dx) {
                            int ix = ox * stride + dx - 1;
                            if (ix < 0 || ix >= w) continue;
                            double prod = k9[3 * dy + dx] * x[(((size_t)in * h + iy) * w + ix) * c_in + ic];
                            acc += prod;
                            sab += fabs(prod);
                        }
                    }
                }
                size_t o = (((size_t)in * ho + oy) * wo + ox) * c_out + oc;
                y[o] = (relu && acc < 0.0) ? 0.0 : acc;
                if (s_abs) s_abs[o] = sab;
            }
        }
    }
    free(wm);
    return 0;
}

/*
 * Integer layer: uint8 activations, int8 weights, int32 bias, exact int64
 * accumulation.  y is int64 so the caller can check that every value fits
 * int32 before comparing with an int32 result.
 */
int patconv_ref_i64(const uint8_t *x, const int8_t *wt, const int16_t *pid, const uint16_t *masks,
                    int P, const int32_t *bias, int relu, int n, int h, int w, int c_in, int c_out,
                    int stride, int64_t *y) {
    if (n < 0 || h < 1 || w < 1 || c_in < 1 || c_out < 1 || (stride != 1 && stride != 2)) return 2;
    int ho = (h + 2 - 3) / stride + 1, wo = (w + 2 - 3) / stride + 1;
    int32_t *wm = (int32_t *)malloc(sizeof(int32_t) * 9 * (size_t)c_in * c_out);
    if (!wm) return 3;
    for (long k = 0; k < (long)c_out * c_in; ++k) {
        int p = pid[k];
        if (p >= P) { free(wm); return 1; }
        for (int t = 0; t < 9; ++t) {
            int keep = (p >= 0) && ((masks[p] >> t) & 1);
            wm[k * 9 + t] = keep ? (int32_t)wt[k * 9 + t] : 0;
        }
    }
    long rows = (long)n * ho;
#pragma omp parallel for schedule(dynamic, 1)
    for (long r = 0; r < rows; ++r) {
        int in = (int)(r / ho), oy = (int)(r % ho);
        for (int ox = 0; ox < wo; ++ox) {
            for (int oc = 0; oc < c_out; ++oc) {
                int64_t acc = bias ? (int64_t)bias[oc] : 0;
                for (int ic = 0; ic < c_in; ++ic) {
                    const int32_t *k9 = wm + ((size_t)oc * c_in + ic) * 9;
                    for (int dy = 0; dy < 3; ++dy) {
                        int iy = oy * stride + dy - 1;
                        if (iy < 0 || iy >= h) continue;
                        for (int dx = 0; dx < 3; ++dx) {
                            int ix = ox * stride + dx - 1;
                            if (ix < 0 || ix >= w) continue;
                            acc += (int64_t)k9[3 * dy + dx] *
                                   (int64_t)x[(((size_t)in * h + iy) * w + ix) * c_in + ic];
                        }
                    }
                }
                size_t o = (((size_t)in * ho + oy) * wo + ox) * c_out + oc;
                y[o] = (relu && acc < 0) ? 0 : acc;
            }
        }
    }
    free(wm);
    return 0;
}

/*
 * Operators fused behind the convolution (paper Sec. 2.2, "universal operator fusion": the
 * operators that follow a convolution -- an element-wise addition, the activation, a pooling, a
 * re-quantisation -- are computed together with it, so the intermediate tensors are never
 * written).  The fused result is by definition what the separate operators give, applied in this
 * order to the convolution's output before any activation:
 *
 *   v = pre[n,oy,ox,oc] (+ residual[n,oy,ox,oc]);   v = relu ? max(v, 0) : v;
 *   pool = 2:  out[n,qy,qx,oc] = max of v over oy in {2qy, 2qy+1}, ox in {2qx, 2qx+1}
 *              (Ho and Wo must be even);   pool = 0: out = v.
 *
 * `pre` is what patconv_ref_f64 returns with relu = 0 (bias included).  Plain loops, double.
 * Returns 0, or 2 for a bad shape.
 */
int patconv_ref_fused_f64(const double *pre, const double *residual, int relu, int pool,
                          int n, int ho, int wo, int c, double *out) {
    if (n < 0 || ho < 1 || wo < 1 || c < 1 || (pool != 0 && pool != 2)) return 2;
    if (pool == 2 && ((ho & 1) || (wo & 1))) return 2;
    const int step = pool == 2 ? 2 : 1;
    const int po = ho / step, pw = wo / step;
    for (int in = 0; in < n; ++in)
        for (int qy = 0; qy < po; ++qy)
            for (int qx = 0; qx < pw; ++qx)
                for (int oc = 0; oc < c; ++oc) {
                    double best = 0.0;
                    int first = 1;
                    for (int dy = 0; dy < step; ++dy)
                        for (int dx = 0; dx < step; ++dx) {
                            size_t i = (((size_t)in * ho + (qy * step + dy)) * wo + (qx * step + dx)) * c + oc;
                            double v = pre[i];
                            if (residual) v += residual[i];
                            if (relu && v < 0.0) v = 0.0;
                            if (first || v > best) best = v;
                            first = 0;
                        }
                    out[(((size_t)in * po + qy) * pw + qx) * c + oc] = best;
                }
    return 0;
}

/*
 * The same for the integer layer, followed, if scale is given, by the re-quantisation to uint8:
 *
 *   q = clamp( rne( (float)v * scale[oc] ) + zero_point, 0, 255 )
 *
 * The product is an fp32 product of the int32 value converted to fp32 (round to nearest even)
 * and the fp32 scale; rne rounds it to the nearest integer, ties to even.  fp32 is the
 * precision in which the device takes this decision, so the oracle takes it in fp32 too: a
 * quantised code is an integer and has to match exactly.  v must fit int32 (returns 4 if not).
 * out_i64 receives v (after pooling) when scale is NULL, out_u8 the codes otherwise.
 */
int patconv_ref_fused_i64(const int64_t *pre, const int32_t *residual, int relu, int pool,
                          int n, int ho, int wo, int c, const float *scale, int zero_point,
                          int64_t *out_i64, uint8_t *out_u8) {
    if (n < 0 || ho < 1 || wo < 1 || c < 1 || (pool != 0 && pool != 2)) return 2;
    if (pool == 2 && ((ho & 1) || (wo & 1))) return 2;
    const int step = pool == 2 ? 2 : 1;
    const int po = ho / step, pw = wo / step;
    for (int in = 0; in < n; ++in)
        for (int qy = 0; qy < po; ++qy)
            for (int qx = 0; qx < pw; ++qx)
                for (int oc = 0; oc < c; ++oc) {
                    int64_t best = 0;
                    int first = 1;
                    for (int dy = 0; dy < step; ++dy)
                        for (int dx = 0; dx < step; ++dx) {
                            size_t i = (((size_t)in * ho + (qy * step + dy)) * wo + (qx * step + dx)) * c + oc;
                            int64_t v = pre[i];
                            if (residual) v += (int64_t)residual[i];
                            if (relu && v < 0) v = 0;
                            if (first || v > best) best = v;
                            first = 0;
                        }
                    if (best > 2147483647LL || best < -2147483648LL) return 4;
                    size_t o = (((size_t)in * po + qy) * pw + qx) * c + oc;
                    if (scale) {
                        volatile float prod = (float)(int32_t)best * scale[oc];   /* one fp32 rounding */
                        float r = nearbyintf(prod);                               /* ties to even */
                        double q = (double)r + (double)zero_point;
                        if (q < 0.0) q = 0.0;
                        if (q > 255.0) q = 255.0;
                        out_u8[o] = (uint8_t)q;
                    } else {
                        out_i64[o] = best;
                    }
                }
    return 0;
}

/*
 * Depthwise pattern-pruned 3x3 convolution (paper Sec. 2.1: pattern pruning "can
 * generalize" beyond the dense 3x3 layer; here every channel has ONE 3x3 kernel of
 * its own, which keeps the 4 weights of its pattern or is removed altogether):
 *
 *   pre[n,oy,ox,c] = bias[c] + sum_{dy,dx} Wm[c,dy,dx] * X[n, oy*s+dy-1, ox*s+dx-1, c]
 *   Wm[c,dy,dx] = W[c,dy,dx] if pid[c] >= 0 and bit (3*dy+dx) of masks[pid[c]] is set, else 0
 *
 * with zero padding 1, stride s in {1,2}, Y = relu ? max(pre, 0) : pre.  Plain loops over
 * the dense 9-tap kernels, double accumulation in the order (dy, dx).
 *   x [n][h][w][c], wt [c][3][3], pid [c], bias [c] or NULL, y [n][ho][wo][c],
 *   s_abs optional, shaped like y: |bias| + sum |Wm * X|.
 * Parity status: pinned (a hand-computed case, the full layer's oracle with a diagonal
 * connectivity, closed forms for constant input, pruned taps and removed channels
 * contributing nothing, linearity, the error scale) -- tests/test_oracle_dwconv_pins.py.
 * Returns 0, 1 for a pattern id outside the library, 2 for a bad shape.
 */
int dwconv_ref_f64(const double *x, const double *wt, const int16_t *pid, const uint16_t *masks, int P,
                   const double *bias, int relu, int n, int h, int w, int c, int stride,
                   double *y, double *s_abs) {
    if (n < 0 || h < 1 || w < 1 || c < 1 || (stride != 1 && stride != 2)) return 2;
    for (int ch = 0; ch < c; ++ch) if (pid[ch] >= P) return 1;
    int ho = (h + 2 - 3) / stride + 1, wo = (w + 2 - 3) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int in = 0; in < n; ++in) {
        for (int oy = 0; oy < ho; ++oy) {
            for (int ox = 0; ox < wo; ++ox) {
                for (int ch = 0; ch < c; ++ch) {
                    double acc = bias ? bias[ch] : 0.0;
                    double sab = bias ? fabs(bias[ch]) : 0.0;
                    const int p = pid[ch];
                    for (int dy = 0; dy < 3; ++dy) {
                        for (int dx = 0; dx < 3; ++dx) {
                            const int keep = (p >= 0) && ((masks[p] >> (3 * dy + dx)) & 1);
                            const int iy = oy * stride + dy - 1, ix = ox * stride + dx - 1;
                            if (!keep || iy < 0 || iy >= h || ix < 0 || ix >= w) continue;
                            const double t = wt[(size_t)ch * 9 + 3 * dy + dx] * x[(((size_t)in * h + iy) * w + ix) * c + ch];
                            acc += t;
                            sab += fabs(t);
                        }
                    }
                    const size_t o = (((size_t)in * ho + oy) * wo + ox) * c + ch;
                    y[o] = (relu && acc < 0.0) ? 0.0 : acc;
                    if (s_abs) s_abs[o] = sab;
                }
            }
        }
    }
    return 0;
}
