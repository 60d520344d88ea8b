/*
 * CPU oracle for the block-pruned matrix product (fully connected layer, 1x1
 * convolution in its matrix form).
 *
 * TEST INFRASTRUCTURE ONLY.  Slow, plain definition that the CUDA library is
 * checked against; it shares no code with that library and is never called by it.
 *
 * What it computes (paper Sec. 2.1 "Block-Based Pruning": the weight matrix of a
 * layer is cut into equal blocks, and inside every block whole rows and whole
 * columns are pruned, independently of the other blocks; a convolution is taken
 * in its matrix form):
 *
 *   W [c_out][k]  cut into blocks of br rows x bc columns; block (i, j) covers rows
 *                 i*br .. and columns j*bc ..; blocks at the right and bottom edge
 *                 may be smaller
 *   row_keep [nbr][nbc][br], col_keep [nbr][nbc][bc]  (bytes, 0 = pruned)
 *   Wm[oc][c] = W[oc][c]  if row_keep[oc/br][c/bc][oc%br] and col_keep[oc/br][c/bc][c%bc]
 *             = 0         otherwise (pruned entries are zeroed explicitly)
 *   pre[m][oc] = bias[oc] + sum_c Wm[oc][c] * X[m][c];   Y = relu ? max(pre, 0) : pre
 *
 * with X [m_rows][k] (one row per pixel of an NHWC activation tensor, or per
 * token).  A plain triple loop over the DENSE masked matrix, accumulating in
 * double in ascending column order; it never sees a compacted layout.  OpenMP
 * splits only the rows of X.
 *
 * Parity status: pinned (a hand-computed case, numpy's matrix product on the
 * masked matrix, the unpruned case against a plain product, pruned rows and
 * columns contributing exactly nothing, linearity, constant inputs in closed
 * form, and the error scale by S == y for non-negative terms and S(x, W, b) ==
 * y(|x|, |W|, |b|)) -- see tests/test_oracle_blockgemm_pins.py.
 */
#include <stdint.h>
#include <stdlib.h>
#include <math.h>

/*
 * x [m_rows][k], w [c_out][k], bias [c_out] or NULL, y [m_rows][c_out],
 * s_abs (optional, shaped like y): |bias| + sum |Wm * X|, the scale of the rounding
 * error of any summation order.
 * Returns 0; 2 for a bad shape; 3 if memory runs out.
 */
int blockgemm_ref_f64(const double *x, const double *w, const uint8_t *row_keep, const uint8_t *col_keep,
                      const double *bias, int relu, long m_rows, int k, int c_out, int br, int bc,
                      double *y, double *s_abs) {
    if (m_rows < 0 || k < 1 || c_out < 1 || br < 1 || bc < 1) return 2;
    const int nbc = (k + bc - 1) / bc;
    double *wm = (double *)malloc(sizeof(double) * (size_t)c_out * k);
    if (!wm) return 3;
    for (int oc = 0; oc < c_out; ++oc) {
        for (int c = 0; c < k; ++c) {
            const long blk = (long)(oc / br) * nbc + c / bc;
            const int keep = row_keep[blk * br + oc % br] && col_keep[blk * bc + c % bc];
            wm[(size_t)oc * k + c] = keep ? w[(size_t)oc * k + c] : 0.0;
        }
    }
#pragma omp parallel for schedule(static)
    for (long m = 0; m < m_rows; ++m) {
        for (int oc = 0; oc < c_out; ++oc) {
            double acc = bias ? bias[oc] : 0.0;
            double sab = bias ? fabs(bias[oc]) : 0.0;
            for (int c = 0; c < k; ++c) {
                const double p = wm[(size_t)oc * k + c] * x[(size_t)m * k + c];
                acc += p;
                sab += fabs(p);
            }
            y[(size_t)m * c_out + oc] = (relu && acc < 0.0) ? 0.0 : acc;
            if (s_abs) s_abs[(size_t)m * c_out + oc] = sab;
        }
    }
    free(wm);
    return 0;
}
