/* CPU checker, TEST INFRASTRUCTURE ONLY: softmax attention restricted to a visibility set,
 * written out as its definition in float64.  Shares no code with the CUDA library.
 *
 * For one scene and one layer, every packed query a (one per parallel field, Sec. 3.3 of
 * the paper: "packed along the sequence length dimension") and every query head h:
 *     g      = h / (Hq / Hkv)                        (grouped-query head mapping)
 *     s_r    = scale * sum_d q[a][h][d] * K[g][r][d]  for every VISIBLE row r
 *     p_r    = exp(s_r - max_r s_r) / sum_r exp(s_r - max_r s_r)
 *     o[d]   = sum_r p_r * V[g][r][d]
 * Invisible rows (independent fields, padding, rows not written yet) take no part at
 * all: their K and V values are never read.  Inputs are the exact fp32 values (bf16
 * inputs are widened by the caller, which is exact).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* q [A][Hq][D], K and V [Hkv][R][D] (row stride D), vis [A][R] (0/1), out [A][Hq][D].
 * Returns the number of threads used, or -1 if a query sees no row at all. */
int fdc_oracle_attention(const float* q, const float* K, const float* V, const uint8_t* vis,
                         int A, int Hq, int Hkv, int R, int D, double scale, double* out,
                         int nthreads)
{
    int G = Hq / Hkv;
    int bad = 0;
    int used = 1;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
    used = nthreads > 0 ? nthreads : omp_get_max_threads();
#endif
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int a = 0; a < A; ++a) {
        for (int h = 0; h < Hq; ++h) {
            int g = h / G;
            const float* qv = q + ((size_t)a * Hq + h) * D;
            const float* Kg = K + (size_t)g * R * D;
            const float* Vg = V + (size_t)g * R * D;
            const uint8_t* va = vis + (size_t)a * R;
            double* o = out + ((size_t)a * Hq + h) * D;
            double* s = (double*)malloc(sizeof(double) * (size_t)R);
            double smax = -INFINITY;
            int nvis = 0;
            for (int r = 0; r < R; ++r) {
                if (!va[r]) continue;
                double acc = 0.0;
                for (int d = 0; d < D; ++d) acc += (double)qv[d] * (double)Kg[(size_t)r * D + d];
                s[r] = scale * acc;
                if (s[r] > smax) smax = s[r];
                ++nvis;
            }
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            if (nvis == 0) {
#pragma omp atomic write
                bad = 1;
                free(s);
                continue;
            }
            double denom = 0.0;
            for (int r = 0; r < R; ++r) {
                if (!va[r]) continue;
                double e = exp(s[r] - smax);
                denom += e;
                for (int d = 0; d < D; ++d) o[d] += e * (double)Vg[(size_t)r * D + d];
            }
            for (int d = 0; d < D; ++d) o[d] /= denom;
            free(s);
        }
    }
    return bad ? -1 : used;
}
