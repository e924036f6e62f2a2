// Fused decode launches: several layers that read the same activations share one row-owner grid.  The SMs
// are dealt out to the layers in proportion to their vector rows and every CTA works on one layer exactly as
// in a launch of its own.
#pragma once
#include "common.cuh"

namespace vptq {

constexpr int MAX_FUSED = 4;                // layers of one fused launch (VPTQ_MAX_FUSED_LAYERS)

// CTAs [cta_begin[l], cta_begin[l + 1]) work on layer l (every layer at least one; leftover SMs go where the
// most rows per CTA remain).  *rows_cta = the most vector rows any CTA gets.  False when there are fewer rows
// than SMs or whole rows would load the SMs less than 80 % evenly.
inline bool split_ctas(const int *rows, int n, int G, int *cta_begin, int *rows_cta)
{
    if (n < 2 || n > MAX_FUSED) return false;
    long long total = 0;
    for (int l = 0; l < n; l++) total += rows[l];
    if (total < G) return false;
    int ctas[MAX_FUSED], used = 0;
    for (int l = 0; l < n; l++) {
        ctas[l] = (int)((long long)G * rows[l] / total);
        if (ctas[l] < 1) ctas[l] = 1;
        used += ctas[l];
    }
    if (used > G) return false;
    for (; used < G; used++) {
        int best = 0;
        for (int l = 1; l < n; l++)
            if (ceil_div(rows[l], ctas[l]) > ceil_div(rows[best], ctas[best])) best = l;
        ctas[best]++;
    }
    int most = 0;
    cta_begin[0] = 0;
    for (int l = 0; l < n; l++) {
        const int per = ceil_div(rows[l], ctas[l]);
        most = most > per ? most : per;
        cta_begin[l + 1] = cta_begin[l] + ctas[l];
    }
    *rows_cta = most;
    return (double)total / ((double)G * most) >= 0.80;
}

// same format apart from the number of output rows, the tables and the column order
inline bool same_geometry(const LayerView &a, const LayerView &b)
{
    return a.N == b.N && a.v == b.v && a.k1 == b.k1 && a.k2 == b.k2 && a.n_out == b.n_out && a.v0 == b.v0 &&
           a.k0 == b.k0 && a.G == b.G && a.has_scale == b.has_scale && a.scale_rows == b.scale_rows &&
           a.x_bf16 == b.x_bf16;
}

}  // namespace vptq
