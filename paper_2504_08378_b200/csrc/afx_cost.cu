// afx_cost_*: the cost model of the swapping pipeline and the greedy parameter search
// (Sec. 4.1 "Elastic and Optimized LLM Execution", Eq. 1-9).  Host arithmetic only.
#include <math.h>

#include "afx.h"

extern "C" afx_status afx_cost_eval(const afx_cost_params* p, afx_cost* out) {
    if (p == nullptr || out == nullptr) return AFX_ERR_INVALID_ARG;
    if (!(p->sp >= 0.0 && p->sp <= 1.0) || !(p->hr >= 0.0 && p->hr <= 1.0) || !(p->si >= 0.0 && p->si <= 1.0) ||
        p->N < 1 || !(p->S_l > 0.0) || !(p->bw_mem > 0.0) || !(p->bw_flash_small > 0.0) || !(p->bw_flash_large > 0.0) ||
        !(p->M_cache >= 0.0) || !(p->M_kv >= 0.0) || p->n_layers < 0)
        return AFX_ERR_INVALID_ARG;
    afx_cost c;
    c.M_cl = p->S_l * (1.0 - p->sp) * p->N;                                             // Eq. 9
    c.M = c.M_cl + p->M_cache + p->M_kv;                                                // Eq. 8
    c.T_load = c.M_cl * (1.0 - p->hr) / p->bw_flash_small;                              // Eq. 3
    c.T_comp = c.M_cl / p->bw_mem;                                                      // Eq. 4
    c.T_onload = p->S_l * (1.0 - p->sp) * (1.0 - p->hr) * (1.0 - p->si) / p->bw_flash_small;  // Eq. 6
    c.T_preload = c.M_cl * (1.0 - p->hr) / p->bw_flash_large;                           // Eq. 7
    c.T_overlap = c.T_onload + (c.T_preload > c.T_comp ? c.T_preload : c.T_comp);       // Eq. 5
    c.T_decode = c.T_load + c.T_overlap + c.T_comp;                                     // Eq. 1
    const int groups = p->n_layers > 0 ? (p->n_layers + p->N - 1) / p->N : 2;
    c.T_token = c.T_load + (groups - 1) * c.T_overlap + c.T_comp;
    *out = c;
    return AFX_OK;
}

// Piecewise-linear reading of a measured table (x ascending); clamped at both ends.
static double table_at(const double* x, const double* y, int n, double at) {
    if (at <= x[0]) return y[0];
    for (int i = 1; i < n; ++i)
        if (at <= x[i]) return y[i - 1] + (y[i] - y[i - 1]) * (at - x[i - 1]) / (x[i] - x[i - 1]);
    return y[n - 1];
}

extern "C" afx_status afx_cost_search(const afx_cost_search_in* in, afx_cost_choice* out) {
    if (in == nullptr || out == nullptr) return AFX_ERR_INVALID_ARG;
    if (!(in->S_m > 0.0) || !(in->S_l > 0.0) || in->n_layers < 1 || !(in->M_max > 0.0) || !(in->M_kv >= 0.0) ||
        !(in->bw_mem > 0.0) || !(in->bw_flash_small > 0.0) || in->n_chunk < 1 || in->chunk_bytes == nullptr ||
        in->chunk_bw == nullptr || !(in->column_bytes > 0.0) || in->n_hr < 1 || in->hr_cache_frac == nullptr ||
        in->hr_value == nullptr || !(in->si >= 0.0 && in->si <= 1.0) || !(in->min_gain >= 0.0) || in->N_max < 1)
        return AFX_ERR_INVALID_ARG;
    for (int i = 1; i < in->n_chunk; ++i)
        if (!(in->chunk_bytes[i] > in->chunk_bytes[i - 1])) return AFX_ERR_INVALID_ARG;
    for (int i = 1; i < in->n_hr; ++i)
        if (!(in->hr_cache_frac[i] > in->hr_cache_frac[i - 1])) return AFX_ERR_INVALID_ARG;
    // 1. the sparsity the memory budget asks for: sp = 1 - M_max / S_m
    double sp = 1.0 - in->M_max / in->S_m;
    if (sp < 0.0) sp = 0.0;
    afx_cost_choice best = {};
    double prev_per_layer = 0.0;
    int stop = AFX_COST_STOP_N_MAX;
    // 2. grow the cross-layer group one layer at a time
    for (int N = 1; N <= in->N_max && N <= in->n_layers; ++N) {
        afx_cost_params p = {};
        p.sp = sp;
        p.si = in->si;
        p.N = N;
        p.n_layers = in->n_layers;
        p.S_l = in->S_l;
        p.bw_mem = in->bw_mem;
        p.bw_flash_small = in->bw_flash_small;
        p.bw_flash_large = table_at(in->chunk_bytes, in->chunk_bw, in->n_chunk, N * in->column_bytes);
        p.M_kv = in->M_kv;
        const double M_cl = in->S_l * (1.0 - sp) * N;
        if (M_cl + in->M_kv > in->M_max) {  // the group alone no longer fits
            if (N == 1) return AFX_ERR_CAPACITY;
            stop = AFX_COST_STOP_MEMORY;
            break;
        }
        p.M_cache = in->M_max - in->M_kv - M_cl;  // what is left goes to the weight cache
        p.hr = table_at(in->hr_cache_frac, in->hr_value, in->n_hr, p.M_cache / in->S_m);
        afx_cost c;
        const afx_status rc = afx_cost_eval(&p, &c);
        if (rc != AFX_OK) return rc;
        const double per_layer = c.T_preload / N;
        if (N > 1 && prev_per_layer > 0.0 && (prev_per_layer - per_layer) < in->min_gain * prev_per_layer) {
            stop = AFX_COST_STOP_GAIN;  // one more layer no longer pays: keep the previous choice
            break;
        }
        best.sp = sp;
        best.N = N;
        best.M_cache = p.M_cache;
        best.hr = p.hr;
        best.bw_flash_large = p.bw_flash_large;
        best.cost = c;
        prev_per_layer = per_layer;
        if (c.T_preload <= c.T_comp) {  // preloading hides behind the computation
            stop = AFX_COST_STOP_BALANCED;
            break;
        }
    }
    best.stop_reason = stop;
    *out = best;
    return AFX_OK;
}
