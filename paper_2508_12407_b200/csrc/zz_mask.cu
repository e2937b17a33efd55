// Layer-mask solver: from per-head importances alpha to the exclusive per-layer mask the rest of
// the library consumes (paper: Section 2.2, Eq. 5; the quantile split of Section 2.1, last
// paragraph).  Host code only.
//
// Eq. 5 charges alpha_ij for every retrieval head that a streaming layer turns into a streaming
// head, and -omega * alpha_ij for every streaming head that a retrieval layer turns into a
// retrieval head.  With a_i = sum of alpha over the retrieval heads of layer i and b_i = the sum over
// its streaming heads, a set T of p streaming layers costs
//     sum_{i in T} a_i - omega * sum_{i not in T} b_i  =  sum_{i in T} (a_i + omega * b_i) - omega * sum_i b_i,
// so the optimum is the p layers with the smallest a_i + omega * b_i: a sort instead of the
// enumeration of all C(L, p) subsets.
#include <algorithm>
#include <cmath>
#include <numeric>
#include <vector>

#include "zigzag.h"

extern "C" int zz_layer_mask_solve(const float* alpha, int32_t n_layers, int32_t n_heads, int32_t n_streaming_layers,
                                   double omega, uint8_t* layer_is_retrieval, uint8_t* head_is_retrieval,
                                   double* cost) {
    if (!alpha || !layer_is_retrieval || n_layers < 1 || n_heads < 1) return ZZ_ERR_INVALID_ARG;
    if (n_streaming_layers < 0 || n_streaming_layers > n_layers) return ZZ_ERR_INVALID_ARG;
    if (!(omega >= 0.0 && omega <= 1.0)) return ZZ_ERR_INVALID_ARG;
    const long long n = (long long)n_layers * n_heads;
    for (long long i = 0; i < n; ++i)
        if (!std::isfinite(alpha[i])) return ZZ_ERR_INVALID_ARG;
    // quantile split: the n_streaming_layers * n_heads heads of smallest alpha are streaming heads
    // (equal alphas: the earlier (layer, head) first)
    std::vector<long long> order(n);
    std::iota(order.begin(), order.end(), 0LL);
    std::stable_sort(order.begin(), order.end(), [&](long long x, long long y) { return alpha[x] < alpha[y]; });
    std::vector<uint8_t> is_r(n, 1);
    const long long n_s_heads = (long long)n_streaming_layers * n_heads;
    for (long long r = 0; r < n_s_heads; ++r) is_r[order[r]] = 0;
    // per-layer masses
    std::vector<double> a(n_layers, 0.0), b(n_layers, 0.0), key(n_layers);
    for (int i = 0; i < n_layers; ++i) {
        for (int j = 0; j < n_heads; ++j) {
            const double v = alpha[(long long)i * n_heads + j];
            if (is_r[(long long)i * n_heads + j]) a[i] += v; else b[i] += v;
        }
        key[i] = a[i] + omega * b[i];
    }
    std::vector<int> lo(n_layers);
    std::iota(lo.begin(), lo.end(), 0);
    std::stable_sort(lo.begin(), lo.end(), [&](int x, int y) { return key[x] < key[y]; });
    for (int i = 0; i < n_layers; ++i) layer_is_retrieval[i] = 1;
    for (int r = 0; r < n_streaming_layers; ++r) layer_is_retrieval[lo[r]] = 0;
    if (head_is_retrieval) std::copy(is_r.begin(), is_r.end(), head_is_retrieval);
    if (cost) {
        double c = 0.0;
        for (int i = 0; i < n_layers; ++i) c += layer_is_retrieval[i] ? -omega * b[i] : a[i];
        *cost = c;
    }
    return ZZ_OK;
}
