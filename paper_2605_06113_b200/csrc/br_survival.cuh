// Empirical-survival realisation of the two-stage prediction interface (Appendix "Estimator
// realizations", paragraph "Empirical-survival"; Eqs. 3-5): both stages are read off the
// empirical CDF of a sorted history of output lengths o_j.  For a request that has produced a
// tokens,
//     p_fin  = #{a < o_j <= a + H} / #{o_j > a},
//     mu_rem = mean of (o_j - a) over a < o_j <= a + H,
//     c_hat  = (1 - p_fin) H + p_fin mu_rem, clipped to [0, H].
// One thread per request: two upper-bound searches in the sorted history and two reads of its
// prefix sums.  A request older than every recorded output (or with no recorded output in the
// window) has p_fin = 0 and keeps the conservative anchor c_hat = H.
#pragma once
#include "br_device.cuh"

namespace br {

struct SurvivalArgs {
    const int32_t *hist;      // [n_hist] output lengths, ascending
    const int64_t *prefix;    // [n_hist + 1] prefix[j] = sum of hist[0 .. j)
    int32_t n_hist, H;
    const int32_t *age;       // [count] tokens produced so far a_i(k)
    int64_t count;
    float *c_hat;             // [count]
    double *p_fin, *mu_rem;   // [count] or NULL
};

// number of history entries <= x
__device__ __forceinline__ int count_le(const int32_t *__restrict__ hist, int n, long long x)
{
    int lo = 0, hi = n;                       // entries [0, lo) are <= x, entries [hi, n) are > x
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if ((long long)__ldg(hist + mid) <= x) lo = mid + 1; else hi = mid;
    }
    return lo;
}

__global__ void __launch_bounds__(256) br_survival_kernel(const SurvivalArgs a)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= a.count) return;
    const long long age = a.age[i];
    const int lo = count_le(a.hist, a.n_hist, age);
    const int hi = count_le(a.hist, a.n_hist, age + a.H);
    const long long c0 = a.n_hist - lo, c1 = hi - lo;
    double p = 0.0, mu = (double)a.H, c = (double)a.H;
    if (c1 > 0) {
        const long long sum1 = (__ldg(a.prefix + hi) - __ldg(a.prefix + lo)) - age * c1;
        p = __ddiv_rn((double)c1, (double)c0);
        mu = __ddiv_rn((double)sum1, (double)c1);
        c = __dadd_rn(__dmul_rn(__dsub_rn(1.0, p), (double)a.H), __dmul_rn(p, mu));
        c = c < 0.0 ? 0.0 : (c > (double)a.H ? (double)a.H : c);
    }
    a.c_hat[i] = (float)c;
    if (a.p_fin) a.p_fin[i] = p;
    if (a.mu_rem) a.mu_rem[i] = mu;
}

}  // namespace br
