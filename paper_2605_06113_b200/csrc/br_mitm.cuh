// Exact Stage-2 subset choice on large windows by meeting in the middle (Algorithms 1 and 2,
// Stage 2; Appendix "Bit-set subset selection").
//
// The score of a candidate subset Q depends on Q only through Delta(Q), and as a function of
// Delta it rises up to a peak and falls after it (Eq. 1: the peak is the safe margin m_g; Eq. 2:
// the kink at which the slope alpha D - beta sum_{passed kinks} d_h stops being positive).  When
// both sides are strictly monotone -- Eq. 1 with G >= 2; Eq. 2 when no segment slope is within
// rounding distance of zero, which the host checks -- the best subset has either the largest
// reachable Delta at or below the peak or the smallest one above it: the two-probe rule of the
// appendix.  The reachable sums are searched exactly: the window is split into its low `ra`
// entries, whose 2^ra subsets are sorted by (size, sum, mask), and its high entries, whose subsets
// are walked one by one; for each of them and each admissible size class one binary search finds
// the neighbours of the peak.  Among subsets of equal Delta, and between the two probes if they
// score the same, the lowest mask wins, as in the enumeration.
#pragma once
#include "br_device.cuh"

namespace br {

constexpr int kMitmMaxLow = 12;                 // the sorted half holds at most 2^12 subsets

struct MitmBest {
    int lo_sum; unsigned lo_mask;               // largest Delta <= peak (lo_sum < 0: none)
    int hi_sum; unsigned hi_mask;               // smallest Delta > peak (hi_sum == INT_MAX: none)
};

__device__ __forceinline__ void mitm_take_lo(MitmBest &b, int sum, unsigned mask)
{
    if (sum > b.lo_sum || (sum == b.lo_sum && mask < b.lo_mask)) { b.lo_sum = sum; b.lo_mask = mask; }
}
__device__ __forceinline__ void mitm_take_hi(MitmBest &b, int sum, unsigned mask)
{
    if (sum < b.hi_sum || (sum == b.hi_sum && mask < b.hi_mask)) { b.hi_sum = sum; b.hi_mask = mask; }
}

// Phase 1: the 2^ra subsets of the low entries as keys (size << 56 | sum << 16 | mask), sorted
// ascending, and the first index of every size class.  nt threads take part (tid < nt); BLOCK:
// barriers are block barriers, else the threads are one warp.
template <bool BLOCK>
__device__ __forceinline__ void mitm_sync() { if (BLOCK) __syncthreads(); else __syncwarp(); }

template <bool BLOCK>
__device__ void mitm_build(const int *win, int ra, unsigned long long *keys, int *cls_off, int tid, int nt)
{
    const int n = 1 << ra;
    for (int m = tid; m < n; m += nt) {
        int sum = 0;
        for (int j = 0; j < ra; ++j) if ((m >> j) & 1) sum += win[j];
        keys[m] = ((unsigned long long)__popc(m) << 56) | ((unsigned long long)(unsigned)sum << 16) | (unsigned)m;
    }
    mitm_sync<BLOCK>();
    // bitonic sort (n is a power of two)
    for (int k2 = 2; k2 <= n; k2 <<= 1) {
        for (int j = k2 >> 1; j > 0; j >>= 1) {
            for (int i = tid; i < n; i += nt) {
                const int p = i ^ j;
                if (p > i) {
                    const unsigned long long x = keys[i], y = keys[p];
                    const bool up = (i & k2) == 0;
                    if ((x > y) == up) { keys[i] = y; keys[p] = x; }
                }
            }
            mitm_sync<BLOCK>();
        }
    }
    // class c starts after C(ra, 0) + ... + C(ra, c - 1) entries
    if (tid == 0) {
        int off = 0, binom = 1;
        for (int c = 0; c <= ra; ++c) { cls_off[c] = off; off += binom; binom = binom * (ra - c) / (c + 1); }
        cls_off[ra + 1] = off;
    }
    mitm_sync<BLOCK>();
}

// Phase 2 for one subset of the high entries (mask_hi, its sum and size): updates b with the
// neighbours of the peak among the admissible classes of the sorted half.
template <typename KEYS, typename OFFS>
__device__ __forceinline__ void mitm_probe(const KEYS keys, const OFFS cls_off, int ra, int lim,
                                           int peak, unsigned mask_hi, int sum_hi, int pop_hi, MitmBest &b)
{
    const int cmax = min(ra, lim - pop_hi);
    const long long target = (long long)peak - sum_hi;              // low-half sums <= target stay at or below the peak
    for (int c = (mask_hi == 0u ? 1 : 0); c <= cmax; ++c) {         // the empty subset is not a candidate
        const int lo = cls_off[c], hi = cls_off[c + 1];
        // u = first entry of the class whose sum exceeds the target
        int a = lo, z = hi;
        while (a < z) {
            const int mid = (a + z) >> 1;
            const long long sm = (long long)((keys[mid] >> 16) & 0xFFFFFFFFFFull);
            if (sm > target) z = mid; else a = mid + 1;
        }
        const int u = a;
        if (u < hi) {
            const unsigned long long e = keys[u];                   // first of its run: the lowest mask with that sum
            mitm_take_hi(b, sum_hi + (int)((e >> 16) & 0xFFFFFFFFFFull), (mask_hi << ra) | (unsigned)(e & 0xFFFFu));
        }
        if (u > lo) {
            const int v = (int)((keys[u - 1] >> 16) & 0xFFFFFFFFFFull);
            int f = u - 1;                                          // walk back to the first entry of the run of sum v
            if (f > lo && (int)((keys[f - 1] >> 16) & 0xFFFFFFFFFFull) == v) {
                int a2 = lo, z2 = f;                                // first entry with sum >= v
                while (a2 < z2) {
                    const int mid = (a2 + z2) >> 1;
                    if ((int)((keys[mid] >> 16) & 0xFFFFFFFFFFull) >= v) z2 = mid; else a2 = mid + 1;
                }
                f = a2;
            }
            mitm_take_lo(b, sum_hi + v, (mask_hi << ra) | (unsigned)(keys[f] & 0xFFFFu));
        }
    }
}

}  // namespace br
