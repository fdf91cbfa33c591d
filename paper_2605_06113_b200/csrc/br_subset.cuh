// Batched exact solver of the Stage-2 subproblem (Algorithm 1 / 2, Stage 2; Appendix
// "Bit-set subset selection"): among the non-empty subsets Q of a window of R requests with
// |Q| <= lim, the one with the highest F_g(Q), lowest mask on ties.  The score depends on Q only
// through Delta(Q), so all 2^R - 1 subsets are enumerated in parallel: one thread block per
// problem, thread t owns the low 8 mask bits, the high bits are walked in Gray-code order so that
// each step changes Delta by one window entry.  Scores are those of the step kernels (Eq. 1 in
// integers, Eq. 2 in fp64 term by term).  Windows beyond the five entries the step kernels handle
// (R up to 20) are what this entry point is for.
#pragma once
#include "br_device.cuh"
#include "br_fscore.cuh"
#include "../../include/br.h"

namespace br {

constexpr int kSubsetMaxR = 20;

struct SubsetArgs {
    FscoreArgs f;           // G, H, fp, aD, beta, d (the other fields are unused)
    int32_t R, first_instance;
    const int32_t *win;     // [N][R]   prompt lengths of the window, bit j of a mask = entry j
    const int64_t *m;       // [N][H+1] margins m_{g,h} of the worker
    const int32_t *lim;     // [N]      largest |Q| (free slots of the worker, at most R)
    uint32_t *best_mask;    // [N]
    double *best_F;         // [N] or NULL
};

__global__ void __launch_bounds__(256) br_subset_kernel(const SubsetArgs a)
{
    __shared__ long long m_s[BR_MAX_H + 1];
    __shared__ int win_s[kSubsetMaxR];
    __shared__ long long red_key[64];
    __shared__ int red_idx[64];
    const int tid = threadIdx.x, R = a.R, H1 = a.f.H + 1;
    const size_t p = (size_t)a.first_instance + blockIdx.x;
    if (tid < H1) m_s[tid] = a.m[p * H1 + tid];
    if (tid < R) win_s[tid] = a.win[p * R + tid];
    __syncthreads();
    int lim = a.lim[p];
    lim = lim < 0 ? 0 : lim;
    const int lowbits = R < 8 ? R : 8, highbits = R - lowbits;
    Best best; best.key = kNoKey; best.idx = kNoIdx;
    if (tid < (1 << lowbits)) {
        int delta = 0;
        for (int j = 0; j < lowbits; ++j) if ((tid >> j) & 1) delta += win_s[j];
        const int cnt_lo = __popc(tid);
        unsigned hi = 0;                                  // Gray code of the step counter
        const unsigned n_hi = 1u << highbits;
        for (unsigned c = 0; c < n_hi; ++c) {
            const unsigned mask = (hi << lowbits) | (unsigned)tid;
            if (mask != 0u && cnt_lo + __popc(hi) <= lim) {
                const long long key = fscore_key(a.f, delta, m_s);
                // masks are not visited in ascending order: keep the lowest among equal scores
                if (key > best.key || (key == best.key && (int)mask < best.idx)) { best.key = key; best.idx = (int)mask; }
            }
            if (c + 1 < n_hi) {
                const int b = __ffs(c + 1) - 1;           // bit that flips between Gray codes c and c + 1
                hi ^= 1u << b;
                delta += ((hi >> b) & 1u) ? win_s[lowbits + b] : -win_s[lowbits + b];
            }
        }
    }
    int phase = 0;
    best = block_argmax(best, red_key, red_idx, phase);
    if (tid == 0) {
        a.best_mask[p] = best.key == kNoKey ? 0u : (unsigned)best.idx;
        if (a.best_F) a.best_F[p] = best.key == kNoKey ? 0.0 : (a.f.fp ? double_of_key(best.key) : (double)best.key);
    }
}

}  // namespace br
