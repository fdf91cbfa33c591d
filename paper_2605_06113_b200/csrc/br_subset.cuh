// Batched exact solver of the Stage-2 subproblem (Algorithm 1 / 2, Stage 2; Appendix
// "Bit-set subset selection"): among the non-empty subsets Q of a window of R requests with
// |Q| <= lim, the one with the highest F_g(Q), lowest mask on ties.  The score depends on Q only
// through Delta(Q), so all 2^R - 1 subsets are enumerated in parallel: one thread block per
// problem, thread t owns the low 8 mask bits, the high bits are walked in Gray-code order so that
// each step changes Delta by one window entry.  Scores are those of the step kernels (Eq. 1 in
// integers, Eq. 2 in fp64 term by term).  Windows of up to 20 entries are enumerated; larger ones
// (up to 32), and any window when the host says the two-probe rule applies, are solved by meeting
// in the middle (br_mitm.cuh).
#pragma once
#include "br_device.cuh"
#include "br_fscore.cuh"
#include "br_mitm.cuh"
#include "../../include/br.h"

namespace br {

constexpr int kSubsetMaxEnum = 20;      // largest window that is enumerated
constexpr int kSubsetMaxR = 32;         // largest window at all (masks are 32 bits)

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
    __shared__ int win_s[kSubsetMaxEnum];
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

// The same problem by meeting in the middle: one thread block per problem.  peak_rule says that
// both sides of the score's peak are strictly monotone (checked on the host).
__global__ void __launch_bounds__(256) br_subset_mitm_kernel(const SubsetArgs a)
{
    __shared__ unsigned long long keys[1 << kMitmMaxLow];
    __shared__ int cls_off[kMitmMaxLow + 2];
    __shared__ long long m_s[BR_MAX_H + 1];
    __shared__ int win_s[kSubsetMaxR];
    __shared__ int red_sum[2][8];
    __shared__ unsigned red_mask[2][8];
    __shared__ int peak_s;
    const int tid = threadIdx.x, R = a.R, H1 = a.f.H + 1;
    const size_t p = (size_t)a.first_instance + blockIdx.x;
    if (tid < H1) m_s[tid] = a.m[p * H1 + tid];
    if (tid < R) win_s[tid] = a.win[p * R + tid];
    __syncthreads();
    int lim = a.lim[p];
    lim = lim < 0 ? 0 : (lim > R ? R : lim);
    if (tid == 0) {
        // the peak: Eq. 1 rises up to m_g; Eq. 2 up to the smallest kink whose passing leaves a
        // slope alpha D - beta sum_{m_h <= kink} d_h that is not positive
        long long peak = 0x7FFFFFFFll;
        if (!a.f.fp) {
            peak = m_s[0];
        } else {
            for (int h = 0; h < H1; ++h) {
                double wsum = 0.0;
                for (int j = 0; j < H1; ++j) if (m_s[j] <= m_s[h]) wsum = __dadd_rn(wsum, a.f.d[j]);
                if (!(a.f.aD > __dmul_rn(a.f.beta, wsum)) && m_s[h] < peak) peak = m_s[h];
            }
        }
        peak_s = peak > 0x7FFFFFFFll ? 0x7FFFFFFF : (peak < 0 ? 0 : (int)peak);
    }
    const int ra = min(kMitmMaxLow, (R + 1) / 2), rb = R - ra;
    mitm_build<true>(win_s, ra, keys, cls_off, tid, blockDim.x);      // ends with a block barrier
    MitmBest b; b.lo_sum = -1; b.lo_mask = 0xFFFFFFFFu; b.hi_sum = 0x7FFFFFFF; b.hi_mask = 0xFFFFFFFFu;
    if (lim >= 1) {
        const int peak = peak_s;
        for (unsigned mh = tid; mh < (1u << rb); mh += blockDim.x) {
            const int ph = __popc(mh);
            if (ph > lim) continue;
            int sh = 0;
            for (unsigned t = mh; t; t &= t - 1) sh += win_s[ra + __ffs(t) - 1];
            mitm_probe(keys, cls_off, ra, lim, peak, mh, sh, ph, b);
        }
    }
    // block reduction: largest lo_sum / smallest hi_sum, lowest mask among equals
    const int lane = tid & 31, warp = tid >> 5;
    for (int o = 16; o > 0; o >>= 1) {
        MitmBest c;
        c.lo_sum = __shfl_xor_sync(kFull, b.lo_sum, o); c.lo_mask = __shfl_xor_sync(kFull, b.lo_mask, o);
        c.hi_sum = __shfl_xor_sync(kFull, b.hi_sum, o); c.hi_mask = __shfl_xor_sync(kFull, b.hi_mask, o);
        mitm_take_lo(b, c.lo_sum, c.lo_mask); mitm_take_hi(b, c.hi_sum, c.hi_mask);
    }
    if (lane == 0) { red_sum[0][warp] = b.lo_sum; red_mask[0][warp] = b.lo_mask; red_sum[1][warp] = b.hi_sum; red_mask[1][warp] = b.hi_mask; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) {
            mitm_take_lo(b, red_sum[0][w], red_mask[0][w]); mitm_take_hi(b, red_sum[1][w], red_mask[1][w]);
        }
        long long bk = kNoKey; unsigned bm = 0u;
        if (b.lo_sum >= 0) { bk = fscore_key(a.f, b.lo_sum, m_s); bm = b.lo_mask; }
        if (b.hi_sum != 0x7FFFFFFF) {
            const long long k2 = fscore_key(a.f, b.hi_sum, m_s);
            if (k2 > bk || (k2 == bk && b.hi_mask < bm)) { bk = k2; bm = b.hi_mask; }
        }
        a.best_mask[p] = bk == kNoKey ? 0u : bm;
        if (a.best_F) a.best_F[p] = bk == kNoKey ? 0.0 : (a.f.fp ? double_of_key(bk) : (double)bk);
    }
}

}  // namespace br
