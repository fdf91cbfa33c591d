// Batched F-score matrix: F_g({i}) for every (request, worker) pair of an instance
// (Eq. 1 in int64, Eq. 2 in fp64).  Margins are staged in shared memory, prompt
// lengths are read with 16-byte loads, the matrix is written with unit stride.
#pragma once
#include "br_device.cuh"
#include "../../include/br.h"

namespace br {

constexpr int kFsTile = 1024;   // requests per thread block

struct FscoreArgs {
    int32_t G, H;
    bool fp;
    double aD, beta;
    double d[BR_MAX_H + 1];
    int32_t n_req, first_instance;
    const int32_t *s;      // [N][n_req]
    const int64_t *Lh;     // [N][G][H+1]
    const int32_t *cap;    // [N][G] or NULL
    double *F;             // [N][n_req][G]
    int32_t *best_g;       // [N][n_req] or NULL
};

__device__ __forceinline__ long long fscore_key(const FscoreArgs &a, int delta, const long long *m)
{
    if (!a.fp) {
        long long over = (long long)delta - m[0];
        over = over > 0 ? over : 0;
        return (long long)delta - (long long)a.G * over;
    }
    const double dl = (double)delta;
    double pen = 0.0;
    for (int h = 0; h <= a.H; ++h) {
        double over = __dsub_rn(dl, (double)m[h]);
        over = over > 0.0 ? over : 0.0;
        pen = __dadd_rn(pen, __dmul_rn(a.d[h], over));
    }
    return key_of_double(__dsub_rn(__dmul_rn(a.aD, dl), __dmul_rn(a.beta, pen)));
}

// Thread t of a block owns worker g = t % G for the whole tile (its margins and discounts stay in
// registers) and walks the requests slice, slice + n_slices, ...: thread t writes elements
// t, t + n_slices * G, ... of the tile's [request][worker] rows, so every store instruction of a
// warp covers consecutive addresses.  HM bounds H at compile time (loops over h unrolled); HM > 16
// stands for any longer horizon: the margins are then read from shared memory in a plain loop.
template <int HM>
__global__ void __launch_bounds__(256) br_fscore_kernel(const FscoreArgs a)
{
    __shared__ long long m_s[BR_MAX_G * (BR_MAX_H + 1)];
    __shared__ long long Mh[BR_MAX_H + 1];
    __shared__ __align__(16) int s_tile[kFsTile];
    __shared__ int cap_s[BR_MAX_G];
    const int tid = threadIdx.x, G = a.G, H = a.H, H1 = a.H + 1;
    const size_t inst = (size_t)a.first_instance + blockIdx.y;
    const int tile0 = blockIdx.x * kFsTile;
    const int n = min(kFsTile, a.n_req - tile0);

    for (int i = tid; i < G * H1; i += blockDim.x) m_s[i] = a.Lh[inst * G * H1 + i];
    for (int g = tid; g < G; g += blockDim.x) cap_s[g] = a.cap ? a.cap[inst * G + g] : 1;
    for (int i = tid * 4; i < n; i += blockDim.x * 4)
        *reinterpret_cast<int4 *>(s_tile + i) =
            *reinterpret_cast<const int4 *>(a.s + inst * a.n_req + tile0 + i);
    __syncthreads();
    if (tid < H1) {
        long long M = m_s[tid];
        for (int g = 1; g < G; ++g) M = max(M, m_s[g * H1 + tid]);
        Mh[tid] = M;
    }
    __syncthreads();
    for (int i = tid; i < G * H1; i += blockDim.x) m_s[i] = Mh[i % H1] - m_s[i];
    __syncthreads();

    double *F = a.F + (inst * a.n_req + tile0) * G;
    const int n_slices = blockDim.x / G;
    const int slice = tid / G, g = tid - slice * G;
    if (slice < n_slices) {
        constexpr bool LONG = HM > 16;
        constexpr int HR = LONG ? 0 : HM;
        double md[HR + 1], dd[HR + 1];
        long long m0 = m_s[g * H1], mmin = m0;
#pragma unroll
        for (int h = 0; h <= HR; ++h) {
            md[h] = h <= H ? (double)m_s[g * H1 + h] : 0.0;
            dd[h] = h <= H ? a.d[h] : 0.0;
            if (h <= H) mmin = min(mmin, m_s[g * H1 + h]);
        }
        if (LONG) for (int h = 1; h <= H; ++h) mmin = min(mmin, m_s[g * H1 + h]);
        const long long Gl = (long long)G;
#pragma unroll 4
        for (int i = slice; i < n; i += n_slices) {
            const int si = s_tile[i];
            double f;
            if (!a.fp) {
                long long over = (long long)si - m0;
                over = over > 0 ? over : 0;
                f = (double)((long long)si - Gl * over);                    // Eq. 1, exact
            } else {
                const double dl = (double)si;
                double pen = 0.0;
                if (LONG) {
                    if ((long long)si > mmin) {
                        for (int h = 0; h <= H; ++h) {
                            double over = __dsub_rn(dl, (double)m_s[g * H1 + h]);
                            over = over > 0.0 ? over : 0.0;
                            pen = __dadd_rn(pen, __dmul_rn(a.d[h], over));
                        }
                    }
                } else if ((long long)si > mmin) {                          // else every (s - m_h)_+ is zero
#pragma unroll
                    for (int h = 0; h <= HR; ++h) {
                        if (h <= H) {
                            double over = __dsub_rn(dl, md[h]);
                            over = over > 0.0 ? over : 0.0;
                            pen = __dadd_rn(pen, __dmul_rn(dd[h], over));
                        }
                    }
                }
                f = __dsub_rn(__dmul_rn(a.aD, dl), __dmul_rn(a.beta, pen)) + 0.0;   // Eq. 2 (-0.0 -> +0.0)
            }
            F[(size_t)i * G + g] = f;
        }
    }
    if (a.best_g) {
        for (int i = tid; i < n; i += blockDim.x) {
            long long bk = kNoKey; int bg = -1;
            for (int g = 0; g < G; ++g) {
                if (cap_s[g] <= 0) continue;
                const long long key = fscore_key(a, s_tile[i], m_s + g * H1);
                if (bg < 0 || key > bk) { bk = key; bg = g; }
            }
            a.best_g[inst * a.n_req + tile0 + i] = bg;
        }
    }
}

}  // namespace br
