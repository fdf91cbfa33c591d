// Pool-bypass dispatch for BR-0 (Appendix "Pool-bypass deployment path for BR-0"): requests are
// routed one at a time, in arrival order, each to argmax_g F_g(s) = alpha s - beta (s - m_g)_+ over
// the workers whose inflight count is below its cap, with m_g = M - L_g taken from *virtual*
// loads (running requests plus those dispatched and not started yet); the chosen worker's virtual load
// and inflight count grow at once, so the next request sees them.  One warp per instance, lane g
// holds worker g (and g + 32): the chain over requests is sequential, the arg-max over workers a
// warp reduction with lowest-g tie-break.
#pragma once
#include "br_device.cuh"
#include "br_fscore.cuh"
#include "../../include/br.h"

namespace br {

struct BypassArgs {
    FscoreArgs f;             // G, H = 0, fp, aD, beta, d[0]
    int32_t n_req, first_instance;
    const int32_t *s;         // [N][n_req] prompt lengths in arrival order
    int64_t *vload;           // [N][G] virtual loads, updated
    int32_t *inflight;        // [N][G] requests running or dispatched per worker, updated
    const int32_t *cap;       // [N][G] inflight cap per worker
    int32_t *g_out;           // [N][n_req] chosen worker, -1 if every worker is at its cap
};

__global__ void __launch_bounds__(128) br_bypass_kernel(const BypassArgs a, int n_inst)
{
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= n_inst) return;
    const size_t inst = (size_t)a.first_instance + row;
    const int G = a.f.G;
    long long L[2] = {0, 0};
    int nfl[2] = {0, 0}, cap[2] = {0, 0};
#pragma unroll
    for (int w = 0; w < 2; ++w) {
        const int g = lane + 32 * w;
        if (g < G) {
            L[w] = a.vload[inst * G + g];
            nfl[w] = a.inflight[inst * G + g];
            cap[w] = a.cap[inst * G + g];
        }
    }
    const int32_t *s = a.s + inst * a.n_req;
    int32_t *out = a.g_out + inst * a.n_req;
#pragma unroll 1
    for (int i = 0; i < a.n_req; ++i) {
        const int si = s[i];
        // envelope M = max_g L_g over all workers (Section 3.1)
        long long mx = L[0];
        if (lane + 32 < G && L[1] > mx) mx = L[1];
        if (lane >= G) mx = (long long)0x8000000000000000ull;
        for (int o = 16; o > 0; o >>= 1) {
            const long long v = __shfl_xor_sync(kFull, mx, o);
            mx = v > mx ? v : mx;
        }
        Best b; b.key = kNoKey; b.idx = kNoIdx;
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            const int g = lane + 32 * w;
            if (g < G && nfl[w] < cap[w]) {
                const long long m = mx - L[w];
                const long long key = fscore_key(a.f, si, &m);
                if (key > b.key) { b.key = key; b.idx = g; }       // w ascends: the lower g is kept on ties
            }
        }
        b = warp_argmax(b);
        const int g = b.key == kNoKey ? -1 : b.idx;
        if (g >= 0 && (g & 31) == lane) { L[g >> 5] += si; nfl[g >> 5] += 1; }
        if (lane == 0) out[i] = g;
    }
#pragma unroll
    for (int w = 0; w < 2; ++w) {
        const int g = lane + 32 * w;
        if (g < G) { a.vload[inst * G + g] = L[w]; a.inflight[inst * G + g] = nfl[w]; }
    }
}

}  // namespace br
