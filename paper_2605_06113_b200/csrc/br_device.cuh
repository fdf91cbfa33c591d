// Device-side building blocks of the routing step: Philox4x32-10, order-preserving
// score keys, warp/block arg-max with lowest-index tie-break.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <type_traits>

namespace br {

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int32_t kEmpty = INT32_MIN;
constexpr long long kNoKey = (long long)0x8000000000000000ull;
constexpr int kNoIdx = 0x7FFFFFFF;

enum : uint32_t { kStreamArrCount = 0, kStreamArrLen = 1, kStreamTerm = 2, kStreamArrOut = 3 };

// ---- range-checked build -------------------------------------------------------------------
// With -DBR_BOUNDS every per-instance array of the step kernels (shared memory and global rows) is
// a Span that knows its length: an index outside it is counted in g_bounds_hits and redirected to
// a sink, so nothing outside the array is touched and the kernel ends normally (no trap, no
// assert).  The host reads the count with br_debug_bounds_hits().  In the normal build span_t<T>
// is a plain pointer and the helpers below vanish.
#ifdef BR_BOUNDS
__device__ unsigned long long g_bounds_sink[8];
__device__ unsigned g_bounds_hits;

template <typename T>
struct Span {
    T *p;
    long long n;
    __device__ Span() : p(nullptr), n(0) {}
    __device__ Span(T *p_, long long n_) : p(p_), n(p_ ? (n_ < 0 ? 0 : n_) : 0) {}
    __device__ explicit operator bool() const { return p != nullptr; }
    __device__ T &operator[](long long i) const
    {
        if (i < 0 || i >= n) { atomicAdd(&g_bounds_hits, 1u); return *reinterpret_cast<T *>(g_bounds_sink); }
        return p[i];
    }
    __device__ Span operator+(long long off) const { return Span(p ? p + off : nullptr, n - off); }
};
template <typename T> using span_t = Span<T>;
template <typename T> __device__ __forceinline__ Span<T> mk_span(T *p, long long n) { return Span<T>(p, n); }
// pointer to a vector of V that covers elements [i, i + sizeof(V) / sizeof(T)) of s
template <typename V, typename T>
__device__ __forceinline__ V *vec_at(const Span<T> &s, long long i)
{
    const long long cnt = (long long)(sizeof(V) / sizeof(T));
    if (i < 0 || i + cnt > s.n) {
        atomicAdd(&g_bounds_hits, 1u);
        return reinterpret_cast<V *>(g_bounds_sink);
    }
    return reinterpret_cast<V *>(const_cast<typename std::remove_const<T>::type *>(s.p) + i);
}
template <typename T> __device__ __forceinline__ T *raw_of(const Span<T> &s) { return s.p; }
#else
template <typename T> using span_t = T *;
template <typename T> __device__ __forceinline__ T *mk_span(T *p, long long) { return p; }
template <typename V, typename T>
__device__ __forceinline__ V *vec_at(T *p, long long i)
{
    return reinterpret_cast<V *>(const_cast<typename std::remove_const<T>::type *>(p) + i);
}
template <typename T> __device__ __forceinline__ T *raw_of(T *p) { return p; }
#endif

// First statements of a step kernel: let the next kernel of the stream start becoming resident,
// then wait until every earlier kernel of the stream has completed and flushed its writes
// (both are no-ops for a launch without programmatic stream serialisation).
__device__ __forceinline__ void stream_order_gate()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Philox4x32-10 (Salmon et al., SC'11): counter (c0..c3), key (k0, k1).
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ uint32_t word_of(const uint4 &v, uint32_t j)
{
    return j == 0 ? v.x : (j == 1 ? v.y : (j == 2 ? v.z : v.w));
}

// fp64 score -> int64 key with the same order and the same sign (0.0 -> 0).
__device__ __forceinline__ long long key_of_double(double f)
{
    const long long b = __double_as_longlong(f + 0.0);      // -0.0 -> +0.0
    return b ^ ((b >> 63) & 0x7FFFFFFFFFFFFFFFll);
}
__device__ __forceinline__ double double_of_key(long long k)
{
    return __longlong_as_double(k ^ ((k >> 63) & 0x7FFFFFFFFFFFFFFFll));
}

struct Best {
    long long key;   // kNoKey if empty
    int idx;         // kNoIdx if empty
};

// arg-max over the warp of (key, idx): largest key, then lowest idx.
__device__ __forceinline__ Best warp_argmax(Best b)
{
    const int hi = (int)(b.key >> 32);
    const unsigned lo = (unsigned)b.key;
    const int mhi = __reduce_max_sync(kFull, hi);
    const bool in1 = (hi == mhi);
    const unsigned mlo = __reduce_max_sync(kFull, in1 ? lo : 0u);
    const bool in2 = in1 && (lo == mlo);
    const unsigned midx = __reduce_min_sync(kFull, in2 ? (unsigned)b.idx : (unsigned)kNoIdx);
    Best r;
    r.key = (long long)(((unsigned long long)(unsigned)mhi << 32) | mlo);
    r.idx = (int)midx;
    return r;
}

// Block-wide arg-max.  red_key/red_idx: shared arrays of 2 * 32 entries; `phase`
// alternates between calls so one barrier per call is enough.
__device__ __forceinline__ Best block_argmax(Best b, long long *red_key, int *red_idx, int &phase)
{
    b = warp_argmax(b);
    const int nwarps = blockDim.x >> 5;
    if (nwarps == 1) return b;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    long long *rk = red_key + phase * 32;
    int *ri = red_idx + phase * 32;
    phase ^= 1;
    if (lane == 0) { rk[warp] = b.key; ri[warp] = b.idx; }
    __syncthreads();
    Best c;
    c.key = lane < nwarps ? rk[lane] : kNoKey;
    c.idx = lane < nwarps ? ri[lane] : kNoIdx;
    return warp_argmax(c);
}

__device__ __forceinline__ void block_sync()
{
    if (blockDim.x == 32) __syncwarp(); else __syncthreads();
}

}  // namespace br
