// The routing-step kernel: one thread block per routing instance.
//
// Phases per decode step k (Section 2.2 model; Algorithms 1 and 2):
//   ARRIVE -> PREDICT (H > 0) -> ROUTE (Stage 1, Stage 2) -> RECORD -> ADVANCE.
// Worker-level state (loads, projected loads, envelope, free slots) lives in shared
// memory; the waiting queue is staged in shared memory with coalesced 16-byte loads;
// every arg-max is a warp-shuffle reduction with a lowest-index tie-break.
#pragma once
#include "br_device.cuh"
#include "../../include/br.h"

namespace br {

struct StepArgs {
    int32_t G, H, B, W, R_max, S_greedy, occ_words;
    int32_t delta_T;
    float gate, c_floor;
    int32_t term_mode;
    uint32_t hazard_thr;
    const uint32_t *arr_cdf;
    int32_t arr_len, arr_period, arr_inst_stride;
    const int32_t *len_tab;
    int32_t len_shift;
    int32_t burst_every, burst_size;
    double aD, beta;
    double d[BR_MAX_H + 1];
    int32_t N, first_instance, n_steps;
    br_worker_state ws;
    br_waiting_queue wq;
    const float *term_probs;
    int32_t *assign_out;
    br_load_out out;
};

// shared-memory footprint of one instance (bytes), mirrored by the host
__host__ __device__ inline size_t step_smem_bytes(int G, int H, int W, int occ_words)
{
    size_t n = 0;
    n += sizeof(long long) * (size_t)G * (H + 1);   // Lh
    n += sizeof(long long) * (size_t)(H + 1);       // Mh
    n += sizeof(long long) * (size_t)G;             // load_new
    n += sizeof(unsigned long long) * (size_t)G * occ_words;
    n += sizeof(long long) * 64;                    // red_key
    n += sizeof(int) * 64 * 2;                      // red_idx, red_val
    n += sizeof(int) * (size_t)W * 2;               // q_s, q_id
    n += sizeof(int) * (size_t)G * 2;               // cap, nact_new
    n += sizeof(int) * 8;                           // scalars
    return (n + 15) & ~(size_t)15;
}

struct BestV {
    long long key;
    int idx;
    int val;
};

// block arg-max carrying a 32-bit payload of the winner
__device__ __forceinline__ BestV block_argmax_v(long long key, int idx, int val, long long *red_key,
                                                int *red_idx, int *red_val, int &phase)
{
    Best b{key, idx};
    Best w = warp_argmax(b);
    const unsigned src = __ballot_sync(kFull, idx == w.idx && key == w.key);
    int v = __shfl_sync(kFull, val, src ? (__ffs(src) - 1) : 0);
    const int nwarps = blockDim.x >> 5;
    if (nwarps == 1) return BestV{w.key, w.idx, v};
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    long long *rk = red_key + phase * 32;
    int *ri = red_idx + phase * 32;
    int *rv = red_val + phase * 32;
    phase ^= 1;
    if (lane == 0) { rk[warp] = w.key; ri[warp] = w.idx; rv[warp] = v; }
    __syncthreads();
    Best c;
    c.key = lane < nwarps ? rk[lane] : kNoKey;
    c.idx = lane < nwarps ? ri[lane] : kNoIdx;
    const int cv = lane < nwarps ? rv[lane] : 0;
    Best w2 = warp_argmax(c);
    const unsigned src2 = __ballot_sync(kFull, c.idx == w2.idx && c.key == w2.key);
    const int v2 = __shfl_sync(kFull, cv, src2 ? (__ffs(src2) - 1) : 0);
    return BestV{w2.key, w2.idx, v2};
}

// Score of admitting total prompt length `delta` to the worker whose margins were
// loaded: Eq. 1 in int64 (FP = false) or Eq. 2 in fp64, term by term in h (FP = true).
// Returned as an order- and sign-preserving int64 key.
template <bool FP, int HM>
struct Scorer {
    long long mi;
    double md[HM + 1];

    __device__ __forceinline__ void load(const long long *Lh, const long long *Mh, int g, int H)
    {
        const int H1 = H + 1;
        if (!FP) {
            mi = Mh[0] - Lh[g * H1];
        } else {
#pragma unroll
            for (int h = 0; h <= HM; ++h)
                md[h] = (h <= H) ? (double)(Mh[h] - Lh[g * H1 + h]) : 0.0;
        }
    }
    __device__ __forceinline__ long long key(const StepArgs &a, int delta) const
    {
        if (!FP) {
            long long over = (long long)delta - mi;
            over = over > 0 ? over : 0;
            return (long long)delta - (long long)a.G * over;
        } else {
            const double dl = (double)delta;
            double pen = 0.0;
#pragma unroll
            for (int h = 0; h <= HM; ++h) {
                if (h <= a.H) {
                    double over = __dsub_rn(dl, md[h]);          // exact: integers below 2^53
                    over = over > 0.0 ? over : 0.0;
                    pen = __dadd_rn(pen, __dmul_rn(a.d[h], over));
                }
            }
            return key_of_double(__dsub_rn(__dmul_rn(a.aD, dl), __dmul_rn(a.beta, pen)));
        }
    }
    __device__ __forceinline__ double value(long long k) const
    {
        return FP ? double_of_key(k) : (double)k;
    }
};

template <bool FP, int HM>
__global__ void __launch_bounds__(512) br_step_kernel(const StepArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, NT = blockDim.x, lane = tid & 31;
    const int G = a.G, H = a.H, B = a.B, W = a.W, H1 = H + 1, A = G * B, OW = a.occ_words;
    const int inst = a.first_instance + blockIdx.x;

    // ---- shared-memory carve-up (sizes match step_smem_bytes) ----
    int *q_s = reinterpret_cast<int *>(smem_raw);                     // 16-byte aligned
    unsigned *q_id = reinterpret_cast<unsigned *>(q_s + W);          // W % 4 == 0
    long long *Lh = reinterpret_cast<long long *>(q_id + W);
    long long *Mh = Lh + (size_t)G * H1;
    long long *load_new = Mh + H1;
    unsigned long long *occ = reinterpret_cast<unsigned long long *>(load_new + G);
    long long *red_key = reinterpret_cast<long long *>(occ + (size_t)G * OW);
    int *red_idx = reinterpret_cast<int *>(red_key + 64);
    int *red_val = red_idx + 64;
    int *cap = red_val + 64;
    int *nact_new = cap + G;
    int *scal = nact_new + G;   // [0] admitted [1] Stage-1 iterations [2] Stage-2 pops [3],[4] status bits
    int phase = 0;
    if (tid < 8) scal[tid] = 0;
    __syncthreads();

    // ---- per-instance global rows ----
    long long *g_load = reinterpret_cast<long long *>(a.ws.load) + (size_t)inst * G;
    int32_t *g_nact = a.ws.nact + (size_t)inst * G;
    unsigned long long *g_occ = reinterpret_cast<unsigned long long *>(a.ws.occ) + (size_t)inst * G * OW;
    int32_t *g_base = a.ws.act_base + (size_t)inst * A;
    uint32_t *g_aid = a.ws.act_id ? a.ws.act_id + (size_t)inst * A : nullptr;
    float *g_chat0 = a.ws.act_chat0 ? a.ws.act_chat0 + (size_t)inst * A : nullptr;
    uint8_t *g_kref = a.ws.act_kref ? a.ws.act_kref + (size_t)inst * A : nullptr;
    int32_t *g_qs = a.wq.s + (size_t)inst * W;
    uint32_t *g_qid = a.wq.id + (size_t)inst * W;

    const unsigned long long seed = a.ws.seed[inst];
    const uint32_t key0 = (uint32_t)seed, key1 = (uint32_t)(seed >> 32);
    int k = a.ws.step[inst];
    uint32_t next_id = a.ws.next_id[inst];
    int n_w = a.wq.n[inst];
    int status = 0;
    if (n_w < 0 || n_w > W) { status |= BR_ST_BAD_STATE; n_w = n_w < 0 ? 0 : W; }   // uniform

    // queue -> shared memory (16-byte loads)
    for (int i = tid * 4; i < n_w; i += NT * 4) {
        const int4 v = *reinterpret_cast<const int4 *>(g_qs + i);
        const uint4 u = *reinterpret_cast<const uint4 *>(g_qid + i);
        *reinterpret_cast<int4 *>(q_s + i) = v;
        *reinterpret_cast<uint4 *>(q_id + i) = u;
    }
    for (int g = tid; g < G; g += NT) {
        int na = g_nact[g];
        if (na < 0 || na > B) { atomicOr(&scal[4], (int)BR_ST_BAD_STATE); na = na < 0 ? 0 : B; }
        cap[g] = B - na;
        if (H == 0) Lh[g] = g_load[g];
    }
    for (int i = tid; i < G * OW; i += NT) occ[i] = g_occ[i];

    for (int it = 0; it < a.n_steps; ++it, ++k) {
        const size_t orow = (size_t)it * a.N + inst;
        const float *probs = a.term_probs ? a.term_probs + orow * (size_t)A * H : nullptr;
        int32_t *assign = a.assign_out + orow * W;
        if (tid < 4) scal[tid] = 0;
        if (H > 0) for (int i = tid; i < G * H1; i += NT) Lh[i] = 0;

        // ================= ARRIVE =================
        int n_arr = 0;
        if (a.arr_cdf) {
            const uint32_t u = philox4x32_10((uint32_t)k, 0u, kStreamArrCount, 0u, key0, key1).x;
            const uint32_t *row = a.arr_cdf +
                ((size_t)inst * a.arr_inst_stride + (size_t)(k % a.arr_period)) * a.arr_len;
            for (int j0 = 0; j0 < a.arr_len; j0 += 32) {
                const int j = j0 + lane;
                const bool ge = (j < a.arr_len) && (u >= row[j]);
                n_arr += __popc(__ballot_sync(kFull, ge));
            }
            if (a.burst_every > 0 && k > 0 && (k % a.burst_every) == 0) n_arr += a.burst_size;
        }
        for (int j = tid; j < n_arr; j += NT) {
            const int pos = n_w + j;
            if (pos < W) {
                const uint4 r = philox4x32_10((uint32_t)k, (uint32_t)j >> 2, kStreamArrLen, 0u, key0, key1);
                q_s[pos] = a.len_tab[word_of(r, j & 3) >> a.len_shift];
                q_id[pos] = next_id + (uint32_t)j;
            }
        }
        const int n_w_old = n_w;
        int n_drop = n_w + n_arr - W;
        n_drop = n_drop > 0 ? n_drop : 0;
        n_w = n_w + n_arr - n_drop;
        next_id += (uint32_t)n_arr;
        if (n_drop) status |= BR_ST_QUEUE_OVERFLOW;
        __syncthreads();

        // ================= PREDICT (H > 0) =================
        if (H > 0) {
            const bool warp_uniform = (B % 32) == 0;
            const int A_up = (A + NT - 1) / NT * NT;
            for (int s0 = tid; s0 < A_up; s0 += NT) {
                const bool inr = s0 < A;
                const int base = inr ? g_base[s0] : kEmpty;
                const bool live = base != kEmpty;
                int cur = 0, nh = -1;
                if (live) {
                    cur = base + k;
                    const float c0 = g_chat0[s0];
                    const int kr = g_kref[s0];
                    const int t = (k - kr) & 255;
                    float c = c0 - (float)t;
                    if (t >= a.delta_T || c < a.c_floor) {
                        const float *q = probs + (size_t)s0 * H;
                        double surv = 1.0, cs = 0.0;
                        for (int h = 0; h < H; ++h) {
                            cs = __dadd_rn(cs, surv);
                            surv = __dmul_rn(surv, __dsub_rn(1.0, (double)q[h]));
                        }
                        const double p_fin = __dsub_rn(1.0, surv);
                        double v;
                        if (p_fin >= (double)a.gate) {
                            v = cs;
                            if (v < (double)a.c_floor) v = (double)a.c_floor;
                            if (v > (double)H) v = (double)H;
                        } else {
                            v = (double)H;
                        }
                        c = (float)v;
                        g_chat0[s0] = c;
                        g_kref[s0] = (uint8_t)(k & 255);
                    }
                    nh = (int)floorf(c);
                    nh = nh < 0 ? 0 : (nh > H ? H : nh);
                }
                const int g = (inr ? s0 : A - 1) / B;
                if (warp_uniform) {
                    for (int h = 0; h <= H; ++h) {
                        const unsigned v = (live && h <= nh) ? (unsigned)(cur + h) : 0u;
                        const unsigned s = __reduce_add_sync(kFull, v);
                        if (lane == 0 && s)
                            atomicAdd(reinterpret_cast<unsigned long long *>(&Lh[g * H1 + h]),
                                      (unsigned long long)s);
                    }
                } else if (live) {
                    for (int h = 0; h <= nh; ++h)
                        atomicAdd(reinterpret_cast<unsigned long long *>(&Lh[g * H1 + h]),
                                  (unsigned long long)(cur + h));
                }
            }
            __syncthreads();
        }
        // envelope M_h = max_g L_g(k+h)
        for (int h = tid; h < H1; h += NT) {
            long long M = Lh[h];
            for (int g = 1; g < G; ++g) M = max(M, Lh[g * H1 + h]);
            Mh[h] = M;
        }
        // assign_out rows start at -1
        for (int i = tid * 4; i < W; i += NT * 4)
            *reinterpret_cast<int4 *>(assign + i) = make_int4(-1, -1, -1, -1);
        __syncthreads();

        Scorer<FP, HM> sc;

        // optional F-score matrix before the first admission
        if (a.out.fscore) {
            double *F = a.out.fscore + orow * (size_t)W * G;
            for (int g = 0; g < G; ++g) {
                sc.load(Lh, Mh, g, H);
                for (int i = tid; i < W; i += NT)
                    F[(size_t)i * G + g] = (i < n_w) ? sc.value(sc.key(a, q_s[i])) : 0.0;
            }
        }

        // ================= ROUTE =================
        int S_tot = 0;
        for (int g = 0; g < G; ++g) S_tot += cap[g];
        int n_left = n_w;                      // waiting requests not yet admitted
        const bool route = (S_tot > 0 && n_w > 0);

        // commit request at queue position i (length s) to worker g; uniform across the block
        auto commit = [&](int i, int s, int g) {
            // every thread has finished reading the state it needs
            __syncthreads();
            if (tid == 0) {
                int slot = -1;
                for (int w = 0; w < OW && slot < 0; ++w) {
                    const unsigned long long fr = ~occ[g * OW + w];
                    if (fr) slot = w * 64 + __ffsll((long long)fr) - 1;
                }
                if (slot >= 0 && slot < B) {
                    occ[g * OW + (slot >> 6)] |= 1ull << (slot & 63);
                    cap[g] -= 1;
                    for (int h = 0; h <= H; ++h) {
                        const long long v = Lh[g * H1 + h] + s;
                        Lh[g * H1 + h] = v;
                        if (v > Mh[h]) Mh[h] = v;
                    }
                    const int sa = g * B + slot;
                    g_base[sa] = s - k;
                    if (g_aid) g_aid[sa] = q_id[i];
                    if (H > 0) {
                        g_chat0[sa] = (float)(H + a.delta_T - 1);
                        g_kref[sa] = (uint8_t)((k + 1 - a.delta_T) & 255);
                    }
                    assign[i] = sa;
                    scal[0] += 1;
                } else {
                    scal[3] |= BR_ST_BAD_STATE;
                }
                q_s[i] = -1;
            }
            __syncthreads();
        };

        // argmax_i F_g({i}) over all waiting requests, earliest position on ties
        auto best_single = [&](int g) -> BestV {
            sc.load(Lh, Mh, g, H);
            long long bk = kNoKey; int bi = kNoIdx, bv = 0;
            for (int i = tid; i < n_w; i += NT) {
                const int s = q_s[i];
                if (s < 0) continue;
                const long long key = sc.key(a, s);
                if (key > bk) { bk = key; bi = i; bv = s; }
            }
            return block_argmax_v(bk, bi, bv, red_key, red_idx, red_val, phase);
        };

        if (route) {
            // ---------- Stage 1: greedy fill ----------
            int guard_iters = 0;
            while (S_tot > a.S_greedy && n_left > 0) {
                if (++guard_iters > W) { status |= BR_ST_ITER_CAP; break; }
                // worker with most free slots; ties: smallest L_g(k), then lowest g
                Best bg{kNoKey, kNoIdx};
                for (int g = lane; g < G; g += 32) {
                    // key: cap (high), -(L) (low, loads < 2^31 by the create-time proof)
                    const long long key = ((long long)cap[g] << 32) |
                                          (long long)(0x7FFFFFFFu - (unsigned)Lh[g * H1]);
                    if (key > bg.key) { bg.key = key; bg.idx = g; }
                }
                bg = warp_argmax(bg);
                const int g = bg.idx;
                const BestV bi = best_single(g);
                if (bi.idx == kNoIdx) break;
                commit(bi.idx, bi.val, g);
                S_tot -= 1; n_left -= 1;
                if (tid == 0) scal[1] += 1;
            }

            // ---------- Stage 2: refined allocation ----------
            guard_iters = 0;
            while (n_left > 0 && S_tot > 0) {
                if (++guard_iters > W + G) { status |= BR_ST_ITER_CAP; break; }
                // worker with (largest cap, largest horizon-min margin, lowest g), cap > 0
                Best bg{kNoKey, kNoIdx};
                for (int g = lane; g < G; g += 32) {
                    if (cap[g] <= 0) continue;
                    long long mm = Mh[0] - Lh[g * H1];
                    for (int h = 1; h <= H; ++h) mm = min(mm, Mh[h] - Lh[g * H1 + h]);
                    const long long key = ((long long)cap[g] << 32) | (long long)(unsigned)mm;
                    if (key > bg.key) { bg.key = key; bg.idx = g; }
                }
                bg = warp_argmax(bg);
                if (bg.idx == kNoIdx) break;
                const int g = bg.idx;
                if (tid == 0) scal[2] += 1;

                // window: the R_max largest waiting requests, earliest first on ties
                int win_i[BR_MAX_RMAX], win_s[BR_MAX_RMAX];
                int nwin = 0;
                long long prev = 0x7FFFFFFFFFFFFFFFll;
#pragma unroll
                for (int r = 0; r < BR_MAX_RMAX; ++r) {
                    if (r < a.R_max && r < n_left) {
                        long long bk = kNoKey; int bi = kNoIdx, bv = 0;
                        for (int i = tid; i < n_w; i += NT) {
                            const int s = q_s[i];
                            if (s < 0) continue;
                            const long long key = ((long long)s << 32) | (long long)(unsigned)(0x7FFFFFFF - i);
                            if (key < prev && key > bk) { bk = key; bi = i; bv = s; }
                        }
                        const BestV w = block_argmax_v(bk, bi, bv, red_key, red_idx, red_val, phase);
                        win_i[r] = w.idx; win_s[r] = w.val; prev = w.key;
                        if (w.idx != kNoIdx) nwin = r + 1;
                    } else {
                        win_i[r] = kNoIdx; win_s[r] = 0;
                    }
                }
                // subsets: lane = mask
                const int lim = min(cap[g], a.R_max);
                sc.load(Lh, Mh, g, H);
                Best bm{kNoKey, kNoIdx};
                if (lane >= 1 && lane < (1 << nwin) && __popc(lane) <= lim) {
                    int delta = 0;
#pragma unroll
                    for (int r = 0; r < BR_MAX_RMAX; ++r)
                        if ((lane >> r) & 1) delta += win_s[r];
                    bm.key = sc.key(a, delta);
                    bm.idx = lane;
                }
                bm = warp_argmax(bm);
                if (bm.idx == kNoIdx) { status |= BR_ST_ITER_CAP; break; }
                if (bm.key <= 0) {
                    // starvation guard: least-bad single request of all of R_wait
                    const BestV bi = best_single(g);
                    if (bi.idx == kNoIdx) break;
                    commit(bi.idx, bi.val, g);
                    S_tot -= 1; n_left -= 1;
                } else {
#pragma unroll
                    for (int r = 0; r < BR_MAX_RMAX; ++r) {
                        if ((bm.idx >> r) & 1) {
                            commit(win_i[r], win_s[r], g);
                            S_tot -= 1; n_left -= 1;
                        }
                    }
                }
            }
        }
        __syncthreads();

        // ================= RECORD =================
        {
            Best mx{kNoKey, kNoIdx}, mn{kNoKey, kNoIdx};
            long long sum = 0;
            for (int g = lane; g < G; g += 32) {
                const long long L = Lh[g * H1];
                if (L > mx.key || mx.idx == kNoIdx) { mx.key = L; mx.idx = g; }
                if (-L > mn.key || mn.idx == kNoIdx) { mn.key = -L; mn.idx = g; }
                sum += L;
            }
            mx = warp_argmax(mx);
            mn = warp_argmax(mn);
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(kFull, sum, o);
            long long *o_load = reinterpret_cast<long long *>(a.out.load) + orow * G;
            for (int g = tid; g < G; g += NT) o_load[g] = Lh[g * H1];
            if (tid == 0) {
                long long *tr = reinterpret_cast<long long *>(a.out.trace) + orow * 3;
                tr[0] = mx.key; tr[1] = -mn.key; tr[2] = sum;
            }
        }

        // ================= queue compaction (stable, in shared memory) =================
        if (tid < 32 && n_left != n_w) {
            int run = 0;
            for (int i0 = 0; i0 < n_w; i0 += 32) {
                const int i = i0 + lane;
                const int s = (i < n_w) ? q_s[i] : -1;
                const unsigned id = (i < n_w) ? q_id[i] : 0u;
                const bool keep = s >= 0;
                const unsigned bal = __ballot_sync(kFull, keep);
                const int dst = run + __popc(bal & ((1u << lane) - 1u));
                __syncwarp();
                if (keep && dst != i) { q_s[dst] = s; q_id[dst] = id; }
                __syncwarp();
                run += __popc(bal);
            }
        }
        n_w = n_left;
        __syncthreads();

        // ================= ADVANCE =================
        for (int g = tid; g < G; g += NT) { load_new[g] = 0; nact_new[g] = 0; }
        __syncthreads();
        {
            const int A4 = A >> 2;
            const int A4_up = (A4 + NT - 1) / NT * NT;
            for (int q4 = tid; q4 < A4_up; q4 += NT) {
                const bool inr = q4 < A4;
                int4 b = make_int4(kEmpty, kEmpty, kEmpty, kEmpty);
                if (inr) b = *reinterpret_cast<const int4 *>(g_base + q4 * 4);
                const bool any = (b.x != kEmpty) | (b.y != kEmpty) | (b.z != kEmpty) | (b.w != kEmpty);
                unsigned part = 0; int cnt = 0; unsigned ended = 0;
                if (any) {
                    uint4 r = make_uint4(0, 0, 0, 0);
                    if (a.term_mode != 0)
                        r = philox4x32_10((uint32_t)k, (uint32_t)q4, kStreamTerm, 0u, key0, key1);
                    int bb[4] = {b.x, b.y, b.z, b.w};
                    const uint32_t rr[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (bb[j] == kEmpty) continue;
                        bool fin = false;
                        if (a.term_mode == 1) fin = rr[j] < a.hazard_thr;
                        else if (a.term_mode == 2)
                            fin = __fmul_rn((float)(rr[j] >> 8), 5.9604644775390625e-8f) <
                                  probs[(size_t)(q4 * 4 + j) * H];
                        if (fin) { ended |= 1u << j; bb[j] = kEmpty; }
                        else { part += (unsigned)(bb[j] + k + 1); cnt += 1; }
                    }
                    if (ended) *reinterpret_cast<int4 *>(g_base + q4 * 4) = make_int4(bb[0], bb[1], bb[2], bb[3]);
                }
                const int g = (inr ? q4 * 4 : A - 4) / B;
                // segmented sums over lanes of the same worker
                const unsigned peers = __match_any_sync(kFull, g);
                const unsigned psum = __reduce_add_sync(peers, part);
                const int pcnt = (int)__reduce_add_sync(peers, (unsigned)cnt);
                if (lane == __ffs(peers) - 1 && inr) {
                    if (psum) atomicAdd(reinterpret_cast<unsigned long long *>(&load_new[g]), (unsigned long long)psum);
                    if (pcnt) atomicAdd(&nact_new[g], pcnt);
                }
                if (ended) {
                    const int slot0 = (q4 * 4) % B;
                    atomicAnd(&occ[g * OW + (slot0 >> 6)], ~((unsigned long long)ended << (slot0 & 63)));
                }
            }
        }
        __syncthreads();
        for (int g = tid; g < G; g += NT) {
            cap[g] = B - nact_new[g];
            if (H == 0) Lh[g] = load_new[g];
        }
        if (tid == 0) {
            if (a.out.counters) {
                uint32_t *c = a.out.counters + orow * 4;
                c[0] = (uint32_t)n_drop; c[1] = (uint32_t)scal[0]; c[2] = (uint32_t)scal[1]; c[3] = (uint32_t)scal[2];
            }
            if (a.out.status) a.out.status[orow] = status | scal[3] | scal[4];
        }
        status = 0;
        __syncthreads();
    }

    // ---- write the snapshot back ----
    for (int g = tid; g < G; g += NT) {
        g_load[g] = load_new[g];
        g_nact[g] = nact_new[g];
    }
    for (int i = tid; i < G * OW; i += NT) g_occ[i] = occ[i];
    for (int i = tid * 4; i < n_w; i += NT * 4) {
        *reinterpret_cast<int4 *>(g_qs + i) = *reinterpret_cast<const int4 *>(q_s + i);
        *reinterpret_cast<uint4 *>(g_qid + i) = *reinterpret_cast<const uint4 *>(q_id + i);
    }
    if (tid == 0) {
        a.ws.step[inst] = k;
        a.ws.next_id[inst] = next_id;
        a.wq.n[inst] = n_w;
    }
}

}  // namespace br
