// BR-0 routing step for small fleets: one warp per instance, no block barrier.
//
// Shapes: G <= 32 workers (lane g owns worker g: free slots, load L_g, occupancy word),
// B <= 64 slots per worker, W <= 512 waiting requests, Eq. 1 scores in 32-bit integers,
// constant-hazard (or no) terminations, no optional outputs.  Everything else runs on
// br_step_kernel.
//
// A lane owns the queue positions (t * 32 + lane) * 4 + j, j < 4: prompt lengths, ids and
// assignments move as 16-byte vectors, and within a lane positions ascend.  For the length of a
// launch the queue lives in shared memory (ids beside it) as packed keys (s << wl | inverted position) so that "largest s, earliest
// arrival" is one integer max; an admitted entry becomes 0x80000000 | slot and a position
// beyond the queue 0x8000FFFF.  Both are negative: they lose every max of keys, and read as
// a prompt length they score below any waiting request (range checked on the host), so the
// scans need no validity test.
//
// Stage 1 and Stage 2 of Algorithm 1 share one loop with one worker selection, one
// single-request arg-max and one admission site (Stage 1 never resumes once S_tot has
// dropped to S_greedy, so the order of the paper's two loops is kept).  For Eq. 1 the
// Stage-2 worker key (cap, m_g) with m_g = M - L_g orders workers like Stage 1's
// (cap, smallest L_g).
#pragma once
#include "br_step.cuh"

namespace br {

constexpr int kSmallBeyond = (int)0x8000FFFFu;   // key of a position beyond the queue (no slot index reaches 0xFFFF)

template <int NT4 /* 128-position groups: W <= 128 * NT4 */, int RM /* window entries kept */>
__global__ void __maxnreg__(NT4 <= 2 ? 72 : 128) br_small_kernel(const StepArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_all[];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5, wpb = blockDim.x >> 5;
    const int row = blockIdx.x * wpb + wib;
    stream_order_gate();
    if (row >= a.N) return;
    const int inst = a.first_instance + row;
    int *q_key_p = reinterpret_cast<int *>(smem_all) + wib * (2 * NT4 * 128);
    const auto q_key = mk_span(q_key_p, NT4 * 128);                                   // [NT4 * 128] packed keys
    const auto q_id = mk_span(reinterpret_cast<unsigned *>(q_key_p + NT4 * 128), NT4 * 128);   // [NT4 * 128] request ids

    const int G = a.G, B = a.B, W = a.W, WL = a.wl, A = G * B;
    const unsigned posmask = (1u << WL) - 1u;
    const unsigned lt = (1u << lane) - 1u;

    const auto g_base = mk_span(a.ws.act_base + (size_t)inst * A, A);
    const auto g_aid = mk_span(a.ws.act_id ? a.ws.act_id + (size_t)inst * A : nullptr, A);
    const auto g_qs = mk_span(a.wq.s + (size_t)inst * W, W);
    const auto g_qid = mk_span(a.wq.id + (size_t)inst * W, W);
    const auto t_len = mk_span(a.len_tab, a.len_tab ? (1ll << (32 - a.len_shift)) : 0);
    const auto t_term = mk_span(a.term_cdf, B);

    const unsigned long long seed = a.ws.seed[inst];
    const uint32_t key0 = (uint32_t)seed, key1 = (uint32_t)(seed >> 32);
    int k = a.ws.step[inst];
    uint32_t next_id = a.ws.next_id[inst];
    int n_w = a.wq.n[inst];
    int status0 = 0;
    if (n_w < 0 || n_w > W) { status0 = BR_ST_BAD_STATE; n_w = n_w < 0 ? 0 : W; }

    // worker state of lane g; lanes beyond G hold cap = -1, L = 0 and a full occupancy word
    const unsigned long long slots = B >= 64 ? ~0ull : ((1ull << B) - 1ull);
    int cap = -1, L = 0;
    unsigned long long occ = ~0ull;
    if (lane < G) {
        int na = a.ws.nact[(size_t)inst * G + lane];
        if (na < 0 || na > B) { status0 = BR_ST_BAD_STATE; na = na < 0 ? 0 : B; }
        cap = B - na;
        L = (int)a.ws.load[(size_t)inst * G + lane];
        occ = a.ws.occ[(size_t)inst * G + lane] | ~slots;
    }

    // ---- the queue moves to shared memory once per launch: packed keys and ids ----
#pragma unroll
    for (int t = 0; t < NT4; ++t) {
        const int p0 = (t * 32 + lane) * 4;
        int4 sv = make_int4(0, 0, 0, 0); uint4 iv = make_uint4(0u, 0u, 0u, 0u);
        if (p0 < W) {
            sv = *vec_at<const int4>(g_qs, p0);
            iv = *vec_at<const uint4>(g_qid, p0);
        }
        int4 kk;
        kk.x = p0 + 0 < n_w ? (sv.x << WL) | (int)(posmask - (unsigned)(p0 + 0)) : kSmallBeyond;
        kk.y = p0 + 1 < n_w ? (sv.y << WL) | (int)(posmask - (unsigned)(p0 + 1)) : kSmallBeyond;
        kk.z = p0 + 2 < n_w ? (sv.z << WL) | (int)(posmask - (unsigned)(p0 + 2)) : kSmallBeyond;
        kk.w = p0 + 3 < n_w ? (sv.w << WL) | (int)(posmask - (unsigned)(p0 + 3)) : kSmallBeyond;
        *vec_at<int4>(q_key, p0) = kk;
        *vec_at<uint4>(q_id, p0) = iv;
    }
    __syncwarp();

#pragma unroll 1
    for (int it = 0; it < a.n_steps; ++it, ++k) {
        const size_t orow = (size_t)it * a.N + inst;          // outputs use the rows of the state (first_instance = 0 when n_steps > 1)
        const auto assign = mk_span(a.assign_out + orow * W, W);
#pragma unroll
        for (int t = 0; t < NT4; ++t) {
            const int p0 = (t * 32 + lane) * 4;
            if (p0 < W) *vec_at<int4>(assign, p0) = make_int4(-1, -1, -1, -1);
        }

        // ================= ARRIVE (Section 2.2) =================
        // One Philox call serves the step: lane 31 draws the arrival count, lane b < 31 the block
        // of prompt-length words of arrivals 4b .. 4b+3.
        int n_arr = 0;
        uint4 rb = make_uint4(0u, 0u, 0u, 0u);
        if (a.arr_cdf) {
            const int kp = a.arr_period == 1 ? 0 : k % a.arr_period;
            const auto rowp = mk_span(a.arr_cdf + ((size_t)inst * a.arr_inst_stride + (size_t)kp) * a.arr_len, a.arr_len);
            const uint32_t r0 = lane < a.arr_len ? rowp[lane] : 0xFFFFFFFFu;
            const uint32_t r1 = lane + 32 < a.arr_len ? rowp[lane + 32] : 0xFFFFFFFFu;
            rb = philox4x32_10((uint32_t)k, lane == 31 ? 0u : (uint32_t)lane,
                               lane == 31 ? kStreamArrCount : kStreamArrLen, 0u, key0, key1);
            const uint32_t u = __shfl_sync(kFull, rb.x, 31);
            n_arr = __popc(__ballot_sync(kFull, lane < a.arr_len && u >= r0)) +
                    __popc(__ballot_sync(kFull, lane + 32 < a.arr_len && u >= r1));
        }
        // constant-hazard draws of this step for worker `lane` (used after routing)
        unsigned long long fin = 0ull;
        if (a.term_mode == 1 && lane < G)
            draw_ending(t_term, B, 1, (uint32_t)k, (uint32_t)lane, key0, key1, &fin);
        // a request that was running before this step and ends at it: its load is asked for now
        const unsigned long long pre = occ & fin & slots;
        const int pj = __ffsll((long long)pre) - 1;
        int pend = 0;
        if (pj >= 0) pend = g_base[lane * B + pj];

        const int n_w_old = n_w;
        const uint32_t id0 = next_id;
        int n_take = W - n_w;
        n_take = n_arr < n_take ? n_arr : n_take;
        const int n_drop = n_arr - n_take;
#pragma unroll 1
        for (int j0 = 0; j0 < n_take; j0 += 32) {
            const int j = j0 + lane;                                   // arrival j: word j % 4 of block j / 4
            const int src = (j >> 2) & 31;
            const uint32_t w0 = __shfl_sync(kFull, rb.x, src), w1 = __shfl_sync(kFull, rb.y, src);
            const uint32_t w2 = __shfl_sync(kFull, rb.z, src), w3 = __shfl_sync(kFull, rb.w, src);
            if (j < n_take) {
                const uint32_t w = (j & 2) ? ((j & 1) ? w3 : w2) : ((j & 1) ? w1 : w0);
                const int s = t_len[w >> a.len_shift];
                const int pos = n_w_old + j;
                q_key[pos] = (s << WL) | (int)(posmask - (unsigned)pos);
                q_id[pos] = id0 + (unsigned)j;
            }
        }
        n_w += n_take;
        next_id += (uint32_t)n_arr;
        __syncwarp();

        // ================= ROUTE (Algorithm 1) =================
        int S_tot = (int)__reduce_add_sync(kFull, (unsigned)(cap > 0 ? cap : 0));
        int M = __reduce_max_sync(kFull, L);
        int n_left = n_w, admitted = 0, s1_iters = 0, s2_pops = 0, status = status0;
        int first_rm = W;                     // lowest queue position admitted so far
        int gw[RM];                           // the RM largest waiting keys, descending
        bool gw_valid = false;
#pragma unroll
        for (int r = 0; r < RM; ++r) gw[r] = 0;

#pragma unroll 1
        for (int iter = 0; n_left > 0 && S_tot > 0; ++iter) {
            if (iter >= 2 * W + G) { status |= BR_ST_ITER_CAP; break; }
            const bool stage1 = S_tot > a.S_greedy;
            // worker: most free slots, then smallest L_g (= largest safe margin), then lowest g
            const int mc = __reduce_max_sync(kFull, cap);
            if (mc <= 0) break;
            const unsigned ml = __reduce_min_sync(kFull, cap == mc ? (unsigned)L : 0xFFFFFFFFu);
            const int g = __ffs(__ballot_sync(kFull, cap == mc && (unsigned)L == ml)) - 1;
            const int m = M - (int)ml;                                  // safe margin m_g (Section 3.1)
            int todo = 0;                                               // window entries to admit (bit r)
            bool single = stage1;
            if (stage1) {
                ++s1_iters;
            } else {
                ++s2_pops;
                if (!gw_valid) {
                    // the RM largest keys: sorted per lane, then merged by RM warp maxima
                    int tk[RM];
#pragma unroll
                    for (int r = 0; r < RM; ++r) tk[r] = 0;
#pragma unroll
                    for (int t = 0; t < NT4; ++t) {
                        const int4 kk = *vec_at<const int4>(q_key, (t * 32 + lane) * 4);
                        const int ke[4] = {kk.x, kk.y, kk.z, kk.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            int x = ke[j];
#pragma unroll
                            for (int r = 0; r < RM - 1; ++r) { const int y = max(tk[r], x); x = min(tk[r], x); tk[r] = y; }
                            tk[RM - 1] = max(tk[RM - 1], x);
                        }
                    }
#pragma unroll
                    for (int r = 0; r < RM; ++r) {
                        const int mx = __reduce_max_sync(kFull, tk[0]);
                        gw[r] = mx;
                        if (tk[0] == mx) {
#pragma unroll
                            for (int q = 0; q < RM - 1; ++q) tk[q] = tk[q + 1];
                            tk[RM - 1] = 0;
                        }
                    }
                    gw_valid = true;
                }
                // subsets of the window, one per lane (lane = mask, bit r = r-th largest request)
                int nwin = a.R_max < n_left ? a.R_max : n_left;
                const int lim = mc < a.R_max ? mc : a.R_max;
                int delta = 0;
#pragma unroll
                for (int r = 0; r < RM; ++r) if ((lane >> r) & 1) delta += gw[r] >> WL;
                int over = delta - m; over = over > 0 ? over : 0;
                int f = delta - G * over;                               // Eq. 1
                if (lane == 0 || lane >= (1 << nwin) || __popc(lane) > lim) f = kEmpty;
                const int mf = __reduce_max_sync(kFull, f);
                if (mf > 0) todo = __ffs(__ballot_sync(kFull, f == mf)) - 1;   // lowest mask on ties
                else single = true;                                     // starvation guard
            }
            int qk = 0;
            if (single) {
                // argmax_i F_g({i}) over all of R_wait, earliest arrival on ties
                int bf = kEmpty, bkey = 0;
#pragma unroll
                for (int t = 0; t < NT4; ++t) {
                    const int4 kk = *vec_at<const int4>(q_key, (t * 32 + lane) * 4);
                    const int ke[4] = {kk.x, kk.y, kk.z, kk.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int s = ke[j] >> WL;
                        int over = s - m; over = over > 0 ? over : 0;
                        const int f = s - G * over;                     // Eq. 1
                        if (f > bf) { bf = f; bkey = ke[j]; }           // positions ascend within a lane
                    }
                }
                const int mf = __reduce_max_sync(kFull, bf);
                const unsigned mp = __reduce_max_sync(kFull, bf == mf ? (unsigned)bkey & posmask : 0u);
                qk = q_key[posmask - mp];
                if (qk <= 0) { status |= BR_ST_BAD_STATE; break; }
                todo = 1;
            }
            // sticky admissions to worker g (lowest free slot), one per set bit of todo
#pragma unroll 1
            for (int r = 0; todo; ++r, todo >>= 1) {
                if (!(todo & 1)) continue;
                if (!single) {
                    qk = gw[0];
#pragma unroll
                    for (int q = 1; q < RM; ++q) if (r == q) qk = gw[q];
                }
                const int s = qk >> WL;
                const int pos = (int)(posmask - ((unsigned)qk & posmask));
                if (lane == g) {
                    const int slot = __ffsll((long long)~occ) - 1;
                    if (slot >= 0) {
                        occ |= 1ull << slot;
                        const int sa = g * B + slot;
                        g_base[sa] = s - k;
                        assign[pos] = sa;
                        q_key[pos] = (int)(0x80000000u | (unsigned)sa);
                        cap -= 1;
                        L += s;
                    } else {                                            // free-slot count and occupancy word disagree
                        status |= BR_ST_BAD_STATE;
                        q_key[pos] = kSmallBeyond;
                        cap = 0;
                    }
                }
                M = max(M, __shfl_sync(kFull, L, g));
                if (qk >= gw[RM - 1]) gw_valid = false;                 // a cached window entry leaves
                first_rm = min(first_rm, pos);
                --S_tot; --n_left; ++admitted;
                __syncwarp();
            }
        }

        // ================= RECORD (Section 3.1) =================
        {
            const auto o_load = mk_span(reinterpret_cast<long long *>(a.out.load) + orow * G, G);
            if (lane < G) o_load[lane] = (long long)L;
            const int mn = (int)__reduce_min_sync(kFull, lane < G ? (unsigned)L : 0xFFFFFFFFu);
            const unsigned lo = __reduce_add_sync(kFull, (unsigned)L & 0xFFFFu);
            const unsigned hi = __reduce_add_sync(kFull, (unsigned)L >> 16);
            status = (int)__reduce_or_sync(kFull, (unsigned)status);
            if (lane == 0) {
                const auto tr = mk_span(reinterpret_cast<long long *>(a.out.trace) + orow * 3, 3);
                tr[0] = (long long)M; tr[1] = (long long)mn;
                tr[2] = ((long long)hi << 16) + (long long)lo;
                if (a.out.counters) {
                    uint32_t *c = a.out.counters + orow * 4;
                    c[0] = (uint32_t)n_drop; c[1] = (uint32_t)admitted; c[2] = (uint32_t)s1_iters; c[3] = (uint32_t)s2_pops;
                }
                if (a.out.status) a.out.status[orow] = status | (n_drop ? BR_ST_QUEUE_OVERFLOW : 0);
            }
        }

        // ============ stable queue compaction in shared memory; ids of the admitted requests ============
        // An entry that moves down by d positions keeps its length and gains d in the inverted
        // position field: its key grows by d.
        {
            int run = 0;                                  // entries kept in the groups before this one
#pragma unroll
            for (int t = 0; t < NT4; ++t) {
                const int p0 = (t * 32 + lane) * 4;
                if (t * 128 >= n_w) break;
                if (t * 128 + 128 <= first_rm) { run += 128; continue; }     // nothing before the first admission moves
                const int4 kk = *vec_at<const int4>(q_key, p0);
                const uint4 ii = *vec_at<const uint4>(q_id, p0);
                const int ke[4] = {kk.x, kk.y, kk.z, kk.w};
                const unsigned idv[4] = {ii.x, ii.y, ii.z, ii.w};
                int below = run;
#pragma unroll
                for (int j = 0; j < 4; ++j) below += __popc(__ballot_sync(kFull, ke[j] > 0) & lt);
                __syncwarp();                             // the group is read before any of it is overwritten
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int pos = p0 + j;
                    if (ke[j] > 0) {
                        if (below != pos) { q_key[below] = ke[j] + (pos - below); q_id[below] = idv[j]; }
                        ++below;
                    } else if (g_aid && ke[j] != kSmallBeyond) {
                        g_aid[ke[j] & 0x7FFFFFFF] = idv[j];
                    }
                }
                run = __shfl_sync(kFull, below, 31);
            }
            for (int j = n_left + lane; j < n_w; j += 32) q_key[j] = kSmallBeyond;   // vacated tail
            __syncwarp();
        }
        n_w = n_left;

        // ================= ADVANCE (Section 2.2) =================
        // L_g(k+1) = L_g(k) - (loads of the requests that end at k) + (number of survivors)
        if (lane < G) {
            unsigned long long e = occ & fin & slots;
            int sub = 0;
            if (pj >= 0) {
                sub = pend + k;
                g_base[lane * B + pj] = kEmpty;
                e &= ~(1ull << pj);
            }
            while (e) {                                   // rare: more than one, or admitted at this very step
                const int j = __ffsll((long long)e) - 1;
                e &= e - 1;
                sub += g_base[lane * B + j] + k;
                g_base[lane * B + j] = kEmpty;
            }
            occ &= ~(fin & slots);
            const int na = __popcll(occ & slots);
            cap = B - na;
            L = L - sub + na;
        }
        __syncwarp();
    }

    // ---- snapshot write-back ----
#pragma unroll
    for (int t = 0; t < NT4; ++t) {
        const int p0 = (t * 32 + lane) * 4;
        if (p0 < W) {
            const int4 kk = *vec_at<const int4>(q_key, p0);
            int4 sv;
            sv.x = kk.x > 0 ? kk.x >> WL : 0; sv.y = kk.y > 0 ? kk.y >> WL : 0;
            sv.z = kk.z > 0 ? kk.z >> WL : 0; sv.w = kk.w > 0 ? kk.w >> WL : 0;
            *vec_at<int4>(g_qs, p0) = sv;
            *vec_at<uint4>(g_qid, p0) = *vec_at<const uint4>(q_id, p0);
        }
    }
    if (lane < G) {
        a.ws.load[(size_t)inst * G + lane] = (long long)L;
        a.ws.nact[(size_t)inst * G + lane] = B - cap;
        a.ws.occ[(size_t)inst * G + lane] = occ & slots;
    }
    if (lane == 0) {
        a.ws.step[inst] = k;
        a.ws.next_id[inst] = next_id;
        a.wq.n[inst] = n_w;
    }
}

}  // namespace br
