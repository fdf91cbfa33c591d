// The general routing-step kernel: an instance is served by 32 to 256 threads (BR-H, large fleets,
// optional outputs; BR-0 on small fleets runs on br_small_kernel).
//
// Phases per decode step k (Section 2.2 model; Algorithms 1 and 2):
//   ARRIVE -> PREDICT (H > 0) -> ROUTE (Stage 1, Stage 2) -> RECORD -> ADVANCE.
//
// Warp 0 is the router.  It keeps the per-worker state (free slots, projected loads
// L_g(k+h), envelope M_h) in registers, one or two workers per lane, and walks the
// sequential admission loop with warp reductions only: no block barrier sits on the
// admission chain.  The waiting queue lives in shared memory as packed 32-bit keys
// (prompt length in the high bits, inverted position in the low bits) so that "largest
// s, earliest arrival" is one integer max.
//
// Loads are advanced incrementally: L_g(k+1) = L_g(k) - sum of the loads of the requests
// that end at k + number of survivors, so ADVANCE touches only the occupancy bit masks,
// one Philox block per worker (the ending slots are walked by geometric gaps), and the few
// slots whose request ends.  Only the horizon
// projection of BR-H streams the per-request state.
#pragma once
#include "br_device.cuh"
#include "br_mitm.cuh"
#include "../../include/br.h"

namespace br {

struct StepArgs {
    int32_t G, H, B, W, R_max, S_greedy, occ_words;
    int32_t wl;                 // log2 of the queue-position field of a packed key
    uint32_t magic_B;           // ceil(2^32 / B): x / B == umulhi(x, magic_B) for x < 2^16
    int32_t delta_T;
    float gate, c_floor;
    int32_t term_mode;
    int32_t pred_mode;          // 1: c_hat = min(remaining steps, H) from act_end (term_mode 3)
    const int32_t *out_tab;     // output lengths of arrivals (term_mode 3)
    int32_t out_shift;
    const uint32_t *term_cdf;   // [B] gap thresholds of the constant hazard
    const uint32_t *arr_cdf;
    int32_t arr_len, arr_period, arr_inst_stride;
    const int32_t *len_tab;
    int32_t len_shift;
    int32_t burst_every, burst_size;
    double aD, beta;
    int32_t peak_ok;            // Eq. 2: every slope alpha D - beta sum_{h in P} d_h is clearly off zero (br_create)
    int32_t big_window;         // R_max > 5: Stage 2 solves its window by meeting in the middle
    double d[BR_MAX_H + 1];
    int32_t N, first_instance, n_steps;
    int32_t tpi, smem_per_inst;  // threads and shared-memory bytes per instance
    int32_t block_sync;          // 1: every barrier is a block barrier (needs full blocks)
    br_worker_state ws;
    br_waiting_queue wq;
    const float *term_probs;
    int32_t *assign_out;
    br_load_out out;
};

// shared-memory footprint of one instance (bytes), mirrored by the host
__host__ __device__ inline size_t step_smem_bytes(int G, int H, int B, int W, int occ_words, bool lifetimes = false,
                                                  bool big_window = false)
{
    size_t n = 0;
    n += 4 * (size_t)W * 2;                      // q_key, q_id
    n += 8 * (size_t)G * occ_words * 2;          // occ, end_mask
    n += 4 * (size_t)G * (H + 1) * 2;            // Lh_s, Ch_s (PREDICT buckets: load sums, counts)
    n += 4 * (size_t)G;                          // sub_load
    n += 8 * (size_t)G * occ_words;              // fin_w
    n += 8 * (size_t)(H + 1) + 4 * (size_t)((H + 2) / 2 * 2);   // md_s (fp64 margins of the selected worker), M_s (envelope)
    n += 2 * 96 + 2 * 32 + 64;                   // end_list, pre_list, scalars
    if (H > 0) n += 2 * (size_t)G * B;           // refresh_list
    n = (n + 15) & ~(size_t)15;
    if (lifetimes) n += 4 * (size_t)W;           // q_o (output lengths of the waiting requests)
    n = (n + 15) & ~(size_t)15;
    if (big_window) n += 8 * (size_t)(1 << 8) + 4 * 16 + 4 * 16;   // sorted half-window subsets, class offsets, window keys
    return (n + 15) & ~(size_t)15;
}

// Order- and sign-preserving key of a score: Eq. 1 in integers (FP = false) or Eq. 2 in
// fp64 evaluated term by term in h (FP = true).
// SL: the horizon is too long for registers; the margins of the selected worker are read from
// shared memory (mds) and the loops over h are not unrolled.
template <bool FP, int HM, bool SL = false>
struct Scorer {
    int mi;                 // Eq. 1 margin
    double md[SL ? 1 : HM + 1];   // Eq. 2 margins
    span_t<double> mds;     // Eq. 2 margins in shared memory (SL)
    int mmin;               // min_h m_{g,h}: at or below it the Eq. 2 penalty is exactly zero

    __device__ __forceinline__ long long key(const StepArgs &a, int delta) const
    {
        if (!FP) {
            int over = delta - mi;
            over = over > 0 ? over : 0;
            return (long long)(delta - a.G * over);        // |F| < 2^31 by the create-time proof
        } else {
            const double dl = (double)delta;
            double pen = 0.0;
            if (SL) {
#pragma unroll 4
                for (int h = 0; h <= a.H; ++h) {
                    double over = __dsub_rn(dl, mds[h]);
                    over = over > 0.0 ? over : 0.0;
                    pen = __dadd_rn(pen, __dmul_rn(a.d[h], over));
                }
            } else {
#pragma unroll
                for (int h = 0; h <= HM; ++h) {
                    if (h <= a.H) {
                        double over = __dsub_rn(dl, md[h]);     // exact: integers below 2^53
                        over = over > 0.0 ? over : 0.0;
                        pen = __dadd_rn(pen, __dmul_rn(a.d[h], over));
                    }
                }
            }
            return key_of_double(__dsub_rn(__dmul_rn(a.aD, dl), __dmul_rn(a.beta, pen)));
        }
    }
    __device__ __forceinline__ static double value(long long k)
    {
        return FP ? double_of_key(k) : (double)k;
    }
};

// warp arg-max of (64-bit key, then largest 32-bit tie value); returns the winning lane
__device__ __forceinline__ int warp_argmax_lane(long long key, unsigned tie, long long &wkey)
{
    const int hi = (int)(key >> 32);
    const unsigned lo = (unsigned)key;
    const int mhi = __reduce_max_sync(kFull, hi);
    const bool in1 = hi == mhi;
    const unsigned mlo = __reduce_max_sync(kFull, in1 ? lo : 0u);
    const bool in2 = in1 && lo == mlo;
    const unsigned mt = __reduce_max_sync(kFull, in2 ? tie : 0u);
    const unsigned who = __ballot_sync(kFull, in2 && tie == mt);
    wkey = (long long)(((unsigned long long)(unsigned)mhi << 32) | mlo);
    return __ffs(who) - 1;
}

// same for 32-bit keys (Eq. 1 scores): largest key, then largest tie value
__device__ __forceinline__ int warp_argmax_lane32(int key, unsigned tie, int &wkey)
{
    const int mk = __reduce_max_sync(kFull, key);
    const bool in1 = key == mk;
    const unsigned mt = __reduce_max_sync(kFull, in1 ? tie : 0u);
    const unsigned who = __ballot_sync(kFull, in1 && tie == mt);
    wkey = mk;
    return __ffs(who) - 1;
}

// Slots of worker g that end at step k under the constant hazard, as bit masks of 64 slots each.
// Slots end independently with one probability, so the ending ones are walked by their gaps:
// cdf[j] = floor(2^32 P(gap <= j)), draw t is word t % 4 of the Philox block (k, g, TERM, t / 4),
// and a word u skips gap = #{j : u >= cdf[j]} slots (cdf ascends: the first j with u < cdf[j]).
template <typename CDF, typename OUT>
__device__ __forceinline__ void draw_ending(const CDF cdf, int B, int OW, uint32_t k,
                                            uint32_t g, uint32_t key0, uint32_t key1,
                                            const OUT out)
{
    for (int w = 0; w < OW; ++w) out[w] = 0ull;
    int pos = 0;
    uint4 r = philox4x32_10(k, g, kStreamTerm, 0u, key0, key1);
#pragma unroll 1
    for (unsigned t = 0; t < (unsigned)B; ++t) {          // every draw moves pos forward
        if (t != 0u && (t & 3u) == 0u) r = philox4x32_10(k, g, kStreamTerm, t >> 2, key0, key1);
        const uint32_t u = word_of(r, t & 3u);
        const int room = B - pos;
        if (u >= cdf[room - 1]) break;                    // the gap reaches past the last slot
        int lo = 0, hi = room - 1;                        // u < cdf[hi]
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (u < cdf[mid]) hi = mid; else lo = mid + 1;
        }
        const int slot = pos + lo;
        out[slot >> 6] |= 1ull << (slot & 63);
        pos = slot + 1;
        if (pos >= B) break;
    }
}

// Loads of classifier output.  A row is read once, by one thread, at a scattered address; left to
// itself the L2 fetches 128 bytes around a missing sector, of which a refresh uses 32 on average,
// so the loads ask for the smallest fetch the instruction set offers (64 bytes).
__device__ __forceinline__ float4 ld_row4(const float *p)
{
    float4 v;
    asm volatile("ld.global.nc.L2::64B.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}
// a whole row of eight probabilities (32-byte aligned) as one 256-bit load
__device__ __forceinline__ void ld_row8(const float *p, float *o)
{
    unsigned r[8];
    asm volatile("ld.global.nc.L2::64B.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]) : "l"(p));
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i] = __uint_as_float(r[i]);
}

// Adds (val, 1) to the prediction bucket `key` (load sum in T, count in C) if key >= 0.  Plain
// shared-memory atomics: combining the lanes of a warp that share a bucket first (match.any and a
// masked reduction) measured 70 % slower than letting the atomics collide.
template <typename TP, typename CP>
__device__ __forceinline__ void bucket_add(const TP T, const CP C, int key, unsigned val, int lane)
{
    (void)lane;
    if (key >= 0) { atomicAdd(&T[key], val); atomicAdd(&C[key], 1u); }
}

constexpr int kRegWin = 5;      // Stage-2 windows of up to five requests are scored one subset per lane
constexpr int kBigWinLow = 8;   // larger windows (up to BR_MAX_RMAX = 16): subsets of the low eight entries are sorted
constexpr int kPassBUnroll = 2;  // classifier rows in flight per thread (4 and 8 measured the same)
constexpr int kUnroll = 2;       // slot quads in flight per thread in the BR-H streaming phase (4 measured the same)
constexpr int kEndList = 96;    // requests ending in one step that are fixed up as one batch

// LEAN > 0: constant-hazard terminations and no optional outputs (score matrix, cycle counters);
// LEAN == 2: in addition the instance is a single warp.  The paths not needed are compiled out,
// which shortens the code every warp walks.
template <bool FP, int HM, int GW, int LEAN>
__global__ void __maxnreg__((FP && HM > 0) ? 128 : 72) br_step_kernel(const StepArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_all[];
    // a.tpi threads serve one instance; a block holds blockDim.x / a.tpi instances (more than one
    // only when tpi == 32, so that an instance-wide barrier is a warp barrier)
    constexpr bool SL = HM > 16;          // long horizons: projected loads, envelope and margins in shared memory
    constexpr int HR = SL ? 0 : HM;       // horizon offsets kept in registers
    const int NT = a.tpi;
    const int tid = threadIdx.x % NT, lane = tid & 31, warp = tid >> 5;
    const int in_block = threadIdx.x / NT, per_block = blockDim.x / NT;
    stream_order_gate();
    if (blockIdx.x * per_block + in_block >= a.N) return;            // whole instance groups only
    unsigned char *smem_raw = smem_all + (size_t)in_block * a.smem_per_inst;
    // Instance-wide barrier.  Single-warp instances that share a block may also be aligned with a
    // block barrier (a.block_sync): the warps then walk the same code at about the same time, which
    // pays off in instruction fetch although no data crosses between them.
    // (Giving wider instances that share a block a named barrier each, so that one never waits for
    // its neighbour, measured 3 % slower on the 1024-instance BR-H batch: instances that walk the
    // phases together share instruction fetch and keep the memory phases aligned.)
    auto inst_sync = [&]() { if (NT == 32 && !a.block_sync) __syncwarp(); else __syncthreads(); };
    const int nwarps = LEAN == 2 ? 1 : (NT >> 5);
    const int term_mode = LEAN ? 1 : a.term_mode;
    const int G = a.G, H = a.H, B = a.B, W = a.W, H1 = H + 1, A = G * B, OW = a.occ_words;
    const int A8 = A >> 3;
    const int WL = a.wl;
    const unsigned posmask = (1u << WL) - 1u;
    const int inst = a.first_instance + blockIdx.x * per_block + in_block;
    const unsigned t_entry = (unsigned)clock64();

    // ---- shared-memory carve-up (sizes match step_smem_bytes) ----
    // (raw carve-up first; every array is then used through a span that knows its length)
    int *q_key_p = reinterpret_cast<int *>(smem_raw);                               // [W]
    unsigned *q_id_p = reinterpret_cast<unsigned *>(q_key_p + W);                   // [W]
    unsigned long long *occ_p = reinterpret_cast<unsigned long long *>(q_id_p + W); // [G][OW]
    unsigned long long *end_mask_p = occ_p + (size_t)G * OW;                        // [G][OW]
    unsigned long long *fin_w_p = end_mask_p + (size_t)G * OW;                      // [G][OW] slots whose draw says "ends"
    double *md_s_p = reinterpret_cast<double *>(fin_w_p + (size_t)G * OW);          // [H1] margins of the selected worker
    int *M_s_p = reinterpret_cast<int *>(md_s_p + H1);                              // [H1 rounded up to even] envelope
    unsigned *Lh_s_p = reinterpret_cast<unsigned *>(M_s_p + (H1 + 1) / 2 * 2);      // [G][H1]
    unsigned *Ch_s_p = Lh_s_p + (size_t)G * H1;                                     // [G][H1]
    unsigned *sub_load_p = Ch_s_p + (size_t)G * H1;                                 // [G]
    unsigned short *end_list_p = reinterpret_cast<unsigned short *>(sub_load_p + G);// [kEndList]
    unsigned short *pre_list_p = end_list_p + kEndList;                             // [32]
    int *scal_p = reinterpret_cast<int *>(pre_list_p + 32);                         // [16]
    unsigned short *refresh_list_p = reinterpret_cast<unsigned short *>(scal_p + 16);   // [A] (H > 0 only)
    // output lengths of the waiting requests (term_mode 3 only), behind everything else
    int *q_o_p = reinterpret_cast<int *>(smem_raw + ((step_smem_bytes(G, H, B, W, OW) + 15) & ~(size_t)15));
    // large Stage-2 windows: sorted subsets of the low half, class offsets, the window's keys
    unsigned long long *bw_keys_p = reinterpret_cast<unsigned long long *>(
        smem_raw + step_smem_bytes(G, H, B, W, OW, !LEAN && a.term_mode == 3));
    int *bw_off_p = reinterpret_cast<int *>(bw_keys_p + (1 << kBigWinLow));
    const bool life = !LEAN && a.term_mode == 3;          // requests carry their output lengths
    const bool bigw = !LEAN && a.big_window != 0;
    const auto q_key = mk_span(q_key_p, W);
    const auto q_id = mk_span(q_id_p, W);
    const auto occ = mk_span(occ_p, G * OW);
    const auto end_mask = mk_span(end_mask_p, G * OW);
    const auto fin_w = mk_span(fin_w_p, G * OW);
    const auto md_s = mk_span(md_s_p, H1);
    const auto M_s = mk_span(M_s_p, H1);
    const auto Lh_s = mk_span(Lh_s_p, 2 * G * H1);        // Ch_s follows it; the two are cleared as one block
    const auto Ch_s = mk_span(Ch_s_p, G * H1);
    const auto sub_load = mk_span(sub_load_p, G);
    const auto end_list = mk_span(end_list_p, kEndList);
    const auto pre_list = mk_span(pre_list_p, 32);
    const auto scal = mk_span(scal_p, 16);
    const auto refresh_list = mk_span(refresh_list_p, H > 0 ? A : 0);
    const auto q_o = mk_span(q_o_p, life ? W : 0);
    const auto bw_keys = mk_span(bw_keys_p, bigw ? (1 << kBigWinLow) : 0);
    const auto bw_off = mk_span(bw_off_p, bigw ? 16 : 0);
    const auto bw_win = mk_span(bw_off_p + 16, bigw ? 16 : 0);
    // scal: [0] queue length after routing, [1] admitted, [2] Stage-1 iterations,
    //       [3] Stage-2 pops, [4] status bits of the step, [5] status bits of the prologue,
    //       [6] requests that ended this step and were not prefetched, [7] prefetched ones,
    //       [8] requests whose c_hat is refreshed at this step,
    //       [9] set when requests that end were found before routing and did not fit the lists

    // ---- per-instance global rows ----
    const auto g_load = mk_span(reinterpret_cast<long long *>(a.ws.load) + (size_t)inst * G, G);
    const auto g_nact = mk_span(a.ws.nact + (size_t)inst * G, G);
    const auto g_occ = mk_span(reinterpret_cast<unsigned long long *>(a.ws.occ) + (size_t)inst * G * OW, G * OW);
    const auto g_base = mk_span(a.ws.act_base + (size_t)inst * A, A);
    const auto g_aid = mk_span(a.ws.act_id ? a.ws.act_id + (size_t)inst * A : nullptr, A);
    const auto g_chat0 = mk_span(a.ws.act_chat0 ? a.ws.act_chat0 + (size_t)inst * A : nullptr, A);
    const auto g_kref = mk_span(a.ws.act_kref ? a.ws.act_kref + (size_t)inst * A : nullptr, A);
    const auto g_end = mk_span(life ? a.ws.act_end + (size_t)inst * A : nullptr, A);
    const auto g_qo = mk_span(life ? a.wq.o + (size_t)inst * W : nullptr, W);
    const auto g_qs = mk_span(a.wq.s + (size_t)inst * W, W);
    const auto g_qid = mk_span(a.wq.id + (size_t)inst * W, W);
    const auto t_len = mk_span(a.len_tab, a.len_tab ? (1ll << (32 - a.len_shift)) : 0);
    const auto t_out = mk_span(a.out_tab, a.out_tab ? (1ll << (32 - a.out_shift)) : 0);
    const auto t_term = mk_span(a.term_cdf, B);

    const unsigned long long seed = a.ws.seed[inst];
    const uint32_t key0 = (uint32_t)seed, key1 = (uint32_t)(seed >> 32);
    int k = a.ws.step[inst];
    uint32_t next_id = a.ws.next_id[inst];
    int n_w = a.wq.n[inst];
    int prologue_status = 0;
    if (n_w < 0 || n_w > W) { prologue_status |= BR_ST_BAD_STATE; n_w = n_w < 0 ? 0 : W; }

    if (tid < 16) scal[tid] = 0;
    // queue -> packed keys and ids in shared memory (16-byte loads).  The first chunks are
    // requested without waiting for the queue length (rows always hold W entries).
    auto fetch_queue = [&](int i) {
        const int4 v = *vec_at<const int4>(g_qs, i);
        const uint4 u = *vec_at<const uint4>(g_qid, i);
        int4 kk;
        kk.x = (v.x << WL) | (int)(posmask - (unsigned)(i + 0));
        kk.y = (v.y << WL) | (int)(posmask - (unsigned)(i + 1));
        kk.z = (v.z << WL) | (int)(posmask - (unsigned)(i + 2));
        kk.w = (v.w << WL) | (int)(posmask - (unsigned)(i + 3));
        *vec_at<int4>(q_key, i) = kk;
        *vec_at<uint4>(q_id, i) = u;
        if (life) *vec_at<int4>(q_o, i) = *vec_at<const int4>(g_qo, i);
    };
    {
        const int i0 = tid * 4, i1 = (NT + tid) * 4;
        if (i0 < W) fetch_queue(i0);
        if (i1 < W) fetch_queue(i1);
    }
    for (int i = (2 * NT + tid) * 4; i < n_w; i += NT * 4) fetch_queue(i);
    for (int i = tid; i < G * OW; i += NT) { occ[i] = g_occ[i]; fin_w[i] = 0ull; }
    for (int i = tid; i < 2 * G * H1; i += NT) Lh_s[i] = 0u;      // Lh_s and Ch_s are adjacent
    for (int i = tid; i < G; i += NT) sub_load[i] = 0u;

    // router registers: lane owns workers lane and lane + 32
    int cap[GW];
    int L[GW][HR + 1];
    int Mh[HR + 1];
    const auto L_s = mk_span(reinterpret_cast<int *>(raw_of(Lh_s)), G * H1);     // SL: the buckets become L_g(k+h) in place
#pragma unroll
    for (int h = 0; h <= HR; ++h) Mh[h] = 0;
#pragma unroll
    for (int w = 0; w < GW; ++w) {
        const int g = lane + 32 * w;
        cap[w] = -1;
#pragma unroll
        for (int h = 0; h <= HR; ++h) L[w][h] = 0;
        if (warp == 0 && g < G) {
            int na = g_nact[g];
            if (na < 0 || na > B) { prologue_status |= BR_ST_BAD_STATE; na = na < 0 ? 0 : B; }
            cap[w] = B - na;
            L[w][0] = (int)g_load[g];
        }
    }
    inst_sync();
    if (prologue_status) atomicOr(&scal[5], prologue_status);

    // this step's constant-hazard draws of workers first, first + stride, ...
    auto draw_fin = [&](int first, int stride) {
#pragma unroll 1
        for (int g = first; g < G; g += stride)
            draw_ending(t_term, B, OW, (uint32_t)k, (uint32_t)g, key0, key1, fin_w + (size_t)g * OW);
    };

    // Per worker word: which running requests end at this step (occupancy & termination draws).
    // Writes end_mask and lists the ending slots; with `prefetch` the first 32 go to pre_list so
    // that their loads can be requested at once by one lane each.
    auto scan_workers = [&](bool prefetch) {
#pragma unroll 1
        for (int idx = tid; idx < G * OW; idx += NT) {
            const int g = idx / OW, x = idx - g * OW;
            const unsigned long long occw = occ[idx];
            const unsigned long long finw = term_mode != 0 ? fin_w[idx] : 0ull;
            unsigned long long ended = occw & finw;
            end_mask[idx] = ended;
            while (ended) {
                const int j = __ffsll((long long)ended) - 1;
                ended &= ended - 1;
                const int sa = g * B + 64 * x + j;
                int at = prefetch ? atomicAdd(&scal[7], 1) : 32;
                if (at < 32) {
                    pre_list[at] = (unsigned short)sa;
                } else {
                    at = atomicAdd(&scal[6], 1);
                    if (at < kEndList) {
                        end_list[at] = (unsigned short)sa;
                    } else {                                         // list full: fix this slot up at once
                        atomicAdd(&sub_load[g], (unsigned)(g_base[sa] + k));
                        // before routing the request still runs (the projection of this step counts
                        // it): its slot is emptied in ADVANCE, found again through end_mask
                        if (prefetch) scal[9] = 1; else g_base[sa] = kEmpty;
                    }
                }
            }
        }
    };

    for (int it = 0; it < a.n_steps; ++it, ++k) {
        const size_t orow = (size_t)it * a.N + inst;
        const auto probs = mk_span(a.term_probs ? a.term_probs + orow * (size_t)A * H : nullptr, (long long)A * H);
        unsigned t_phase[7];
        const bool timing = !LEAN && a.out.phase_cycles != nullptr && tid == 0;
        if (timing) t_phase[0] = (unsigned)clock64();

        // ================= ARRIVE =================
        // the arrival-count row is requested first; a single-warp block draws the termination
        // words while that load is in flight
        uint32_t row0 = 0xFFFFFFFFu, row1 = 0xFFFFFFFFu;
        span_t<const uint32_t> row = mk_span((const uint32_t *)nullptr, 0);
        if (a.arr_cdf) {
            row = mk_span(a.arr_cdf + ((size_t)inst * a.arr_inst_stride + (size_t)(k % a.arr_period)) * a.arr_len, a.arr_len);
            if (lane < a.arr_len) row0 = row[lane];
            if (lane + 32 < a.arr_len) row1 = row[lane + 32];
        }
        // A single-warp instance also resolves, right away, which of the requests already
        // running end at this step, and requests their loads: the values are used only after
        // routing, so that memory latency is off the step's critical path.
        const bool have_pre = (nwarps == 1 && term_mode == 1);
        int pend = 0, n_pre = 0;
        if (have_pre) {
            draw_fin(tid, NT);
            __syncwarp();
            scan_workers(true);
            __syncwarp();
            n_pre = min(scal[7], 32);
            if (tid < n_pre) pend = g_base[pre_list[tid]];
        }
        int n_arr = 0;
        if (a.arr_cdf) {
            const uint32_t u = philox4x32_10((uint32_t)k, 0u, kStreamArrCount, 0u, key0, key1).x;
            n_arr = __popc(__ballot_sync(kFull, lane < a.arr_len && u >= row0)) +
                    __popc(__ballot_sync(kFull, lane + 32 < a.arr_len && u >= row1));
            for (int j0 = 64; j0 < a.arr_len; j0 += 32) {
                const int j = j0 + lane;
                const bool ge = (j < a.arr_len) && (u >= row[j]);
                n_arr += __popc(__ballot_sync(kFull, ge));
            }
            if (a.burst_every > 0 && k > 0 && (k % a.burst_every) == 0) n_arr += a.burst_size;
        }
        const int n_w_old = n_w;
        const uint32_t id0 = next_id;             // id of arrival 0 of this step
        for (int j = tid; j < n_arr; j += NT) {
            const int pos = n_w_old + j;
            if (pos < W) {
                const uint4 r = philox4x32_10((uint32_t)k, (uint32_t)j >> 2, kStreamArrLen, 0u, key0, key1);
                const int s = t_len[word_of(r, j & 3) >> a.len_shift];
                q_key[pos] = (s << WL) | (int)(posmask - (unsigned)pos);
                q_id[pos] = id0 + (unsigned)j;
                if (life) {
                    const uint4 ro = philox4x32_10((uint32_t)k, (uint32_t)j >> 2, kStreamArrOut, 0u, key0, key1);
                    q_o[pos] = t_out[word_of(ro, j & 3) >> a.out_shift];
                }
            }
        }
        int n_drop = n_w + n_arr - W;
        n_drop = n_drop > 0 ? n_drop : 0;
        n_w = n_w + n_arr - n_drop;
        next_id += (uint32_t)n_arr;
        if (timing) t_phase[1] = (unsigned)clock64();

        // ============ PREDICT (H > 0): c_hat maintenance + horizon projection ============
        // Every running request adds (cur, 1) to the bucket (worker, floor(c_hat)); the router turns
        // the buckets into L_g(k+h) = sum_{j >= h} T_j + h * sum_{j >= h} C_j by suffix sums.
        // Pass A streams the per-request state and settles the requests that only age; the ones due
        // for a refresh are listed, and pass B reads their classifier rows with independent loads.
        if (HM > 0 && H > 0 && !LEAN && a.pred_mode == 1) {
            // perfect lookahead: c_hat = min(r_i(k), H) with r_i(k) = act_end - k + 1 steps still to run
            const int A4 = A >> 2;
#pragma unroll 2
            for (int q0 = 0; q0 < A4; q0 += NT) {
                const int q4 = q0 + tid;
                const bool inr = q4 < A4;
                const int4 bq = inr ? *vec_at<const int4>(g_base, 4 * q4) : make_int4(kEmpty, kEmpty, kEmpty, kEmpty);
                const int4 eq = inr ? *vec_at<const int4>(g_end, 4 * q4) : make_int4(0, 0, 0, 0);
                const int bs4[4] = {bq.x, bq.y, bq.z, bq.w};
                const int en4[4] = {eq.x, eq.y, eq.z, eq.w};
                const int g = (int)__umulhi((unsigned)(4 * q4), a.magic_B);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const bool live = bs4[j] != kEmpty;
                    int nh = en4[j] - k + 1;
                    nh = nh < 0 ? 0 : (nh > H ? H : nh);
                    bucket_add(Lh_s, Ch_s, live ? g * H1 + nh : -1, live ? (unsigned)(bs4[j] + k) : 0u, lane);
                }
            }
        } else if (HM > 0 && H > 0) {
            const int A4 = A >> 2;
#pragma unroll 1
            for (int q_base = 0; q_base < A4; q_base += NT * kUnroll) {
                int4 bq[kUnroll]; float4 cq[kUnroll]; unsigned kq[kUnroll];
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    const int q4 = q_base + u * NT + tid;
                    const bool inr = q4 < A4;
                    bq[u] = inr ? *vec_at<const int4>(g_base, 4 * q4) : make_int4(kEmpty, kEmpty, kEmpty, kEmpty);
                    cq[u] = inr ? *vec_at<const float4>(g_chat0, 4 * q4) : make_float4(0.f, 0.f, 0.f, 0.f);
                    kq[u] = inr ? *vec_at<const unsigned>(g_kref, 4 * q4) : 0u;
                }
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    const int q4 = q_base + u * NT + tid;
                    const int bs4[4] = {bq[u].x, bq[u].y, bq[u].z, bq[u].w};
                    const float c04[4] = {cq[u].x, cq[u].y, cq[u].z, cq[u].w};
                    const int g = (int)__umulhi((unsigned)(4 * q4), a.magic_B);      // slot / B
                    // which of the four requests are due for a refresh; one list append per quad and warp
                    bool due4[4]; float c4[4]; unsigned dm4[4];
                    int n_due = 0;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const bool live = bs4[j] != kEmpty;
                        const int t = (k - (int)((kq[u] >> (8 * j)) & 0xFFu)) & 255;
                        c4[j] = c04[j] - (float)t;
                        due4[j] = live && (t >= a.delta_T || c4[j] < a.c_floor);
                        dm4[j] = __ballot_sync(kFull, due4[j]);
                        n_due += __popc(dm4[j]);
                    }
                    if (n_due) {                                             // uniform over the warp
                        int at = 0;
                        if (lane == 0) at = atomicAdd(&scal[8], n_due);
                        at = __shfl_sync(kFull, at, 0);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            if (due4[j]) refresh_list[at + __popc(dm4[j] & ((1u << lane) - 1u))] = (unsigned short)(4 * q4 + j);
                            at += __popc(dm4[j]);
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const bool settle = bs4[j] != kEmpty && !due4[j];
                        int nh = (int)floorf(c4[j]);
                        nh = nh < 0 ? 0 : (nh > H ? H : nh);
                        bucket_add(Lh_s, Ch_s, settle ? g * H1 + nh : -1, settle ? (unsigned)(bs4[j] + k) : 0u, lane);
                    }
                }
            }
            inst_sync();
            const int n_ref = scal[8];
            // Pass B: the classifier row of every request on the list.  The loop runs the same number of
            // rounds on every lane.
#pragma unroll kPassBUnroll
            for (int e0 = 0; e0 < n_ref; e0 += NT) {
                const int e = e0 + tid;
                int key = -1;
                unsigned cur = 0u;
                if (e < n_ref) {
                    const int s0 = refresh_list[e];
                    const auto q = probs + (long long)s0 * H;
                    double v = (double)H;                               // gate closed: the conservative anchor
                    if (SL) {
                        // long classifier rows stay in memory: p_fin and c* in one pass
                        double surv = 1.0, cs = 0.0;
                        for (int h = 0; h < H; ++h) {
                            cs = __dadd_rn(cs, surv);
                            surv = __dmul_rn(surv, __dsub_rn(1.0, (double)q[h]));
                        }
                        if (__dsub_rn(1.0, surv) >= (double)a.gate) v = cs;
                    } else {
                        float qv[HR > 0 ? HR : 1];
                        if (HR == 8 && H == 8 && (reinterpret_cast<size_t>(raw_of(probs)) & 31) == 0) {
                            ld_row8(reinterpret_cast<const float *>(vec_at<const double4>(q, 0)), qv);
                        } else if ((H & 3) == 0) {
#pragma unroll
                            for (int h = 0; h < HR; h += 4) {
                                if (h < H) {
                                    const float4 qq = ld_row4(reinterpret_cast<const float *>(vec_at<const float4>(q, h)));
                                    qv[h] = qq.x; qv[h + 1] = qq.y; qv[h + 2] = qq.z; qv[h + 3] = qq.w;
                                }
                            }
                        } else {
#pragma unroll
                            for (int h = 0; h < HR; ++h) if (h < H) qv[h] = q[h];
                        }
                        // p_fin = 1 - prod (1 - q_h) <= sum q_h for probabilities: when the fp32 sum is
                        // clearly below the gate the fp64 product cannot reach it and is not evaluated
                        float qsum = 0.0f, qmin = 0.0f;
#pragma unroll
                        for (int h = 0; h < HR; ++h) if (h < H) { qsum += qv[h]; qmin = fminf(qmin, qv[h]); }
                        double p_fin = 0.0;
                        if (!(qmin >= 0.0f && qsum * 1.0001f < a.gate)) {
                            double surv = 1.0;
#pragma unroll
                            for (int h = 0; h < HR; ++h)
                                if (h < H) surv = __dmul_rn(surv, __dsub_rn(1.0, (double)qv[h]));
                            p_fin = __dsub_rn(1.0, surv);
                        }
                        if (p_fin >= (double)a.gate) {
                            // gate open: E[min(r, H)] = sum_h prod_{j<h} (1 - q_j)
                            double sv = 1.0, cs = 0.0;
#pragma unroll
                            for (int h = 0; h < HR; ++h) {
                                if (h < H) {
                                    cs = __dadd_rn(cs, sv);
                                    sv = __dmul_rn(sv, __dsub_rn(1.0, (double)qv[h]));
                                }
                            }
                            v = cs;
                        }
                    }
                    if (v < (double)a.c_floor) v = (double)a.c_floor;   // clipped to [floor, H]
                    if (v > (double)H) v = (double)H;
                    const float c = (float)v;
                    cur = (unsigned)(g_base[s0] + k);
                    g_chat0[s0] = c;
                    g_kref[s0] = (uint8_t)(k & 255);
                    int nh = (int)floorf(c);
                    nh = nh < 0 ? 0 : (nh > H ? H : nh);
                    key = (int)__umulhi((unsigned)s0, a.magic_B) * H1 + nh;
                }
                bucket_add(Lh_s, Ch_s, key, cur, lane);
            }
        }
        inst_sync();                                              // B1
        if (timing) t_phase[2] = (unsigned)clock64();

        if (warp == 0) {
            // ================= ROUTE (warp 0 only, warp-synchronous) =================
            if (SL) {
                // buckets -> L_g(k+h) in place (each lane owns the rows of its workers), then the envelope
                // with the lanes spread over h
#pragma unroll
                for (int w = 0; w < GW; ++w) {
                    const int g = lane + 32 * w;
                    if (g < G) {
                        int accT = 0, accC = 0;
                        for (int h = H; h >= 0; --h) {
                            accT += (int)Lh_s[g * H1 + h]; accC += (int)Ch_s[g * H1 + h];
                            L_s[g * H1 + h] = accT + h * accC;
                        }
                        L[w][0] = accT;
                    }
                }
                __syncwarp();
                for (int h = lane; h <= H; h += 32) {
                    int v = L_s[h];
                    for (int g = 1; g < G; ++g) v = max(v, L_s[g * H1 + h]);
                    M_s[h] = v;
                }
                __syncwarp();
                Mh[0] = M_s[0];
            } else {
                if (H > 0) {
#pragma unroll
                    for (int w = 0; w < GW; ++w) {
                        const int g = lane + 32 * w;
                        int accT = 0, accC = 0;
#pragma unroll
                        for (int h = HR; h >= 0; --h) {
                            if (g < G && h <= H) { accT += (int)Lh_s[g * H1 + h]; accC += (int)Ch_s[g * H1 + h]; }
                            L[w][h] = (g < G && h <= H) ? accT + h * accC : 0;
                        }
                    }
                }
#pragma unroll
                for (int h = 0; h <= HR; ++h) {
                    int v = L[0][h];
#pragma unroll
                    for (int w = 1; w < GW; ++w) v = max(v, L[w][h]);
                    Mh[h] = (h <= H) ? __reduce_max_sync(kFull, v) : 0;
                }
            }

            Scorer<FP, HM, SL> sc;
            sc.mds = md_s;
            // margins of worker g -> every lane's scorer
            auto load_margins = [&](int g) {
                const int src = g & 31;
                const int set = g >> 5;
                if (!FP) {
                    int mine = Mh[0] - L[0][0];
#pragma unroll
                    for (int w = 1; w < GW; ++w) if (set == w) mine = Mh[0] - L[w][0];
                    sc.mi = __shfl_sync(kFull, mine, src);
                } else if (SL) {
                    int mmin = 0x7FFFFFFF;
                    __syncwarp();                          // earlier readers of md_s are done
                    for (int h = lane; h <= H; h += 32) {
                        const int mh = M_s[h] - L_s[g * H1 + h];
                        md_s[h] = (double)mh;
                        mmin = min(mmin, mh);
                    }
                    sc.mmin = __reduce_min_sync(kFull, mmin);
                    __syncwarp();
                } else {
                    int mmin = 0x7FFFFFFF;
#pragma unroll
                    for (int h = 0; h <= HR; ++h) {
                        int mine = Mh[h] - L[0][h];
#pragma unroll
                        for (int w = 1; w < GW; ++w) if (set == w) mine = Mh[h] - L[w][h];
                        const int mh = __shfl_sync(kFull, mine, src);
                        sc.md[h] = (double)mh;
                        if (h <= H) mmin = min(mmin, mh);
                    }
                    sc.mmin = mmin;
                }
            };

            // optional F-score matrix before the first admission
            if (!LEAN && a.out.fscore) {
                double *F = a.out.fscore + orow * (size_t)W * G;
                for (int g = 0; g < G; ++g) {
                    load_margins(g);
                    for (int i = lane; i < W; i += 32)
                        F[(size_t)i * G + g] = (i < n_w) ? sc.value(sc.key(a, q_key[i] >> WL)) : 0.0;
                }
            }

            int S_tot = 0;
#pragma unroll
            for (int w = 0; w < GW; ++w) S_tot += cap[w] > 0 ? cap[w] : 0;
            S_tot = (int)__reduce_add_sync(kFull, (unsigned)S_tot);
            int n_left = n_w;
            int admitted = 0, s1_iters = 0, s2_pops = 0, status = 0;
            const int n_tiles = (n_w + 31) >> 5;

            // Stage-2 window state: each lane's five largest waiting keys, sorted, built by the first
            // pop of the step and kept up to date as requests are admitted
            int wt0 = 0, wt1 = 0, wt2 = 0, wt3 = 0, wt4 = 0;
            bool w_built = false, w_trunc = false;
            constexpr bool w_keep = FP;
            int gw[kRegWin] = {0, 0, 0, 0, 0};
            bool gw_valid = false;

            // argmax_i F_g({i}) over all waiting requests, earliest arrival on ties.
            // Returns the packed key of the winner (0 if none).
            auto best_single = [&]() -> int {
                if (!FP) {
                    int bk = kEmpty; int bkey = 0;
#pragma unroll 4
                    for (int t = 0; t < n_tiles; ++t) {
                        const int idx = (t << 5) + lane;
                        const int qk = idx < n_w ? q_key[idx] : 0;
                        if (qk > 0) {
                            const int f = (int)sc.key(a, qk >> WL);
                            // within a lane positions ascend, so strict > keeps the earliest
                            if (f > bk) { bk = f; bkey = qk; }
                        }
                    }
                    int wk;
                    const int src = warp_argmax_lane32(bk, (unsigned)bkey & posmask, wk);
                    const int res = __shfl_sync(kFull, bkey, src);
                    return res > 0 ? res : 0;
                } else if (!SL && a.peak_ok) {
                    // Eq. 2 is concave and piecewise linear in s with kinks at the m_{g,h}: it rises up
                    // to s* = the smallest kink at which the slope alpha D - beta sum_{m_h <= kink} d_h
                    // is no longer positive, and falls after it.  br_create has checked that no such
                    // slope is within rounding distance of zero, so the fp64 scores of integer lengths
                    // are strictly ordered on either side, and the arg-max is the largest s <= s* or the
                    // smallest s > s* (earliest arrival among equal lengths): two integer scans and two
                    // evaluations of Eq. 2.
                    double mine = 0.0;
#pragma unroll
                    for (int h = 0; h <= HR; ++h) if (lane == h) mine = sc.md[h];
                    double wsum = 0.0;
#pragma unroll
                    for (int h = 0; h <= HR; ++h) if (h <= H && sc.md[h] <= mine) wsum = __dadd_rn(wsum, a.d[h]);
                    const bool past = lane <= H && !(a.aD > __dmul_rn(a.beta, wsum));
                    const int sstar = (int)__reduce_min_sync(kFull, past ? (unsigned)(int)mine : 0x7FFFFFFFu);
                    const int thr = sstar >= (1 << (31 - WL)) ? 0x7FFFFFFF : ((sstar << WL) | (int)posmask);
                    int below = 0; unsigned above = 0x7FFFFFFFu;
#pragma unroll 4
                    for (int t = 0; t < n_tiles; ++t) {
                        const int idx = (t << 5) + lane;
                        const int qk = idx < n_w ? q_key[idx] : 0;
                        if (qk > 0) {
                            if (qk <= thr) below = max(below, qk);
                            else above = min(above, (unsigned)qk ^ posmask);
                        }
                    }
                    const int ka = __reduce_max_sync(kFull, below);
                    const unsigned ab = __reduce_min_sync(kFull, above);
                    const int kb = ab == 0x7FFFFFFFu ? 0 : (int)(ab ^ posmask);
                    const long long fa = ka > 0 ? sc.key(a, ka >> WL) : kNoKey;
                    const long long fb = kb > 0 ? sc.key(a, kb >> WL) : kNoKey;
                    if (fa > fb) return ka;
                    if (fb > fa) return kb;
                    if (ka <= 0) return 0;
                    return ((unsigned)ka & posmask) > ((unsigned)kb & posmask) ? ka : kb;
                } else {
                    // Horizon-safe requests (s <= min_h m_{g,h}) score alpha D s exactly, which grows
                    // with s: of those only the largest key per lane is scored; the others in full.
                    long long bk = kNoKey; int bkey = 0, best_safe = 0;
#pragma unroll 2
                    for (int t = 0; t < n_tiles; ++t) {
                        const int idx = (t << 5) + lane;
                        const int qk = idx < n_w ? q_key[idx] : 0;
                        if (qk > 0) {
                            if ((qk >> WL) <= sc.mmin) {
                                best_safe = max(best_safe, qk);
                            } else {
                                const long long f = sc.key(a, qk >> WL);
                                if (f > bk) { bk = f; bkey = qk; }
                            }
                        }
                    }
                    if (best_safe > 0) {
                        const long long f = sc.key(a, best_safe >> WL);
                        if (f > bk || (f == bk && ((unsigned)best_safe & posmask) > ((unsigned)bkey & posmask))) {
                            bk = f; bkey = best_safe;
                        }
                    }
                    long long wk;
                    const int src = warp_argmax_lane(bk, (unsigned)bkey & posmask, wk);
                    const int res = __shfl_sync(kFull, bkey, src);
                    return wk == kNoKey ? 0 : res;
                }
            };

            // sticky admission of the request with packed key qk to worker g
            auto commit = [&](int qk, int g) {
                const int s = qk >> WL;
                const int pos = (int)(posmask - ((unsigned)qk & posmask));
                const int src = g & 31, set = g >> 5;
                if (lane == src) {
                    int slot = -1;
                    for (int w = 0; w < OW && slot < 0; ++w) {
                        const unsigned long long fr = ~occ[g * OW + w];
                        if (fr) slot = w * 64 + __ffsll((long long)fr) - 1;
                    }
                    if (slot >= 0 && slot < B) {
                        occ[g * OW + (slot >> 6)] |= 1ull << (slot & 63);
                        const int sa = g * B + slot;
                        g_base[sa] = s - k;
                        if (H > 0 && g_chat0) {
                            g_chat0[sa] = (float)(H + a.delta_T - 1);
                            g_kref[sa] = (uint8_t)((k + 1 - a.delta_T) & 255);
                        }
                        if (life) g_end[sa] = k + q_o[pos] - 1;          // runs at steps k .. k + o_i - 1
                        if (g_aid) g_aid[sa] = q_id[pos];
                        q_key[pos] = (int)(0x80000000u | (unsigned)sa);
                    } else {
                        status |= BR_ST_BAD_STATE;
                        q_key[pos] = -1;                  // gone, no slot
                    }
#pragma unroll
                    for (int w = 0; w < GW; ++w) {
                        if (set == w) {
                            cap[w] -= 1;
#pragma unroll
                            for (int h = 0; h <= HR; ++h) if (h <= H) L[w][h] += s;
                        }
                    }
                }
                // envelope: only worker g grew, so M_h = max(M_h, L_g(k+h))
                if (SL) {
                    for (int h = lane; h <= H; h += 32) {
                        const int v = L_s[g * H1 + h] + s;
                        L_s[g * H1 + h] = v;
                        M_s[h] = max(M_s[h], v);
                    }
                    __syncwarp();
                    Mh[0] = M_s[0];
                }
#pragma unroll
                for (int h = 0; h <= HR; ++h) {
                    if (!SL && h <= H) {
                        int mine = L[0][h];
#pragma unroll
                        for (int w = 1; w < GW; ++w) if (set == w) mine = L[w][h];
                        Mh[h] = max(Mh[h], __shfl_sync(kFull, mine, src));
                    }
                }
                if (!w_keep && qk >= gw[kRegWin - 1]) gw_valid = false;   // one of the cached largest keys leaves
                if (w_keep && w_built && lane == (pos & 31)) {
                    if (wt0 == qk) { wt0 = wt1; wt1 = wt2; wt2 = wt3; wt3 = wt4; wt4 = 0; }
                    else if (wt1 == qk) { wt1 = wt2; wt2 = wt3; wt3 = wt4; wt4 = 0; }
                    else if (wt2 == qk) { wt2 = wt3; wt3 = wt4; wt4 = 0; }
                    else if (wt3 == qk) { wt3 = wt4; wt4 = 0; }
                    else if (wt4 == qk) { wt4 = 0; }
                }
                __syncwarp();
                S_tot -= 1; n_left -= 1; admitted += 1;
            };

            if (S_tot > 0 && n_w > 0) {
                // ---------- Stage 1: greedy fill ----------
#pragma unroll 1
                while (S_tot > a.S_greedy && n_left > 0) {
                    if (s1_iters >= W) { status |= BR_ST_ITER_CAP; break; }
                    ++s1_iters;
                    // most free slots; ties: smallest L_g(k), then lowest g
                    int bc = cap[0], bl = L[0][0], bg = lane;
#pragma unroll
                    for (int w = 1; w < GW; ++w)
                        if (cap[w] > bc || (cap[w] == bc && L[w][0] < bl)) { bc = cap[w]; bl = L[w][0]; bg = lane + 32 * w; }
                    const int mc = __reduce_max_sync(kFull, bc);
                    const unsigned ml = __reduce_min_sync(kFull, bc == mc ? (unsigned)bl : 0xFFFFFFFFu);
                    const unsigned mg = __reduce_min_sync(kFull, (bc == mc && (unsigned)bl == ml) ? (unsigned)bg : 0xFFFFFFFFu);
                    const int g = (int)mg;
                    load_margins(g);
                    const int qk = best_single();
                    if (qk <= 0) break;
                    commit(qk, g);
                }
            }
            if (timing) t_phase[3] = (unsigned)clock64();
            if (S_tot > 0 && n_left > 0) {
                // ---------- Stage 2: refined allocation ----------
#pragma unroll 1
                while (n_left > 0 && S_tot > 0) {
                    if (s2_pops >= W + G) { status |= BR_ST_ITER_CAP; break; }
                    ++s2_pops;
                    // (largest cap, largest horizon-min margin, lowest g) among cap > 0
                    int bc = -1, bm = -1, bg = 0x7FFFFFFF;
#pragma unroll
                    for (int w = 0; w < GW; ++w) {
                        int mm = Mh[0] - L[w][0];
                        if (SL) {
                            const int g = lane + 32 * w;
                            if (g < G)
                                for (int h = 1; h <= H; ++h) mm = min(mm, M_s[h] - L_s[g * H1 + h]);
                        }
#pragma unroll
                        for (int h = 1; h <= HR; ++h) if (h <= H) mm = min(mm, Mh[h] - L[w][h]);
                        if (cap[w] > 0 && (cap[w] > bc || (cap[w] == bc && mm > bm))) { bc = cap[w]; bm = mm; bg = lane + 32 * w; }
                    }
                    const int mc = __reduce_max_sync(kFull, bc);
                    if (mc <= 0) break;
                    const int mm2 = __reduce_max_sync(kFull, bc == mc ? bm : -1);
                    const unsigned mg = __reduce_min_sync(kFull, (bc == mc && bm == mm2) ? (unsigned)bg : 0xFFFFFFFFu);
                    const int g = (int)mg;
                    load_margins(g);

                    if (!LEAN && a.big_window) {
                        // ---- windows of 6 to 16 requests (Appendix "Bit-set subset selection") ----
                        // the R_max largest keys, one warp maximum per entry (keys are distinct)
                        const int R = min(a.R_max, n_left);
                        int thr = 0x7FFFFFFF;
                        for (int r = 0; r < R; ++r) {
                            int best = 0;
#pragma unroll 4
                            for (int t = 0; t < n_tiles; ++t) {
                                const int idx = (t << 5) + lane;
                                const int x = idx < n_w ? q_key[idx] : 0;
                                if (x < thr) best = max(best, x);
                            }
                            thr = __reduce_max_sync(kFull, best);
                            if (lane == 0) bw_win[r] = thr;
                        }
                        __syncwarp();
                        // prompt lengths of the window in shared memory (reusing the key slots' upper half is
                        // not needed: lengths are recomputed from the keys)
                        const int lim = min(mc, R);
                        const int ra = min(kBigWinLow, (R + 1) / 2), rb = R - ra;
                        // sorted subsets of the low entries (as prompt lengths)
                        {
                            const int n = 1 << ra;
                            for (int m = lane; m < n; m += 32) {
                                int sum = 0;
                                for (int j = 0; j < ra; ++j) if ((m >> j) & 1) sum += bw_win[j] >> WL;
                                bw_keys[m] = ((unsigned long long)__popc(m) << 56) | ((unsigned long long)(unsigned)sum << 16) | (unsigned)m;
                            }
                            __syncwarp();
                            for (int k2 = 2; k2 <= n; k2 <<= 1) {
                                for (int j = k2 >> 1; j > 0; j >>= 1) {
                                    for (int i = lane; i < n; i += 32) {
                                        const int p = i ^ j;
                                        if (p > i) {
                                            const unsigned long long x = bw_keys[i], y = bw_keys[p];
                                            const bool up = (i & k2) == 0;
                                            if ((x > y) == up) { bw_keys[i] = y; bw_keys[p] = x; }
                                        }
                                    }
                                    __syncwarp();
                                }
                            }
                            if (lane == 0) {
                                int off = 0, binom = 1;
                                for (int c = 0; c <= ra; ++c) { bw_off[c] = off; off += binom; binom = binom * (ra - c) / (c + 1); }
                                bw_off[ra + 1] = off;
                            }
                            __syncwarp();
                        }
                        // the peak of the score in Delta
                        int peak;
                        if (!FP) {
                            peak = sc.mi;
                        } else {
                            double mine = 0.0;
#pragma unroll
                            for (int h = 0; h <= HR; ++h) if (lane == h) mine = sc.md[h];
                            double wsum = 0.0;
#pragma unroll
                            for (int h = 0; h <= HR; ++h) if (h <= H && sc.md[h] <= mine) wsum = __dadd_rn(wsum, a.d[h]);
                            const bool past = lane <= H && !(a.aD > __dmul_rn(a.beta, wsum));
                            peak = (int)__reduce_min_sync(kFull, past ? (unsigned)(int)mine : 0x7FFFFFFFu);
                        }
                        MitmBest b; b.lo_sum = -1; b.lo_mask = 0xFFFFFFFFu; b.hi_sum = 0x7FFFFFFF; b.hi_mask = 0xFFFFFFFFu;
                        for (unsigned mh = lane; mh < (1u << rb); mh += 32) {
                            const int ph = __popc(mh);
                            if (ph > lim) continue;
                            int sh = 0;
                            for (unsigned t = mh; t; t &= t - 1) sh += bw_win[ra + __ffs(t) - 1] >> WL;
                            mitm_probe(bw_keys, bw_off, ra, lim, peak, mh, sh, ph, b);
                        }
                        // warp reduction: largest sum at or below the peak, smallest above it, lowest mask among equals
                        {
                            const int ls = __reduce_max_sync(kFull, b.lo_sum);
                            const unsigned lm = __reduce_min_sync(kFull, b.lo_sum == ls ? b.lo_mask : 0xFFFFFFFFu);
                            const int hs = __reduce_min_sync(kFull, b.hi_sum);
                            const unsigned hm = __reduce_min_sync(kFull, b.hi_sum == hs ? b.hi_mask : 0xFFFFFFFFu);
                            b.lo_sum = ls; b.lo_mask = lm; b.hi_sum = hs; b.hi_mask = hm;
                        }
                        long long bk = kNoKey; unsigned bmask = 0u;
                        if (b.lo_sum >= 0) { bk = sc.key(a, b.lo_sum); bmask = b.lo_mask; }
                        if (b.hi_sum != 0x7FFFFFFF) {
                            const long long k2 = sc.key(a, b.hi_sum);
                            if (k2 > bk || (k2 == bk && b.hi_mask < bmask)) { bk = k2; bmask = b.hi_mask; }
                        }
                        if (bk == kNoKey) { status |= BR_ST_ITER_CAP; break; }
                        if (bk <= 0) {
                            const int qk = best_single();                   // starvation guard
                            if (qk <= 0) break;
                            commit(qk, g);
                        } else {
                            for (int r = 0; r < R; ++r)
                                if ((bmask >> r) & 1u) commit(bw_win[r], g);
                        }
                        continue;
                    }

                    // window: the R_max largest waiting requests, earliest first on ties
                    int win[kRegWin];
                    int nwin = 0;
                    if (!w_keep) {
                        // Eq. 1 kernels cache the five largest keys of the queue; the cache stays valid
                        // until one of them is admitted (the guard mostly admits small requests)
                        if (!gw_valid) {
                            int t0 = 0, t1 = 0, t2 = 0, t3 = 0, t4 = 0;
#pragma unroll 4
                            for (int t = 0; t < n_tiles; ++t) {
                                const int idx = (t << 5) + lane;
                                int x = idx < n_w ? q_key[idx] : 0;
                                int y;
                                y = max(t0, x); x = min(t0, x); t0 = y;
                                y = max(t1, x); x = min(t1, x); t1 = y;
                                y = max(t2, x); x = min(t2, x); t2 = y;
                                y = max(t3, x); x = min(t3, x); t3 = y;
                                t4 = max(t4, x);
                            }
#pragma unroll
                            for (int r = 0; r < kRegWin; ++r) {
                                const int m = __reduce_max_sync(kFull, t0);
                                gw[r] = m;
                                if (t0 == m) { t0 = t1; t1 = t2; t2 = t3; t3 = t4; t4 = 0; }
                            }
                            gw_valid = true;
                        }
#pragma unroll
                        for (int r = 0; r < kRegWin; ++r) {
                            win[r] = (r < a.R_max && r < n_left) ? gw[r] : 0;
                            if (win[r] > 0) nwin = r + 1;
                        }
                    } else {
                        // Eq. 2 kernels keep every lane's sorted candidates across pops and merge the
                        // heads.  A list that runs dry although its lane holds more keys (possible only
                        // after several admissions from one lane) forces a rebuild.
#pragma unroll 1
                        for (int attempt = 0; attempt < 2; ++attempt) {
                            if (!w_built) {
                                int t0 = 0, t1 = 0, t2 = 0, t3 = 0, t4 = 0, cnt = 0;
#pragma unroll 4
                                for (int t = 0; t < n_tiles; ++t) {
                                    const int idx = (t << 5) + lane;
                                    int x = idx < n_w ? q_key[idx] : 0;
                                    cnt += x > 0;
                                    int y;
                                    y = max(t0, x); x = min(t0, x); t0 = y;
                                    y = max(t1, x); x = min(t1, x); t1 = y;
                                    y = max(t2, x); x = min(t2, x); t2 = y;
                                    y = max(t3, x); x = min(t3, x); t3 = y;
                                    t4 = max(t4, x);
                                }
                                wt0 = t0; wt1 = t1; wt2 = t2; wt3 = t3; wt4 = t4;
                                w_trunc = cnt > 5;
                                w_built = true;
                            }
                            int h0 = wt0, h1 = wt1, h2 = wt2, h3 = wt3, h4 = wt4;
                            bool dry = false;
                            nwin = 0;
#pragma unroll
                            for (int r = 0; r < kRegWin; ++r) {
                                win[r] = 0;
                                if (r < a.R_max && r < n_left) {
                                    dry = dry || (h0 == 0 && w_trunc);
                                    const int m = __reduce_max_sync(kFull, h0);
                                    win[r] = m;
                                    if (m > 0) nwin = r + 1;
                                    if (h0 == m) { h0 = h1; h1 = h2; h2 = h3; h3 = h4; h4 = 0; }
                                }
                            }
                            if (!__any_sync(kFull, dry)) break;
                            w_built = false;
                        }
                    }
                    // subsets of the window: lane = mask, lowest mask on ties
                    const int lim = min(mc, a.R_max);
                    long long fk = kNoKey;
                    if (lane >= 1 && lane < (1 << nwin) && __popc(lane) <= lim) {
                        int delta = 0;
#pragma unroll
                        for (int r = 0; r < kRegWin; ++r)
                            if ((lane >> r) & 1) delta += win[r] >> WL;
                        fk = sc.key(a, delta);
                    }
                    long long wk;
                    int best_mask;
                    if (!FP) {                          // Eq. 1 scores fit 32 bits
                        int wk32;
                        best_mask = warp_argmax_lane32(fk == kNoKey ? kEmpty : (int)fk, 31u - (unsigned)lane, wk32);
                        wk = wk32 == kEmpty ? kNoKey : (long long)wk32;
                    } else {
                        best_mask = warp_argmax_lane(fk, 31u - (unsigned)lane, wk);
                    }
                    if (wk == kNoKey) { status |= BR_ST_ITER_CAP; break; }
                    if (wk <= 0) {
                        // starvation guard: least-bad single request of all of R_wait
                        const int qk = best_single();
                        if (qk <= 0) break;
                        commit(qk, g);
                    } else {
#pragma unroll
                        for (int r = 0; r < kRegWin; ++r)
                            if ((best_mask >> r) & 1) commit(win[r], g);
                    }
                }
            }
            if (timing) t_phase[4] = (unsigned)clock64();

            // ================= RECORD =================
            {
                int mx = L[0][0], mn = cap[0] >= 0 ? L[0][0] : 0x7FFFFFFF;
                long long sum = cap[0] >= 0 ? (long long)L[0][0] : 0;
                const auto o_load = mk_span(reinterpret_cast<long long *>(a.out.load) + orow * G, G);
                if (cap[0] >= 0) o_load[lane] = L[0][0];
#pragma unroll
                for (int w = 1; w < GW; ++w) {
                    if (cap[w] >= 0) {
                        mx = max(mx, L[w][0]); mn = min(mn, L[w][0]); sum += L[w][0];
                        o_load[lane + 32 * w] = L[w][0];
                    }
                }
                mx = __reduce_max_sync(kFull, mx);
                mn = __reduce_min_sync(kFull, mn);
                for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(kFull, sum, o);
                status = (int)__reduce_or_sync(kFull, (unsigned)status);
                if (lane == 0) {
                    const auto tr = mk_span(reinterpret_cast<long long *>(a.out.trace) + orow * 3, 3);
                    tr[0] = mx; tr[1] = mn; tr[2] = sum;
                    scal[0] = n_left; scal[1] = admitted; scal[2] = s1_iters; scal[3] = s2_pops;
                    scal[4] = status | (n_drop ? BR_ST_QUEUE_OVERFLOW : 0);
                }
            }
        } else if (term_mode == 1) {
            // warps 1.. draw this step's termination words while warp 0 routes
            draw_fin(tid - 32, NT - 32);
        }
        inst_sync();                                              // B2: admissions visible

        // ============ queue compaction and assignments (warp 0) ============
        // A lane owns four consecutive positions of every group of 128 (16-byte accesses to the keys,
        // the ids and the assignment row); an entry's new position is the count of kept entries before it.
        if (warp == 0) {
            const auto assign = mk_span(a.assign_out + orow * W, W);
            int run = 0;
            const int n_before = n_w;          // queue length after ARRIVE
            const unsigned lt = (1u << lane) - 1u;
#pragma unroll 1
            for (int i0 = 0; i0 < W; i0 += 128) {
                const int p0 = i0 + lane * 4;
                if (i0 >= n_before) {
                    // the rest of the row is beyond the queue: only assignments remain
                    if (p0 < W) *vec_at<int4>(assign, p0) = make_int4(-1, -1, -1, -1);
                    continue;
                }
                int4 kk = make_int4(0, 0, 0, 0); uint4 ii = make_uint4(0u, 0u, 0u, 0u); int4 oo = make_int4(0, 0, 0, 0);
                if (p0 < W) {
                    kk = *vec_at<const int4>(q_key, p0);
                    ii = *vec_at<const uint4>(q_id, p0);
                    if (life) oo = *vec_at<const int4>(q_o, p0);
                }
                int ke[4] = {kk.x, kk.y, kk.z, kk.w};
                const unsigned idv[4] = {ii.x, ii.y, ii.z, ii.w};
                const int ov[4] = {oo.x, oo.y, oo.z, oo.w};
                int as[4];
                int below = run, total = 0;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (p0 + j >= n_before) ke[j] = 0;                  // beyond the queue
                    const unsigned bal = __ballot_sync(kFull, ke[j] > 0);
                    below += __popc(bal & lt);
                    total += __popc(bal);
                    const int sa = ke[j] & 0x7FFFFFFF;
                    const bool gone = ke[j] < 0 && sa < A;
                    as[j] = gone ? sa : -1;
                    if (have_pre && gone) {
                        // a request admitted at this step may also end at it
                        const int g = (int)__umulhi((unsigned)sa, a.magic_B), slot = sa - g * B;
                        if ((fin_w[g * OW + (slot >> 6)] >> (slot & 63)) & 1ull) {
                            atomicOr(&end_mask[g * OW + (slot >> 6)], 1ull << (slot & 63));
                            const int at = atomicAdd(&scal[6], 1);
                            if (at < kEndList) {
                                end_list[at] = (unsigned short)sa;
                            } else {
                                atomicAdd(&sub_load[g], (unsigned)(g_base[sa] + k));
                                g_base[sa] = kEmpty;
                            }
                        }
                    }
                }
                if (p0 < W) *vec_at<int4>(assign, p0) = make_int4(as[0], as[1], as[2], as[3]);
                __syncwarp();                                           // the group is read before any of it is overwritten
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (ke[j] > 0) {
                        const int i = p0 + j, dst = below;
                        const int sv = ke[j] >> WL;
                        if (dst != i) { q_key[dst] = (sv << WL) | (int)(posmask - (unsigned)dst); q_id[dst] = idv[j]; }
                        if (dst != i || i >= n_w_old) { g_qs[dst] = sv; g_qid[dst] = idv[j]; }
                        if (life) {
                            if (dst != i) q_o[dst] = ov[j];
                            if (dst != i || i >= n_w_old) g_qo[dst] = ov[j];
                        }
                        ++below;
                    }
                }
                __syncwarp();
                run += total;
            }
        }
        n_w = scal[0];
        if (timing) t_phase[5] = (unsigned)clock64();

        // ================= ADVANCE =================
        // Only the occupancy masks, the termination draws and the few ending slots are touched.
        if (!have_pre) {
            if (term_mode == 2) {
                // Bernoulli(term_probs[slot][0]) per running request: 24-bit uniform below the probability
                const float sc24 = 5.9604644775390625e-8f;
#pragma unroll 1
                for (int q8 = tid; q8 < A8; q8 += NT) {
                    const int a0 = q8 << 3;
                    const int g = a0 / B, slot0 = a0 - g * B;
                    const unsigned ob = (unsigned)(occ[g * OW + (slot0 >> 6)] >> (slot0 & 63)) & 0xFFu;
                    unsigned fb = 0;
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        if (!((ob >> (4 * half)) & 0xFu)) continue;
                        const uint4 r = philox4x32_10((uint32_t)k, (uint32_t)(q8 * 2 + half), kStreamTerm, 0u, key0, key1);
                        const uint32_t rr[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int jj = 4 * half + j;
                            if ((ob >> jj) & 1u) {
                                const float q = probs[(size_t)(a0 + jj) * H];
                                if (__fmul_rn((float)(rr[j] >> 8), sc24) < q) fb |= 1u << jj;
                            }
                        }
                    }
                    *vec_at<unsigned char>(mk_span(reinterpret_cast<unsigned char *>(raw_of(fin_w)), (long long)G * OW * 8), (long long)g * OW * 8 + (slot0 >> 3)) = (unsigned char)fb;
                }
                inst_sync();
            } else if (term_mode == 3) {
                // a request ends with its o_i-th step: act_end == k
#pragma unroll 1
                for (int q8 = tid; q8 < A8; q8 += NT) {
                    const int a0 = q8 << 3;
                    const int g = a0 / B, slot0 = a0 - g * B;
                    const unsigned ob = (unsigned)(occ[g * OW + (slot0 >> 6)] >> (slot0 & 63)) & 0xFFu;
                    unsigned fb = 0;
                    if (ob) {
                        const int4 e0 = *vec_at<const int4>(g_end, a0);
                        const int4 e1 = *vec_at<const int4>(g_end, a0 + 4);
                        const int en[8] = {e0.x, e0.y, e0.z, e0.w, e1.x, e1.y, e1.z, e1.w};
#pragma unroll
                        for (int j = 0; j < 8; ++j) if (((ob >> j) & 1u) && en[j] == k) fb |= 1u << j;
                    }
                    *vec_at<unsigned char>(mk_span(reinterpret_cast<unsigned char *>(raw_of(fin_w)), (long long)G * OW * 8), (long long)g * OW * 8 + (slot0 >> 3)) = (unsigned char)fb;
                }
                inst_sync();
            }
            scan_workers(false);
        }
        inst_sync();
        {
            // the requests that ended: subtract their load from the worker, free the slot
            if (tid < n_pre) {
                const int sa = pre_list[tid];
                g_base[sa] = kEmpty;
                atomicAdd(&sub_load[sa / B], (unsigned)(pend + k));
            }
            const int n_end = min(scal[6], kEndList);
            for (int e = tid; e < n_end; e += NT) {
                const int sa = end_list[e];
                const int cur = g_base[sa] + k;
                g_base[sa] = kEmpty;
                atomicAdd(&sub_load[sa / B], (unsigned)cur);
            }
            if (have_pre && scal[9]) {
                // more requests ended than the lists hold: the rest were subtracted when they were
                // found, their slots are emptied here (the instance is one warp; the listed slots
                // have been read by now)
                __syncwarp();
#pragma unroll 1
                for (int idx = tid; idx < G * OW; idx += NT) {
                    const int g = idx / OW, x = idx - g * OW;
                    unsigned long long ended = end_mask[idx];
                    while (ended) {
                        const int j = __ffsll((long long)ended) - 1;
                        ended &= ended - 1;
                        g_base[g * B + 64 * x + j] = kEmpty;
                    }
                }
            }
        }
        inst_sync();                                              // B3

        if (warp == 0) {
            // L_g(k+1) = L_g(k) - (loads of the requests that ended) + (number of survivors)
#pragma unroll
            for (int w = 0; w < GW; ++w) {
                const int g = lane + 32 * w;
                if (g < G) {
                    int na = 0;
                    for (int x = 0; x < OW; ++x) {
                        const unsigned long long o = occ[g * OW + x] & ~end_mask[g * OW + x];
                        occ[g * OW + x] = o;
                        na += __popcll(o);
                    }
                    cap[w] = B - na;
                    L[w][0] = L[w][0] - (int)sub_load[g] + na;
                    sub_load[g] = 0u;
                }
            }
            if (lane == 0) {
                if (a.out.counters) {
                    uint32_t *c = a.out.counters + orow * 4;
                    c[0] = (uint32_t)n_drop; c[1] = (uint32_t)scal[1]; c[2] = (uint32_t)scal[2]; c[3] = (uint32_t)scal[3];
                }
                if (a.out.status) a.out.status[orow] = scal[4] | scal[5];
                scal[6] = 0; scal[7] = 0; scal[8] = 0; scal[9] = 0;
                if (timing) {
                    t_phase[6] = (unsigned)clock64();
                    uint32_t *pc = a.out.phase_cycles + orow * 8;
#pragma unroll
                    for (int p = 0; p < 6; ++p) pc[p] = (uint32_t)(t_phase[p + 1] - t_phase[p]);
                    pc[6] = it == 0 ? (uint32_t)(t_phase[0] - t_entry) : 0u;
                    pc[7] = 0u;
                }
            }
        }
        if (it + 1 < a.n_steps) {
            for (int i = tid; i < 2 * G * H1; i += NT) Lh_s[i] = 0u;
            inst_sync();
        }
    }

    // ---- write the snapshot back ----
    if (warp == 0) {
#pragma unroll
        for (int w = 0; w < GW; ++w) {
            const int g = lane + 32 * w;
            if (g < G) {
                g_load[g] = (long long)L[w][0];
                g_nact[g] = B - cap[w];
                for (int x = 0; x < OW; ++x) g_occ[g * OW + x] = occ[g * OW + x];   // updated by this lane
            }
        }
    }
    if (tid == 0) {
        a.ws.step[inst] = k;
        a.ws.next_id[inst] = next_id;
        a.wq.n[inst] = n_w;
        if (a.out.phase_cycles)      // time from kernel entry to here, for the last step's row
            a.out.phase_cycles[((size_t)(a.n_steps - 1) * a.N + inst) * 8 + 7] = (uint32_t)((unsigned)clock64() - t_entry);
    }
}

}  // namespace br
