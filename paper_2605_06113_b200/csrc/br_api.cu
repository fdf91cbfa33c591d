// C-ABI entry points of the BalanceRoute routing library (declared in include/br.h).
// Host side only validates, fills the kernel argument block and launches.
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <atomic>
#include <new>

#include "br_step.cuh"
#include "br_small.cuh"
#include "br_fscore.cuh"
#include "br_subset.cuh"
#include "br_bypass.cuh"
#include "br_survival.cuh"

using br::StepArgs;

struct br_ctx {
    int32_t G, H;
    br_params p;              // resolved parameters
    StepArgs base;            // constant part of the kernel arguments
    int threads;              // threads per instance for large batches
    int threads_small;        // ... for batches of a few instances (latency path)
    int inst_per_block;       // single-warp instances per thread block
    bool small_ok;            // the fleet shape fits br_small_kernel
    bool two_probe_ok;        // both sides of the score's peak are strictly monotone up to Delta = 32 s_max
    size_t smem;
    // latency path
    cudaGraph_t graph;
    cudaGraphExec_t graph_exec;
    cudaStream_t graph_stream;
    // host-buffer path
    void *stage;
    size_t stage_bytes;
    cudaStream_t pipe[3];     // copy-in, kernel and copy-out streams of the chunked host-buffer step
    cudaEvent_t pipe_ev[2 * 8 + 2];
    bool pipe_ready;
};

namespace {

thread_local char g_cuda_msg[256] = "no CUDA error recorded";

int cuda_fail(cudaError_t e, const char *what)
{
    snprintf(g_cuda_msg, sizeof(g_cuda_msg), "%s: %s", what, cudaGetErrorString(e));
    return BR_ECUDA;
}
#define BR_CUDA(call)                                      \
    do {                                                   \
        cudaError_t e__ = (call);                          \
        if (e__ != cudaSuccess) return cuda_fail(e__, #call); \
    } while (0)

// For calls made after work has been queued on `stream`: on failure the stream is drained first,
// so that no copy still reads or writes the caller's buffers (or the shared staging) when the error
// is reported.
#define BR_CUDA_DRAIN(call, stream)                        \
    do {                                                   \
        cudaError_t e__ = (call);                          \
        if (e__ != cudaSuccess) {                          \
            cudaStreamSynchronize(stream);                 \
            return cuda_fail(e__, #call);                  \
        }                                                  \
    } while (0)

inline bool misaligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; }

typedef void (*step_kernel_t)(const StepArgs);

// lean: 0 general, 1 constant hazard and no optional outputs, 2 the same on a single warp
template <int GW>
step_kernel_t pick_kernel_gw(bool fp, int H, int lean)
{
    if (!fp) return lean == 2 ? br::br_step_kernel<false, 0, GW, 2> : br::br_step_kernel<false, 0, GW, 0>;
    if (H == 0) return br::br_step_kernel<true, 0, GW, 0>;
    if (H <= 4) return lean ? br::br_step_kernel<true, 4, GW, 1> : br::br_step_kernel<true, 4, GW, 0>;
    if (H <= 8) return lean ? br::br_step_kernel<true, 8, GW, 1> : br::br_step_kernel<true, 8, GW, 0>;
    if (H <= 16) return lean ? br::br_step_kernel<true, 16, GW, 1> : br::br_step_kernel<true, 16, GW, 0>;
    // longer horizons (up to BR_MAX_H): projected loads and margins live in shared memory
    return lean ? br::br_step_kernel<true, BR_MAX_H, GW, 1> : br::br_step_kernel<true, BR_MAX_H, GW, 0>;
}

step_kernel_t pick_kernel(bool fp, int H, int G, int lean)
{
    return G <= 32 ? pick_kernel_gw<1>(fp, H, lean) : pick_kernel_gw<2>(fp, H, lean);
}

int check_step_args(const br_ctx *ctx, const br_instance_batch *b, const br_worker_state *ws,
                    const br_waiting_queue *wq, const float *term_probs, const int32_t *assign_out,
                    const br_load_out *out)
{
    if (!ctx || !b || !ws || !wq || !out) return BR_EINVAL;
    if (b->n_instances < 0 || b->first_instance < 0) return BR_EINVAL;
    const int n_steps = b->n_steps <= 0 ? 1 : b->n_steps;
    if (n_steps > 1 && b->first_instance != 0) return BR_EINVAL;
    if (!ws->load || !ws->nact || !ws->occ || !ws->act_base || !ws->step || !ws->seed || !ws->next_id)
        return BR_EINVAL;
    if (!wq->s || !wq->id || !wq->n) return BR_EINVAL;
    if (!assign_out || !out->load || !out->trace) return BR_EINVAL;
    const bool classifier = ctx->H > 0 && ctx->p.pred_mode == 0;
    if (classifier && (!ws->act_chat0 || !ws->act_kref || !term_probs)) return BR_EINVAL;
    if (ctx->p.term_mode == 2 && !term_probs) return BR_EINVAL;
    if (ctx->p.term_mode == 3 && (!ws->act_end || !wq->o || misaligned(ws->act_end, 16) || misaligned(wq->o, 16)))
        return BR_EINVAL;
    if (misaligned(ws->act_base, 16) || misaligned(wq->s, 16) || misaligned(wq->id, 16) ||
        misaligned(assign_out, 16) || misaligned(ws->load, 8) || misaligned(ws->occ, 8) ||
        misaligned(out->load, 8) || misaligned(out->trace, 8) || misaligned(ws->seed, 8) ||
        (term_probs && misaligned(term_probs, 16)) || (out->fscore && misaligned(out->fscore, 8)) ||
        (classifier && (misaligned(ws->act_chat0, 16) || misaligned(ws->act_kref, 4))))
        return BR_EINVAL;
    return BR_OK;
}

// Launch with programmatic stream serialisation: the blocks of this launch may become resident
// while the previous kernel of the stream is still draining.  Both step kernels open with
// griddepcontrol.wait, which returns only when every earlier kernel of the stream has completed
// and its writes are visible, so only launch latency and block scheduling overlap.
cudaError_t launch_overlapped(step_kernel_t kern, int blocks, int threads, size_t smem, cudaStream_t stream,
                              const StepArgs &a, bool overlap)
{
    if (!overlap) {                      // plain launch (stream capture)
        kern<<<blocks, threads, smem, stream>>>(a);
        return cudaGetLastError();
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)blocks); cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, a);
}

int launch_step(br_ctx *ctx, const br_instance_batch *b, const br_worker_state *ws,
                const br_waiting_queue *wq, const float *term_probs, int32_t *assign_out,
                const br_load_out *out, cudaStream_t stream, bool overlap = true)
{
    StepArgs a = ctx->base;
    a.N = b->n_instances;
    a.first_instance = b->first_instance;
    a.n_steps = b->n_steps <= 0 ? 1 : b->n_steps;
    a.ws = *ws;
    a.wq = *wq;
    a.term_probs = term_probs;
    a.assign_out = assign_out;
    a.out = *out;
    // few instances: the launch is latency-bound, so spread each instance over more warps
    const int tpi = b->n_instances <= 64 ? ctx->threads_small : ctx->threads;
    if (tpi == 32 && ctx->small_ok && !out->fscore && !out->phase_cycles) {
        // BR-0 on a small fleet: the one-warp-per-instance kernel
        int wpb = ctx->inst_per_block;
        if (wpb > b->n_instances) wpb = b->n_instances;
        const int nt4 = ctx->p.W <= 128 ? 1 : (ctx->p.W <= 256 ? 2 : 4);
        const bool r4 = ctx->p.R_max <= 4;
        step_kernel_t kern = nt4 == 1 ? (r4 ? br::br_small_kernel<1, 4> : br::br_small_kernel<1, 5>)
                           : nt4 == 2 ? (r4 ? br::br_small_kernel<2, 4> : br::br_small_kernel<2, 5>)
                                      : (r4 ? br::br_small_kernel<4, 4> : br::br_small_kernel<4, 5>);
        a.tpi = 32;
        const int blocks = (b->n_instances + wpb - 1) / wpb;
        cudaError_t e = launch_overlapped(kern, blocks, 32 * wpb, (size_t)wpb * nt4 * 128 * 2 * sizeof(int), stream, a, overlap);
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(e, "br_step launch");
        return BR_OK;
    }
    const int lean = (ctx->p.term_mode == 1 && !out->fscore && !out->phase_cycles && !ctx->base.big_window)
                         ? (tpi == 32 ? 2 : 1) : 0;
    step_kernel_t kern = pick_kernel(ctx->p.score_mode == 1, ctx->H, ctx->G, lean);
    // instances are packed several to a block: single-warp ones always, wider ones only in full
    // blocks (their barriers are block barriers)
    int per_block = ctx->inst_per_block;
    if (tpi > 32) { while (per_block > 1 && (per_block * tpi > 256 || b->n_instances % per_block != 0)) --per_block; }
    if (per_block > b->n_instances) per_block = b->n_instances;
    while (per_block > 1 && ctx->smem * per_block > 48 * 1024) --per_block;
    if (tpi > 32 && per_block > 1 && b->n_instances % per_block != 0) per_block = 1;
    a.tpi = tpi;
    a.block_sync = (per_block > 1 && b->n_instances % per_block == 0) ? 1 : 0;
    a.smem_per_inst = (int32_t)ctx->smem;
    const int blocks = (b->n_instances + per_block - 1) / per_block;
    if (ctx->smem * per_block > 48 * 1024) {
        // beyond the default limit: opt the kernel in (br_create has checked the device maximum)
        cudaError_t eo = cudaFuncSetAttribute((const void *)kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)(ctx->smem * per_block));
        if (eo != cudaSuccess) return cuda_fail(eo, "cudaFuncSetAttribute(shared memory)");
    }
    cudaError_t e = launch_overlapped(kern, blocks, tpi * per_block, ctx->smem * per_block, stream, a, overlap);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "br_step launch");
    return BR_OK;
}

}  // namespace

extern "C" {

int br_version(void) { return BR_VERSION; }

const char *br_strerror(int status)
{
    switch (status) {
    case BR_OK: return "ok";
    case BR_EINVAL: return "invalid argument (null or misaligned pointer, or size outside the compiled limits)";
    case BR_ERANGE: return "value range too large for the device integer packing";
    case BR_ECUDA: return g_cuda_msg;
    case BR_ENOMEM: return "allocation failed";
    case BR_ESTATE: return "call order violated";
    case BR_ELIMIT: return "batch needs more staging than the built-in no-allocation buffer holds (BR_STATIC_STAGE_BYTES)";
    default: return "unknown status";
    }
}

int br_create(int32_t G, int32_t H, const br_params *params, br_ctx **out)
{
    if (!params || !out) return BR_EINVAL;
    if (G < 1 || G > BR_MAX_G || H < 0 || H > BR_MAX_H) return BR_EINVAL;
    br_params p = *params;
    if (p.B < 8 || p.B > BR_MAX_B || (p.B % 8) != 0) return BR_EINVAL;
    if (p.W < 4 || p.W > BR_MAX_W || (p.W % 4) != 0) return BR_EINVAL;
    if (p.R_max <= 0) p.R_max = 4;
    if (p.R_max > BR_MAX_RMAX) return BR_EINVAL;
    if (p.S_greedy < 0) p.S_greedy = 2 * G;
    if (p.delta_T <= 0) p.delta_T = H / 2 > 1 ? H / 2 : 1;
    if (p.delta_T > 128) return BR_EINVAL;
    if (p.gate < 0.0f) p.gate = 0.5f;
    if (p.c_floor < 0.0f) p.c_floor = 1.0f;
    if (p.score_mode < 0) p.score_mode = (H == 0) ? 0 : 1;
    if (p.score_mode > 1 || (p.score_mode == 0 && H != 0)) return BR_EINVAL;
    if (p.term_mode < 0 || p.term_mode > 3 || (p.term_mode == 2 && H == 0)) return BR_EINVAL;
    if (p.term_mode == 1 && !p.term_cdf) return BR_EINVAL;
    if (p.pred_mode < 0) p.pred_mode = 0;
    if (p.pred_mode > 1 || (p.pred_mode == 1 && (H == 0 || p.term_mode != 3))) return BR_EINVAL;
    if (p.term_mode == 3 && p.arr_cdf && (!p.out_tab || p.out_tab_log2 < 0 || p.out_tab_log2 > 24)) return BR_EINVAL;
    if (p.arr_cdf) {
        if (p.arr_len < 1 || p.arr_period < 1 || p.arr_inst_stride < 0 || !p.len_tab) return BR_EINVAL;
        if (p.len_tab_log2 < 0 || p.len_tab_log2 > 24) return BR_EINVAL;
        if (p.burst_every < 0 || p.burst_size < 0) return BR_EINVAL;
    }
    int wl = 2;
    while ((1 << wl) < p.W) ++wl;
    if (p.s_max <= 0) p.s_max = (1 << (31 - wl)) - 1 < (1 << 20) ? (1 << (31 - wl)) - 1 : (1 << 20);
    // range proofs for the 32-bit device arithmetic:
    //   packed queue keys  s * 2^wl + position        < 2^31
    //   loads and partial sums  B * (s_max + 2^22)     < 2^31   (requests older than 2^22 steps are not supported)
    //   Eq. 1 scores  G * R_max * s_max                < 2^31
    if ((long long)p.s_max >= (1ll << (31 - wl))) return BR_ERANGE;
    if ((long long)p.B * ((long long)p.s_max + (1ll << 22)) >= (1ll << 31)) return BR_ERANGE;
    if ((long long)G * p.R_max * (long long)p.s_max >= (1ll << 31)) return BR_ERANGE;
    if (p.score_mode == 1) {
        if (!(p.alpha > 0.0) || !(p.gamma > 0.0) || !(p.gamma <= 1.0) || !(p.beta >= 0.0) ||
            !isfinite(p.alpha) || !isfinite(p.beta))
            return BR_EINVAL;
    }
    const int A = G * p.B;
    int threads_small, threads_large;
    if (p.threads > 0) {
        if (p.threads % 32 != 0 || p.threads > 256) return BR_EINVAL;
        threads_small = threads_large = p.threads;
    } else {
        const int work = A * (H > 0 ? 2 : 1);
        int w = (work + 4095) / 4096;
        threads_large = 32 * (w < 1 ? 1 : (w > 8 ? 8 : w));
        w = (work + 1023) / 1024;
        threads_small = 32 * (w < 1 ? 1 : (w > 8 ? 8 : w));
    }

    br_ctx *ctx = new (std::nothrow) br_ctx();
    if (!ctx) return BR_ENOMEM;
    memset(ctx, 0, sizeof(*ctx));
    ctx->G = G; ctx->H = H; ctx->p = p;
    ctx->threads = threads_large; ctx->threads_small = threads_small;
    ctx->inst_per_block = p.inst_per_block > 0 ? (p.inst_per_block > 8 ? 8 : p.inst_per_block) : 4;
    StepArgs &a = ctx->base;
    a.G = G; a.H = H; a.B = p.B; a.W = p.W; a.R_max = p.R_max; a.S_greedy = p.S_greedy;
    a.occ_words = (p.B + 63) / 64;
    a.wl = wl;
    a.magic_B = (uint32_t)(((1ull << 32) + (unsigned)p.B - 1) / (unsigned)p.B);
    a.delta_T = p.delta_T; a.gate = p.gate; a.c_floor = p.c_floor;
    a.term_mode = p.term_mode; a.term_cdf = p.term_cdf;
    a.pred_mode = p.pred_mode; a.out_tab = p.out_tab; a.out_shift = 32 - p.out_tab_log2;
    a.arr_cdf = p.arr_cdf; a.arr_len = p.arr_len; a.arr_period = p.arr_period;
    a.arr_inst_stride = p.arr_inst_stride;
    a.len_tab = p.len_tab; a.len_shift = 32 - p.len_tab_log2;
    a.burst_every = p.burst_every; a.burst_size = p.burst_size;
    // d = (1, gamma, ..., gamma^H) by repeated multiplication; D = 1^T d left to right
    volatile double D = 0.0;
    for (int h = 0; h <= BR_MAX_H; ++h) a.d[h] = 0.0;
    if (p.score_mode == 1) {
        for (int h = 0; h <= H; ++h) {
            volatile double dh = (h == 0) ? 1.0 : a.d[h - 1] * p.gamma;
            a.d[h] = dh;
            D = D + dh;
        }
        volatile double aD = p.alpha * D;
        a.aD = aD; a.beta = p.beta;
        // The single-request arg-max may use the concavity of Eq. 2 only if no segment slope
        // alpha D - beta sum_{h in P} d_h (P any set of passed kinks) is within rounding distance of
        // zero: then fp64 scores of integer lengths are strictly ordered on both sides of the peak.
        // The 2^(H+1) slopes are enumerated for H <= 16; longer horizons score every request.
        a.peak_ok = 0;
        if (H <= 16) {
            const int n = H + 1;
            double min_abs = 1e300;
            for (unsigned mask = 0; mask < (1u << n); ++mask) {
                double w = 0.0;
                for (int h = 0; h < n; ++h) if (mask >> h & 1u) w += a.d[h];
                const double sl = fabs(a.aD - p.beta * w);
                if (sl < min_abs) min_abs = sl;
            }
            const double err = 4.0 * (H + 5) * 1.1102230246251565e-16 * (a.aD + p.beta * D) * (double)p.s_max;
            a.peak_ok = (min_abs > err && min_abs > 1e-9) ? 1 : 0;
            // the same for subsets of up to 32 requests (Delta <= 32 s_max): the two-probe rule of the
            // large-window solvers
            ctx->two_probe_ok = min_abs > 32.0 * err && min_abs > 1e-9;
        }
    } else {
        a.d[0] = 1.0; a.aD = 1.0; a.beta = (double)G; a.peak_ok = 0;
        ctx->two_probe_ok = G >= 2;            // Eq. 1 falls with slope -(G - 1) beyond the margin
    }
    // Stage-2 windows beyond five requests are solved by meeting in the middle, which rests on the
    // two-probe rule
    a.big_window = p.R_max > br::kRegWin ? 1 : 0;
    if (a.big_window && !ctx->two_probe_ok) { delete ctx; return BR_EINVAL; }
    ctx->smem = br::step_smem_bytes(G, H, p.B, p.W, a.occ_words, p.term_mode == 3, a.big_window != 0);
    if (ctx->smem > 227 * 1024) { delete ctx; return BR_EINVAL; }      // one instance must fit a thread block's shared memory
    // br_small_kernel: Eq. 1, one worker per lane, one occupancy word, at most 512 waiting requests,
    // arrivals served by one Philox call, and negative queue keys scoring below every waiting request
    ctx->small_ok = p.score_mode == 0 && G <= 32 && p.B <= 64 && p.W <= 512 && p.term_mode <= 1 && p.R_max <= br::kRegWin &&
                    p.burst_every == 0 && (!p.arr_cdf || p.arr_len <= 64) &&
                    (long long)(G - 1) * p.s_max + 65536 < (1ll << (31 - wl));
    *out = ctx;
    return BR_OK;
}

int br_step(br_ctx *ctx, const br_instance_batch *batch, br_worker_state *ws, br_waiting_queue *wq,
            const float *term_probs, int32_t *assign_out, br_load_out *out)
{
    int rc = check_step_args(ctx, batch, ws, wq, term_probs, assign_out, out);
    if (rc != BR_OK) return rc;
    if (batch->n_instances == 0) return BR_OK;
    return launch_step(ctx, batch, ws, wq, term_probs, assign_out, out, (cudaStream_t)batch->stream);
}

int br_graph_capture(br_ctx *ctx, const br_instance_batch *batch, br_worker_state *ws,
                     br_waiting_queue *wq, const float *term_probs, int32_t *assign_out,
                     br_load_out *out)
{
    int rc = check_step_args(ctx, batch, ws, wq, term_probs, assign_out, out);
    if (rc != BR_OK) return rc;
    if (batch->n_instances == 0) return BR_EINVAL;
    if (ctx->graph_exec) { cudaGraphExecDestroy(ctx->graph_exec); ctx->graph_exec = nullptr; }
    if (ctx->graph) { cudaGraphDestroy(ctx->graph); ctx->graph = nullptr; }
    cudaStream_t cap;
    BR_CUDA(cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking));
    cudaError_t e = cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal);
    if (e != cudaSuccess) { cudaStreamDestroy(cap); return cuda_fail(e, "cudaStreamBeginCapture"); }
    rc = launch_step(ctx, batch, ws, wq, term_probs, assign_out, out, cap, false);
    e = cudaStreamEndCapture(cap, &ctx->graph);
    cudaStreamDestroy(cap);
    if (rc != BR_OK) return rc;
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamEndCapture");
    BR_CUDA(cudaGraphInstantiate(&ctx->graph_exec, ctx->graph, 0));
    ctx->graph_stream = (cudaStream_t)batch->stream;
    return BR_OK;
}

int br_graph_step(br_ctx *ctx)
{
    if (!ctx) return BR_EINVAL;
    if (!ctx->graph_exec) return BR_ESTATE;
    BR_CUDA(cudaGraphLaunch(ctx->graph_exec, ctx->graph_stream));
    return BR_OK;
}

namespace {

// One block of the staging area of the host-buffer entry points: a [N][row] array that goes up
// before the kernel (in), comes down after it (out), or both.
struct StageBlk { size_t bytes; void **dev; void *host; bool in, out; };
constexpr int kStageBlks = 23;

struct StagePlan {
    StageBlk blk[kStageBlks];
    br_worker_state dws; br_waiting_queue dwq; br_load_out dout;
    float *d_probs; int32_t *d_assign;
    size_t total;               // bytes, every block padded to 256
};

// Validates the host pointers of a host-buffer step and lists its blocks (device addresses are
// assigned by the caller once it knows where the staging area is).
int plan_host_step(const br_ctx *ctx, const br_instance_batch *batch, br_worker_state *hws, br_waiting_queue *hwq,
                   const float *h_probs, int32_t *h_assign, br_load_out *hout, StagePlan *pl)
{
    if (!ctx || !batch || !hws || !hwq || !hout) return BR_EINVAL;
    if (batch->n_instances < 0 || batch->first_instance != 0 || batch->n_steps > 1) return BR_EINVAL;
    if (!hws->load || !hws->nact || !hws->occ || !hws->act_base || !hws->step || !hws->seed ||
        !hws->next_id || !hwq->s || !hwq->id || !hwq->n || !h_assign || !hout->load || !hout->trace)
        return BR_EINVAL;
    const bool pred = ctx->H > 0 && ctx->p.pred_mode == 0;
    const bool life = ctx->p.term_mode == 3;
    if (pred && (!hws->act_chat0 || !hws->act_kref || !h_probs)) return BR_EINVAL;
    if (ctx->p.term_mode == 2 && !h_probs) return BR_EINVAL;
    if (life && (!hws->act_end || !hwq->o)) return BR_EINVAL;
    const size_t N = (size_t)batch->n_instances;
    const size_t G = ctx->G, H = ctx->H, B = ctx->p.B, W = ctx->p.W, A = G * B;
    const size_t OW = (B + 63) / 64;
    memset(&pl->dws, 0, sizeof(pl->dws)); memset(&pl->dwq, 0, sizeof(pl->dwq)); memset(&pl->dout, 0, sizeof(pl->dout));
    pl->d_probs = nullptr; pl->d_assign = nullptr;
    const StageBlk blks[kStageBlks] = {
        {N * G * 8, (void **)&pl->dws.load, hws->load, true, true},
        {N * G * 4, (void **)&pl->dws.nact, hws->nact, true, true},
        {N * G * OW * 8, (void **)&pl->dws.occ, hws->occ, true, true},
        {N * A * 4, (void **)&pl->dws.act_base, hws->act_base, true, true},
        {hws->act_id ? N * A * 4 : 0, (void **)&pl->dws.act_id, hws->act_id, true, true},
        {pred ? N * A * 4 : 0, (void **)&pl->dws.act_chat0, hws->act_chat0, true, true},
        {pred ? N * A : 0, (void **)&pl->dws.act_kref, hws->act_kref, true, true},
        {life ? N * A * 4 : 0, (void **)&pl->dws.act_end, hws->act_end, true, true},
        {N * 4, (void **)&pl->dws.step, hws->step, true, true},
        {N * 8, (void **)&pl->dws.seed, hws->seed, true, false},
        {N * 4, (void **)&pl->dws.next_id, hws->next_id, true, true},
        {N * W * 4, (void **)&pl->dwq.s, hwq->s, true, true},
        {N * W * 4, (void **)&pl->dwq.id, hwq->id, true, true},
        {life ? N * W * 4 : 0, (void **)&pl->dwq.o, hwq->o, true, true},
        {N * 4, (void **)&pl->dwq.n, hwq->n, true, true},
        {h_probs ? N * A * H * 4 : 0, (void **)&pl->d_probs, (void *)h_probs, true, false},
        {N * W * 4, (void **)&pl->d_assign, h_assign, false, true},
        {N * G * 8, (void **)&pl->dout.load, hout->load, false, true},
        {N * 3 * 8, (void **)&pl->dout.trace, hout->trace, false, true},
        {hout->status ? N * 4 : 0, (void **)&pl->dout.status, hout->status, false, true},
        {hout->counters ? N * 16 : 0, (void **)&pl->dout.counters, hout->counters, false, true},
        {hout->fscore ? N * W * G * 8 : 0, (void **)&pl->dout.fscore, hout->fscore, false, true},
        {hout->phase_cycles ? N * 32 : 0, (void **)&pl->dout.phase_cycles, hout->phase_cycles, false, true},
    };
    pl->total = 0;
    for (int i = 0; i < kStageBlks; ++i) { pl->blk[i] = blks[i]; pl->total += (blks[i].bytes + 255) & ~(size_t)255; }
    return BR_OK;
}

}  // namespace

int br_step_host(br_ctx *ctx, const br_instance_batch *batch, br_worker_state *hws,
                 br_waiting_queue *hwq, const float *h_probs, int32_t *h_assign, br_load_out *hout,
                 int64_t *h2d_bytes, int64_t *d2h_bytes)
{
    StagePlan pl;
    int rc = plan_host_step(ctx, batch, hws, hwq, h_probs, h_assign, hout, &pl);
    if (rc != BR_OK) return rc;
    const size_t N = (size_t)batch->n_instances;
    if (N == 0) return BR_OK;
    cudaStream_t st = (cudaStream_t)batch->stream;
    typedef StageBlk Blk;
    Blk (&blks)[kStageBlks] = pl.blk;
    br_worker_state &dws = pl.dws; br_waiting_queue &dwq = pl.dwq; br_load_out &dout = pl.dout;
    float *&d_probs = pl.d_probs; int32_t *&d_assign = pl.d_assign;
    const size_t total = pl.total;
    if (total > ctx->stage_bytes) {
        if (ctx->stage) { cudaFree(ctx->stage); ctx->stage = nullptr; ctx->stage_bytes = 0; }
        cudaError_t e = cudaMalloc(&ctx->stage, total);
        if (e != cudaSuccess) { cuda_fail(e, "cudaMalloc(staging)"); return BR_ENOMEM; }
        ctx->stage_bytes = total;
    }
    // per-instance row size of every block (all blocks are [N][row] arrays)
    size_t off = 0; int64_t up = 0, down = 0;
    for (Blk &b : blks) {
        if (!b.bytes) continue;
        *b.dev = (char *)ctx->stage + off;
        off += (b.bytes + 255) & ~(size_t)255;
        if (b.in) up += (int64_t)b.bytes;
        if (b.out) down += (int64_t)b.bytes;
    }
    br_instance_batch db = *batch; db.n_steps = 1;
    rc = check_step_args(ctx, &db, &dws, &dwq, d_probs, d_assign, &dout);
    if (rc != BR_OK) return rc;
    // Large batches go through in chunks of instances on three streams: the upload of chunk c + 1,
    // the kernel of chunk c and the download of chunk c - 1 overlap (the two copy directions use
    // separate engines).  Every chunk is a contiguous range of rows of every array.  Only the
    // large arrays are cut into chunks (a copy call costs microseconds of host time): the small
    // ones go up whole before the first chunk and come down whole after the last.
    const int n_chunks = N >= 512 ? 4 : 1;              // measured best of 2..8 on 4096 instances of the c3 shape
    const size_t kBig = (size_t)1 << 20;
    if (n_chunks > 1 && !ctx->pipe_ready) {
        for (int i = 0; i < 3; ++i) BR_CUDA(cudaStreamCreateWithFlags(&ctx->pipe[i], cudaStreamNonBlocking));
        for (int i = 0; i < 2 * 8 + 2; ++i) BR_CUDA(cudaEventCreateWithFlags(&ctx->pipe_ev[i], cudaEventDisableTiming));
        ctx->pipe_ready = true;
    }
    // once copies are queued an error drains the device before it is reported (the copies use the
    // caller's buffers and up to three streams)
#define BR_HOST_STEP(call)                                            \
    do {                                                              \
        cudaError_t e__ = (call);                                     \
        if (e__ != cudaSuccess) { cudaDeviceSynchronize(); return cuda_fail(e__, #call); } \
    } while (0)
    cudaStream_t s_in = st, s_k = st, s_out = st;
    if (n_chunks > 1) {
        s_in = ctx->pipe[0]; s_k = ctx->pipe[1]; s_out = ctx->pipe[2];
        BR_CUDA(cudaEventRecord(ctx->pipe_ev[16], st));              // everything queued on the caller's stream first
        BR_CUDA(cudaStreamWaitEvent(s_in, ctx->pipe_ev[16], 0));
        BR_CUDA(cudaStreamWaitEvent(s_k, ctx->pipe_ev[16], 0));
        BR_CUDA(cudaStreamWaitEvent(s_out, ctx->pipe_ev[16], 0));
    }
    if (n_chunks > 1)
        for (Blk &b : blks)
            if (b.bytes && b.in && b.bytes < kBig)
                BR_HOST_STEP(cudaMemcpyAsync(*b.dev, b.host, b.bytes, cudaMemcpyHostToDevice, s_in));
    for (int c = 0; c < n_chunks; ++c) {
        const size_t i0 = N * (size_t)c / n_chunks, i1 = N * (size_t)(c + 1) / n_chunks;
        for (Blk &b : blks) {
            if (!b.bytes || !b.in || (n_chunks > 1 && b.bytes < kBig)) continue;
            const size_t row = b.bytes / N;
            BR_HOST_STEP(cudaMemcpyAsync((char *)*b.dev + i0 * row, (const char *)b.host + i0 * row, (i1 - i0) * row,
                                    cudaMemcpyHostToDevice, s_in));
        }
        if (n_chunks > 1) {
            BR_CUDA(cudaEventRecord(ctx->pipe_ev[c], s_in));
            BR_CUDA(cudaStreamWaitEvent(s_k, ctx->pipe_ev[c], 0));
        }
        br_instance_batch cb = db;
        cb.first_instance = (int32_t)i0; cb.n_instances = (int32_t)(i1 - i0);
        rc = launch_step(ctx, &cb, &dws, &dwq, d_probs, d_assign, &dout, s_k);   // rows are addressed through first_instance
        if (rc != BR_OK) { cudaDeviceSynchronize(); return rc; }
        if (n_chunks > 1) {
            BR_CUDA(cudaEventRecord(ctx->pipe_ev[8 + c], s_k));
            BR_CUDA(cudaStreamWaitEvent(s_out, ctx->pipe_ev[8 + c], 0));
        }
        for (Blk &b : blks) {
            if (!b.bytes || !b.out || (n_chunks > 1 && b.bytes < kBig)) continue;
            const size_t row = b.bytes / N;
            BR_HOST_STEP(cudaMemcpyAsync((char *)b.host + i0 * row, (const char *)*b.dev + i0 * row, (i1 - i0) * row,
                                    cudaMemcpyDeviceToHost, s_out));
        }
    }
    if (n_chunks > 1)
        for (Blk &b : blks)                              // s_out has waited for the last kernel
            if (b.bytes && b.out && b.bytes < kBig)
                BR_HOST_STEP(cudaMemcpyAsync(b.host, *b.dev, b.bytes, cudaMemcpyDeviceToHost, s_out));
    if (n_chunks > 1) {
        BR_CUDA(cudaEventRecord(ctx->pipe_ev[17], s_out));
        BR_CUDA(cudaStreamWaitEvent(st, ctx->pipe_ev[17], 0));
    }
    BR_CUDA(cudaStreamSynchronize(st));
#undef BR_HOST_STEP
    if (h2d_bytes) *h2d_bytes = up;
    if (d2h_bytes) *d2h_bytes = down;
    return BR_OK;
}

/* ---- host-buffer step without any allocation ------------------------------------------- */

// Staging for br_step_host_static.  It lives in the library image: every GPU that loads the
// library holds these bytes until the process exits, and every call on a device shares them.
static __device__ __align__(256) unsigned char g_static_stage[BR_STATIC_STAGE_BYTES];

namespace {
constexpr int kMaxDevices = 64;
// device address of g_static_stage, per device (looked up once; two threads that race on the first
// call both store the same address).  cudaDeviceReset invalidates it: the library does not support
// being used across a device reset.
std::atomic<void *> g_static_stage_ptr[kMaxDevices];

// In host code `g_static_stage` is only a handle; the address a kernel or a copy can use
// has to be asked for, once per device, with that device current.
int static_stage_address(void **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) return BR_EINVAL;
    void *ptr = g_static_stage_ptr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        e = cudaGetSymbolAddress((void **)&ptr, g_static_stage);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(g_static_stage)");
        g_static_stage_ptr[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return BR_OK;
}
}  // namespace

int br_step_host_static(br_ctx *ctx, const br_instance_batch *batch, br_worker_state *hws,
                        br_waiting_queue *hwq, const float *h_probs, int32_t *h_assign,
                        br_load_out *hout, int64_t *h2d_bytes, int64_t *d2h_bytes)
{
    if (hout && hout->fscore) return BR_EINVAL;         // the score matrix is not offered on this path
    StagePlan pl;
    int rc = plan_host_step(ctx, batch, hws, hwq, h_probs, h_assign, hout, &pl);
    if (rc != BR_OK) return rc;
    const size_t N = (size_t)batch->n_instances;
    if (N == 0) return BR_OK;
    cudaStream_t st = (cudaStream_t)batch->stream;
    typedef StageBlk Blk;
    Blk (&blks)[kStageBlks] = pl.blk;
    br_worker_state &dws = pl.dws; br_waiting_queue &dwq = pl.dwq; br_load_out &dout = pl.dout;
    float *&d_probs = pl.d_probs; int32_t *&d_assign = pl.d_assign;
    const size_t total = pl.total;
    if (total > (size_t)BR_STATIC_STAGE_BYTES) return BR_ELIMIT;      // nothing was touched

    void *stage = nullptr;
    rc = static_stage_address(&stage);
    if (rc != BR_OK) return rc;

    size_t off = 0, out_begin = 0, out_end = 0;
    int64_t up = 0, down = 0;
    for (Blk &b : blks) {
        if (!b.bytes) continue;
        *b.dev = (char *)stage + off;
        if (!b.in) { if (!out_end) out_begin = off; out_end = off + ((b.bytes + 255) & ~(size_t)255); }
        off += (b.bytes + 255) & ~(size_t)255;
        if (b.in) { BR_CUDA_DRAIN(cudaMemcpyAsync(*b.dev, b.host, b.bytes, cudaMemcpyHostToDevice, st), st); up += (int64_t)b.bytes; }
    }
    // the buffer still holds the previous call's results: the output blocks start from zero
    if (out_end > out_begin) BR_CUDA_DRAIN(cudaMemsetAsync((char *)stage + out_begin, 0, out_end - out_begin, st), st);
    br_instance_batch db = *batch; db.n_steps = 1;
    rc = check_step_args(ctx, &db, &dws, &dwq, d_probs, d_assign, &dout);
    if (rc == BR_OK) rc = launch_step(ctx, &db, &dws, &dwq, d_probs, d_assign, &dout, st);
    if (rc != BR_OK) { cudaStreamSynchronize(st); return rc; }
    for (Blk &b : blks) {
        if (!b.bytes || !b.out) continue;
        BR_CUDA_DRAIN(cudaMemcpyAsync(b.host, *b.dev, b.bytes, cudaMemcpyDeviceToHost, st), st);
        down += (int64_t)b.bytes;
    }
    BR_CUDA(cudaStreamSynchronize(st));
    if (h2d_bytes) *h2d_bytes = up;
    if (d2h_bytes) *d2h_bytes = down;
    return BR_OK;
}

int br_fscore(br_ctx *ctx, const br_instance_batch *batch, const int32_t *s, int32_t n_requests,
              const int64_t *Lh, const int32_t *cap, double *F, int32_t *best_g)
{
    if (!ctx || !batch || !s || !Lh || !F) return BR_EINVAL;
    if (batch->n_instances < 0 || n_requests < 0 || (n_requests % 4) != 0) return BR_EINVAL;
    if (misaligned(s, 16) || misaligned(Lh, 8) || misaligned(F, 8)) return BR_EINVAL;
    if (batch->n_instances == 0 || n_requests == 0) return BR_OK;
    br::FscoreArgs a;
    a.G = ctx->G; a.H = ctx->H; a.fp = ctx->p.score_mode == 1;
    a.aD = ctx->base.aD; a.beta = ctx->base.beta;
    for (int h = 0; h <= BR_MAX_H; ++h) a.d[h] = ctx->base.d[h];
    a.n_req = n_requests; a.first_instance = batch->first_instance;
    a.s = s; a.Lh = Lh; a.cap = cap; a.F = F; a.best_g = best_g;
    const int tiles = (n_requests + br::kFsTile - 1) / br::kFsTile;
    dim3 grid(tiles, batch->n_instances);
    void (*kern)(const br::FscoreArgs) = ctx->H == 0 ? br::br_fscore_kernel<0> : ctx->H <= 4 ? br::br_fscore_kernel<4>
                                       : ctx->H <= 8 ? br::br_fscore_kernel<8>
                                       : ctx->H <= 16 ? br::br_fscore_kernel<16> : br::br_fscore_kernel<BR_MAX_H>;
    kern<<<grid, 256, 0, (cudaStream_t)batch->stream>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "br_fscore launch");
    return BR_OK;
}

int br_best_subset(br_ctx *ctx, const br_instance_batch *batch, const int32_t *win, int32_t R,
                   const int64_t *margins, const int32_t *lim, uint32_t *best_mask, double *best_F)
{
    if (!ctx || !batch || !win || !margins || !lim || !best_mask) return BR_EINVAL;
    if (batch->n_instances < 0 || batch->first_instance < 0 || R < 1 || R > br::kSubsetMaxR) return BR_EINVAL;
    if (misaligned(win, 4) || misaligned(margins, 8) || misaligned(lim, 4) || misaligned(best_mask, 4) ||
        (best_F && misaligned(best_F, 8)))
        return BR_EINVAL;
    if (batch->n_instances == 0) return BR_OK;
    br::SubsetArgs a;
    memset(&a, 0, sizeof(a));
    a.f.G = ctx->G; a.f.H = ctx->H; a.f.fp = ctx->p.score_mode == 1;
    a.f.aD = ctx->base.aD; a.f.beta = ctx->base.beta;
    for (int h = 0; h <= BR_MAX_H; ++h) a.f.d[h] = ctx->base.d[h];
    a.R = R; a.first_instance = batch->first_instance;
    a.win = win; a.m = margins; a.lim = lim; a.best_mask = best_mask; a.best_F = best_F;
    // windows of 13 requests and more meet in the middle when the two-probe rule holds; without it
    // only enumeration is exact, which stops at 20 requests
    if (R > br::kSubsetMaxEnum && !ctx->two_probe_ok) return BR_EINVAL;
    if (R > 12 && ctx->two_probe_ok)
        br::br_subset_mitm_kernel<<<batch->n_instances, 256, 0, (cudaStream_t)batch->stream>>>(a);
    else
        br::br_subset_kernel<<<batch->n_instances, 256, 0, (cudaStream_t)batch->stream>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "br_best_subset launch");
    return BR_OK;
}

int br_bypass_dispatch(br_ctx *ctx, const br_instance_batch *batch, const int32_t *s, int32_t n_requests,
                       int64_t *virtual_load, int32_t *inflight, const int32_t *inflight_cap, int32_t *worker_out)
{
    if (!ctx || !batch || !s || !virtual_load || !inflight || !inflight_cap || !worker_out) return BR_EINVAL;
    if (ctx->H != 0) return BR_EINVAL;                       // the pool-bypass path exists for BR-0 only
    if (batch->n_instances < 0 || batch->first_instance < 0 || n_requests < 0) return BR_EINVAL;
    if (misaligned(s, 4) || misaligned(virtual_load, 8) || misaligned(inflight, 4) ||
        misaligned(inflight_cap, 4) || misaligned(worker_out, 4))
        return BR_EINVAL;
    if (batch->n_instances == 0 || n_requests == 0) return BR_OK;
    br::BypassArgs a;
    memset(&a, 0, sizeof(a));
    a.f.G = ctx->G; a.f.H = 0; a.f.fp = ctx->p.score_mode == 1;
    a.f.aD = ctx->base.aD; a.f.beta = ctx->base.beta;
    for (int h = 0; h <= BR_MAX_H; ++h) a.f.d[h] = ctx->base.d[h];
    a.n_req = n_requests; a.first_instance = batch->first_instance;
    a.s = s; a.vload = virtual_load; a.inflight = inflight; a.cap = inflight_cap; a.g_out = worker_out;
    const int blocks = (batch->n_instances + 3) / 4;
    br::br_bypass_kernel<<<blocks, 128, 0, (cudaStream_t)batch->stream>>>(a, batch->n_instances);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "br_bypass_dispatch launch");
    return BR_OK;
}

int br_survival_chat(br_ctx *ctx, void *stream, const int32_t *hist_sorted, const int64_t *hist_prefix,
                     int32_t n_hist, const int32_t *age, int64_t count, float *c_hat, double *p_fin,
                     double *mu_rem)
{
    if (!ctx || !hist_sorted || !hist_prefix || !age || !c_hat) return BR_EINVAL;
    if (ctx->H < 1 || n_hist < 1 || count < 0) return BR_EINVAL;
    if (misaligned(hist_sorted, 4) || misaligned(hist_prefix, 8) || misaligned(age, 4) || misaligned(c_hat, 4) ||
        (p_fin && misaligned(p_fin, 8)) || (mu_rem && misaligned(mu_rem, 8)))
        return BR_EINVAL;
    if (count == 0) return BR_OK;
    br::SurvivalArgs a;
    a.hist = hist_sorted; a.prefix = hist_prefix; a.n_hist = n_hist; a.H = ctx->H;
    a.age = age; a.count = count; a.c_hat = c_hat; a.p_fin = p_fin; a.mu_rem = mu_rem;
    const int64_t blocks = (count + 255) / 256;
    if (blocks > 0x7FFFFFFF) return BR_EINVAL;
    br::br_survival_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "br_survival_chat launch");
    return BR_OK;
}

#ifdef BR_BOUNDS
namespace {
// indexes a four-element span at -1, 4 and 7 (one read, two writes): all three land in the sink
__global__ void bounds_selftest_kernel(int *four)
{
    const auto s = br::mk_span(four, 4);
    const int v = s[-1];
    s[4] = v + 1;
    *br::vec_at<int4>(s, 4) = make_int4(1, 2, 3, 4);
    s[3] = 7;                                             // in range: not counted
}
}  // namespace
#endif

int br_debug_bounds_hits(void)
{
#ifdef BR_BOUNDS
    unsigned h = 0;
    BR_CUDA(cudaDeviceSynchronize());
    BR_CUDA(cudaMemcpyFromSymbol(&h, br::g_bounds_hits, sizeof(h)));
    return (int)(h > 0x7FFFFFFFu ? 0x7FFFFFFFu : h);
#else
    return -1;
#endif
}

int br_debug_bounds_selftest(int32_t *four_ints)
{
#ifdef BR_BOUNDS
    if (!four_ints) return BR_EINVAL;
    const int before = br_debug_bounds_hits();
    if (before < 0) return before;
    bounds_selftest_kernel<<<1, 1>>>(four_ints);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "bounds self-test launch");
    const int after = br_debug_bounds_hits();
    return after < 0 ? after : after - before;
#else
    (void)four_ints;
    return -1;
#endif
}

int br_destroy(br_ctx *ctx)
{
    if (!ctx) return BR_OK;
    if (ctx->graph_exec) cudaGraphExecDestroy(ctx->graph_exec);
    if (ctx->graph) cudaGraphDestroy(ctx->graph);
    if (ctx->stage) cudaFree(ctx->stage);
    if (ctx->pipe_ready) {
        for (int i = 0; i < 3; ++i) cudaStreamDestroy(ctx->pipe[i]);
        for (int i = 0; i < 2 * 8 + 2; ++i) cudaEventDestroy(ctx->pipe_ev[i]);
    }
    delete ctx;
    return BR_OK;
}

}  // extern "C"
