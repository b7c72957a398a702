// C entry points of libchoco: argument checks, allocation, and the order in which one step
// enqueues its kernels.  No arithmetic of the method lives here.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"
#include "internal.h"

using namespace choco;

namespace {

int fail_cuda(choco_ctx* ctx, cudaError_t e)
{
    if (ctx) ctx->last_cuda_error = (int)e;
    return CHOCO_ERR_CUDA;
}

template <typename T>
cudaError_t dev_alloc(choco_ctx* ctx, T** out, int64_t count)
{
    void* p = nullptr;
    const size_t bytes = (size_t)(count > 0 ? count : 1) * sizeof(T);
    cudaError_t e = cudaMalloc(&p, bytes);
    if (e != cudaSuccess) return e;
    e = cudaMemset(p, 0, bytes);
    if (e != cudaSuccess) { cudaFree(p); return e; }
    if (ctx->nallocs >= (int)(sizeof(ctx->allocs) / sizeof(ctx->allocs[0]))) { cudaFree(p); return cudaErrorMemoryAllocation; }
    ctx->allocs[ctx->nallocs++] = p;
    *out = (T*)p;
    return cudaSuccess;
}

int64_t round_up(int64_t v, int64_t m) { return (v + m - 1) / m * m; }

// Assumption 1 plus the CSR rules of choco.h
int check_w(int32_t n, const int32_t* rp, const int32_t* col, const float* val)
{
    if (rp[0] != 0) return CHOCO_ERR_BAD_W;
    for (int32_t i = 0; i < n; ++i) {
        if (rp[i + 1] <= rp[i]) return CHOCO_ERR_BAD_W;
        double sum = 0.0;
        bool diag = false;
        for (int32_t e = rp[i]; e < rp[i + 1]; ++e) {
            if (col[e] < 0 || col[e] >= n) return CHOCO_ERR_BAD_W;
            if (e > rp[i] && col[e] <= col[e - 1]) return CHOCO_ERR_BAD_W;
            if (!(val[e] >= 0.0f && val[e] <= 1.0f)) return CHOCO_ERR_BAD_W;
            if (col[e] == i) diag = true;
            sum += (double)val[e];
        }
        if (!diag || std::fabs(sum - 1.0) > 1e-5) return CHOCO_ERR_BAD_W;
    }
    // symmetry: every (i, j, w) needs a (j, i, w')
    for (int32_t i = 0; i < n; ++i)
        for (int32_t e = rp[i]; e < rp[i + 1]; ++e) {
            const int32_t j = col[e];
            bool found = false;
            for (int32_t f = rp[j]; f < rp[j + 1]; ++f)
                if (col[f] == i) { found = std::fabs((double)val[f] - (double)val[e]) <= 1e-6; break; }
            if (!found) return CHOCO_ERR_BAD_W;
        }
    return CHOCO_OK;
}

bool is_pow2(int64_t v) { return v > 0 && (v & (v - 1)) == 0; }

float qsgd_tau(int64_t len, int32_t s, bool biased)
{
    if (!biased) return 1.0f;
    const double a = (double)len / ((double)s * (double)s);
    const double b = std::sqrt((double)len) / (double)s;
    return (float)(1.0 + (a < b ? a : b));
}

// Raise the device's persisting-L2 carve-out so that the context's hot arena (messages, range
// records, per-tile tables) can stay resident while the dense arrays stream past; kernels then
// carry an access-policy window over it as a launch attribute.  Best effort: failures are
// ignored, the results do not depend on it.  The limit is never lowered here.
void reserve_hot_l2(choco_ctx* ctx, void* base, int64_t bytes)
{
    int dev = 0, max_persist = 0, max_window = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return;
    cudaDeviceGetAttribute(&max_persist, cudaDevAttrMaxPersistingL2CacheSize, dev);
    cudaDeviceGetAttribute(&max_window, cudaDevAttrMaxAccessPolicyWindowSize, dev);
    if (max_persist <= 0 || max_window <= 0 || bytes <= 0) { cudaGetLastError(); return; }
    const size_t want = std::min<size_t>((size_t)bytes, (size_t)max_persist / 4 * 3);
    size_t have = 0;
    cudaDeviceGetLimit(&have, cudaLimitPersistingL2CacheSize);
    if (have < want) cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, want);
    have = 0;
    cudaDeviceGetLimit(&have, cudaLimitPersistingL2CacheSize);
    cudaGetLastError(); // best effort
    if (have == 0) return;
    const size_t window = std::min<size_t>((size_t)bytes, (size_t)max_window);
    const double ratio = (double)have / (double)window;
    ctx->dv.hot_base = base;
    ctx->dv.hot_bytes = (int64_t)window;
    ctx->dv.hot_ratio = ratio >= 1.0 ? 1.0f : (float)ratio;
    ctx->hot_l2 = true;
}

__global__ void bump_step_kernel(unsigned long long* step) { *step += 1ull; }

bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }
bool aligned4(const void* p) { return ((uintptr_t)p & 3u) == 0; }

// The update of a step in chunks of rows (choco_sgd_step_host): chunk c waits for `ready[c]` and
// records `done[c]` on the step's stream.
struct RowChunks {
    int count, rows_per_chunk;
    cudaEvent_t* ready;
    cudaEvent_t* done;
};

int step_body(choco_ctx* ctx, float* X, float* Xhat, float* S, const float* G, float* M, float eta,
              float gamma, float lambda, float beta, void* stream, const RowChunks* chunks = nullptr)
{
    if (!ctx || !X || !Xhat || !S) return CHOCO_ERR_INVALID_ARG;
    if (ctx->timed_out) return CHOCO_ERR_TIMEOUT; // the arrays are no valid state any more
    if (!aligned4(X) || !aligned4(Xhat) || !aligned4(S) || !aligned4(G) || !aligned4(M))
        return CHOCO_ERR_MISALIGNED;
    cudaStream_t st = (cudaStream_t)stream;
    Dev dv = ctx->dv; // by value: the dense message buffers are swapped per step
    {
        const choco_ctx::DenseBuf &cur = ctx->dbuf[ctx->msg_cur], &nxt = ctx->dbuf[ctx->msg_cur ^ 1];
        dv.msg_bits = cur.bits; dv.msg_scale = cur.scale; dv.msg_norms = cur.norms;
        dv.msg_levels = cur.levels; dv.msg_dense = cur.dense;
        dv.nxt_bits = nxt.bits; dv.nxt_scale = nxt.scale; dv.nxt_norms = nxt.norms;
        dv.nxt_levels = nxt.levels; dv.nxt_dense = nxt.dense;
    }
    StepArgs a;
    a.X = X; a.Xhat = Xhat; a.S = S; a.G = G; a.M = M;
    a.eta = eta; a.gamma = gamma; a.lambda = lambda; a.beta = beta;
    a.step = ctx->step;
    a.step_dev = ctx->dev_step ? ctx->step_dev : nullptr;
    a.launches = &ctx->launches;
    a.vec = (dv.ld % 4 == 0) && aligned16(X) && aligned16(Xhat) && aligned16(S) &&
            (!G || aligned16(G)) && (!M || aligned16(M));
    if (ctx->last_x != X || ctx->last_xhat != Xhat) ctx->prepared = false;

    cudaError_t e = cudaSuccess;
    const bool sparse = dv.kind == CHOCO_Q_TOPK || dv.kind == CHOCO_Q_RANDK;
    const bool was_prepared = ctx->prepared;
    if (sparse) {
        if (!was_prepared) e = launch_select_prepare(dv, a, st);
        if (e == cudaSuccess) e = launch_select_emit(dv, a, was_prepared, st);
        if (e == cudaSuccess && dv.rescue && dv.kind == CHOCO_Q_TOPK) e = launch_select_rescue(dv, a, st);
    } else if (!was_prepared) {
        e = launch_compress_dense(dv, a, st);
    }
    // the update kernel can collect the next step's candidates from the x' - x^' it holds
    const bool emit = ctx->carry_enabled && apply_can_emit(dv, a);
    const bool prof = ctx->prof_ev && ctx->prof_n < ctx->prof_cap &&
                      (ctx->prof_stride <= 1 || ctx->steps_enqueued % (uint64_t)ctx->prof_stride == 0);
    if (e == cudaSuccess && prof) e = cudaEventRecord(ctx->prof_ev[2 * ctx->prof_n], st);
    if (chunks) {
        for (int c = 0; c < chunks->count && e == cudaSuccess; ++c) {
            a.row0 = c * chunks->rows_per_chunk;
            a.rows = std::min(chunks->rows_per_chunk, dv.n - a.row0);
            e = cudaStreamWaitEvent(st, chunks->ready[c], 0);
            if (e == cudaSuccess) e = launch_apply(dv, a, emit, st);
            if (e == cudaSuccess) e = cudaEventRecord(chunks->done[c], st);
        }
        a.row0 = 0;
        a.rows = 0;
    } else if (e == cudaSuccess) {
        e = launch_apply(dv, a, emit, st);
    }
    if (e == cudaSuccess && prof) {
        e = cudaEventRecord(ctx->prof_ev[2 * ctx->prof_n + 1], st);
        ctx->prof_n += 1;
    }
    if (e == cudaSuccess && emit && dv.kind == CHOCO_Q_SIGN) {
        e = launch_next_sign_scale(dv, st);
        ctx->launches += 1;
    }
    if (e == cudaSuccess && ctx->dev_step) {
        bump_step_kernel<<<1, 1, 0, st>>>(ctx->step_dev);
        e = cudaGetLastError();
        ctx->launches += 1;
    }
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    ctx->msg_last = ctx->msg_cur;
    if (emit && !sparse) ctx->msg_cur ^= 1; // the next step's messages sit in the other buffer
    ctx->prepared = emit;
    ctx->last_x = X;
    ctx->last_xhat = Xhat;
    ctx->step += 1;
    ctx->steps_enqueued += 1;
    return CHOCO_OK;
}

// The host-side fields a step changes, to undo a capture that failed.
struct HostState {
    uint64_t step, steps_enqueued;
    bool prepared;
    int msg_cur, msg_last;
    const float *last_x, *last_xhat;
    unsigned long long launches;
};

// A step call: small problems replay their steady-state step from a CUDA graph captured the
// second time a set of arguments is seen (a step there is a few short kernels, and launching
// them one by one takes longer than running them); everything else is enqueued kernel by kernel.
int run_step(choco_ctx* ctx, float* X, float* Xhat, float* S, const float* G, float* M, float eta,
             float gamma, float lambda, float beta, void* stream)
{
    if (!ctx || !X || !Xhat || !S) return CHOCO_ERR_INVALID_ARG;
    if (ctx->timed_out) return CHOCO_ERR_TIMEOUT;
    cudaStream_t st = (cudaStream_t)stream;
    uint64_t mode = 0;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    // the legacy default stream (NULL or cudaStreamLegacy) cannot be captured
    if (!ctx->graphs_ok || st == nullptr || st == cudaStreamLegacy || !step_repeats(ctx, X, Xhat, &mode) ||
        cudaStreamIsCapturing(st, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone)
        return step_body(ctx, X, Xhat, S, G, M, eta, gamma, lambda, beta, stream);
    // A set of arguments is captured the second time it is seen: a caller that passes new
    // arrays every step (a fresh gradient tensor, say) never pays for a capture.
    int slot = -1;
    for (int i = 0; i < ctx->ngraphs; ++i) {
        const choco_step_graph& g = ctx->graphs[i];
        if (g.X == X && g.Xhat == Xhat && g.S == S && g.G == G && g.M == M && g.eta == eta && g.gamma == gamma &&
            g.lambda == lambda && g.beta == beta && g.mode == mode) { slot = i; break; }
    }
    if (slot >= 0 && ctx->graphs[slot].exec) {
        choco_step_graph& g = ctx->graphs[slot];
        const cudaError_t e = cudaGraphLaunch(g.exec, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
        g.last_use = ++ctx->graph_clock;
        advance_after_replay(ctx, ctx->launches_per_step);
        ctx->graph_replays += 1;
        return CHOCO_OK;
    }
    if (slot < 0) { // first sighting: remember it, enqueue kernel by kernel
        slot = ctx->ngraphs;
        if (slot < kCtxGraphs) {
            ctx->ngraphs += 1;
        } else {
            slot = 0;
            for (int i = 1; i < kCtxGraphs; ++i)
                if (ctx->graphs[i].last_use < ctx->graphs[slot].last_use) slot = i;
            if (ctx->graphs[slot].exec) cudaGraphExecDestroy(ctx->graphs[slot].exec);
        }
        ctx->graphs[slot] = {X, Xhat, S, G, M, eta, gamma, lambda, beta, mode, nullptr, ++ctx->graph_clock};
        return step_body(ctx, X, Xhat, S, G, M, eta, gamma, lambda, beta, stream);
    }
    const HostState before = {ctx->step, ctx->steps_enqueued, ctx->prepared, ctx->msg_cur, ctx->msg_last,
                              ctx->last_x, ctx->last_xhat, ctx->launches};
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    bool ok = cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) == cudaSuccess;
    if (ok) {
        const int rc = step_body(ctx, X, Xhat, S, G, M, eta, gamma, lambda, beta, stream);
        const cudaError_t e = cudaStreamEndCapture(st, &graph);
        ok = rc == CHOCO_OK && e == cudaSuccess && graph != nullptr;
    }
    if (ok) ok = cudaGraphInstantiate(&exec, graph, 0) == cudaSuccess;
    if (graph) cudaGraphDestroy(graph);
    if (ok) ok = cudaGraphLaunch(exec, st) == cudaSuccess;
    if (!ok) { // put the host state back, give graphs up for this context, enqueue the step as usual
        cudaGetLastError();
        if (exec) cudaGraphExecDestroy(exec);
        ctx->step = before.step; ctx->steps_enqueued = before.steps_enqueued; ctx->prepared = before.prepared;
        ctx->msg_cur = before.msg_cur; ctx->msg_last = before.msg_last; ctx->last_x = before.last_x;
        ctx->last_xhat = before.last_xhat; ctx->launches = before.launches;
        ctx->graphs_ok = false;
        return step_body(ctx, X, Xhat, S, G, M, eta, gamma, lambda, beta, stream);
    }
    ctx->launches_per_step = ctx->launches - before.launches;
    ctx->graphs[slot].exec = exec;
    ctx->graphs[slot].last_use = ++ctx->graph_clock;
    return CHOCO_OK;
}

// For calls that have just synchronised `st`: did a bounded wait inside a kernel run out?
int check_device_timeouts(choco_ctx* ctx, cudaStream_t st)
{
    if (ctx->timed_out) return CHOCO_ERR_TIMEOUT;
    unsigned long long t = 0;
    cudaError_t e = cudaMemcpyAsync(&t, &ctx->dv.stats->timeouts, sizeof(t), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    if (t != 0) {
        ctx->timed_out = true;
        return CHOCO_ERR_TIMEOUT;
    }
    return CHOCO_OK;
}

} // namespace

namespace choco {

bool step_repeats(const choco_ctx* c, const float* X, const float* Xhat, uint64_t* mode)
{
    if (c->steps_enqueued == 0) return false; // the first step also sets the kernels up
    const StepArgs none = {};
    const bool carries = c->carry_enabled && apply_can_emit(c->dv, none);
    if (c->prepared != carries) return false;
    if (c->prepared && (c->last_x != X || c->last_xhat != Xhat)) return false;
    if (c->prof_ev && c->prof_n < c->prof_cap) return false;
    *mode = (uint64_t)((c->prepared ? 1 : 0) | (c->msg_cur << 1));
    return true;
}

void advance_after_replay(choco_ctx* c, unsigned long long launches)
{
    const bool sparse = c->dv.kind == CHOCO_Q_TOPK || c->dv.kind == CHOCO_Q_RANDK;
    c->msg_last = c->msg_cur;
    if (c->prepared && !sparse) c->msg_cur ^= 1; // the step wrote the next messages into the other buffer
    c->step += 1;
    c->steps_enqueued += 1;
    c->launches += launches;
}

} // namespace choco

extern "C" {

int choco_init(choco_ctx** out, int32_t n, int64_t d, int64_t ld, const int32_t* w_row_ptr,
               const int32_t* w_col, const float* w_val, const choco_params* p, uint64_t seed)
{
    if (!out || !w_row_ptr || !w_col || !w_val || !p) return CHOCO_ERR_INVALID_ARG;
    *out = nullptr;
    if (n < 1 || d < 1 || ld < d) return CHOCO_ERR_INVALID_ARG;
    if (d >= (int64_t)1 << 31) return CHOCO_ERR_TOO_LARGE;
    if (n > 65535) return CHOCO_ERR_TOO_LARGE; // rows index gridDim.y
    const int rcw = check_w(n, w_row_ptr, w_col, w_val);
    if (rcw) return rcw;
    const int32_t nnz = w_row_ptr[n];
    switch (p->kind) {
    case CHOCO_Q_IDENTITY:
    case CHOCO_Q_SIGN:
        break;
    case CHOCO_Q_TOPK:
    case CHOCO_Q_RANDK:
        if (p->k < 1 || p->k > d) return CHOCO_ERR_INVALID_ARG;
        break;
    case CHOCO_Q_QSGD:
        if (!is_pow2(p->s) || p->s < 2 || p->s > 32768) return CHOCO_ERR_INVALID_ARG;
        if (p->bucket < 0) return CHOCO_ERR_INVALID_ARG;
        if (p->bucket != 0 && !(is_pow2(p->bucket) && p->bucket >= 128 && p->bucket <= 1024))
            return CHOCO_ERR_UNSUPPORTED;
        break;
    default:
        return CHOCO_ERR_INVALID_ARG;
    }

    choco_ctx* ctx = new (std::nothrow) choco_ctx();
    if (!ctx) return CHOCO_ERR_ALLOC;
    std::memset(ctx, 0, sizeof(*ctx));
    ctx->params = *p;
    ctx->carry_enabled = true;
    ctx->graphs_ok = (int64_t)n * d <= kGraphCoords;
    // gsgd_b and random_a key their generator with the step number, which a captured kernel
    // argument would freeze: such contexts keep it in device memory and bump it there
    ctx->dev_step = ctx->graphs_ok && (p->kind == CHOCO_Q_QSGD || p->kind == CHOCO_Q_RANDK);
    Dev& dv = ctx->dv;
    dv.n = n; dv.d = d; dv.ld = ld; dv.kind = p->kind; dv.seed = seed;
    dv.wait_polls = kSpinLimit;
    dv.nesterov = 0;
    for (uint32_t r = 0; r < 10; ++r) {
        dv.round_key[r][0] = (uint32_t)seed + r * 0x9E3779B9u;
        dv.round_key[r][1] = (uint32_t)(seed >> 32) + r * 0xBB67AE85u;
    }
    dv.ntiles = (d + kTile - 1) / kTile;
    dv.nspans = (d + kSpan - 1) / kSpan;
    dv.nchunks = (d + kChunk - 1) / kChunk;

    cudaError_t e = cudaGetDevice(&ctx->device);
    int32_t *rp = nullptr, *col = nullptr;
    float* wv = nullptr;
    if (e == cudaSuccess) e = dev_alloc(ctx, &rp, n + 1);
    if (e == cudaSuccess) e = dev_alloc(ctx, &col, nnz);
    if (e == cudaSuccess) e = dev_alloc(ctx, &wv, nnz);
    if (e == cudaSuccess) e = cudaMemcpy(rp, w_row_ptr, sizeof(int32_t) * (n + 1), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(col, w_col, sizeof(int32_t) * nnz, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(wv, w_val, sizeof(float) * nnz, cudaMemcpyHostToDevice);
    dv.row_ptr = rp; dv.col = col; dv.wval = wv;
    {
        // for every CSR entry (j -> i): where j sits in row i, and the weight row i holds for it
        std::vector<int32_t> pos(nnz);
        std::vector<float> rw(nnz);
        int32_t maxdeg = 0;
        for (int32_t j = 0; j < n; ++j) {
            maxdeg = std::max(maxdeg, w_row_ptr[j + 1] - w_row_ptr[j]);
            for (int32_t e2 = w_row_ptr[j]; e2 < w_row_ptr[j + 1]; ++e2) {
                const int32_t i = w_col[e2];
                for (int32_t f = w_row_ptr[i]; f < w_row_ptr[i + 1]; ++f)
                    if (w_col[f] == j) { pos[e2] = f - w_row_ptr[i]; rw[e2] = w_val[f]; break; }
            }
        }
        dv.maxdeg = maxdeg;
        int32_t* dpos = nullptr;
        float* drw = nullptr;
        if (e == cudaSuccess) e = dev_alloc(ctx, &dpos, nnz);
        if (e == cudaSuccess) e = dev_alloc(ctx, &drw, nnz);
        if (e == cudaSuccess) e = cudaMemcpy(dpos, pos.data(), sizeof(int32_t) * nnz, cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemcpy(drw, rw.data(), sizeof(float) * nnz, cudaMemcpyHostToDevice);
        dv.rd_pos = dpos; dv.rd_w = drw;
    }
    if (e == cudaSuccess) e = dev_alloc(ctx, &dv.stats, 1);
    if (e == cudaSuccess) e = dev_alloc(ctx, &ctx->step_dev, 1); // zeroed, as the step counter is

    const int64_t nwords = (d + 31) / 32;
    if (p->kind == CHOCO_Q_TOPK || p->kind == CHOCO_Q_RANDK) {
        dv.k = p->k;
        dv.rescue = (p->kind == CHOCO_Q_TOPK && d >= kRescueMinD) ? 1 : 0;
        dv.kpitch = round_up(p->k, 4);
        // candidates per row: aimed at 2.5 k, with room for a bound that was guessed low
        int64_t cap = 6 * p->k > p->k + 8192 ? 6 * p->k : p->k + 8192;
        dv.cap = round_up(cap < d ? cap : d, 4); // rows of the candidate arrays stay 16-byte aligned
        {
            // slots of three times a tile's share of the 3 k candidates the bound aims at first
            // (a tile cannot have more than kTile), and room for 2 k candidates behind them
            const int64_t share = (9 * p->k + dv.ntiles - 1) / dv.ntiles;
            const int64_t slot = std::min<int64_t>(kTile, std::max<int64_t>(16, round_up(share, 8)));
            dv.cand_slot_alloc = (uint32_t)slot;
            dv.cand_slot = 0;
            const int64_t behind = std::min<int64_t>(dv.cap, std::max<int64_t>(2 * p->k, 2048));
            dv.cand_pitch = std::max<int64_t>(dv.cap, round_up(dv.ntiles * slot + behind, 4));
        }
        {
            // One arena for what one kernel writes and the next reads back within a step.  Its
            // head (range records, messages, per-tile tables) is read with dependent loads by
            // the update kernel: steps ask the L2 cache to keep that part resident while the
            // dense arrays stream past it (measured: keeping the candidates too does not pay).
            const int64_t b_rec = round_up((int64_t)n * dv.ntiles * dv.maxdeg * 16, 256);
            const int64_t b_msg = round_up(n * dv.kpitch * 4, 256);
            const int64_t b_tp = round_up(n * (dv.ntiles + 1) * 4, 256);
            const int64_t b_cand = round_up(n * dv.cand_pitch * 4, 256);
            const int64_t b_seg = round_up(n * dv.ntiles * 4, 256);
            const int64_t b_row = round_up((int64_t)n * 4, 256);
            const int64_t total = b_rec + 2 * b_msg + b_tp + 2 * b_cand + 2 * b_seg + 6 * b_row;
            unsigned char* arena = nullptr;
            if (e == cudaSuccess) e = dev_alloc(ctx, &arena, total);
            unsigned char* q = arena;
            dv.rec = (uint4*)q; q += b_rec;
            dv.msg_idx = (uint32_t*)q; q += b_msg;
            dv.msg_val = (float*)q; q += b_msg;
            dv.tile_ptr = (uint32_t*)q; q += b_tp;
            dv.seg_off = (uint32_t*)q; q += b_seg;
            dv.seg_cnt = (uint32_t*)q; q += b_seg;
            dv.row_lo = (uint32_t*)q; q += b_row;
            dv.row_count = (uint32_t*)q; q += b_row;
            dv.row_flags = (uint32_t*)q; q += b_row;
            dv.row_aim = (uint32_t*)q; q += b_row;
            dv.row_above = (uint32_t*)q; q += b_row;
            dv.row_ovf = (uint32_t*)q; q += b_row;
            const int64_t hot = q - arena; // the candidates behind it are written once, read once
            dv.cand_idx = (uint32_t*)q; q += b_cand;
            dv.cand_val = (uint32_t*)q; q += b_cand;
            if (e == cudaSuccess) reserve_hot_l2(ctx, arena, hot);
        }
        if (e == cudaSuccess) e = dev_alloc(ctx, &dv.hist, (int64_t)n * kHistBins);
        if (e == cudaSuccess) e = dev_alloc(ctx, &dv.tile_a, n * dv.ntiles);
        if (e == cudaSuccess) e = dev_alloc(ctx, &dv.tile_b, n * dv.ntiles);
        if (e == cudaSuccess) e = dev_alloc(ctx, &dv.tile_c, n * dv.ntiles);
        {
            // the emit kernel keeps in shared memory, in this order of preference and as far
            // as the budget allows: slab prefixes, per-tile arrays, a cache of the keys
            // every piece a multiple of 16 bytes, so that the key cache behind them can be the
            // destination of bulk copies; 16 bytes in front for their barrier
            dv.slab_pitch = round_up(dv.cap / 32 + 2, 4);
            const int64_t tpitch = round_up(dv.ntiles, 4);
            int64_t left = kEmitSmemBudget - 16;
            dv.emit_slabs_smem = 2 * dv.slab_pitch * 4 <= left ? 1 : 0;
            if (dv.emit_slabs_smem) left -= 2 * dv.slab_pitch * 4;
            dv.emit_tiles_smem = 3 * tpitch * 4 <= left ? 1 : 0;
            if (dv.emit_tiles_smem) left -= 3 * tpitch * 4;
            dv.emit_masks_smem = 2 * dv.slab_pitch * 4 <= left ? 1 : 0;
            if (dv.emit_masks_smem) left -= 2 * dv.slab_pitch * 4;
            dv.emit_keys_cap = std::min<int64_t>(dv.cap, (left / 8) & ~(int64_t)3); // value bits and index per candidate
            dv.emit_smem_bytes = kEmitSmemBudget - left + dv.emit_keys_cap * 8;
            // Few rows leave most SMs idle in a kernel with one block per row: let a cluster of
            // 2 or 4 blocks serve each row, as long as all clusters still run at once.
            int nsm = 0;
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&nsm, cudaDevAttrMultiProcessorCount, ctx->device);
            dv.emit_cluster = n * 4 <= nsm ? 4 : (n * 2 <= nsm ? 2 : 1);
            // (rows with few candidates are served faster by one block: the cluster's barriers
            // and exchanges cost more than the shared work saves; measured on d = 272 474, k = 2 724)
            if (dv.cap < 32768) dv.emit_cluster = 1;
            // candidates per block: what fits beside the fixed arrays, no more than a row can have
            const int64_t budget_words = kEmitSmemBudget / 4;
            int64_t cl = ((budget_words - 5152) * 8 / 17) & ~(int64_t)31; // 2.125 words per candidate
            dv.emit_cap_local = std::min<int64_t>(cl, round_up(dv.cap, 32));
            // the cluster kernel gathers tile by tile: the update kernel may then place a tile's
            // candidates in the tile's own slot instead of reserving room with an atomic add
            dv.cand_slot = (p->kind == CHOCO_Q_TOPK && dv.emit_cluster > 1) ? dv.cand_slot_alloc : 0u;
            if (e == cudaSuccess) e = dev_alloc(ctx, &dv.spill_key, n * dv.cand_pitch);
            if (e == cudaSuccess) e = dev_alloc(ctx, &dv.spill_idx, n * dv.cand_pitch);
            if (e == cudaSuccess) e = dev_alloc(ctx, &dv.slab_a, n * dv.slab_pitch);
            if (e == cudaSuccess) e = dev_alloc(ctx, &dv.slab_b, n * dv.slab_pitch);
            if (e == cudaSuccess) e = dev_alloc(ctx, &dv.slab_c, n * dv.slab_pitch);
            if (e == cudaSuccess) e = dev_alloc(ctx, &dv.slab_d, n * dv.slab_pitch);
        }
        ctx->msg_bytes_per_worker = (p->kind == CHOCO_Q_TOPK ? 8 : 4) * p->k;
    } else if (p->kind == CHOCO_Q_SIGN) {
        dv.wpitch = round_up(nwords, 4);
        for (int b = 0; b < 2; ++b) {
            if (e == cudaSuccess) e = dev_alloc(ctx, &ctx->dbuf[b].bits, n * dv.wpitch);
            if (e == cudaSuccess) e = dev_alloc(ctx, &ctx->dbuf[b].scale, n);
        }
        if (e == cudaSuccess) e = dev_alloc(ctx, &dv.partial, n * dv.nchunks);
        if (e == cudaSuccess) e = dev_alloc(ctx, &dv.partial2, n * dv.nchunks);
        ctx->msg_bytes_per_worker = 4 * nwords + 4;
    } else if (p->kind == CHOCO_Q_QSGD) {
        dv.s = p->s;
        dv.bucket = p->bucket;
        int w = 1;
        while ((1 << w) < p->s) w *= 2;
        dv.wbits = w;
        const int64_t blen = p->bucket > 0 ? p->bucket : d;
        dv.nbuckets = (d + blen - 1) / blen;
        dv.npitch = round_up(dv.nbuckets, 4);
        dv.bucket_shift = 0;
        while (p->bucket > 0 && (1 << dv.bucket_shift) < p->bucket) ++dv.bucket_shift;
        dv.tail_bucket = (p->bucket > 0 && d % blen != 0) ? dv.nbuckets - 1 : -1;
        dv.tau_full = qsgd_tau(blen, p->s, p->qsgd_biased != 0);
        dv.tau_tail = qsgd_tau(d % blen ? d % blen : blen, p->s, p->qsgd_biased != 0);
        dv.wpitch = round_up(nwords, 4);
        const int64_t lbytes = (d * w + 7) / 8;
        dv.lpitch = round_up(lbytes, 16) + 16;
        for (int b = 0; b < 2; ++b) {
            if (e == cudaSuccess) e = dev_alloc(ctx, &ctx->dbuf[b].bits, n * dv.wpitch);
            if (e == cudaSuccess) e = dev_alloc(ctx, &ctx->dbuf[b].norms, n * dv.npitch);
            if (e == cudaSuccess) e = dev_alloc(ctx, &ctx->dbuf[b].levels, n * dv.lpitch);
        }
        if (e == cudaSuccess) e = dev_alloc(ctx, &dv.partial, n * dv.nchunks);
        if (e == cudaSuccess) e = dev_alloc(ctx, &dv.partial2, n * dv.nchunks);
        ctx->msg_bytes_per_worker = 4 * dv.nbuckets + 4 * nwords + lbytes;
    } else {
        dv.dpitch = round_up(d, 4);
        for (int b = 0; b < 2; ++b)
            if (e == cudaSuccess) e = dev_alloc(ctx, &ctx->dbuf[b].dense, n * dv.dpitch);
        ctx->msg_bytes_per_worker = 4 * d;
    }
    ctx->cons_blocks = (d + 255) / 256;
    if (e == cudaSuccess) e = dev_alloc(ctx, &ctx->cons_scratch, ctx->cons_blocks);
    if (e == cudaSuccess) e = dev_alloc(ctx, &ctx->cons_out, 1);
    if (e != cudaSuccess) {
        for (int i = 0; i < ctx->nallocs; ++i) cudaFree(ctx->allocs[i]);
        const bool oom = e == cudaErrorMemoryAllocation;
        delete ctx;
        return oom ? CHOCO_ERR_ALLOC : CHOCO_ERR_CUDA;
    }
    *out = ctx;
    return CHOCO_OK;
}

int choco_destroy(choco_ctx* ctx)
{
    if (!ctx) return CHOCO_ERR_INVALID_ARG;
    cudaDeviceSynchronize();
    for (int i = 0; i < ctx->ngraphs; ++i)
        if (ctx->graphs[i].exec) cudaGraphExecDestroy(ctx->graphs[i].exec);
    if (ctx->hot_l2) { cudaCtxResetPersistingL2Cache(); cudaGetLastError(); }
    for (int i = 0; i < ctx->nallocs; ++i) cudaFree(ctx->allocs[i]);
    for (int i = 0; i < 4; ++i)
        if (ctx->stage[i]) cudaFree(ctx->stage[i]);
    if (ctx->host_in) {
        cudaStreamDestroy(ctx->host_in);
        cudaStreamDestroy(ctx->host_out);
        for (cudaEvent_t ev : ctx->host_ev)
            if (ev) cudaEventDestroy(ev);
    }
    if (ctx->prof_ev) {
        for (int i = 0; i < 2 * ctx->prof_cap; ++i) cudaEventDestroy(ctx->prof_ev[i]);
        delete[] ctx->prof_ev;
    }
    delete ctx;
    return CHOCO_OK;
}

int choco_gossip_step(choco_ctx* ctx, float* X, float* Xhat, float* S, float gamma, void* stream)
{
    return run_step(ctx, X, Xhat, S, nullptr, nullptr, 0.f, gamma, 0.f, 0.f, stream);
}

int choco_sgd_step(choco_ctx* ctx, float* X, float* Xhat, float* S, const float* G, float eta,
                   float gamma, void* stream)
{
    if (!G) return CHOCO_ERR_INVALID_ARG;
    return run_step(ctx, X, Xhat, S, G, nullptr, eta, gamma, 0.f, 0.f, stream);
}

int choco_sgd_momentum_step(choco_ctx* ctx, float* X, float* Xhat, float* S, const float* G,
                            float* M, float eta, float gamma, float lambda, float beta,
                            void* stream)
{
    if (!G || !M) return CHOCO_ERR_INVALID_ARG;
    return run_step(ctx, X, Xhat, S, G, M, eta, gamma, lambda, beta, stream);
}

int choco_sgd_step_host(choco_ctx* ctx, float* X, float* Xhat, float* S, const float* G,
                        float eta, float gamma, void* stream)
{
    if (!ctx || !X || !Xhat || !S) return CHOCO_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const int n = ctx->dv.n;
    const size_t row_bytes = (size_t)ctx->dv.ld * sizeof(float);
    const size_t bytes = (size_t)n * row_bytes;
    for (int i = 0; i < 4; ++i)
        if (!ctx->stage[i]) {
            cudaError_t e = cudaMalloc((void**)&ctx->stage[i], bytes);
            if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return CHOCO_ERR_ALLOC; }
        }
    if (!ctx->host_in) {
        cudaError_t e = cudaStreamCreateWithFlags(&ctx->host_in, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->host_out, cudaStreamNonBlocking);
        for (cudaEvent_t& ev : ctx->host_ev)
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
    }
    // Uploads on one stream, downloads on another, kernels on the caller's: the messages need all
    // of X and X^, but a row's update needs only its own s and g, and its results can leave while
    // later rows are still being uploaded and updated (the link carries both directions at once).
    cudaEvent_t fork = ctx->host_ev[0], xh_in = ctx->host_ev[1], join = ctx->host_ev[2];
    cudaEvent_t* ready = ctx->host_ev + 3;
    cudaEvent_t* done = ready + kHostChunks;
    RowChunks chunks;
    chunks.rows_per_chunk = (n + kHostChunks - 1) / kHostChunks;
    chunks.count = (n + chunks.rows_per_chunk - 1) / chunks.rows_per_chunk;
    chunks.ready = ready;
    chunks.done = done;
    auto rows_of = [&](int c, size_t* off, size_t* len) {
        const int r0 = c * chunks.rows_per_chunk, cnt = std::min(chunks.rows_per_chunk, n - r0);
        *off = (size_t)r0 * (size_t)ctx->dv.ld; // in floats
        *len = (size_t)cnt * row_bytes;          // in bytes
    };
    cudaError_t e = cudaEventRecord(fork, st);   // what the caller enqueued before comes first
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->host_in, fork, 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->host_out, fork, 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->stage[0], X, bytes, cudaMemcpyHostToDevice, ctx->host_in);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->stage[1], Xhat, bytes, cudaMemcpyHostToDevice, ctx->host_in);
    if (e == cudaSuccess) e = cudaEventRecord(xh_in, ctx->host_in);
    for (int c = 0; c < chunks.count && e == cudaSuccess; ++c) {
        size_t off, len;
        rows_of(c, &off, &len);
        e = cudaMemcpyAsync(ctx->stage[2] + off, S + off, len, cudaMemcpyHostToDevice, ctx->host_in);
        if (e == cudaSuccess && G) e = cudaMemcpyAsync(ctx->stage[3] + off, G + off, len, cudaMemcpyHostToDevice, ctx->host_in);
        if (e == cudaSuccess) e = cudaEventRecord(ready[c], ctx->host_in);
    }
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, xh_in, 0);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    ctx->prepared = false; // the staging contents changed
    const bool carry = ctx->carry_enabled;
    ctx->carry_enabled = false; // the next call overwrites the staging buffers anyway
    const int rc = step_body(ctx, ctx->stage[0], ctx->stage[1], ctx->stage[2], G ? ctx->stage[3] : nullptr,
                            nullptr, eta, gamma, 0.f, 0.f, stream, &chunks);
    ctx->carry_enabled = carry;
    if (rc) {
        cudaDeviceSynchronize(); // the side streams may still be copying
        return rc;
    }
    float* dst[3] = {X, Xhat, S};
    for (int c = 0; c < chunks.count && e == cudaSuccess; ++c) {
        size_t off, len;
        rows_of(c, &off, &len);
        e = cudaStreamWaitEvent(ctx->host_out, done[c], 0);
        for (int i = 0; i < 3 && e == cudaSuccess; ++i)
            e = cudaMemcpyAsync(dst[i] + off, ctx->stage[i] + off, len, cudaMemcpyDeviceToHost, ctx->host_out);
    }
    if (e == cudaSuccess) e = cudaEventRecord(join, ctx->host_out);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, join, 0);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) { cudaDeviceSynchronize(); return fail_cuda(ctx, e); }
    ctx->prepared = false;
    return check_device_timeouts(ctx, st);
}

int choco_invalidate(choco_ctx* ctx)
{
    if (!ctx) return CHOCO_ERR_INVALID_ARG;
    ctx->prepared = false;
    return CHOCO_OK;
}

int choco_set_carry(choco_ctx* ctx, int32_t enable)
{
    if (!ctx) return CHOCO_ERR_INVALID_ARG;
    ctx->carry_enabled = enable != 0;
    ctx->prepared = false;
    return CHOCO_OK;
}

int choco_set_rescue(choco_ctx* ctx, int32_t enable)
{
    if (!ctx) return CHOCO_ERR_INVALID_ARG;
    if (ctx->dv.kind != CHOCO_Q_TOPK) return enable ? CHOCO_ERR_UNSUPPORTED : CHOCO_OK;
    ctx->dv.rescue = enable ? 1 : 0;
    ctx->dv_epoch += 1;
    // the kernels a step enqueues change: no captured step stands for it any more
    for (int i = 0; i < ctx->ngraphs; ++i)
        if (ctx->graphs[i].exec) { cudaGraphExecDestroy(ctx->graphs[i].exec); }
    ctx->ngraphs = 0;
    return CHOCO_OK;
}

int choco_set_select_blocks(choco_ctx* ctx, int32_t blocks)
{
    if (!ctx || !(blocks == 1 || blocks == 2 || blocks == 4)) return CHOCO_ERR_INVALID_ARG;
    if (ctx->dv.kind != CHOCO_Q_TOPK && ctx->dv.kind != CHOCO_Q_RANDK) return CHOCO_ERR_UNSUPPORTED;
    ctx->dv.emit_cluster = blocks;
    ctx->dv.cand_slot = (ctx->dv.kind == CHOCO_Q_TOPK && blocks > 1) ? ctx->dv.cand_slot_alloc : 0u;
    ctx->prepared = false; // candidates collected by the last step lie in the other arrangement
    ctx->dv_epoch += 1;
    // the kernels a step enqueues change: no captured step stands for it any more
    for (int i = 0; i < ctx->ngraphs; ++i)
        if (ctx->graphs[i].exec) cudaGraphExecDestroy(ctx->graphs[i].exec);
    ctx->ngraphs = 0;
    return CHOCO_OK;
}

int choco_debug_set_candidate_slot(choco_ctx* ctx, int32_t slot)
{
    if (!ctx || slot < 1) return CHOCO_ERR_INVALID_ARG;
    if (ctx->dv.kind != CHOCO_Q_TOPK || ctx->dv.emit_cluster <= 1) return CHOCO_ERR_UNSUPPORTED;
    ctx->dv.cand_slot = (uint32_t)slot < ctx->dv.cand_slot_alloc ? (uint32_t)slot : ctx->dv.cand_slot_alloc;
    ctx->prepared = false;
    ctx->dv_epoch += 1;
    for (int i = 0; i < ctx->ngraphs; ++i)
        if (ctx->graphs[i].exec) cudaGraphExecDestroy(ctx->graphs[i].exec);
    ctx->ngraphs = 0;
    return CHOCO_OK;
}

int choco_set_nesterov(choco_ctx* ctx, int32_t enable)
{
    if (!ctx) return CHOCO_ERR_INVALID_ARG;
    ctx->dv.nesterov = enable ? 1 : 0;
    ctx->dv_epoch += 1;
    // captured steps hold the old parameter block
    for (int i = 0; i < ctx->ngraphs; ++i)
        if (ctx->graphs[i].exec) cudaGraphExecDestroy(ctx->graphs[i].exec);
    ctx->ngraphs = 0;
    return CHOCO_OK;
}

int choco_set_graphs(choco_ctx* ctx, int32_t enable)
{
    if (!ctx) return CHOCO_ERR_INVALID_ARG;
    if (enable && !ctx->graphs_ok && (ctx->dv.kind == CHOCO_Q_QSGD || ctx->dv.kind == CHOCO_Q_RANDK) &&
        !ctx->dev_step) {
        // from now on the kernels read the step number from device memory: bring it up to date
        const unsigned long long v = ctx->step;
        cudaError_t e = cudaDeviceSynchronize();
        if (e == cudaSuccess) e = cudaMemcpy(ctx->step_dev, &v, sizeof(v), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
        ctx->dev_step = true;
    }
    ctx->graphs_ok = enable != 0;
    return CHOCO_OK;
}

int choco_get_step(const choco_ctx* ctx, uint64_t* t)
{
    if (!ctx || !t) return CHOCO_ERR_INVALID_ARG;
    *t = ctx->step;
    return CHOCO_OK;
}

int choco_set_step(choco_ctx* ctx, uint64_t t)
{
    if (!ctx) return CHOCO_ERR_INVALID_ARG;
    if (t >> 56) return CHOCO_ERR_TOO_LARGE;
    if (ctx->dev_step) {
        const unsigned long long v = t;
        cudaError_t e = cudaDeviceSynchronize();
        if (e == cudaSuccess) e = cudaMemcpy(ctx->step_dev, &v, sizeof(v), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
    }
    ctx->step = t;
    ctx->prepared = false;
    return CHOCO_OK;
}

int choco_message_bytes(const choco_ctx* ctx, int64_t* per_worker, int64_t* total)
{
    if (!ctx) return CHOCO_ERR_INVALID_ARG;
    if (per_worker) *per_worker = ctx->msg_bytes_per_worker;
    if (total) *total = ctx->msg_bytes_per_worker * ctx->dv.n;
    return CHOCO_OK;
}

int choco_get_message(const choco_ctx* ctx, int32_t worker, int32_t plane, const void** dev_ptr,
                      int64_t* nbytes)
{
    if (!ctx || !dev_ptr || !nbytes || worker < 0 || worker >= ctx->dv.n || plane < 0 || plane > 2)
        return CHOCO_ERR_INVALID_ARG;
    Dev dv = ctx->dv;
    {
        const choco_ctx::DenseBuf& last = ctx->dbuf[ctx->msg_last];
        dv.msg_bits = last.bits; dv.msg_scale = last.scale; dv.msg_norms = last.norms;
        dv.msg_levels = last.levels; dv.msg_dense = last.dense;
    }
    const int64_t nwords = (dv.d + 31) / 32;
    *dev_ptr = nullptr;
    *nbytes = 0;
    switch (dv.kind) {
    case CHOCO_Q_TOPK:
    case CHOCO_Q_RANDK:
        if (plane == 0) { *dev_ptr = dv.msg_idx + worker * dv.kpitch; *nbytes = 4 * dv.k; }
        if (plane == 1) { *dev_ptr = dv.msg_val + worker * dv.kpitch; *nbytes = 4 * dv.k; }
        break;
    case CHOCO_Q_SIGN:
        if (plane == 0) { *dev_ptr = dv.msg_bits + worker * dv.wpitch; *nbytes = 4 * nwords; }
        if (plane == 1) { *dev_ptr = dv.msg_scale + worker; *nbytes = 4; }
        break;
    case CHOCO_Q_QSGD:
        if (plane == 0) { *dev_ptr = dv.msg_bits + worker * dv.wpitch; *nbytes = 4 * nwords; }
        if (plane == 1) { *dev_ptr = dv.msg_norms + worker * dv.npitch; *nbytes = 4 * dv.nbuckets; }
        if (plane == 2) { *dev_ptr = dv.msg_levels + worker * dv.lpitch; *nbytes = (dv.d * dv.wbits + 7) / 8; }
        break;
    default:
        if (plane == 1) { *dev_ptr = dv.msg_dense + worker * dv.dpitch; *nbytes = 4 * dv.d; }
        break;
    }
    return CHOCO_OK;
}

int choco_read_message(choco_ctx* ctx, int32_t worker, int32_t plane, void* host_dst,
                       int64_t capacity, int64_t* nbytes, void* stream)
{
    if (!host_dst || capacity < 0) return CHOCO_ERR_INVALID_ARG;
    const void* src = nullptr;
    const int rc = choco_get_message(ctx, worker, plane, &src, nbytes);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = cudaStreamSynchronize(st);
    if (e == cudaSuccess && *nbytes > 0 && *nbytes <= capacity)
        e = cudaMemcpy(host_dst, src, (size_t)*nbytes, cudaMemcpyDeviceToHost);
    return e == cudaSuccess ? check_device_timeouts(ctx, st) : fail_cuda(ctx, e);
}

int choco_consensus_error(choco_ctx* ctx, const float* X, double* out, void* stream)
{
    if (!ctx || !X || !out) return CHOCO_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = launch_consensus(X, ctx->dv.n, ctx->dv.d, ctx->dv.ld, ctx->cons_scratch,
                                     ctx->cons_blocks, ctx->cons_out, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out, ctx->cons_out, sizeof(double), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    return e == cudaSuccess ? check_device_timeouts(ctx, st) : fail_cuda(ctx, e);
}

int choco_get_stats(choco_ctx* ctx, choco_stats* out, void* stream)
{
    if (!ctx || !out) return CHOCO_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    Stats h;
    cudaError_t e = cudaMemcpyAsync(&h, ctx->dv.stats, sizeof(h), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    out->steps = ctx->steps_enqueued;
    out->prepared_rows = h.prepared_rows;
    out->recompressed_rows = h.recompressed_rows;
    out->exact_rows = h.exact_rows;
    out->device_timeouts = h.timeouts;
    out->kernel_launches = ctx->launches;
    out->graph_replays = ctx->graph_replays;
    out->rescued_rows = h.rescued_rows;
    if (h.timeouts != 0) ctx->timed_out = true;
    return ctx->timed_out ? CHOCO_ERR_TIMEOUT : CHOCO_OK;
}

int choco_debug_set_wait_polls(choco_ctx* ctx, uint32_t polls)
{
    if (!ctx) return CHOCO_ERR_INVALID_ARG;
    ctx->dv.wait_polls = polls > kSpinLimit ? kSpinLimit : polls;
    ctx->dv_epoch += 1;
    // the bound is a kernel argument: no captured step stands for it any more
    for (int i = 0; i < ctx->ngraphs; ++i)
        if (ctx->graphs[i].exec) cudaGraphExecDestroy(ctx->graphs[i].exec);
    ctx->ngraphs = 0;
    return CHOCO_OK;
}

int choco_profile_enable(choco_ctx* ctx, int32_t max_steps)
{
    if (!ctx || max_steps < 1 || max_steps > 100000) return CHOCO_ERR_INVALID_ARG;
    if (ctx->prof_ev) {
        for (int i = 0; i < 2 * ctx->prof_cap; ++i) cudaEventDestroy(ctx->prof_ev[i]);
        delete[] ctx->prof_ev;
        ctx->prof_ev = nullptr;
    }
    ctx->prof_ev = new (std::nothrow) cudaEvent_t[2 * (size_t)max_steps];
    if (!ctx->prof_ev) return CHOCO_ERR_ALLOC;
    ctx->prof_cap = 0;
    ctx->prof_n = 0;
    for (int i = 0; i < 2 * max_steps; ++i) {
        cudaError_t e = cudaEventCreate(&ctx->prof_ev[i]);
        if (e != cudaSuccess) {
            for (int j = 0; j < i; ++j) cudaEventDestroy(ctx->prof_ev[j]);
            delete[] ctx->prof_ev;
            ctx->prof_ev = nullptr;
            return fail_cuda(ctx, e);
        }
    }
    ctx->prof_cap = max_steps;
    return CHOCO_OK;
}

int choco_profile_set_stride(choco_ctx* ctx, int32_t stride)
{
    if (!ctx || stride < 1) return CHOCO_ERR_INVALID_ARG;
    ctx->prof_stride = stride;
    return CHOCO_OK;
}

int choco_profile_read(choco_ctx* ctx, int32_t* steps_recorded, double* update_ms_total,
                       void* stream)
{
    if (!ctx || !steps_recorded || !update_ms_total) return CHOCO_ERR_INVALID_ARG;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    double total = 0.0;
    for (int i = 0; e == cudaSuccess && i < ctx->prof_n; ++i) {
        float ms = 0.f;
        e = cudaEventElapsedTime(&ms, ctx->prof_ev[2 * i], ctx->prof_ev[2 * i + 1]);
        total += (double)ms;
    }
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    *steps_recorded = ctx->prof_n;
    *update_ms_total = total;
    ctx->prof_n = 0;
    return CHOCO_OK;
}

const char* choco_strerror(int code)
{
    switch (code) {
    case CHOCO_OK: return "ok";
    case CHOCO_ERR_INVALID_ARG: return "invalid argument";
    case CHOCO_ERR_BAD_W: return "mixing matrix violates Assumption 1 or the CSR rules";
    case CHOCO_ERR_ALLOC: return "allocation failed";
    case CHOCO_ERR_CUDA: return "CUDA runtime error";
    case CHOCO_ERR_MISALIGNED: return "pointer not 4-byte aligned";
    case CHOCO_ERR_UNSUPPORTED: return "unsupported configuration";
    case CHOCO_ERR_TOO_LARGE: return "size exceeds a documented limit";
    case CHOCO_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out; the state arrays are invalid";
    default: return "unknown error";
    }
}

int choco_last_cuda_error(const choco_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }

} // extern "C"
