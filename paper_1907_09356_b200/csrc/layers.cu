// Per-layer compression (Section 5, "Setup": every compression scheme is applied to every
// layer separately): the flat parameter vector is cut into consecutive layers and each layer is
// its own vector for Q.  This file holds host code only.  A layered context owns one ordinary
// context per layer, with d = the layer's length and the shared row pitch; a step runs the
// layers' steps on column slices of the caller's arrays.  The layers are independent of each
// other, so their kernels are spread over a few internal streams that fork from and join the
// caller's stream.
//
// Many small layers make a step launch-bound (two or three launches per layer).  For top_a,
// scaled sign and gsgd_b with blocks the steady-state step of ALL layers is therefore enqueued
// as two or three launches whose blocks look their layer up in a table (combined_step below);
// the layers' contexts only lend their parameters and buffers, and their host-side bookkeeping
// is advanced by hand.  For the other operators the steady-state step is captured once into a
// CUDA graph per set of arguments (array pointers, step sizes, message-buffer parity) and
// replayed with one launch.  gsgd_b with one norm per layer and random_a key their generator
// with the step number, which a captured kernel argument would freeze: their contexts keep the
// step number in device memory and bump it there after every step.
#include <algorithm>
#include <cstring>
#include <new>
#include <utility>
#include <vector>

#include "common.cuh"
#include "internal.h"

namespace {

constexpr int kLayerStreams = 16;
constexpr size_t kMaxGraphs = 32; // cached step graphs per layered context (least recently used goes)

struct StepGraph {
    float *X, *Xhat, *S;
    const float* G;
    float* M;
    float eta, gamma, lambda, beta;
    uint64_t mode; // hash over the layers of (compression carried, message buffer in use)
    cudaGraphExec_t exec;
    uint64_t last_use;
};

// the host-side fields of a context that a step changes
struct HostState {
    uint64_t step, steps_enqueued;
    bool prepared;
    int msg_cur, msg_last;
    const float *last_x, *last_xhat;
    unsigned long long launches;
};

HostState save_state(const choco_ctx* c)
{
    return {c->step, c->steps_enqueued, c->prepared, c->msg_cur, c->msg_last, c->last_x, c->last_xhat, c->launches};
}

void restore_state(choco_ctx* c, const HostState& h)
{
    c->step = h.step; c->steps_enqueued = h.steps_enqueued; c->prepared = h.prepared;
    c->msg_cur = h.msg_cur; c->msg_last = h.msg_last; c->last_x = h.last_x; c->last_xhat = h.last_xhat;
    c->launches = h.launches;
}

} // namespace

struct choco_layers {
    int32_t n;
    int32_t n_layers;
    int64_t ld;
    std::vector<int64_t> off;      // n_layers + 1
    std::vector<choco_ctx*> ctx;   // one per layer
    // combined launches over all layers (top_a, scaled sign, gsgd_b with blocks)
    bool combine;                  // the operator has them
    choco::Dev* devs_dev[2];       // the layers' parameters, one copy per message-buffer parity
    int64_t* off_dev;
    uint64_t devs_epoch;           // sum of the contexts' parameter epochs the copies were made from
    uint32_t align_key;            // alignment of the state arrays the groups below were made for
    bool groups_valid;
    choco::LayerTable tiles_al, tiles_ua; // layers whose rows are 16-byte aligned / the others the kernels take
    choco::LayerTable rows;               // all of those, for the launches over rows
    choco::LayerTable rows_small, rows_large; // the same split by row length (top_a: two block sizes)
    std::vector<int32_t> grouped, rest;   // layers served by the combined launches / by their own context
    size_t emit_smem_small, emit_smem_large;
    uint64_t combined_steps;
    cudaStream_t side[kLayerStreams];
    cudaEvent_t fork;
    cudaEvent_t join[kLayerStreams];
    int nside;
    bool graphs_ok;                              // steady-state steps may be captured and replayed
    std::vector<StepGraph> graphs;
    std::vector<unsigned long long> launches_per_step; // per layer, in the captured steady state
    uint64_t use_clock;
    uint64_t replays;
};

namespace {

void free_groups(choco_layers* L)
{
    L->tiles_al.entries = L->tiles_ua.entries = L->rows.entries = 0;
    L->rows_small.entries = L->rows_large.entries = 0;
    L->groups_valid = false;
}

void destroy_layers(choco_layers* L)
{
    if (!L) return;
    cudaDeviceSynchronize();
    free_groups(L);
    for (int p = 0; p < 2; ++p)
        if (L->devs_dev[p]) cudaFree(L->devs_dev[p]);
    if (L->off_dev) cudaFree(L->off_dev);
    for (choco_ctx* c : L->ctx)
        if (c) choco_destroy(c);
    for (StepGraph& g : L->graphs)
        if (g.exec) cudaGraphExecDestroy(g.exec);
    for (int s = 0; s < L->nside; ++s) {
        if (L->side[s]) cudaStreamDestroy(L->side[s]);
        if (L->join[s]) cudaEventDestroy(L->join[s]);
    }
    if (L->fork) cudaEventDestroy(L->fork);
    delete L;
}

int eager_step(choco_layers* L, float* X, float* Xhat, float* S, const float* G, float* M, float eta,
               float gamma, float lambda, float beta, void* stream)
{
    cudaStream_t st = (cudaStream_t)stream;
    const bool fan = L->nside > 1 && L->n_layers > 1;
    if (fan) {
        if (cudaEventRecord(L->fork, st) != cudaSuccess) return CHOCO_ERR_CUDA;
        for (int s = 0; s < L->nside; ++s)
            if (cudaStreamWaitEvent(L->side[s], L->fork, 0) != cudaSuccess) return CHOCO_ERR_CUDA;
    }
    int rc = CHOCO_OK;
    for (int32_t l = 0; l < L->n_layers && rc == CHOCO_OK; ++l) {
        const int64_t o = L->off[l];
        void* lst = fan ? (void*)L->side[l % L->nside] : stream;
        if (M)
            rc = choco_sgd_momentum_step(L->ctx[l], X + o, Xhat + o, S + o, G + o, M + o, eta, gamma, lambda,
                                         beta, lst);
        else if (G)
            rc = choco_sgd_step(L->ctx[l], X + o, Xhat + o, S + o, G + o, eta, gamma, lst);
        else
            rc = choco_gossip_step(L->ctx[l], X + o, Xhat + o, S + o, gamma, lst);
    }
    if (fan) { // join even after an error so that the caller's stream stays ordered behind the layers
        for (int s = 0; s < L->nside; ++s) {
            if (cudaEventRecord(L->join[s], L->side[s]) != cudaSuccess) return CHOCO_ERR_CUDA;
            if (cudaStreamWaitEvent(st, L->join[s], 0) != cudaSuccess) return CHOCO_ERR_CUDA;
        }
    }
    return rc;
}

// A captured step can stand for the next one if every layer's step repeats; `mode` receives a
// hash of what selects the kernels and message buffers of the layers, part of a graph's key.
bool steady(const choco_layers* L, const float* X, const float* Xhat, uint64_t* mode)
{
    uint64_t h = 1469598103934665603ull;
    for (int32_t l = 0; l < L->n_layers; ++l) {
        uint64_t m = 0;
        if (!choco::step_repeats(L->ctx[l], X + L->off[l], Xhat + L->off[l], &m)) return false;
        h = (h ^ m) * 1099511628211ull;
    }
    *mode = h;
    return true;
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }
bool aligned8(const void* p) { return ((uintptr_t)p & 7u) == 0; }

// The device copies of the layers' parameters: layer l at parity p reads its messages from the
// layer's buffer p and writes the next ones to buffer p ^ 1 (dense operators).
int upload_devs(choco_layers* L)
{
    std::vector<choco::Dev> host((size_t)L->n_layers);
    for (int p = 0; p < 2; ++p) {
        for (int32_t l = 0; l < L->n_layers; ++l) {
            choco::Dev dv = L->ctx[l]->dv;
            const choco_ctx::DenseBuf &cur = L->ctx[l]->dbuf[p], &nxt = L->ctx[l]->dbuf[p ^ 1];
            dv.msg_bits = cur.bits; dv.msg_scale = cur.scale; dv.msg_norms = cur.norms;
            dv.msg_levels = cur.levels; dv.msg_dense = cur.dense;
            dv.nxt_bits = nxt.bits; dv.nxt_scale = nxt.scale; dv.nxt_norms = nxt.norms;
            dv.nxt_levels = nxt.levels; dv.nxt_dense = nxt.dense;
            host[(size_t)l] = dv;
        }
        if (cudaMemcpy(L->devs_dev[p], host.data(), sizeof(choco::Dev) * host.size(), cudaMemcpyHostToDevice) != cudaSuccess)
            return CHOCO_ERR_CUDA;
    }
    uint64_t epoch = 0;
    for (const choco_ctx* c : L->ctx) epoch += c->dv_epoch;
    L->devs_epoch = epoch;
    return CHOCO_OK;
}

// Sort the layers into the launches that can serve them, for state arrays of this alignment.
int make_groups(choco_layers* L, const float* X, const float* Xhat, const float* S, const float* G, const float* M)
{
    free_groups(L);
    L->grouped.clear();
    L->rest.clear();
    const bool sparse = L->ctx[0]->dv.kind == CHOCO_Q_TOPK;
    size_t emit_smem[2] = {0, 0};
    auto add = [](choco::LayerTable& t, int32_t l, int64_t off, int64_t dl, uint32_t blocks) {
        const int e = t.entries++;
        t.layer[e] = l;
        t.d[e] = (int32_t)dl;
        t.off[e] = off;
        t.first_block[e + 1] = t.first_block[e] + blocks;
    };
    L->tiles_al.first_block[0] = L->tiles_ua.first_block[0] = L->rows.first_block[0] = 0u;
    L->rows_small.first_block[0] = L->rows_large.first_block[0] = 0u;
    for (int32_t l = 0; l < L->n_layers; ++l) {
        const int64_t o = L->off[l], dl = L->off[l + 1] - L->off[l];
        const void* ptr[5] = {X + o, Xhat + o, S + o, G ? G + o : nullptr, M ? M + o : nullptr};
        bool a16 = L->ld % 4 == 0, a8 = L->ld % 2 == 0;
        for (const void* q : ptr) { a16 = a16 && aligned16(q); a8 = a8 && aligned8(q); }
        const bool al_ok = a16 && dl % 4 == 0;
        if (!sparse && !al_ok && !a8) { L->rest.push_back(l); continue; } // rows at odd elements: the layer's own context
        const uint32_t tiles = (uint32_t)((dl + choco::kTile - 1) / choco::kTile);
        add(al_ok ? L->tiles_al : L->tiles_ua, l, o, dl, tiles);
        add(L->rows, l, o, dl, (uint32_t)L->n);
        const int big = dl > choco::kSmallRow ? 1 : 0;
        add(big ? L->rows_large : L->rows_small, l, o, dl, (uint32_t)L->n);
        L->grouped.push_back(l);
        emit_smem[big] = std::max<size_t>(emit_smem[big], (size_t)L->ctx[l]->dv.emit_smem_bytes);
    }
    L->emit_smem_small = emit_smem[0];
    L->emit_smem_large = emit_smem[1];
    L->groups_valid = true;
    return CHOCO_OK;
}

uint32_t alignment_key(const choco_layers* L, const float* X, const float* Xhat, const float* S, const float* G,
                       const float* M)
{
    auto low = [](const void* q) { return (uint32_t)((uintptr_t)q & 15u); };
    return low(X) | (low(Xhat) << 4) | (low(S) << 8) | (low(G) << 12) | (low(M) << 16) | ((G ? 1u : 0u) << 20) |
           ((M ? 1u : 0u) << 21) | (1u << 31);
}

// Can this step be enqueued as the combined launches?  Every layer must be in the state that
// repeats: its compression prepared by the last step on these very arrays, no row rescue, no
// per-step events, and all layers at the same step and message-buffer parity.
bool combinable(const choco_layers* L, const float* X, const float* Xhat)
{
    if (!L->combine) return false;
    const choco_ctx* c0 = L->ctx[0];
    for (int32_t l = 0; l < L->n_layers; ++l) {
        const choco_ctx* c = L->ctx[l];
        if (c->timed_out || c->steps_enqueued == 0 || !c->carry_enabled || !c->prepared || c->dv.rescue) return false;
        if (c->dv.emit_cluster > 1) return false; // (the launch over all layers selects with one block per row)
        if (c->last_x != X + L->off[l] || c->last_xhat != Xhat + L->off[l]) return false;
        if (c->prof_ev && c->prof_n < c->prof_cap) return false;
        if (c->step != c0->step || c->msg_cur != c0->msg_cur) return false;
    }
    return true;
}

int combined_step(choco_layers* L, float* X, float* Xhat, float* S, const float* G, float* M, float eta, float gamma,
                  float lambda, float beta, void* stream)
{
    using namespace choco;
    cudaStream_t st = (cudaStream_t)stream;
    uint64_t epoch = 0;
    for (const choco_ctx* c : L->ctx) epoch += c->dv_epoch;
    if (epoch != L->devs_epoch) {
        cudaDeviceSynchronize(); // no kernel may still be reading the copies (rare: a setter was called)
        const int rc = upload_devs(L);
        if (rc != CHOCO_OK) return rc;
    }
    const uint32_t key = alignment_key(L, X, Xhat, S, G, M);
    if (!L->groups_valid || key != L->align_key) {
        const int rc = make_groups(L, X, Xhat, S, G, M);
        if (rc != CHOCO_OK) return rc;
        L->align_key = key;
    }
    choco_ctx* c0 = L->ctx[0];
    const Dev& proto = c0->dv;
    unsigned long long launches = 0;
    StepArgs a;
    a.X = X; a.Xhat = Xhat; a.S = S; a.G = G; a.M = M;
    a.eta = eta; a.gamma = gamma; a.lambda = lambda; a.beta = beta;
    a.step = c0->step;
    a.step_dev = nullptr;
    a.vec = false;
    a.launches = &launches;
    LayerSet ls;
    ls.devs = L->devs_dev[c0->msg_cur];
    ls.ld = L->ld;
    cudaError_t e = cudaSuccess;
    if (proto.kind == CHOCO_Q_TOPK) {
        if (L->rows_small.entries) {
            e = launch_select_emit_layers(L->rows_small, ls, L->n, L->emit_smem_small, true, a, st);
            launches += 1;
        }
        if (e == cudaSuccess && L->rows_large.entries) {
            e = launch_select_emit_layers(L->rows_large, ls, L->n, L->emit_smem_large, false, a, st);
            launches += 1;
        }
        for (const auto& g : {std::make_pair(&L->tiles_al, true), std::make_pair(&L->tiles_ua, false)}) {
            if (e != cudaSuccess || g.first->entries == 0) continue;
            e = launch_update_bulk_layers(*g.first, ls, L->n, a, g.second, st);
            launches += 1;
        }
    } else {
        for (const auto& g : {std::make_pair(&L->tiles_al, true), std::make_pair(&L->tiles_ua, false)}) {
            if (e != cudaSuccess || g.first->entries == 0) continue;
            e = launch_update_dense_bulk_layers(proto, *g.first, ls, a, g.second, st);
            launches += 1;
        }
        if (e == cudaSuccess && proto.kind == CHOCO_Q_SIGN && L->rows.entries) {
            e = launch_sign_scale_layers(L->rows, ls, L->n, st);
            launches += 1;
        }
    }
    if (e != cudaSuccess) { c0->last_cuda_error = (int)e; return CHOCO_ERR_CUDA; }
    // the layers the combined kernels do not take (rows that start at odd elements) run their own step
    int rc = CHOCO_OK;
    for (int32_t l : L->rest) {
        const int64_t o = L->off[l];
        if (M) rc = choco_sgd_momentum_step(L->ctx[l], X + o, Xhat + o, S + o, G + o, M + o, eta, gamma, lambda, beta, stream);
        else if (G) rc = choco_sgd_step(L->ctx[l], X + o, Xhat + o, S + o, G + o, eta, gamma, stream);
        else rc = choco_gossip_step(L->ctx[l], X + o, Xhat + o, S + o, gamma, stream);
        if (rc != CHOCO_OK) return rc;
    }
    for (int32_t l : L->grouped) choco::advance_after_replay(L->ctx[l], 0);
    if (!L->grouped.empty()) L->ctx[L->grouped[0]]->launches += launches;
    L->combined_steps += 1;
    return CHOCO_OK;
}

int layers_step(choco_layers* L, float* X, float* Xhat, float* S, const float* G, float* M, float eta,
                float gamma, float lambda, float beta, void* stream)
{
    if (!L || !X || !Xhat || !S) return CHOCO_ERR_INVALID_ARG;
    for (const choco_ctx* c : L->ctx)
        if (c->timed_out) return CHOCO_ERR_TIMEOUT;
    if (combinable(L, X, Xhat)) return combined_step(L, X, Xhat, S, G, M, eta, gamma, lambda, beta, stream);
    cudaStream_t st = (cudaStream_t)stream;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    uint64_t mode = 0;
    if (!L->graphs_ok || L->n_layers < 2 || cudaStreamIsCapturing(st, &cap) != cudaSuccess ||
        cap != cudaStreamCaptureStatusNone || !steady(L, X, Xhat, &mode))
        return eager_step(L, X, Xhat, S, G, M, eta, gamma, lambda, beta, stream);

    // A set of arguments is captured the second time it is seen: a caller that passes new
    // arrays every step (a fresh gradient tensor, say) never pays for a capture.
    StepGraph* hit = nullptr;
    for (StepGraph& g : L->graphs)
        if (g.X == X && g.Xhat == Xhat && g.S == S && g.G == G && g.M == M && g.eta == eta && g.gamma == gamma &&
            g.lambda == lambda && g.beta == beta && g.mode == mode) { hit = &g; break; }
    if (hit && hit->exec) {
        if (cudaGraphLaunch(hit->exec, st) != cudaSuccess) return CHOCO_ERR_CUDA;
        hit->last_use = ++L->use_clock;
        for (int32_t l = 0; l < L->n_layers; ++l) choco::advance_after_replay(L->ctx[l], L->launches_per_step[l]);
        L->replays += 1;
        return CHOCO_OK;
    }
    if (!hit) { // first sighting: remember it, enqueue kernel by kernel
        const StepGraph g = {X, Xhat, S, G, M, eta, gamma, lambda, beta, mode, nullptr, ++L->use_clock};
        if (L->graphs.size() < kMaxGraphs) {
            L->graphs.push_back(g);
        } else {
            size_t oldest = 0;
            for (size_t i = 1; i < L->graphs.size(); ++i)
                if (L->graphs[i].last_use < L->graphs[oldest].last_use) oldest = i;
            if (L->graphs[oldest].exec) cudaGraphExecDestroy(L->graphs[oldest].exec);
            L->graphs[oldest] = g;
        }
        return eager_step(L, X, Xhat, S, G, M, eta, gamma, lambda, beta, stream);
    }

    // capture this step; on any failure put the host state back and run it eagerly
    std::vector<HostState> before(L->n_layers);
    for (int32_t l = 0; l < L->n_layers; ++l) before[l] = save_state(L->ctx[l]);
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    bool ok = cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) == cudaSuccess;
    if (ok) {
        const int rc = eager_step(L, X, Xhat, S, G, M, eta, gamma, lambda, beta, stream);
        const cudaError_t e = cudaStreamEndCapture(st, &graph);
        ok = rc == CHOCO_OK && e == cudaSuccess && graph != nullptr;
    }
    if (ok) ok = cudaGraphInstantiate(&exec, graph, 0) == cudaSuccess;
    if (graph) cudaGraphDestroy(graph);
    if (ok) ok = cudaGraphLaunch(exec, st) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        if (exec) cudaGraphExecDestroy(exec);
        for (int32_t l = 0; l < L->n_layers; ++l) restore_state(L->ctx[l], before[l]);
        L->graphs_ok = false; // do not try again on this context
        return eager_step(L, X, Xhat, S, G, M, eta, gamma, lambda, beta, stream);
    }
    L->launches_per_step.resize(L->n_layers);
    for (int32_t l = 0; l < L->n_layers; ++l) L->launches_per_step[l] = L->ctx[l]->launches - before[l].launches;
    hit->exec = exec;
    hit->last_use = ++L->use_clock;
    return CHOCO_OK;
}

} // namespace

extern "C" {

int choco_layers_init(choco_layers** out, int32_t n, int32_t n_layers, const int64_t* layer_off, int64_t ld,
                      const int32_t* w_row_ptr, const int32_t* w_col, const float* w_val, const choco_params* p,
                      int64_t a_num, int64_t a_den, uint64_t seed)
{
    if (!out || !layer_off || !p) return CHOCO_ERR_INVALID_ARG;
    *out = nullptr;
    if (n_layers < 1 || layer_off[0] != 0) return CHOCO_ERR_INVALID_ARG;
    for (int32_t l = 0; l < n_layers; ++l)
        if (layer_off[l + 1] <= layer_off[l]) return CHOCO_ERR_INVALID_ARG;
    if (ld < layer_off[n_layers]) return CHOCO_ERR_INVALID_ARG;
    const bool sparse = p->kind == CHOCO_Q_TOPK || p->kind == CHOCO_Q_RANDK;
    if (sparse && (a_num < 1 || a_den < a_num)) return CHOCO_ERR_INVALID_ARG;

    choco_layers* L = new (std::nothrow) choco_layers();
    if (!L) return CHOCO_ERR_ALLOC;
    L->n = n; L->n_layers = n_layers; L->ld = ld;
    L->off.assign(layer_off, layer_off + n_layers + 1);
    L->ctx.assign(n_layers, nullptr);
    L->nside = 0; L->fork = nullptr;
    L->graphs_ok = true;
    L->use_clock = 0; L->replays = 0;
    // Combined launches pay where a step is bound by its launches: few blocks per layer.  Their
    // kernels read the layer's parameters from shared instead of constant memory, which costs
    // large layers more than the saved launches bring (measured on 161 layers of 25.6 M
    // coordinates in all: 14 - 20 % slower than a launch per layer).
    int64_t total_blocks = 0;
    for (int32_t l = 0; l < n_layers; ++l)
        total_blocks += (layer_off[l + 1] - layer_off[l] + choco::kTile - 1) / choco::kTile * n;
    L->combine = n_layers <= choco::kMaxComboLayers && total_blocks <= 32768 &&
                 (p->kind == CHOCO_Q_TOPK || p->kind == CHOCO_Q_SIGN || (p->kind == CHOCO_Q_QSGD && p->bucket > 0));
    L->devs_dev[0] = L->devs_dev[1] = nullptr;
    L->off_dev = nullptr;
    L->devs_epoch = ~0ull;
    L->align_key = 0;
    L->groups_valid = false;
    L->tiles_al.entries = L->tiles_ua.entries = L->rows.entries = 0;
    L->rows_small.entries = L->rows_large.entries = 0;
    L->emit_smem_small = L->emit_smem_large = 0;
    L->combined_steps = 0;
    std::memset(L->side, 0, sizeof(L->side));
    std::memset(L->join, 0, sizeof(L->join));
    for (int32_t l = 0; l < n_layers; ++l) {
        const int64_t dl = layer_off[l + 1] - layer_off[l];
        choco_params pl = *p;
        if (sparse) {
            // floor(a d_l) in integers, but never an empty message
            const int64_t k = (int64_t)(((__int128)dl * a_num) / a_den);
            pl.k = k < 1 ? 1 : k;
        }
        const int rc = choco_init(&L->ctx[l], n, dl, ld, w_row_ptr, w_col, w_val, &pl, seed + (uint64_t)l);
        if (rc != CHOCO_OK) { destroy_layers(L); return rc; }
        // gsgd_b and random_a key their generator with the step number: these contexts keep it
        // in device memory, where a replayed graph finds the current value
        // (operators whose steady-state step is enqueued as combined launches are never captured)
        L->ctx[l]->dev_step = !L->combine && (p->kind == CHOCO_Q_QSGD || p->kind == CHOCO_Q_RANDK);
        L->ctx[l]->graphs_ok = false; // the layered step is captured as a whole, not layer by layer
    }
    if (L->combine) {
        L->graphs_ok = false; // steady-state steps are a few launches already
        bool okc = cudaMalloc((void**)&L->devs_dev[0], sizeof(choco::Dev) * (size_t)n_layers) == cudaSuccess &&
                   cudaMalloc((void**)&L->devs_dev[1], sizeof(choco::Dev) * (size_t)n_layers) == cudaSuccess &&
                   true;
        if (!okc) { destroy_layers(L); return CHOCO_ERR_ALLOC; }
    }
    bool ok = cudaEventCreateWithFlags(&L->fork, cudaEventDisableTiming) == cudaSuccess;
    for (int s = 0; s < kLayerStreams && ok; ++s) {
        ok = cudaStreamCreateWithFlags(&L->side[s], cudaStreamNonBlocking) == cudaSuccess &&
             cudaEventCreateWithFlags(&L->join[s], cudaEventDisableTiming) == cudaSuccess;
        L->nside = s + 1;
    }
    if (!ok) { destroy_layers(L); return CHOCO_ERR_CUDA; }
    *out = L;
    return CHOCO_OK;
}

int choco_layers_destroy(choco_layers* L)
{
    destroy_layers(L);
    return CHOCO_OK;
}

int choco_layers_gossip_step(choco_layers* L, float* X, float* Xhat, float* S, float gamma, void* stream)
{
    return layers_step(L, X, Xhat, S, nullptr, nullptr, 0.f, gamma, 0.f, 0.f, stream);
}

int choco_layers_sgd_step(choco_layers* L, float* X, float* Xhat, float* S, const float* G, float eta,
                          float gamma, void* stream)
{
    if (!G) return CHOCO_ERR_INVALID_ARG;
    return layers_step(L, X, Xhat, S, G, nullptr, eta, gamma, 0.f, 0.f, stream);
}

int choco_layers_sgd_momentum_step(choco_layers* L, float* X, float* Xhat, float* S, const float* G, float* M,
                                   float eta, float gamma, float lambda, float beta, void* stream)
{
    if (!G || !M) return CHOCO_ERR_INVALID_ARG;
    return layers_step(L, X, Xhat, S, G, M, eta, gamma, lambda, beta, stream);
}

int choco_layers_message_bytes(const choco_layers* L, int64_t* per_worker, int64_t* total)
{
    if (!L) return CHOCO_ERR_INVALID_ARG;
    int64_t pw = 0;
    for (choco_ctx* c : L->ctx) {
        int64_t a = 0, b = 0;
        const int rc = choco_message_bytes(c, &a, &b);
        if (rc != CHOCO_OK) return rc;
        pw += a;
    }
    if (per_worker) *per_worker = pw;
    if (total) *total = pw * L->n;
    return CHOCO_OK;
}

int choco_layers_get_layer(const choco_layers* L, int32_t layer, choco_ctx** ctx, int64_t* offset, int64_t* length)
{
    if (!L || layer < 0 || layer >= L->n_layers) return CHOCO_ERR_INVALID_ARG;
    if (ctx) *ctx = L->ctx[layer];
    if (offset) *offset = L->off[layer];
    if (length) *length = L->off[layer + 1] - L->off[layer];
    return CHOCO_OK;
}

int choco_layers_set_graphs(choco_layers* L, int32_t enable, uint64_t* replays)
{
    if (!L) return CHOCO_ERR_INVALID_ARG;
    if (replays) *replays = L->replays;
    if (enable >= 0) L->graphs_ok = enable != 0;
    return CHOCO_OK;
}

int choco_layers_combined_steps(const choco_layers* L, uint64_t* steps)
{
    if (!L || !steps) return CHOCO_ERR_INVALID_ARG;
    *steps = L->combined_steps;
    return CHOCO_OK;
}

int choco_layers_invalidate(choco_layers* L)
{
    if (!L) return CHOCO_ERR_INVALID_ARG;
    for (choco_ctx* c : L->ctx) choco_invalidate(c);
    return CHOCO_OK;
}

int choco_layers_set_step(choco_layers* L, uint64_t t)
{
    if (!L) return CHOCO_ERR_INVALID_ARG;
    for (choco_ctx* c : L->ctx) {
        const int rc = choco_set_step(c, t);
        if (rc != CHOCO_OK) return rc;
    }
    return CHOCO_OK;
}

int choco_layers_set_nesterov(choco_layers* L, int32_t enable)
{
    if (!L) return CHOCO_ERR_INVALID_ARG;
    for (choco_ctx* c : L->ctx) {
        const int rc = choco_set_nesterov(c, enable); // (bumps the parameter epoch: the copies are uploaded again)
        if (rc != CHOCO_OK) return rc;
    }
    // captured steps hold the old parameter blocks
    for (StepGraph& g : L->graphs)
        if (g.exec) cudaGraphExecDestroy(g.exec);
    L->graphs.clear();
    return CHOCO_OK;
}

} // extern "C"
