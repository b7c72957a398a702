// Internal layout of a libchoco context and the launchers of its kernels.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/choco.h"

namespace choco {

// Row flags of the selection pipeline (top-k, random-k).
constexpr uint32_t kRowExact = 1u;    // candidates unusable: run the exact one-block selection
constexpr uint32_t kRowRescue = 2u;   // candidates unusable: collect afresh with grid-wide kernels
constexpr uint32_t kRowRefine = 4u;   // the first digit's bin is too full: resolve the next 11 bits
constexpr int64_t kRescueMinD = (int64_t)1 << 22; // rows this long are rescued rather than selected by one block

constexpr uint32_t kSpinLimit = 1u << 22;   // polls a kernel spends on a wait before it gives up

constexpr int64_t kEmitSmemBudget = 200 * 1024; // dynamic shared memory the emit kernel may use
constexpr int kSmallRow = 4096;       // rows up to this length are selected by small blocks, several per SM
constexpr int kHistBins = 2048;       // first radix digit: top 11 bits of the ordering key

struct Stats {
    unsigned long long prepared_rows;
    unsigned long long recompressed_rows;
    unsigned long long exact_rows;
    unsigned long long timeouts;   // bounded device waits that ran out
    unsigned long long rescued_rows; // rows whose candidates were collected afresh after a miss
};

// A range of device memory that a launch asks the L2 cache to keep resident.
struct HotRange {
    void* base;
    size_t bytes;
    float ratio;
};

// Everything the kernels need; passed by value.
struct Dev {
    int32_t n;
    int32_t kind;
    int64_t d;
    int64_t ld;
    int64_t ntiles;              // ceil(d / kTile): tiles of the sparse path
    int64_t nspans;              // ceil(d / kSpan): blocks per row of the dense kernels
    int64_t nchunks;             // ceil(d / 1024)
    // W (CSR)
    const int32_t* row_ptr;
    const int32_t* col;
    const float* wval;
    // reader-oriented view of the messages (sparse Q): for worker i, tile t and position r in
    // i's CSR row, rec[(i * ntiles + t) * maxdeg + r] = {j, first entry of j's message in the
    // tile, number of entries, bits of w_ij}; unused positions keep a zero count
    int32_t maxdeg;              // longest CSR row (diagonal included)
    const int32_t* rd_pos;       // [nnz] for entry (j, i): position of j in row i
    const float* rd_w;           // [nnz] for entry (j, i): w_ij as row i stores it
    uint4* rec;                  // [n, ntiles, maxdeg]
    // generator
    uint64_t seed;
    uint32_t round_key[10][2];   // Philox4x32-10 key schedule of `seed`: key + r * (0x9E3779B9, 0xBB67AE85)
    // sparse messages: idx / val [n, kpitch], tile_ptr [n, ntiles + 1]
    int64_t k;
    int64_t kpitch;
    uint32_t* msg_idx;
    float* msg_val;
    uint32_t* tile_ptr;
    // selection workspace
    int32_t rescue;              // top-k: a row that misses is re-collected by grid-wide kernels
    int64_t cap;                 // candidate capacity per row
    uint32_t* hist;              // [n, kHistBins]
    uint32_t* row_lo;            // [n] lower bound of the ordering key for candidates
    uint32_t* row_count;         // [n] candidates collected
    uint32_t* row_aim;           // [n] rank the next bound aims at, in units of k / 256
    uint32_t* row_flags;         // [n]
    uint32_t* row_above;         // [n] keys above the first digit's bin (while a row is refined)
    uint32_t* cand_idx;          // [n, cand_pitch]
    uint32_t* cand_val;          // [n, cand_pitch] value bits (top-k) or random word (random-k)
    // Where a tile's candidates go.  cand_slot == 0: wherever an atomic add on row_count puts
    // them (the row's candidates end up contiguous, tiles in arrival order).  cand_slot > 0
    // (update kernel, when the selection kernel gathers tile by tile anyway): tile t owns
    // [t * cand_slot, (t + 1) * cand_slot) and needs no reservation; a tile with more candidates
    // reserves room behind the slots, [ntiles * cand_slot, cand_pitch), through row_ovf.
    int64_t cand_pitch;          // row stride of the candidate arrays (>= cap, a multiple of 4)
    uint32_t cand_slot;          // slot per tile in use, or 0
    uint32_t cand_slot_alloc;    // slot per tile the arrays were sized for
    uint32_t* row_ovf;           // [n] candidates placed behind the slots
    uint32_t* spill_key;         // [n, cand_pitch] a row's candidates in tile order, for the cluster kernel
    uint32_t* spill_idx;         //                 when a block's share does not fit its shared memory
    uint32_t* seg_off;           // [n, ntiles] first candidate of a tile
    uint32_t* seg_cnt;           // [n, ntiles]
    uint32_t* tile_a;            // [n, ntiles] scratch
    uint32_t* tile_b;            // [n, ntiles] scratch
    uint32_t* tile_c;            // [n, ntiles] scratch
    // emit kernel: where its working arrays live (shared memory as far as it fits)
    int64_t slab_pitch;          // cap / 32 + 2: slabs of 32 candidates per row
    uint32_t* slab_a;            // [n, slab_pitch] scratch (used when not in shared memory)
    uint32_t* slab_b;            // [n, slab_pitch]
    uint32_t* slab_c;            // [n, slab_pitch] ballot of the keys above the k-th, per slab
    uint32_t* slab_d;            // [n, slab_pitch] ballot of the keys equal to it
    int32_t emit_slabs_smem;     // slab arrays in shared memory
    int32_t emit_tiles_smem;     // per-tile arrays in shared memory
    int32_t emit_masks_smem;     // slab ballots in shared memory
    int64_t emit_keys_cap;       // candidate keys cached in shared memory up to this many
    int64_t emit_smem_bytes;     // dynamic shared memory of the emit kernel
    int32_t emit_cluster;        // blocks that serve one row together (a thread-block cluster); 1 = one block
    int64_t emit_cap_local;      // candidates one block of the cluster can hold in shared memory
    Stats* stats;
    uint32_t wait_polls;         // bound of the kernels' first wait for their staged copies
    int32_t nesterov;            // momentum steps use the look-ahead direction (choco_set_nesterov)
    // what steps ask the L2 cache to keep resident (sparse Q): messages, range records, tables
    void* hot_base;
    int64_t hot_bytes;
    float hot_ratio;
    // dense messages
    int64_t wpitch;              // sign-plane words per row (multiple of 4)
    uint32_t* msg_bits;          // [n, wpitch]
    float* msg_scale;            // sign: [n]
    int64_t nbuckets;            // qsgd blocks per row
    int64_t npitch;              // floats per row of msg_norms
    float* msg_norms;            // qsgd: [n, npitch]
    int64_t lpitch;              // bytes per row of msg_levels (multiple of 16)
    uint8_t* msg_levels;         // qsgd: [n, lpitch]
    int64_t dpitch;              // identity: floats per row of msg_dense
    float* msg_dense;            // identity: [n, dpitch]
    // the other message buffer of the dense operators: the update kernel writes the next
    // step's messages there while it reads this step's from msg_* (the host swaps them)
    uint32_t* nxt_bits;
    float* nxt_scale;
    float* nxt_norms;
    uint8_t* nxt_levels;
    float* nxt_dense;
    // qsgd parameters
    int32_t s;
    int32_t bucket;              // 0 = whole row
    int32_t wbits;               // level field width
    int32_t bucket_shift;        // log2(bucket) when bucket > 0
    int64_t tail_bucket;         // index of the ragged last block, or -1 if the last one is full
    float tau_full;              // tau of a full block (or of the whole row)
    float tau_tail;              // tau of the ragged last block
    // norm workspace
    float* partial;              // [n, nchunks] per-1024 partial sums
    float* partial2;             // [n, nchunks] ping-pong for the tree
};

inline HotRange hot_range_of(const Dev& dv) { return {dv.hot_base, (size_t)dv.hot_bytes, dv.hot_ratio}; }

struct StepArgs {
    float* X;
    float* Xhat;
    float* S;
    const float* G;              // may be null
    float* M;                    // momentum memory, may be null
    float eta, gamma, lambda, beta;
    uint64_t step;
    const unsigned long long* step_dev; // if set, the step number is read from here instead
    bool vec;                    // rows 16-byte aligned: 128-bit accesses
    unsigned long long* launches; // host counter of kernels enqueued (not used on the device)
    // an update launch may serve the workers [row0, row0 + rows) only (rows == 0: all of them)
    int32_t row0 = 0;
    int32_t rows = 0;
};

// One launch over the tiles (or rows) of several layers of a layered context.  The table comes
// as a kernel argument (constant memory): a block finds its entry by bisection over first_block
// (launches over tiles) or as blockIdx.x / n (launches over rows) and can request its tiles at
// once; the rest of the layer's parameters it reads from devs[layer[entry]] in device memory.
constexpr int kHostChunks = 8;     // choco_sgd_step_host moves and updates the rows in this many chunks
constexpr int kMaxComboLayers = 512;
struct LayerTable {
    int32_t entries;                            // layers served by this launch
    uint32_t first_block[kMaxComboLayers + 1];  // blocks (of a row) before each entry's, then the total
    int32_t layer[kMaxComboLayers];             // the layer an entry stands for
    int32_t d[kMaxComboLayers];                 // its length
    int64_t off[kMaxComboLayers];               // its first coordinate
};
struct LayerSet {
    const Dev* devs;      // per layer, device memory: the layer's parameters for this step
    int64_t ld;           // row pitch of the state arrays
};

#ifdef __CUDACC__
// The step number that keys the generator.  A context may keep it in device memory (and bump it
// there after every step) so that a captured launch sequence stays valid from step to step.
__device__ __forceinline__ uint64_t step_of(const StepArgs& a)
{
    return a.step_dev ? (uint64_t)*a.step_dev : a.step;
}
#endif

// selection (top-k / random-k)
cudaError_t launch_select_prepare(const Dev& dv, const StepArgs& a, cudaStream_t st);
// fused: the candidates came from the previous step's update kernel (statistics only)
cudaError_t launch_select_emit(const Dev& dv, const StepArgs& a, bool fused, cudaStream_t st);
// dv.rescue: rows that the emit kernel flagged get fresh histograms, a bound and a candidate
// list from the dense row (all SMs), then their emit; six launches that do nothing otherwise
cudaError_t launch_select_rescue(const Dev& dv, const StepArgs& a, cudaStream_t st);
// dense compressors
cudaError_t launch_compress_dense(const Dev& dv, const StepArgs& a, cudaStream_t st);
// update kernel; emit: also collect the next step's top-k candidates (if apply_can_emit)
bool apply_can_emit(const Dev& dv, const StepArgs& a);
cudaError_t launch_update_bulk(const Dev& dv, const StepArgs& a, bool emit, cudaStream_t st);
bool update_dense_can_emit(const Dev& dv);
cudaError_t launch_update_dense(const Dev& dv, const StepArgs& a, bool emit, cudaStream_t st);
bool update_dense_bulk_usable(const Dev& dv, const StepArgs& a);
cudaError_t launch_update_dense_bulk(const Dev& dv, const StepArgs& a, bool emit, cudaStream_t st);
// sign: finish the tree over the partial sums the update kernel left and set nxt_scale
cudaError_t launch_next_sign_scale(const Dev& dv, cudaStream_t st);
cudaError_t launch_apply(const Dev& dv, const StepArgs& a, bool emit, cudaStream_t st);
// the same kernels over several layers at once (see LayerTable): every layer of a launch shares
// kind, level width, block of the norm, row count n and alignment class
cudaError_t launch_update_dense_bulk_layers(const Dev& proto, const LayerTable& tab, const LayerSet& ls, const StepArgs& a,
                                            bool aligned, cudaStream_t st);
cudaError_t launch_sign_scale_layers(const LayerTable& tab, const LayerSet& ls, int32_t n, cudaStream_t st);
cudaError_t launch_update_bulk_layers(const LayerTable& tab, const LayerSet& ls, int32_t n, const StepArgs& a, bool aligned,
                                      cudaStream_t st);
// `small`: every row of the table is at most kSmallRow long (blocks of kSelThreadsSmall threads)
cudaError_t launch_select_emit_layers(const LayerTable& tab, const LayerSet& ls, int32_t n, size_t smem_bytes, bool small,
                                      const StepArgs& a, cudaStream_t st);
// metrics
cudaError_t launch_consensus(const float* X, int32_t n, int64_t d, int64_t ld, double* scratch,
                             int64_t nblocks, double* out, cudaStream_t st);

} // namespace choco

struct choco_ctx;
namespace choco {
// True if the context's next step will enqueue the same kernels, on the same buffers, as its
// last one did: its compression was prepared by the last step on these very arrays (operators
// that carry it across steps), or it compresses afresh every step; and no per-step events are
// asked for.  *mode receives what else selects kernels and message buffers.
bool step_repeats(const choco_ctx* ctx, const float* X, const float* Xhat, uint64_t* mode);
// The host-side effects of one step call, for a step that was replayed from a graph.
void advance_after_replay(choco_ctx* ctx, unsigned long long launches);
} // namespace choco

// A captured steady-state step of one context, kept for replay (small problems, where a step
// is a few short kernels and their launches dominate).  exec == nullptr: the arguments were
// seen once and will be captured when they come again.
struct choco_step_graph {
    float *X, *Xhat, *S;
    const float* G;
    float* M;
    float eta, gamma, lambda, beta;
    uint64_t mode;               // (compression carried, message buffer in use)
    cudaGraphExec_t exec;
    uint64_t last_use;
};
constexpr int kCtxGraphs = 16;   // per context; the least recently used one is replaced
constexpr int64_t kGraphCoords = (int64_t)1 << 22; // contexts with n d up to this replay graphs

struct choco_ctx {
    choco::Dev dv;
    choco_params params;
    uint64_t step;
    unsigned long long* step_dev; // device copy of `step`, kept equal to it while dev_step is set
    bool dev_step;               // kernels read the step number from step_dev (layered contexts)
    uint64_t steps_enqueued;
    int device;
    int last_cuda_error;
    bool prepared;               // next step's candidates/messages already formed
    bool carry_enabled;          // steps may prepare the next step's compression
    const float* last_x;
    const float* last_xhat;
    int64_t msg_bytes_per_worker;
    // dense operators: two sets of message buffers; msg_cur is read by the next update
    // kernel, msg_last holds the message applied most recently (choco_get_message)
    struct DenseBuf { uint32_t* bits; float* scale; float* norms; uint8_t* levels; float* dense; } dbuf[2];
    int msg_cur, msg_last;
    bool timed_out;              // a synchronising call saw device_timeouts != 0: steps refuse
    uint64_t dv_epoch;           // bumped whenever a setter changes `dv` (a layered context keeps device copies)
    bool hot_l2;                 // the context asked for persisting L2 lines (reset on destroy)
    // host staging for choco_sgd_step_host: device copies of X, X^, S, G; two streams that carry the
    // uploads and the downloads beside the caller's stream; events that order them per chunk of rows
    float* stage[4];
    cudaStream_t host_in, host_out;
    cudaEvent_t host_ev[3 + 2 * choco::kHostChunks]; // fork, X and X^ uploaded, join; per chunk: uploaded, updated
    // consensus scratch
    double* cons_scratch;
    int64_t cons_blocks;
    double* cons_out;
    unsigned long long launches;
    // optional event pairs around the update kernel
    cudaEvent_t* prof_ev;
    int prof_cap, prof_n, prof_stride;
    // replay of captured steady-state steps (see choco_step_graph)
    bool graphs_ok;
    choco_step_graph graphs[kCtxGraphs];
    int ngraphs;
    uint64_t graph_clock, graph_replays;
    unsigned long long launches_per_step; // kernels in a captured step
    // all device allocations, for choco_destroy
    void* allocs[64];
    int nallocs;
};
