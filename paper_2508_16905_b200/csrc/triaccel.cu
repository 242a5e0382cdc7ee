// Host side of the Tri-Accel optimizer pass: C ABI, planner, launches.  See include/triaccel.h
// for the contract of every entry point.
#include "../../include/triaccel.h"

#include <algorithm>
#include <deque>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "kernels.cuh"
#include "pipeline.cuh"

namespace {

thread_local char g_create_error[256] = "";

struct GuardRec {          // a buffer allocated between guard words: what cudaMalloc returned, what the library uses, its size
    void *raw, *user;
    size_t bytes;
};

struct DeviceBuffers {
    ta::Item *items = nullptr;
    uint32_t *item_lo = nullptr;
    uint64_t *seg_off = nullptr, *seg_len = nullptr, *seg_k = nullptr;
    ta::LayerState *state = nullptr;
    ta::LayerScratch *scratch = nullptr;
    ta::Status *status = nullptr;
    unsigned long long *barrier = nullptr;        // fused launch: [0] grid-barrier arrivals, [1] last launch with non-finite input
    ta::FusedWarpHead *warp_head = nullptr;       // fused launch: the plan's records per warp, per block, per (block, layer)
    ta::FusedBlockHead *block_head = nullptr;
    ta::FusedBlockLayer *block_layer = nullptr;
    ta::FusedSlot *slot_table = nullptr;
    ta::FusedPartial *part = nullptr;             // fused launch: block partials, grouped by layer
    double *p_s1 = nullptr, *p_s2 = nullptr, *p_sa = nullptr, *p_mass = nullptr;
    float *p_piv = nullptr;
    uint32_t *p_amax = nullptr, *p_amin = nullptr, *p_bad = nullptr;
    uint2 *window = nullptr;                      // top-k: per layer, the level-1 bins the next sweep collects candidates in
    uint32_t *hist = nullptr;
    ta::SelectState *sel = nullptr;
    uint32_t *mask = nullptr;
    uint32_t *cand_count = nullptr, *cand_val = nullptr, *cand_idx = nullptr, *batch_seg = nullptr;
    // layer-pipelined pass (TA_FLAG_INPUTS_FINITE): its own items, task queues and counters
    ta::PipeTask *pipe_tasks_sweep = nullptr, *pipe_tasks_apply = nullptr, *pipe_tasks_hold = nullptr;
    uint32_t *pipe_batch_lo = nullptr;
    ta::BatchSums *pipe_bsum = nullptr;
    uint32_t *pipe_layer_done = nullptr, *pipe_layer_ready = nullptr;
    ta::PipeControl *pipe_ctl = nullptr;
    // power iteration support: per-item partial sums, per-layer coefficients and norms
    double *pw_part = nullptr;
    float *pw_coef = nullptr, *pw_norm = nullptr;
    // host-tensor staging (ta_step_host)
    float *mom = nullptr;                         // SGD momentum buffer [n_total], only when momentum != 0
    float *st_w = nullptr, *st_hz = nullptr;
    void *st_g = nullptr;
    uint16_t *st_c = nullptr;
};

}  // namespace

struct ta_handle {
    int device = 0;
    int sm_count = 0;
    uint32_t L = 0;
    uint64_t n_total = 0;
    ta_hparams hp{};
    std::vector<ta_segment> table;
    std::vector<uint64_t> seg_k;
    uint32_t n_items = 0, n_batches = 0, item_elems = 0;
    uint64_t mask_words = 0;
    bool topk = false;
    bool ring_asked = false;          // the top-k sweep's shared-memory ring has been allowed on this device
    bool stepped = false;
    uint64_t last_step = 0;
    uint64_t launches = 0;
    cudaStream_t last_stream = nullptr;
    std::vector<cudaEvent_t> events;      // 4 per timed step: before sweep, after sweep, after decisions, after update
    uint32_t timed_cap = 0, timed_used = 0;
    bool expire_next_wait = false;        // test aid: the next one-launch step waits for arrivals that never come
    bool fused_ok = false;                // small dense models: sweep + decisions + update in one cooperative launch ...
    bool fused_split = false;             // ... or as two dependent launches over the same plan (the default)
    int fused_grid = 0;                   // blocks of the one-launch grid (all resident)
    uint32_t fused_cap_w = 0, fused_cap_g = 0;                           // shared-memory slots per warp: weights, gradients
    uint32_t fused_block_layers = 0, fused_block_runs = 0, fused_slots = 0, fused_parts = 0;   // table sizes of the plan
    size_t fused_smem = 0;
    unsigned long long barrier_base = 0;  // barrier arrivals of all fused launches so far
    unsigned long long fused_launches = 0;// fused launches since the arrival counters were last cleared
    bool sharded = false;                 // this handle holds the flat range [range_lo, range_hi) of a model spread over ranks
    uint64_t range_lo = 0, range_hi = 0;
    uint64_t pending_step = 0;            // shard: step of a ta_shard_sweep whose ta_shard_apply has not come yet
    bool pending = false, pending_has_hz = false;
    bool pipe_ok = false;                 // large dense models with TA_FLAG_INPUTS_FINITE: the layer-pipelined launch
    uint32_t pipe_batches = 0;
    int pipe_per_sm = 0;
    unsigned long long pipe_base_s = 0, pipe_base_a = 0;
    uint32_t pipe_launches = 0;
    std::vector<GuardRec> guards;         // TA_FLAG_GUARD_WORKSPACES: the buffers allocated by ta_create, with their guard words
    std::vector<ta::Item> items_host;     // the plan, kept for the pipelined host path
    cudaStream_t copy_back = nullptr;     // ta_step_host: device-to-host copies run beside the host-to-device ones
    std::vector<cudaEvent_t> chunk_done;
    cudaEvent_t decided = nullptr;
    DeviceBuffers d;
    char err[256] = "";
};

namespace {

int fail(ta_handle *h, int code, const char *fmt, const char *detail = "")
{
    char *dst = h ? h->err : g_create_error;
    snprintf(dst, 256, fmt, detail);
    return code;
}

#define TA_CUDA(h, call)                                                          \
    do {                                                                          \
        cudaError_t e__ = (call);                                                 \
        if (e__ != cudaSuccess) {                                                 \
            char *dst__ = (h) ? (h)->err : g_create_error;                        \
            snprintf(dst__, 256, "%s failed: %s", #call, cudaGetErrorString(e__)); \
            return e__ == cudaErrorMemoryAllocation ? TA_ERR_NOMEM : TA_ERR_CUDA; \
        }                                                                         \
    } while (0)

// A library-owned buffer allocated with guard words on both sides (TA_FLAG_GUARD_WORKSPACES): a kernel that writes
// outside a workspace is caught by ta_test_check_guards instead of corrupting its neighbour silently.
constexpr size_t kGuardBytes = 256;
constexpr int kGuardFill = 0xA5;
thread_local std::vector<GuardRec> *g_guard_sink = nullptr;      // set while ta_create allocates for a guarded handle

template <typename T> cudaError_t dev_alloc(T **p, size_t count)
{
    const size_t bytes = std::max<size_t>(count, 1) * sizeof(T);
    if (!g_guard_sink) return cudaMalloc(reinterpret_cast<void **>(p), bytes);
    char *raw = nullptr;
    cudaError_t e = cudaMalloc(reinterpret_cast<void **>(&raw), bytes + 2 * kGuardBytes);
    if (e != cudaSuccess) return e;
    e = cudaMemset(raw, kGuardFill, kGuardBytes);
    if (e == cudaSuccess) e = cudaMemset(raw + kGuardBytes + bytes, kGuardFill, kGuardBytes);
    *p = reinterpret_cast<T *>(raw + kGuardBytes);
    g_guard_sink->push_back(GuardRec{raw, *p, bytes});
    return e;
}

void free_all(DeviceBuffers &d, const std::vector<GuardRec> &guards = {})
{
    void *ptrs[] = {d.pipe_tasks_sweep, d.pipe_tasks_apply, d.pipe_tasks_hold, d.pipe_batch_lo, d.pipe_bsum, d.pipe_layer_done, d.pipe_layer_ready, d.pipe_ctl,
                    d.warp_head, d.block_head, d.block_layer, d.slot_table, d.part, d.mom, d.pw_part, d.pw_coef, d.pw_norm, d.barrier, d.items, d.item_lo, d.seg_off, d.seg_len, d.seg_k, d.state, d.scratch, d.status, d.p_s1, d.p_s2, d.p_piv,
                    d.p_sa, d.p_mass, d.p_amax, d.p_amin, d.p_bad, d.window, d.hist, d.sel, d.mask, d.cand_count, d.cand_val, d.cand_idx, d.batch_seg, d.st_w, d.st_hz,
                    d.st_g, d.st_c};
    for (void *p : ptrs) {
        if (!p) continue;
        void *raw = p;
        for (const GuardRec &g : guards)
            if (g.user == p) raw = g.raw;
        cudaFree(raw);
    }
    d = DeviceBuffers{};
}

// Elements per work item: the largest size that still gives every warp slot of the GPU a few
// items, so that thousands of tiny tensors and a few huge ones both keep all SMs busy.
uint32_t choose_item_elems(uint64_t n_params, int sm_count)
{
    const uint64_t want_items = (uint64_t)sm_count * ta::kWarps * 4;
    uint32_t best = 512;
    for (uint32_t cand : {1024u, 2048u, 4096u, 8192u, 16384u})
        if (n_params / cand >= want_items) best = cand;
    return best;
}

// The work items of the multi-kernel pass: every layer (the part of it inside [range_lo, range_hi)) cut on a global
// grid of item_elems elements, in buffer order; eight consecutive items make a batch, one per warp of a block.
// topk: a layer of at least one full batch starts on a batch boundary, so that its batches hold one layer only and
// can count their histogram in shared memory (the padding items are empty).  item_lo[l] is the first item of layer l,
// batch_seg[b] the layer of a batch whose items all lie in one layer, else kMixedBatch.
struct ItemPlan {
    std::vector<ta::Item> items;
    std::vector<uint32_t> item_lo, batch_seg;
    bool too_many = false;
};

ItemPlan plan_items(const ta_segment *table, uint32_t L, uint32_t item_elems, bool topk, uint64_t range_lo, uint64_t range_hi)
{
    ItemPlan pl;
    pl.item_lo.assign(L + 1, 0u);
    std::vector<ta::Item> &items = pl.items;
    for (uint32_t l = 0; l < L; ++l) {
        pl.item_lo[l] = (uint32_t)items.size();
        // a shard holds the part of every layer that lies inside its range (possibly nothing)
        const uint64_t b = std::max<uint64_t>(table[l].offset, range_lo), e = std::min<uint64_t>(table[l].offset + table[l].length, range_hi);
        if (e <= b) continue;
        const uint64_t layer_items = (e - 1) / item_elems - b / item_elems + 1;
        if (topk && layer_items >= (uint64_t)ta::kWarps && l > 0)
            while (items.size() % ta::kWarps) items.push_back(ta::Item{b, 0u, l - 1});
        pl.item_lo[l] = (uint32_t)items.size();
        for (uint64_t p = b; p < e;) {
            const uint64_t next = std::min(e, (p / item_elems + 1) * (uint64_t)item_elems);
            items.push_back(ta::Item{p, (uint32_t)(next - p), l});
            p = next;
        }
        if (items.size() > 0x7FFFFFFFull) { pl.too_many = true; return pl; }
    }
    pl.item_lo[L] = (uint32_t)items.size();
    const uint32_t n_items = (uint32_t)items.size(), n_batches = (n_items + ta::kWarps - 1) / ta::kWarps;
    pl.batch_seg.assign(n_batches, ta::kMixedBatch);
    for (uint32_t bt = 0; bt < n_batches; ++bt) {
        uint32_t seg = ta::kMixedBatch;
        bool uniform = true;
        for (uint32_t i = bt * ta::kWarps; i < std::min(n_items, (bt + 1) * ta::kWarps); ++i) {
            if (items[i].len == 0) continue;
            if (seg == ta::kMixedBatch) seg = items[i].seg;
            else if (seg != items[i].seg) uniform = false;
        }
        pl.batch_seg[bt] = uniform ? seg : ta::kMixedBatch;
    }
    return pl;
}

int grid_for(const ta_handle *h)
{
    const long long cap = (long long)h->sm_count * 8;
    return (int)std::max<long long>(1, std::min<long long>(h->n_batches, cap));
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

ta::Hyper hyper_of(const ta_hparams &hp)
{
    ta::Hyper y;
    y.beta = hp.beta; y.tau_low = hp.tau_low; y.tau_high = hp.tau_high; y.tau_curv = hp.tau_curv;
    y.alpha = hp.alpha; y.num_probes = hp.num_probes; y.t_ctrl = hp.t_ctrl; y.topk_ppm = hp.topk_ppm;
    return y;
}

// Launches a kernel of the multi-kernel pass so that its blocks may be scheduled while the kernel before it in the
// stream drains (its first instruction waits for that kernel's completion, so nothing else changes): the launch
// latency between the three or four dependent kernels of a step is hidden behind the previous kernel's tail.
template <typename... KArgs, typename... Args>
cudaError_t launch_after(void (*kernel)(KArgs...), unsigned grid, size_t smem, cudaStream_t s, Args... args)
{
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(ta::kThreads); cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

template <int P, bool BF16, bool TOPK> void launch_sweep(ta_handle *h, const ta::SweepArgs &a, cudaStream_t s)
{
    // the top-k sweeps stage their rows in a ring of shared memory (beyond the 48 KB a launch gets without asking)
    const size_t ring = TOPK ? ta::sweep_ring_bytes(P) : 0;
    if (TOPK && !h->ring_asked) {           // per device and kernel; a handle has one of each
        cudaFuncSetAttribute(ta::k_sweep<P, BF16, TOPK>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ring);
        h->ring_asked = true;
    }
    // the second sweep of a top-k step usually finds nothing to repeat: one resident wave of blocks, which walk the
    // batches in a loop, starts (and ends) faster than a block per batch and is as fast when there is work
    const unsigned grid = TOPK && a.redo ? (unsigned)std::min<long long>(grid_for(h), (long long)h->sm_count * 2) : (unsigned)grid_for(h);
    launch_after(ta::k_sweep<P, BF16, TOPK>, grid, ring, s, a);
    ++h->launches;
}

template <bool BF16> bool dispatch_sweep(ta_handle *h, int P, const ta::SweepArgs &a, cudaStream_t s)
{
    const bool topk = h->topk && P > 0;
    switch (P) {
    case 0: launch_sweep<0, BF16, false>(h, a, s); return true;
    case 1: topk ? launch_sweep<1, BF16, true>(h, a, s) : launch_sweep<1, BF16, false>(h, a, s); return true;
    case 2: topk ? launch_sweep<2, BF16, true>(h, a, s) : launch_sweep<2, BF16, false>(h, a, s); return true;
    case 4: topk ? launch_sweep<4, BF16, true>(h, a, s) : launch_sweep<4, BF16, false>(h, a, s); return true;
    case 8: topk ? launch_sweep<8, BF16, true>(h, a, s) : launch_sweep<8, BF16, false>(h, a, s); return true;
    default: return false;
    }
}

// Update + cast over the items [item_begin, item_begin + item_count) (item_begin a multiple of the batch size).
void launch_apply(ta_handle *h, float *w, const void *g, uint16_t *c, uint32_t item_begin, uint32_t item_count, cudaStream_t s)
{
    if (item_count == 0) return;
    const uint32_t batches = (item_count + ta::kWarps - 1) / ta::kWarps;
    ta::ApplyArgs aa{h->d.items + item_begin, item_count, batches, w, g, c, h->d.state, h->d.status,
                     h->d.mom, h->hp.momentum, h->hp.weight_decay};
    const int grid = (int)std::min<long long>(batches, (long long)h->sm_count * 8);
    const bool bf16 = h->hp.grad_dtype == TA_GRAD_BF16, mom = h->d.mom != nullptr;
    if (bf16 && mom) launch_after(ta::k_apply<true, true>, (unsigned)grid, 0, s, aa);
    else if (bf16) launch_after(ta::k_apply<true, false>, (unsigned)grid, 0, s, aa);
    else if (mom) launch_after(ta::k_apply<false, true>, (unsigned)grid, 0, s, aa);
    else launch_after(ta::k_apply<false, false>, (unsigned)grid, 0, s, aa);
    ++h->launches;
}

template <int P, bool BF16, int MODE> const void *fused_fn() { return reinterpret_cast<const void *>(&ta::k_fused<P, BF16, MODE>); }

template <int MODE> const void *fused_kernel_mode(int P, bool bf16)
{
    switch (P) {
    case 0: return bf16 ? fused_fn<0, true, MODE>() : fused_fn<0, false, MODE>();
    case 1: return bf16 ? fused_fn<1, true, MODE>() : fused_fn<1, false, MODE>();
    case 2: return bf16 ? fused_fn<2, true, MODE>() : fused_fn<2, false, MODE>();
    case 4: return bf16 ? fused_fn<4, true, MODE>() : fused_fn<4, false, MODE>();
    case 8: return bf16 ? fused_fn<8, true, MODE>() : fused_fn<8, false, MODE>();
    default: return nullptr;
    }
}
const void *fused_kernel(int P, bool bf16) { return fused_kernel_mode<ta::kWholeStep>(P, bf16); }
const void *sweep_half_kernel(int P, bool bf16) { return fused_kernel_mode<ta::kSweepHalf>(P, bf16); }
const void *update_half_kernel(bool bf16) { return bf16 ? fused_fn<0, true, ta::kUpdateHalf>() : fused_fn<0, false, ta::kUpdateHalf>(); }

constexpr int kFusedSmemMax = 226 * 1024;         // dynamic shared memory a block may ask for (227 KB opt-in limit minus the static part)
constexpr uint64_t kRunOverhead = 256;            // cost of starting a run, in elements: reductions and partial rows
constexpr uint64_t kMinWarpCost = 512;            // a warp is given at least this much work

// The plan of the one-launch path: every layer is cut into runs so that each of n_warps warps gets a list of
// consecutive runs of equal total cost (elements plus a constant per run).  Cuts lie on the global grid of
// 128-element rows, so only the first and the last row of a layer can be partial.
struct RunPlan {
    std::vector<ta::Item> runs;
    std::vector<uint32_t> item_lo, warp_lo;           // first run of every layer / warp
    std::vector<uint32_t> part_lo, block_part_lo;     // block partials: first of every layer, first of every block
    std::vector<ta::FusedWarpHead> warp_head;
    std::vector<ta::FusedBlockHead> block_head;
    std::vector<ta::FusedBlockLayer> block_layer;
    std::vector<ta::FusedSlot> slot_table;            // [n_warps][max_slots]
    uint32_t n_warps = 0, n_part = 0;
    uint32_t max_slots = 0, max_warp_runs = 0, max_block_runs = 0, max_block_layers = 0;
};

RunPlan plan_runs(const ta_segment *table, uint32_t L, uint64_t max_warps)
{
    RunPlan pl;
    uint64_t cost = 0;
    for (uint32_t l = 0; l < L; ++l) cost += table[l].length + kRunOverhead;
    uint64_t n_warps = std::min<uint64_t>(max_warps, (cost + kMinWarpCost - 1) / kMinWarpCost);
    n_warps = std::max<uint64_t>(ta::kWarps, (n_warps + ta::kWarps - 1) / ta::kWarps * ta::kWarps);
    const double target = (double)cost / (double)n_warps;
    pl.n_warps = (uint32_t)n_warps;
    pl.item_lo.resize(L + 1);
    std::vector<uint32_t> run_warp;
    uint64_t cum = 0, warp = 0;
    for (uint32_t l = 0; l < L; ++l) {
        pl.item_lo[l] = (uint32_t)pl.runs.size();
        const uint64_t b = table[l].offset, e = b + table[l].length;
        cum += kRunOverhead;
        for (uint64_t p = b; p < e;) {
            const double room = target * (double)(warp + 1) - (double)cum;
            uint64_t q = e;
            if (warp + 1 < n_warps && room < (double)(e - p)) {
                q = (p + (uint64_t)std::max(room, 0.0) + 64) / 128 * 128;        // nearest row boundary
                if (q <= p) q = (p / 128 + 1) * 128;
                if (q > e) q = e;
            }
            pl.runs.push_back(ta::Item{p, (uint32_t)(q - p), l});
            run_warp.push_back((uint32_t)warp);
            cum += q - p;
            p = q;
            while (warp + 1 < n_warps && (double)cum >= target * (double)(warp + 1) - 64.0) ++warp;      // this warp is full
        }
    }
    pl.item_lo[L] = (uint32_t)pl.runs.size();
    pl.warp_lo.assign(n_warps + 1, (uint32_t)pl.runs.size());
    for (size_t r = pl.runs.size(); r-- > 0;) pl.warp_lo[run_warp[r]] = (uint32_t)r;
    for (size_t wq = n_warps; wq-- > 0;) pl.warp_lo[wq] = std::min(pl.warp_lo[wq], pl.warp_lo[wq + 1]);   // warps without runs
    for (uint64_t wq = 0; wq < n_warps; ++wq) {
        uint64_t slots = 0;       // rows the warp visits, partial ones included
        for (uint32_t r = pl.warp_lo[wq]; r < pl.warp_lo[wq + 1]; ++r)
            slots += (pl.runs[r].begin + pl.runs[r].len - 1) / 128 - pl.runs[r].begin / 128 + 1;
        pl.max_slots = std::max<uint32_t>(pl.max_slots, (uint32_t)slots);
        pl.max_warp_runs = std::max(pl.max_warp_runs, pl.warp_lo[wq + 1] - pl.warp_lo[wq]);
    }
    // every block writes one partial per layer it touches; in (block, layer) order these are grouped by layer
    const uint64_t n_blocks = n_warps / ta::kWarps;
    pl.block_part_lo.resize(n_blocks);
    std::vector<uint32_t> per_layer(L, 0);
    for (uint64_t blk = 0; blk < n_blocks; ++blk) {
        const uint32_t lo = pl.warp_lo[blk * ta::kWarps], hi = pl.warp_lo[(blk + 1) * ta::kWarps];
        pl.block_part_lo[blk] = pl.n_part;
        if (hi <= lo) continue;
        const uint32_t lf = pl.runs[lo].seg, ll = pl.runs[hi - 1].seg;
        pl.max_block_layers = std::max(pl.max_block_layers, ll - lf + 1);
        pl.max_block_runs = std::max(pl.max_block_runs, hi - lo);
        for (uint32_t l = lf; l <= ll; ++l) ++per_layer[l];
        pl.n_part += ll - lf + 1;
    }
    pl.part_lo.resize(L + 1);
    pl.part_lo[0] = 0;
    for (uint32_t l = 0; l < L; ++l) pl.part_lo[l + 1] = pl.part_lo[l] + per_layer[l];
    // the records the kernel reads: per warp its slots, per block its runs and layers
    pl.warp_head.assign(n_warps, ta::FusedWarpHead{0, 0, 0, 0});
    pl.slot_table.assign((size_t)n_warps * pl.max_slots, ta::FusedSlot{0, 0, 0, 0});
    for (uint64_t wq = 0; wq < n_warps; ++wq) {
        uint32_t n = 0;
        for (uint32_t r = pl.warp_lo[wq]; r < pl.warp_lo[wq + 1]; ++r) {
            const uint64_t b = pl.runs[r].begin, e = b + pl.runs[r].len;
            for (uint64_t row = b / 128; row <= (e - 1) / 128; ++row) {
                const uint64_t r0 = row * 128;
                const uint32_t lo = b > r0 ? (uint32_t)(b - r0) : 0u, hi = e < r0 + 128 ? (uint32_t)(e - r0) : 128u;
                pl.slot_table[wq * pl.max_slots + n++] = ta::FusedSlot{(uint32_t)row, lo | (hi << 16), r - pl.warp_lo[wq], pl.runs[r].seg};
            }
        }
        pl.warp_head[wq] = ta::FusedWarpHead{pl.warp_lo[wq], n, 0, 0};
    }
    pl.block_head.resize(n_blocks);
    pl.block_layer.resize(pl.n_part);
    for (uint64_t blk = 0; blk < n_blocks; ++blk) {
        const uint32_t lo = pl.warp_lo[blk * ta::kWarps], hi = pl.warp_lo[(blk + 1) * ta::kWarps];
        const uint32_t lf = hi > lo ? pl.runs[lo].seg : 0u, nl = hi > lo ? pl.runs[hi - 1].seg - lf + 1 : 0u;
        pl.block_head[blk] = ta::FusedBlockHead{lo, hi, lf, nl, pl.block_part_lo[blk], 0, 0, 0};
        for (uint32_t q = 0; q < nl; ++q) {
            const uint32_t l = lf + q;
            ta::FusedBlockLayer bl{};
            bl.n = (double)table[l].length;
            bl.part_lo = pl.part_lo[l];
            bl.part_hi = pl.part_lo[l + 1];
            bl.own = pl.item_lo[l] >= lo ? 1u : 0u;
            bl.run_lo = std::max(pl.item_lo[l], lo);
            bl.run_hi = std::min(pl.item_lo[l + 1], hi);
            pl.block_layer[pl.block_part_lo[blk] + q] = bl;
        }
    }
    return pl;
}

// The plan of the layer-pipelined pass: batches of kPipeCells cells of kPipeItemElems elements cut on a global grid,
// every batch inside one layer, and the task queues.  A step with decisions: the sweep tasks in buffer order, and the
// apply tasks layer by layer, within a layer the last batch first.  A step without decisions: one single-pass task
// per batch, in buffer order.
struct PipePlan {
    std::vector<uint32_t> batch_lo;
    std::vector<ta::PipeTask> sweep, apply, hold;
};

PipePlan plan_pipe(const ta_segment *table, uint32_t L)
{
    PipePlan pl;
    pl.batch_lo.resize(L + 1);
    std::vector<ta::PipeTask> batches;         // in buffer order; the kind is filled in per queue
    const uint64_t cells = ta::kPipeCells;     // cells of kPipeItemElems elements per batch
    for (uint32_t l = 0; l < L; ++l) {
        pl.batch_lo[l] = (uint32_t)batches.size();
        const uint64_t b = table[l].offset, e = b + table[l].length;
        for (uint64_t p = b; p < e;) {
            const uint64_t next = std::min<uint64_t>(e, (p / ta::kPipeItemElems + cells) * (uint64_t)ta::kPipeItemElems);
            batches.push_back(ta::PipeTask{p, (uint32_t)(next - p), l, (uint32_t)batches.size(), 0u, 0u, 0u});
            p = next;
        }
        for (uint32_t i = pl.batch_lo[l]; i < batches.size(); ++i) batches[i].layer_batches = (uint32_t)batches.size() - pl.batch_lo[l];
    }
    pl.batch_lo[L] = (uint32_t)batches.size();
    auto task_of = [&](uint32_t b, uint32_t kind) {
        ta::PipeTask t = batches[b];
        t.seg_type |= kind << 30;
        return t;
    };
    pl.hold.reserve(batches.size());
    pl.sweep.reserve(batches.size());
    pl.apply.reserve(batches.size());
    for (uint32_t b = 0; b < batches.size(); ++b) {
        pl.hold.push_back(task_of(b, ta::kTaskBoth));
        pl.sweep.push_back(task_of(b, ta::kTaskSweep));
    }
    for (uint32_t l = 0; l < L; ++l)
        for (uint32_t b = pl.batch_lo[l + 1]; b-- > pl.batch_lo[l];) pl.apply.push_back(task_of(b, ta::kTaskApply));
    return pl;
}

template <int P, bool BF16> const void *pipe_fn() { return reinterpret_cast<const void *>(&ta::k_pipe<P, BF16>); }

const void *pipe_kernel(int P, bool bf16)
{
    switch (P) {
    case 0: return bf16 ? pipe_fn<0, true>() : pipe_fn<0, false>();
    case 1: return bf16 ? pipe_fn<1, true>() : pipe_fn<1, false>();
    case 2: return bf16 ? pipe_fn<2, true>() : pipe_fn<2, false>();
    case 4: return bf16 ? pipe_fn<4, true>() : pipe_fn<4, false>();
    case 8: return bf16 ? pipe_fn<8, true>() : pipe_fn<8, false>();
    default: return nullptr;
    }
}

constexpr uint64_t kFusedMaxParams = 16ull << 20;      // models up to ~16 M parameters (ResNet-18 scale) take the one-launch path

// A bounded wait inside a kernel ran out (a block of a cooperative launch never arrived): the step that
// hit it is incomplete.  Reports it once and re-arms the barrier.
int check_device_error(ta_handle *h)
{
    ta::Status s;
    TA_CUDA(h, cudaMemcpy(&s, h->d.status, sizeof(s), cudaMemcpyDeviceToHost));
    if (!s.device_error) return TA_OK;
    s.device_error = 0u;
    TA_CUDA(h, cudaMemcpy(h->d.status, &s, sizeof(s), cudaMemcpyHostToDevice));
    if (h->d.barrier) TA_CUDA(h, cudaMemset(h->d.barrier, 0, 4 * sizeof(unsigned long long)));

    h->barrier_base = 0;
    h->fused_launches = 0;
    if (h->pipe_ok) {
        TA_CUDA(h, cudaMemset(h->d.pipe_ctl, 0, sizeof(ta::PipeControl)));
        TA_CUDA(h, cudaMemset(h->d.pipe_layer_done, 0, h->L * sizeof(uint32_t)));
        TA_CUDA(h, cudaMemset(h->d.pipe_layer_ready, 0, h->L * sizeof(uint32_t)));
        h->pipe_base_s = h->pipe_base_a = 0;
        h->pipe_launches = 0;
    }
    return fail(h, TA_ERR_CUDA, "a bounded device-side wait ran out during the last step; its results are incomplete");
}

int default_mem_reader(void *, uint64_t *free_b, uint64_t *total_b)
{
    size_t f = 0, t = 0;
    if (cudaMemGetInfo(&f, &t) != cudaSuccess) return 1;
    *free_b = f;
    *total_b = t;
    return 0;
}

struct StateHeader {
    uint64_t magic, n_total, last_step, mask_words;
    uint32_t L, stepped;
    ta_hparams hp;
};
constexpr uint64_t kStateMagic = 0x5441535441544531ull;   // "TASTATE1"

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

const char *ta_last_error(const ta_handle *h) { return h ? h->err : g_create_error; }

static int create_impl(const ta_segment *table, uint32_t L, uint64_t n_total, const ta_hparams *hp, uint64_t range_lo,
                       uint64_t range_hi, bool sharded, ta_handle **out)
{
    if (out) *out = nullptr;
    g_create_error[0] = 0;
    if (!table || !hp || !out || L == 0) return fail(nullptr, TA_ERR_ARG, "ta_create: NULL argument or empty table");
    if (hp->struct_size != sizeof(ta_hparams)) return fail(nullptr, TA_ERR_ARG, "ta_create: hp.struct_size does not match this library");
    if (!(hp->beta >= 0.f && hp->beta < 1.f)) return fail(nullptr, TA_ERR_ARG, "ta_create: beta must be in [0,1)");
    if (!(hp->tau_low <= hp->tau_high)) return fail(nullptr, TA_ERR_ARG, "ta_create: tau_low must not exceed tau_high");
    if (!(hp->alpha >= 0.f)) return fail(nullptr, TA_ERR_ARG, "ta_create: alpha must be >= 0");
    if (hp->num_probes != 1 && hp->num_probes != 2 && hp->num_probes != 4 && hp->num_probes != 8)
        return fail(nullptr, TA_ERR_ARG, "ta_create: num_probes must be 1, 2, 4 or 8");
    if (hp->topk_ppm == 0 || hp->topk_ppm > 1000000u) return fail(nullptr, TA_ERR_ARG, "ta_create: topk_ppm must be in [1, 1000000]");
    if (hp->t_ctrl == 0) return fail(nullptr, TA_ERR_ARG, "ta_create: t_ctrl must be >= 1");
    if (hp->grad_dtype != TA_GRAD_F32 && hp->grad_dtype != TA_GRAD_BF16) return fail(nullptr, TA_ERR_ARG, "ta_create: unknown grad_dtype");
    if (!(hp->momentum >= 0.f && hp->momentum < 1.f)) return fail(nullptr, TA_ERR_ARG, "ta_create: momentum must be in [0,1)");
    if (!(hp->weight_decay >= 0.f) || !(hp->weight_decay < 1e30f)) return fail(nullptr, TA_ERR_ARG, "ta_create: weight_decay must be finite and >= 0");
    if (hp->flags & ~(uint32_t)(TA_FLAG_INPUTS_FINITE | TA_FLAG_NO_ONE_LAUNCH | TA_FLAG_GUARD_WORKSPACES | TA_FLAG_COOPERATIVE_LAUNCH)) return fail(nullptr, TA_ERR_ARG, "ta_create: unknown bit in flags");
    if (n_total % 4 != 0) return fail(nullptr, TA_ERR_ARG, "ta_create: n_total must be a multiple of 4");
    uint64_t end = 0, n_params = 0;
    for (uint32_t l = 0; l < L; ++l) {
        if (table[l].length == 0 || table[l].length > 0xFFFFFFFEull)
            return fail(nullptr, TA_ERR_ARG, "ta_create: segment length out of range");
        if (table[l].offset < end) return fail(nullptr, TA_ERR_ARG, "ta_create: segments must be ascending and non-overlapping");
        end = table[l].offset + table[l].length;
        n_params += table[l].length;
    }
    if (end > n_total) return fail(nullptr, TA_ERR_ARG, "ta_create: a segment reaches beyond n_total");
    if (sharded) {
        if (range_lo % 128 || range_hi % 128 || range_lo >= range_hi || range_hi > (n_total + 127) / 128 * 128)
            return fail(nullptr, TA_ERR_ARG, "ta_create_shard: the range must be non-empty, inside the buffer and cut on multiples of 128 elements");
        if (hp->topk_ppm < 1000000u) return fail(nullptr, TA_ERR_ARG, "ta_create_shard: the top-k mask is not available on a sharded model");
    }

    ta_handle *h = new (std::nothrow) ta_handle;
    if (!h) return fail(nullptr, TA_ERR_NOMEM, "ta_create: out of host memory");
    auto bail = [&](int code) {
        snprintf(g_create_error, 256, "%s", h->err);
        g_guard_sink = nullptr;
        free_all(h->d, h->guards);
        delete h;
        return code;
    };
    if (hp->flags & TA_FLAG_GUARD_WORKSPACES) g_guard_sink = &h->guards;
#define TA_TRY(call)                                                                 \
    do {                                                                             \
        cudaError_t e__ = (call);                                                    \
        if (e__ != cudaSuccess) {                                                    \
            snprintf(h->err, 256, "%s failed: %s", #call, cudaGetErrorString(e__));  \
            return bail(e__ == cudaErrorMemoryAllocation ? TA_ERR_NOMEM : TA_ERR_CUDA); \
        }                                                                            \
    } while (0)

    TA_TRY(cudaGetDevice(&h->device));
    cudaDeviceProp prop;
    TA_TRY(cudaGetDeviceProperties(&prop, h->device));
    if (prop.major < 10) {
        snprintf(h->err, 256, "ta_create: device is sm_%d%d; this library is built for sm_100a only", prop.major, prop.minor);
        return bail(TA_ERR_CUDA);
    }
    h->sm_count = prop.multiProcessorCount;
    h->L = L;
    h->n_total = n_total;
    h->hp = *hp;
    h->table.assign(table, table + L);
    h->topk = hp->topk_ppm < 1000000u;
    h->mask_words = h->topk ? (n_total + 31) / 32 : 0;
    h->sharded = sharded;
    h->range_lo = sharded ? range_lo : 0;
    h->range_hi = sharded ? range_hi : n_total;

    // one-launch path for small dense models: needs a cooperative launch with every block resident
    int fused_per_sm = 0;
    {
        int coop = 0;
        TA_TRY(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, h->device));
        if (coop && !sharded && !(hp->flags & TA_FLAG_NO_ONE_LAUNCH) && !h->topk && hp->momentum == 0.f && hp->weight_decay == 0.f &&
            n_params <= kFusedMaxParams) {
            const bool bf16 = hp->grad_dtype == TA_GRAD_BF16;
            h->fused_ok = true;
            h->fused_split = !(hp->flags & TA_FLAG_COOPERATIVE_LAUNCH);
            fused_per_sm = 1 << 20;
            for (int P : {0, (int)hp->num_probes}) {
                int per_sm = 0;
                const void *fn = h->fused_split ? sweep_half_kernel(P, bf16) : fused_kernel(P, bf16);
                TA_TRY(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kFusedSmemMax));
                TA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, ta::kThreads, 0));
                fused_per_sm = std::min(fused_per_sm, per_sm);
            }
            if (h->fused_split) {
                int per_sm = 0;
                TA_TRY(cudaFuncSetAttribute(update_half_kernel(bf16), cudaFuncAttributeMaxDynamicSharedMemorySize, kFusedSmemMax));
                TA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, update_half_kernel(bf16), ta::kThreads, 0));
                fused_per_sm = std::min(fused_per_sm, per_sm);
            }
            if (fused_per_sm < 1) h->fused_ok = false;
        }
    }

    // plan: items cut on a global grid of item_elems elements, clipped to each layer
    h->item_elems = choose_item_elems(n_params, h->sm_count);
    std::vector<ta::Item> items;
    std::vector<uint32_t> item_lo(L + 1);
    RunPlan run_plan;
    std::vector<uint64_t> seg_off(L), seg_len(L);
    h->seg_k.resize(L);
    for (uint32_t l = 0; l < L; ++l) {
        seg_off[l] = table[l].offset;
        seg_len[l] = table[l].length;
        uint64_t k = (table[l].length * (uint64_t)hp->topk_ppm + 999999ull) / 1000000ull;
        h->seg_k[l] = k < 1 ? 1 : k;
    }
    if (h->fused_ok) {
        // one-launch path: the items are the runs of a plan that gives every resident warp the same amount of work;
        // what is left of the SM's shared memory, after the per-block tables, holds weight rows first, then gradient rows
        RunPlan pl = plan_runs(table, L, (uint64_t)h->sm_count * fused_per_sm * ta::kWarps);
        const size_t tables = (size_t)pl.max_block_layers * (sizeof(ta::LayerState) + sizeof(ta::FusedBlockLayer) + 8) +
                              (size_t)pl.max_block_runs * sizeof(ta::FusedPartial) + (size_t)ta::kWarps * pl.max_slots * sizeof(ta::FusedSlot);
        const long long per_block = std::min<long long>(kFusedSmemMax, (228ll * 1024) / fused_per_sm - 1024) - 512 /* static */ - (long long)tables;
        const long long rows_fit = per_block / (ta::kWarps * 512);
        if (rows_fit < 0 || tables > 64 * 1024 || n_total >= (1ull << 38)) {
            h->fused_ok = false;
        } else {
            // weights first, then gradients; a model whose weights do not all fit gains nothing from a part of
            // them (its update is bound by the write-back of what it writes): it keeps nothing in shared memory
            h->fused_cap_w = (uint32_t)std::min<long long>(pl.max_slots, rows_fit);
            h->fused_cap_g = (uint32_t)std::min<long long>(pl.max_slots, rows_fit - h->fused_cap_w);
            if (h->fused_cap_w < pl.max_slots) h->fused_cap_w = h->fused_cap_g = 0;
            if (h->fused_split) h->fused_cap_w = h->fused_cap_g = 0;      // nothing survives in shared memory between two launches
            h->fused_block_layers = pl.max_block_layers;
            h->fused_block_runs = pl.max_block_runs;
            h->fused_slots = pl.max_slots;
            h->fused_parts = pl.n_part;
            h->fused_smem = (size_t)ta::kWarps * 512 * (h->fused_cap_w + h->fused_cap_g) + tables;
            h->fused_grid = (int)(pl.n_warps / ta::kWarps);
            items = pl.runs;
            item_lo = pl.item_lo;
            run_plan = std::move(pl);
        }
    }
    std::vector<uint32_t> batch_seg;
    if (!h->fused_ok) {
        ItemPlan ip = plan_items(table, L, h->item_elems, h->topk, h->range_lo, h->range_hi);
        if (ip.too_many) { snprintf(h->err, 256, "ta_create: too many work items"); return bail(TA_ERR_ARG); }
        items = std::move(ip.items);
        item_lo = std::move(ip.item_lo);
        batch_seg = std::move(ip.batch_seg);
    }
    h->items_host = items;
    h->n_items = (uint32_t)items.size();
    h->n_batches = (h->n_items + ta::kWarps - 1) / ta::kWarps;
    if (h->fused_ok) batch_seg.assign(h->n_batches, ta::kMixedBatch);        // the one-launch path keeps no histogram

    DeviceBuffers &d = h->d;
    TA_TRY(dev_alloc(&d.items, items.size()));
    TA_TRY(dev_alloc(&d.item_lo, L + 1));
    TA_TRY(dev_alloc(&d.seg_off, L));
    TA_TRY(dev_alloc(&d.seg_len, L));
    TA_TRY(dev_alloc(&d.seg_k, L));
    TA_TRY(dev_alloc(&d.state, L));
    TA_TRY(dev_alloc(&d.scratch, L));
    TA_TRY(dev_alloc(&d.status, 1));
    TA_TRY(dev_alloc(&d.p_s1, h->n_items));
    TA_TRY(dev_alloc(&d.p_s2, h->n_items));
    TA_TRY(dev_alloc(&d.p_piv, h->n_items));
    TA_TRY(dev_alloc(&d.p_amax, h->n_items));
    TA_TRY(dev_alloc(&d.p_amin, h->n_items));
    TA_TRY(dev_alloc(&d.p_bad, h->n_items));
    if (h->topk) {
        TA_TRY(dev_alloc(&d.p_sa, h->n_items));
        TA_TRY(dev_alloc(&d.p_mass, h->n_items));
        TA_TRY(dev_alloc(&d.window, L));
        {
            std::vector<uint2> none(L, make_uint2(1u, 0u));          // no guess before the first step with curvature
            TA_TRY(cudaMemcpy(d.window, none.data(), L * sizeof(uint2), cudaMemcpyHostToDevice));
        }
        TA_TRY(dev_alloc(&d.hist, (size_t)L * ta::kHistBins));
        TA_TRY(dev_alloc(&d.sel, L));
        TA_TRY(dev_alloc(&d.mask, 2 * h->mask_words));           // the current mask and the one being built
        TA_TRY(dev_alloc(&d.cand_count, L));
        TA_TRY(dev_alloc(&d.cand_val, n_total));
        TA_TRY(dev_alloc(&d.cand_idx, n_total));
        TA_TRY(dev_alloc(&d.batch_seg, h->n_batches));
        TA_TRY(cudaMemset(d.cand_count, 0, (size_t)L * sizeof(uint32_t)));

        TA_TRY(cudaMemcpy(d.batch_seg, batch_seg.data(), batch_seg.size() * sizeof(uint32_t), cudaMemcpyHostToDevice));
        TA_TRY(cudaMemset(d.hist, 0, (size_t)L * ta::kHistBins * sizeof(uint32_t)));
        TA_TRY(cudaMemset(d.sel, 0, (size_t)L * sizeof(ta::SelectState)));
        TA_TRY(cudaMemset(d.mask, 0, 2 * h->mask_words * sizeof(uint32_t)));
    }
    TA_TRY(cudaMemcpy(d.items, items.data(), items.size() * sizeof(ta::Item), cudaMemcpyHostToDevice));
    TA_TRY(cudaMemcpy(d.item_lo, item_lo.data(), (L + 1) * sizeof(uint32_t), cudaMemcpyHostToDevice));
    TA_TRY(cudaMemcpy(d.seg_off, seg_off.data(), L * sizeof(uint64_t), cudaMemcpyHostToDevice));
    TA_TRY(cudaMemcpy(d.seg_len, seg_len.data(), L * sizeof(uint64_t), cudaMemcpyHostToDevice));
    TA_TRY(cudaMemcpy(d.seg_k, h->seg_k.data(), L * sizeof(uint64_t), cudaMemcpyHostToDevice));
    std::vector<ta::LayerState> init(L);
    for (auto &s : init) {
        std::memset(&s, 0, sizeof(s));
        s.code = TA_CODE_BF16;        // BF16 is the default mode (Sec. 3.1)
        s.eta_scale = 1.0f;
        s.eta = hp->eta0;
        s.topk_mass = 0.0;
    }
    TA_TRY(cudaMemcpy(d.state, init.data(), L * sizeof(ta::LayerState), cudaMemcpyHostToDevice));
    TA_TRY(cudaMemset(d.scratch, 0, L * sizeof(ta::LayerScratch)));
    TA_TRY(cudaMemset(d.status, 0, sizeof(ta::Status)));
    if (hp->momentum != 0.f) {
        if (sharded) { snprintf(h->err, 256, "ta_create_shard: momentum is not available on a sharded model"); return bail(TA_ERR_ARG); }
        TA_TRY(dev_alloc(&d.mom, n_total));
        TA_TRY(cudaMemset(d.mom, 0, n_total * sizeof(float)));
    }
    if (h->fused_ok) {
        TA_TRY(dev_alloc(&d.barrier, 4));          // arrivals, non-finite flag; two more flags for the two-launch form
        TA_TRY(cudaMemset(d.barrier, 0, 4 * sizeof(unsigned long long)));

        TA_TRY(dev_alloc(&d.warp_head, run_plan.warp_head.size()));
        TA_TRY(cudaMemcpy(d.warp_head, run_plan.warp_head.data(), run_plan.warp_head.size() * sizeof(ta::FusedWarpHead), cudaMemcpyHostToDevice));
        TA_TRY(dev_alloc(&d.block_head, run_plan.block_head.size()));
        TA_TRY(cudaMemcpy(d.block_head, run_plan.block_head.data(), run_plan.block_head.size() * sizeof(ta::FusedBlockHead), cudaMemcpyHostToDevice));
        TA_TRY(dev_alloc(&d.block_layer, run_plan.block_layer.size()));
        TA_TRY(cudaMemcpy(d.block_layer, run_plan.block_layer.data(), run_plan.block_layer.size() * sizeof(ta::FusedBlockLayer), cudaMemcpyHostToDevice));
        TA_TRY(dev_alloc(&d.slot_table, run_plan.slot_table.size()));
        TA_TRY(cudaMemcpy(d.slot_table, run_plan.slot_table.data(), run_plan.slot_table.size() * sizeof(ta::FusedSlot), cudaMemcpyHostToDevice));
        TA_TRY(dev_alloc(&d.part, 2 * (size_t)h->fused_parts));      // the two-launch form alternates between two sets
        // the occupancy the plan counted on must hold with the shared memory it asks for
        const bool bf16 = hp->grad_dtype == TA_GRAD_BF16;
        for (int P : {0, (int)hp->num_probes}) {
            int per_sm = 0;
            TA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, h->fused_split ? sweep_half_kernel(P, bf16) : fused_kernel(P, bf16), ta::kThreads, h->fused_smem));
            if ((long long)per_sm * h->sm_count < h->fused_grid) {
                snprintf(h->err, 256, "ta_create: the one-launch grid of %d blocks is not resident (%d per SM)", h->fused_grid, per_sm);
                return bail(TA_ERR_CUDA);
            }
        }
    }
    if ((hp->flags & TA_FLAG_INPUTS_FINITE) && !sharded && !h->fused_ok && !h->topk && hp->momentum == 0.f && hp->weight_decay == 0.f) {
        // the layer-pipelined launch: its own (finer) items, the two task queues and the per-layer counters
        const PipePlan pl = plan_pipe(table, L);
        if (L < (1u << 30) && pl.sweep.size() < 0xFFFFFFFFull) {
            const bool bf16 = hp->grad_dtype == TA_GRAD_BF16;
            int per_sm = 1 << 20;
            for (int P : {0, (int)hp->num_probes}) {
                int v = 0;
                TA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&v, pipe_kernel(P, bf16), ta::kThreads, 0));
                per_sm = std::min(per_sm, v);
            }
            if (per_sm >= 1) {
                h->pipe_ok = true;
                h->pipe_per_sm = per_sm;
                h->pipe_batches = pl.batch_lo[L];
                const size_t bytes = pl.sweep.size() * sizeof(ta::PipeTask);
                TA_TRY(dev_alloc(&d.pipe_tasks_sweep, pl.sweep.size()));
                TA_TRY(cudaMemcpy(d.pipe_tasks_sweep, pl.sweep.data(), bytes, cudaMemcpyHostToDevice));
                TA_TRY(dev_alloc(&d.pipe_tasks_apply, pl.apply.size()));
                TA_TRY(cudaMemcpy(d.pipe_tasks_apply, pl.apply.data(), bytes, cudaMemcpyHostToDevice));
                TA_TRY(dev_alloc(&d.pipe_tasks_hold, pl.hold.size()));
                TA_TRY(cudaMemcpy(d.pipe_tasks_hold, pl.hold.data(), bytes, cudaMemcpyHostToDevice));
                TA_TRY(dev_alloc(&d.pipe_batch_lo, L + 1));
                TA_TRY(cudaMemcpy(d.pipe_batch_lo, pl.batch_lo.data(), (L + 1) * sizeof(uint32_t), cudaMemcpyHostToDevice));
                TA_TRY(dev_alloc(&d.pipe_bsum, h->pipe_batches));
                TA_TRY(dev_alloc(&d.pipe_layer_done, L));
                TA_TRY(dev_alloc(&d.pipe_layer_ready, L));
                TA_TRY(dev_alloc(&d.pipe_ctl, 1));
                TA_TRY(cudaMemset(d.pipe_layer_done, 0, L * sizeof(uint32_t)));
                TA_TRY(cudaMemset(d.pipe_layer_ready, 0, L * sizeof(uint32_t)));
                TA_TRY(cudaMemset(d.pipe_ctl, 0, sizeof(ta::PipeControl)));
            }
        }
    }
    TA_TRY(cudaDeviceSynchronize());
#undef TA_TRY
    g_guard_sink = nullptr;
    *out = h;
    return TA_OK;
}

int ta_create(const ta_segment *table, uint32_t L, uint64_t n_total, const ta_hparams *hp, ta_handle **out)
{
    return create_impl(table, L, n_total, hp, 0, n_total, false, out);
}

int ta_create_shard(const ta_segment *table, uint32_t L, uint64_t n_total, const ta_hparams *hp, uint64_t range_lo,
                    uint64_t range_hi, ta_handle **out)
{
    return create_impl(table, L, n_total, hp, range_lo, range_hi, true, out);
}

int ta_destroy(ta_handle *h)
{
    if (!h) return TA_OK;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(h->device);
    if (h->last_stream || h->stepped) cudaStreamSynchronize(h->last_stream);
    for (cudaEvent_t e : h->events) cudaEventDestroy(e);
    if (h->copy_back) { cudaStreamSynchronize(h->copy_back); cudaStreamDestroy(h->copy_back); }
    for (cudaEvent_t e : h->chunk_done) cudaEventDestroy(e);
    if (h->decided) cudaEventDestroy(h->decided);
    free_all(h->d, h->guards);
    cudaSetDevice(prev);
    delete h;
    return TA_OK;
}

int ta_set_lr(ta_handle *h, float eta0)
{
    if (!h) return TA_ERR_ARG;
    if (!(eta0 == eta0)) return fail(h, TA_ERR_ARG, "ta_set_lr: eta0 is NaN");
    h->hp.eta0 = eta0;
    return TA_OK;
}

const char *ta_path(const ta_handle *h)
{
    if (!h) return "";
    if (h->sharded) return "sharded: sweep, record exchange, update";
    if (h->pipe_ok) return "pipelined launch";
    if (h->fused_ok) return h->fused_split ? "two dependent launches" : "one cooperative launch";
    return h->topk ? "separate kernels with top-k selection" : "separate kernels";
}

int ta_launch_count(ta_handle *h, uint64_t *count)
{
    if (!h || !count) return TA_ERR_ARG;
    *count = h->launches;
    return TA_OK;
}

int ta_test_expire_next_wait(ta_handle *h)
{
    if (!h) return TA_ERR_ARG;
    if (!h->fused_ok || h->fused_split) return fail(h, TA_ERR_STATE, "ta_test_expire_next_wait: this handle does not use the one-launch path");
    h->expire_next_wait = true;
    return TA_OK;
}

int ta_test_check_guards(ta_handle *h)
{
    if (!h) return TA_ERR_ARG;
    if (!(h->hp.flags & TA_FLAG_GUARD_WORKSPACES)) return fail(h, TA_ERR_STATE, "ta_test_check_guards: the handle was created without TA_FLAG_GUARD_WORKSPACES");
    TA_CUDA(h, cudaStreamSynchronize(h->last_stream));
    unsigned char host[2 * kGuardBytes];
    for (size_t i = 0; i < h->guards.size(); ++i) {
        const GuardRec &g = h->guards[i];
        TA_CUDA(h, cudaMemcpy(host, g.raw, kGuardBytes, cudaMemcpyDeviceToHost));
        TA_CUDA(h, cudaMemcpy(host + kGuardBytes, static_cast<char *>(g.raw) + kGuardBytes + g.bytes, kGuardBytes, cudaMemcpyDeviceToHost));
        for (size_t b = 0; b < 2 * kGuardBytes; ++b) {
            if (host[b] != (unsigned char)kGuardFill) {
                snprintf(h->err, 256, "a guard word %s workspace %zu (%zu bytes) was overwritten", b < kGuardBytes ? "in front of" : "behind", i, g.bytes);
                return TA_ERR_STATE;
            }
        }
    }
    return TA_OK;
}

int ta_plan_one_launch(const ta_segment *table, uint32_t L, uint32_t warps, ta_run *out, uint32_t cap,
                       uint32_t *n_runs, uint32_t *warps_used, uint32_t *max_rows)
{
    if (!table || L == 0 || warps == 0 || !n_runs) return fail(nullptr, TA_ERR_ARG, "ta_plan_one_launch: table, L, warps and n_runs are required");
    uint64_t end = 0;
    for (uint32_t l = 0; l < L; ++l) {
        if (table[l].length == 0 || table[l].length > 0xFFFFFFFEull)
            return fail(nullptr, TA_ERR_ARG, "ta_plan_one_launch: segment length out of range");
        if (table[l].offset < end) return fail(nullptr, TA_ERR_ARG, "ta_plan_one_launch: segments must be ascending and non-overlapping");
        end = table[l].offset + table[l].length;
    }
    const RunPlan pl = plan_runs(table, L, warps);
    *n_runs = (uint32_t)pl.runs.size();
    if (warps_used) {
        uint32_t used = 0;
        for (uint32_t wq = 0; wq < pl.n_warps; ++wq) used += pl.warp_lo[wq + 1] > pl.warp_lo[wq] ? 1u : 0u;
        *warps_used = used;
    }
    if (max_rows) *max_rows = pl.max_slots;
    if (pl.runs.size() > cap || (!out && cap)) return fail(nullptr, TA_ERR_ARG, "ta_plan_one_launch: out is too small for the plan");
    for (uint32_t wq = 0; wq < pl.n_warps; ++wq)
        for (uint32_t r = pl.warp_lo[wq]; r < pl.warp_lo[wq + 1]; ++r)
            out[r] = ta_run{pl.runs[r].begin, pl.runs[r].len, pl.runs[r].seg, wq, 0u};
    return TA_OK;
}

int ta_plan_pipeline(const ta_segment *table, uint32_t L, uint32_t with_decisions, ta_task *out, uint64_t cap, uint64_t *n_tasks)
{
    if (!table || L == 0 || !n_tasks) return fail(nullptr, TA_ERR_ARG, "ta_plan_pipeline: table, L and n_tasks are required");
    uint64_t end = 0;
    for (uint32_t l = 0; l < L; ++l) {
        if (table[l].length == 0 || table[l].length > 0xFFFFFFFEull)
            return fail(nullptr, TA_ERR_ARG, "ta_plan_pipeline: segment length out of range");
        if (table[l].offset < end) return fail(nullptr, TA_ERR_ARG, "ta_plan_pipeline: segments must be ascending and non-overlapping");
        end = table[l].offset + table[l].length;
    }
    const PipePlan pl = plan_pipe(table, L);
    std::vector<ta::PipeTask> tasks = with_decisions ? pl.sweep : pl.hold;
    if (with_decisions) tasks.insert(tasks.end(), pl.apply.begin(), pl.apply.end());
    *n_tasks = tasks.size();
    if (tasks.size() > cap || (!out && cap)) return fail(nullptr, TA_ERR_ARG, "ta_plan_pipeline: out is too small for the queues");
    for (size_t i = 0; i < tasks.size() && out; ++i)
        out[i] = ta_task{tasks[i].begin, tasks[i].len, tasks[i].seg_type & 0x3FFFFFFFu, tasks[i].seg_type >> 30, 0u};
    return TA_OK;
}

int ta_plan_items(const ta_segment *table, uint32_t L, uint32_t sm_count, uint32_t topk, ta_run *out, uint64_t cap,
                  uint64_t *n_items, uint32_t *item_elems)
{
    if (!table || L == 0 || !n_items || sm_count == 0) return fail(nullptr, TA_ERR_ARG, "ta_plan_items: table, L, sm_count and n_items are required");
    uint64_t end = 0, n_params = 0;
    for (uint32_t l = 0; l < L; ++l) {
        if (table[l].length == 0 || table[l].length > 0xFFFFFFFEull)
            return fail(nullptr, TA_ERR_ARG, "ta_plan_items: segment length out of range");
        if (table[l].offset < end) return fail(nullptr, TA_ERR_ARG, "ta_plan_items: segments must be ascending and non-overlapping");
        end = table[l].offset + table[l].length;
        n_params += table[l].length;
    }
    const uint32_t elems = choose_item_elems(n_params, (int)sm_count);
    const ItemPlan pl = plan_items(table, L, elems, topk != 0, 0, ~0ull);
    if (pl.too_many) return fail(nullptr, TA_ERR_ARG, "ta_plan_items: too many work items");
    *n_items = pl.items.size();
    if (item_elems) *item_elems = elems;
    if (pl.items.size() > cap || (!out && cap)) return fail(nullptr, TA_ERR_ARG, "ta_plan_items: out is too small for the items");
    for (size_t i = 0; i < pl.items.size() && out; ++i)
        out[i] = ta_run{pl.items[i].begin, pl.items[i].len, pl.items[i].seg, (uint32_t)(i % ta::kWarps),
                        pl.batch_seg[i / ta::kWarps] == ta::kMixedBatch ? 0u : 1u};
    return TA_OK;
}

int ta_timing_begin(ta_handle *h, uint32_t max_steps)
{
    if (!h) return TA_ERR_ARG;
    if (max_steps > 4096) return fail(h, TA_ERR_ARG, "ta_timing_begin: at most 4096 steps");
    while (h->events.size() < 4 * (size_t)max_steps) {
        cudaEvent_t e;
        TA_CUDA(h, cudaEventCreate(&e));
        h->events.push_back(e);
    }
    h->timed_cap = max_steps;
    h->timed_used = 0;
    return TA_OK;
}

int ta_timing_end(ta_handle *h, double *ms_sweep, double *ms_decide, double *ms_update, uint32_t *steps)
{
    if (!h || !ms_sweep || !ms_decide || !ms_update || !steps) return TA_ERR_ARG;
    TA_CUDA(h, cudaStreamSynchronize(h->last_stream));
    double acc[3] = {0.0, 0.0, 0.0};
    for (uint32_t i = 0; i < h->timed_used; ++i)
        for (int k = 0; k < 3; ++k) {
            float ms = 0.f;
            TA_CUDA(h, cudaEventElapsedTime(&ms, h->events[4 * (size_t)i + k], h->events[4 * (size_t)i + k + 1]));
            acc[k] += ms;
        }
    *ms_sweep = acc[0]; *ms_decide = acc[1]; *ms_update = acc[2];
    *steps = h->timed_used;
    h->timed_cap = 0;
    h->timed_used = 0;
    return TA_OK;
}

// The whole step; with defer_apply the update kernel is left to the caller (launch_apply), who may run it
// piecewise while the weights are still arriving from the host.
static int step_impl(ta_handle *h, float *w, const void *g, const float *Hz, uint16_t *c, uint64_t probe_seed,
                     uint64_t step, void *stream, bool defer_apply)
{
    if (!h) return TA_ERR_ARG;
    if (!w || !g || !c) return fail(h, TA_ERR_ARG, "ta_step: w, g and c must not be NULL");
    if (!aligned16(w) || !aligned16(g) || !aligned16(c) || !aligned16(Hz))
        return fail(h, TA_ERR_ALIGN, "ta_step: every device pointer must be 16-byte aligned");
    if (step >= (1ull << 32)) return fail(h, TA_ERR_ARG, "ta_step: step must be below 2^32");
    if (h->stepped && step <= h->last_step) return fail(h, TA_ERR_STATE, "ta_step: step must increase from call to call");
    if (h->sharded) return fail(h, TA_ERR_STATE, "ta_step: this handle holds a shard; use ta_shard_sweep and ta_shard_apply");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool bf16 = h->hp.grad_dtype == TA_GRAD_BF16;
    const int P = Hz ? (int)h->hp.num_probes : 0;
    const bool topk = h->topk && Hz;
    DeviceBuffers &d = h->d;

    const bool timed = h->timed_used < h->timed_cap;
    cudaEvent_t *ev = timed ? &h->events[4 * (size_t)h->timed_used] : nullptr;
    if (timed) cudaEventRecord(ev[0], s);

    if (h->pipe_ok && !defer_apply) {
        const bool control = (step % h->hp.t_ctrl) == 0;
        ta::PipeArgs pa{};
        pa.tasks_s = control ? d.pipe_tasks_sweep : d.pipe_tasks_hold;
        pa.tasks_a = d.pipe_tasks_apply;
        pa.n_s = h->pipe_batches;
        pa.n_a = control ? h->pipe_batches : 0u;
        pa.batch_lo = d.pipe_batch_lo; pa.seg_len = d.seg_len; pa.bsum = d.pipe_bsum;
        pa.layer_done = d.pipe_layer_done; pa.layer_ready = d.pipe_layer_ready; pa.ctl = d.pipe_ctl;
        pa.base_s = h->pipe_base_s; pa.base_a = h->pipe_base_a; pa.epoch = h->pipe_launches + 1;
        pa.w = w; pa.g = g; pa.hz = Hz; pa.c = c; pa.n_total = h->n_total; pa.seed = probe_seed; pa.step32 = (uint32_t)step;
        pa.state = d.state; pa.scratch = d.scratch; pa.status = d.status;
        pa.dp.hp = hyper_of(h->hp); pa.dp.eta0 = h->hp.eta0; pa.dp.has_hz = Hz ? 1u : 0u;
        pa.dp.control = control ? 1u : 0u; pa.dp.topk = 0u;
        pa.L = h->L; pa.step = step;
        const unsigned grid = (unsigned)std::min<long long>((long long)h->sm_count * h->pipe_per_sm, pa.n_s);
        void *args[] = {&pa};
        TA_CUDA(h, cudaLaunchKernel(pipe_kernel(P, bf16), dim3(grid), dim3(ta::kThreads), args, 0, s));
        h->pipe_base_s += (unsigned long long)pa.n_s + grid;     // every block draws exactly one ticket past the end of each queue
        h->pipe_base_a += (unsigned long long)pa.n_a + grid;
        ++h->pipe_launches;
        ++h->launches;
        if (timed) { cudaEventRecord(ev[1], s); cudaEventRecord(ev[2], s); cudaEventRecord(ev[3], s); ++h->timed_used; }
        h->stepped = true;
        h->last_step = step;
        h->last_stream = s;
        return TA_OK;
    }

    if (h->fused_ok) {
        ta::FusedArgs fa{};
        fa.runs = d.items; fa.n_runs = h->n_items;
        fa.g = g; fa.hz = Hz; fa.n_total = h->n_total; fa.seed = probe_seed; fa.step32 = (uint32_t)step;
        fa.w = w; fa.c = c;
        fa.warp_head = d.warp_head; fa.block_head = d.block_head; fa.block_layer = d.block_layer; fa.slot_table = d.slot_table;
        fa.part = d.part; fa.n_part = h->fused_parts;
        fa.state = d.state; fa.status = d.status;
        fa.dp.hp = hyper_of(h->hp); fa.dp.eta0 = h->hp.eta0; fa.dp.has_hz = Hz ? 1u : 0u;
        fa.dp.control = (step % h->hp.t_ctrl) == 0 ? 1u : 0u; fa.dp.topk = 0u;
        fa.L = h->L; fa.cap_w = h->fused_cap_w; fa.cap_g = h->fused_cap_g;
        fa.max_slots = h->fused_slots; fa.max_block_runs = h->fused_block_runs; fa.max_block_layers = h->fused_block_layers;
        fa.step = step; fa.barrier = d.barrier; fa.barrier_base = h->barrier_base; fa.flag = d.barrier + 1;
        fa.epoch = h->fused_launches + 1;
        if (h->fused_split) {
            // two dependent launches: the sweep of this step may run beside the update of the step before (it touches
            // none of its data), so partials and the non-finite flag alternate between two sets
            const unsigned long long parity = h->fused_launches & 1ull;
            fa.part = d.part + parity * h->fused_parts;
            fa.flag = d.barrier + 2 + parity;
            fa.early_weights = 0u;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = dim3((unsigned)h->fused_grid); cfg.blockDim = dim3(ta::kThreads);
            cfg.dynamicSmemBytes = h->fused_smem; cfg.stream = s; cfg.attrs = attr; cfg.numAttrs = 1;
            void *args[] = {&fa};
            TA_CUDA(h, cudaLaunchKernelExC(&cfg, sweep_half_kernel(P, bf16), args));
            if (timed) { cudaEventRecord(ev[1], s); cudaEventRecord(ev[2], s); }
            TA_CUDA(h, cudaLaunchKernelExC(&cfg, update_half_kernel(bf16), args));
            ++h->fused_launches;
            h->launches += 2;
            if (timed) { cudaEventRecord(ev[3], s); ++h->timed_used; }
            h->stepped = true;
            h->last_step = step;
            h->last_stream = s;
            return TA_OK;
        }
        fa.early_weights = 0u;
      // the weight copies start after the sweep (measured faster than starting them with its first loads)
        if (h->expire_next_wait) { fa.barrier_base += 1ull << 40; h->expire_next_wait = false; }
        const int grid = h->fused_grid;
        void *args[] = {&fa};
        TA_CUDA(h, cudaLaunchCooperativeKernel(fused_kernel(P, bf16), dim3(grid), dim3(ta::kThreads), args, h->fused_smem, s));
        h->barrier_base += (unsigned long long)grid;
        ++h->fused_launches;
        ++h->launches;
        if (timed) { cudaEventRecord(ev[1], s); cudaEventRecord(ev[2], s); cudaEventRecord(ev[3], s); ++h->timed_used; }
        h->stepped = true;
        h->last_step = step;
        h->last_stream = s;
        return TA_OK;
    }

    ta::SweepArgs sa{};
    sa.items = d.items; sa.n_items = h->n_items; sa.n_batches = h->n_batches;
    sa.g = g; sa.hz = Hz; sa.n_total = h->n_total; sa.seed = probe_seed; sa.step = (uint32_t)step;
    sa.p_s1 = d.p_s1; sa.p_s2 = d.p_s2; sa.p_sa = d.p_sa; sa.p_piv = d.p_piv;
    sa.p_amax = d.p_amax; sa.p_amin = d.p_amin; sa.p_bad = d.p_bad;
    sa.hist = d.hist; sa.batch_seg = d.batch_seg;
    sa.mask2 = d.mask; sa.mask_words = h->mask_words; sa.window = d.window; sa.sel = d.sel;
    sa.cand_count = d.cand_count; sa.cand_val = d.cand_val; sa.cand_idx = d.cand_idx; sa.seg_off = d.seg_off;
    sa.p_mass = d.p_mass; sa.status = d.status; sa.redo = 0u;
    if (topk) TA_CUDA(h, cudaMemsetAsync(&d.status->redo_layers, 0, sizeof(uint32_t), s));
    const bool ok = bf16 ? dispatch_sweep<true>(h, P, sa, s) : dispatch_sweep<false>(h, P, sa, s);
    if (!ok) return fail(h, TA_ERR_ARG, "ta_step: unsupported probe count");
    if (timed) cudaEventRecord(ev[1], s);

    ta::DecideArgs da{};
    da.item_lo = d.item_lo; da.seg_len = d.seg_len; da.items = d.items;
    da.p_s1 = d.p_s1; da.p_s2 = d.p_s2; da.p_sa = d.p_sa; da.p_piv = d.p_piv;
    da.p_amax = d.p_amax; da.p_amin = d.p_amin; da.p_bad = d.p_bad;
    da.scratch = d.scratch; da.state = d.state; da.status = d.status;
    da.hp = hyper_of(h->hp); da.eta0 = h->hp.eta0; da.L = h->L;
    da.has_hz = Hz ? 1u : 0u; da.control = (step % h->hp.t_ctrl) == 0 ? 1u : 0u; da.topk = topk ? 1u : 0u;
    da.step = step;
    da.hist = d.hist; da.sel = d.sel; da.cand_count = d.cand_count; da.seg_k = d.seg_k; da.window = d.window;
    launch_after(ta::k_decide, h->L, 0, s, da);
    ++h->launches;

    if (topk) {
        // layers whose selection window missed are swept once more with the exact bin (nothing to do in the common case)
        sa.redo = 1u;
        if (!(bf16 ? dispatch_sweep<true>(h, P, sa, s) : dispatch_sweep<false>(h, P, sa, s)))
            return fail(h, TA_ERR_ARG, "ta_step: unsupported probe count");
        const int grid = grid_for(h);
        ta::ResolveArgs ra{d.item_lo, d.seg_off, d.seg_len, d.cand_count, d.cand_val, d.cand_idx, d.cand_count, d.mask,
                           h->mask_words, d.p_mass, d.scratch, d.sel, d.state, d.status};
        // the update needs nothing from the resolve step: both run in one launch (k_apply_resolve)
        if (timed) cudaEventRecord(ev[2], s);
        ta::ApplyArgs aa{d.items, h->n_items, h->n_batches, w, g, c, d.state, d.status, d.mom, h->hp.momentum, h->hp.weight_decay};
        const unsigned blocks = (unsigned)h->L + (unsigned)grid;
        const bool mom = d.mom != nullptr;
        if (bf16 && mom) launch_after(ta::k_apply_resolve<true, true>, blocks, 0, s, aa, ra, h->L);
        else if (bf16) launch_after(ta::k_apply_resolve<true, false>, blocks, 0, s, aa, ra, h->L);
        else if (mom) launch_after(ta::k_apply_resolve<false, true>, blocks, 0, s, aa, ra, h->L);
        else launch_after(ta::k_apply_resolve<false, false>, blocks, 0, s, aa, ra, h->L);
        ++h->launches;
        if (timed) { cudaEventRecord(ev[3], s); ++h->timed_used; }
        TA_CUDA(h, cudaGetLastError());
        h->stepped = true;
        h->last_step = step;
        h->last_stream = s;
        return TA_OK;
    }

    if (timed) cudaEventRecord(ev[2], s);
    if (!defer_apply) launch_apply(h, w, g, c, 0, h->n_items, s);
    if (timed) { cudaEventRecord(ev[3], s); ++h->timed_used; }

    TA_CUDA(h, cudaGetLastError());
    h->stepped = true;
    h->last_step = step;
    h->last_stream = s;
    return TA_OK;
}

int ta_step(ta_handle *h, float *w, const void *g, const float *Hz, uint16_t *c, uint64_t probe_seed, uint64_t step,
            void *stream)
{
    return step_impl(h, w, g, Hz, c, probe_seed, step, stream, false);
}

int ta_step_host(ta_handle *h, float *w_host, const void *g_host, const float *Hz_host, uint16_t *c_host,
                 uint64_t probe_seed, uint64_t step, void *stream)
{
    if (!h) return TA_ERR_ARG;
    if (!w_host || !g_host || !c_host) return fail(h, TA_ERR_ARG, "ta_step_host: w, g and c must not be NULL");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    DeviceBuffers &d = h->d;
    const size_t n = h->n_total;
    const size_t g_bytes = n * (h->hp.grad_dtype == TA_GRAD_BF16 ? 2 : 4);
    if (!d.st_w) {
        TA_CUDA(h, dev_alloc(&d.st_w, n));
        TA_CUDA(h, cudaMalloc(&d.st_g, std::max<size_t>(g_bytes, 16)));
        TA_CUDA(h, dev_alloc(&d.st_c, n));
        TA_CUDA(h, dev_alloc(&d.st_hz, n * h->hp.num_probes));
    }
    if (!h->fused_ok && !h->topk && h->n_items >= 64 * ta::kWarps) {
        // Large dense model: the statistics need only g and Hz, so they are copied first and the sweep and the
        // decisions run while the weights are still on their way.  The weights then arrive in chunks; each
        // chunk is updated as soon as it is there and travels back on a second stream while the next one comes in.
        constexpr uint32_t kChunks = 16;
        if (!h->copy_back) {
            TA_CUDA(h, cudaStreamCreateWithFlags(&h->copy_back, cudaStreamNonBlocking));
            TA_CUDA(h, cudaEventCreateWithFlags(&h->decided, cudaEventDisableTiming));
            for (uint32_t k = 0; k < kChunks; ++k) {
                cudaEvent_t e;
                TA_CUDA(h, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
                h->chunk_done.push_back(e);
            }
        }
        TA_CUDA(h, cudaMemcpyAsync(d.st_g, g_host, g_bytes, cudaMemcpyHostToDevice, s));
        if (Hz_host) TA_CUDA(h, cudaMemcpyAsync(d.st_hz, Hz_host, n * 4 * h->hp.num_probes, cudaMemcpyHostToDevice, s));
        const int rc = step_impl(h, d.st_w, d.st_g, Hz_host ? d.st_hz : nullptr, d.st_c, probe_seed, step, stream, true);
        if (rc != TA_OK) return rc;
        std::vector<ta::LayerState> st(h->L);
        ta::Status status;
        TA_CUDA(h, cudaMemcpyAsync(st.data(), d.state, h->L * sizeof(ta::LayerState), cudaMemcpyDeviceToHost, s));
        TA_CUDA(h, cudaMemcpyAsync(&status, d.status, sizeof(status), cudaMemcpyDeviceToHost, s));
        TA_CUDA(h, cudaEventRecord(h->decided, s));
        // chunk boundaries on whole batches of items
        uint32_t bounds[kChunks + 1];
        for (uint32_t k = 0; k <= kChunks; ++k)
            bounds[k] = k == kChunks ? h->n_items : (uint32_t)((uint64_t)h->n_items * k / kChunks) / ta::kWarps * ta::kWarps;
        auto elem_begin = [&](uint32_t k) { return h->items_host[bounds[k]].begin; };
        auto elem_end = [&](uint32_t k) { return k + 1 == kChunks ? h->items_host.back().begin + h->items_host.back().len : h->items_host[bounds[k + 1]].begin; };
        for (uint32_t k = 0; k < kChunks; ++k) {
            const uint64_t b = elem_begin(k), e = elem_end(k);
            TA_CUDA(h, cudaMemcpyAsync(d.st_w + b, w_host + b, (e - b) * 4, cudaMemcpyHostToDevice, s));
            launch_apply(h, d.st_w, d.st_g, d.st_c, bounds[k], bounds[k + 1] - bounds[k], s);
            TA_CUDA(h, cudaEventRecord(h->chunk_done[k], s));
        }
        TA_CUDA(h, cudaGetLastError());
        TA_CUDA(h, cudaEventSynchronize(h->decided));          // codes and the skip flag are on the host now
        if (!status.skipped) {
            uint32_t l = 0;
            for (uint32_t k = 0; k < kChunks; ++k) {
                const uint64_t b = elem_begin(k), e = elem_end(k);
                TA_CUDA(h, cudaStreamWaitEvent(h->copy_back, h->chunk_done[k], 0));
                TA_CUDA(h, cudaMemcpyAsync(w_host + b, d.st_w + b, (e - b) * 4, cudaMemcpyDeviceToHost, h->copy_back));
                // 16-bit copies: the parts of FP16 / BF16 layers that lie in this chunk
                while (l < h->L && h->table[l].offset + h->table[l].length <= b) ++l;
                for (uint32_t j = l; j < h->L && h->table[j].offset < e; ++j) {
                    if (st[j].code >= TA_CODE_FP32) continue;
                    const uint64_t cb = std::max<uint64_t>(b, h->table[j].offset);
                    const uint64_t ce = std::min<uint64_t>(e, h->table[j].offset + h->table[j].length);
                    if (ce > cb) TA_CUDA(h, cudaMemcpyAsync(c_host + cb, d.st_c + cb, (ce - cb) * 2, cudaMemcpyDeviceToHost, h->copy_back));
                }
            }
        }
        TA_CUDA(h, cudaStreamSynchronize(s));
        TA_CUDA(h, cudaStreamSynchronize(h->copy_back));
        return TA_OK;
    }
    TA_CUDA(h, cudaMemcpyAsync(d.st_w, w_host, n * 4, cudaMemcpyHostToDevice, s));
    TA_CUDA(h, cudaMemcpyAsync(d.st_g, g_host, g_bytes, cudaMemcpyHostToDevice, s));
    if (Hz_host) TA_CUDA(h, cudaMemcpyAsync(d.st_hz, Hz_host, n * 4 * h->hp.num_probes, cudaMemcpyHostToDevice, s));
    const int rc = ta_step(h, d.st_w, d.st_g, Hz_host ? d.st_hz : nullptr, d.st_c, probe_seed, step, stream);
    if (rc != TA_OK) return rc;
    // the new master weights of every layer, and the 16-bit copy of the layers that keep one
    std::vector<ta::LayerState> st(h->L);
    ta::Status status;
    TA_CUDA(h, cudaMemcpyAsync(st.data(), d.state, h->L * sizeof(ta::LayerState), cudaMemcpyDeviceToHost, s));
    TA_CUDA(h, cudaMemcpyAsync(&status, d.status, sizeof(status), cudaMemcpyDeviceToHost, s));
    TA_CUDA(h, cudaStreamSynchronize(s));
    if (!status.skipped) {
        const uint64_t first = h->table.front().offset, last = h->table.back().offset + h->table.back().length;
        TA_CUDA(h, cudaMemcpyAsync(w_host + first, d.st_w + first, (last - first) * 4, cudaMemcpyDeviceToHost, s));
        for (uint32_t l = 0; l < h->L;) {
            if (st[l].code >= TA_CODE_FP32) { ++l; continue; }
            uint32_t r = l;      // run of adjacent layers that keep a copy: one transfer (gaps hold stale staging data, so stop at gaps)
            while (r + 1 < h->L && st[r + 1].code < TA_CODE_FP32 &&
                   h->table[r + 1].offset == h->table[r].offset + h->table[r].length) ++r;
            const uint64_t b = h->table[l].offset, e = h->table[r].offset + h->table[r].length;
            TA_CUDA(h, cudaMemcpyAsync(c_host + b, d.st_c + b, (e - b) * 2, cudaMemcpyDeviceToHost, s));
            l = r + 1;
        }
        TA_CUDA(h, cudaStreamSynchronize(s));
    }
    return TA_OK;
}

int ta_shard_sweep(ta_handle *h, const void *g_local, const float *Hz_local, uint64_t probe_seed, uint64_t step,
                   ta_layer_record *records_out, void *stream)
{
    if (!h) return TA_ERR_ARG;
    if (!h->sharded) return fail(h, TA_ERR_STATE, "ta_shard_sweep: the handle was not made by ta_create_shard");
    if (!g_local || !records_out) return fail(h, TA_ERR_ARG, "ta_shard_sweep: g and records_out must not be NULL");
    if (!aligned16(g_local) || !aligned16(Hz_local) || (reinterpret_cast<uintptr_t>(records_out) & 7u))
        return fail(h, TA_ERR_ALIGN, "ta_shard_sweep: g and Hz must be 16-byte aligned, records_out 8-byte aligned");
    if (step >= (1ull << 32)) return fail(h, TA_ERR_ARG, "ta_shard_sweep: step must be below 2^32");
    if (h->stepped && step <= h->last_step) return fail(h, TA_ERR_STATE, "ta_shard_sweep: step must increase from call to call");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    DeviceBuffers &d = h->d;
    const bool bf16 = h->hp.grad_dtype == TA_GRAD_BF16;
    const int P = Hz_local ? (int)h->hp.num_probes : 0;
    const uint64_t local_n = h->range_hi - h->range_lo;
    // the kernels index by flat element (the probes depend on it): the local buffers are addressed through bases moved
    // back by the start of the range; only elements inside the range are ever touched
    ta::SweepArgs sa{};
    sa.items = d.items; sa.n_items = h->n_items; sa.n_batches = h->n_batches;
    sa.g = static_cast<const char *>(g_local) - h->range_lo * (bf16 ? 2 : 4);
    sa.hz = Hz_local ? Hz_local - h->range_lo : nullptr;
    sa.n_total = local_n; sa.seed = probe_seed; sa.step = (uint32_t)step;
    sa.p_s1 = d.p_s1; sa.p_s2 = d.p_s2; sa.p_sa = d.p_sa; sa.p_piv = d.p_piv;
    sa.p_amax = d.p_amax; sa.p_amin = d.p_amin; sa.p_bad = d.p_bad;
    if (h->n_items) {
        if (!(bf16 ? dispatch_sweep<true>(h, P, sa, s) : dispatch_sweep<false>(h, P, sa, s)))
            return fail(h, TA_ERR_ARG, "ta_shard_sweep: unsupported probe count");
    }
    ta::DecideArgs da{};
    da.item_lo = d.item_lo; da.seg_len = d.seg_len; da.items = d.items;
    da.p_s1 = d.p_s1; da.p_s2 = d.p_s2; da.p_sa = d.p_sa; da.p_piv = d.p_piv;
    da.p_amax = d.p_amax; da.p_amin = d.p_amin; da.p_bad = d.p_bad;
    da.has_hz = Hz_local ? 1u : 0u; da.L = h->L;
    da.record_out = reinterpret_cast<ta::LayerRecord *>(records_out);
    ta::k_decide<<<h->L, ta::kThreads, 0, s>>>(da);
    ++h->launches;
    TA_CUDA(h, cudaGetLastError());
    h->pending_step = step;
    h->pending = true;
    h->pending_has_hz = Hz_local != nullptr;
    h->last_stream = s;
    return TA_OK;
}

int ta_shard_apply(ta_handle *h, float *w_local, const void *g_local, uint16_t *c_local, const ta_layer_record *records_all,
                   uint32_t world, void *stream)
{
    if (!h) return TA_ERR_ARG;
    if (!h->sharded) return fail(h, TA_ERR_STATE, "ta_shard_apply: the handle was not made by ta_create_shard");
    if (!w_local || !g_local || !c_local || !records_all || world == 0) return fail(h, TA_ERR_ARG, "ta_shard_apply: NULL argument");
    if (!aligned16(w_local) || !aligned16(g_local) || !aligned16(c_local) || (reinterpret_cast<uintptr_t>(records_all) & 7u))
        return fail(h, TA_ERR_ALIGN, "ta_shard_apply: w, g and c must be 16-byte aligned, records_all 8-byte aligned");
    if (!h->pending) return fail(h, TA_ERR_STATE, "ta_shard_apply: no ta_shard_sweep is waiting for its records");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    DeviceBuffers &d = h->d;
    const bool bf16 = h->hp.grad_dtype == TA_GRAD_BF16;
    const uint64_t step = h->pending_step;
    ta::k_merge_records<<<(h->L + ta::kThreads - 1) / ta::kThreads, ta::kThreads, 0, s>>>(
        reinterpret_cast<const ta::LayerRecord *>(records_all), world, h->L, d.scratch);
    ta::DecideArgs da{};
    da.scratch = d.scratch; da.state = d.state; da.status = d.status;
    da.hp = hyper_of(h->hp); da.eta0 = h->hp.eta0; da.L = h->L;
    da.has_hz = h->pending_has_hz ? 1u : 0u; da.control = (step % h->hp.t_ctrl) == 0 ? 1u : 0u; da.topk = 0u;
    da.step = step;
    ta::k_commit<<<1, ta::kThreads, 0, s>>>(da);
    h->launches += 2;
    launch_apply(h, w_local - h->range_lo, static_cast<const char *>(g_local) - h->range_lo * (bf16 ? 2 : 4), c_local - h->range_lo, 0, h->n_items, s);
    TA_CUDA(h, cudaGetLastError());
    h->stepped = true;
    h->last_step = step;
    h->pending = false;
    h->last_stream = s;
    return TA_OK;
}

int ta_power_iterate(ta_handle *h, const float *u, const float *Hu, const float *V, const float *lambda_V, uint32_t m,
                     float *u_next, float *lambda_out, float *norm_out, void *stream)
{
    if (!h) return TA_ERR_ARG;
    if (!u || !Hu || !u_next || !lambda_out) return fail(h, TA_ERR_ARG, "ta_power_iterate: u, Hu, u_next and lambda_out must not be NULL");
    if (m > (uint32_t)ta::kMaxEigs) return fail(h, TA_ERR_ARG, "ta_power_iterate: at most TA_MAX_EIGS deflated vectors");
    if (m > 0 && (!V || !lambda_V)) return fail(h, TA_ERR_ARG, "ta_power_iterate: V and lambda_V are needed when m > 0");
    if (!aligned16(u) || !aligned16(Hu) || !aligned16(V) || !aligned16(u_next))
        return fail(h, TA_ERR_ALIGN, "ta_power_iterate: every flat device buffer must be 16-byte aligned");
    DeviceBuffers &d = h->d;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (!d.pw_part) {
        TA_CUDA(h, dev_alloc(&d.pw_part, (size_t)ta::kMaxEigs * h->n_items));
        TA_CUDA(h, dev_alloc(&d.pw_coef, (size_t)ta::kMaxEigs * h->L));
        TA_CUDA(h, dev_alloc(&d.pw_norm, h->L));
    }
    float *norm = norm_out ? norm_out : d.pw_norm;
    ta::PowerArgs pa{d.items, h->n_items, h->n_batches, u, Hu, V, h->n_total, m, h->L, d.pw_part, d.pw_coef, norm, u_next};
    ta::PowerLayerArgs la{d.item_lo, h->n_items, m, h->L, d.pw_part, lambda_V, d.pw_coef, lambda_out, norm};
    const int grid = grid_for(h);
    if (m > 0) {
        ta::k_power<0><<<grid, ta::kThreads, 0, s>>>(pa);
        ta::k_power_layer<0><<<h->L, ta::kThreads, 0, s>>>(la);
        h->launches += 2;
    }
    ta::k_power<1><<<grid, ta::kThreads, 0, s>>>(pa);
    ta::k_power_layer<1><<<h->L, ta::kThreads, 0, s>>>(la);
    ta::k_power<2><<<grid, ta::kThreads, 0, s>>>(pa);
    h->launches += 3;
    TA_CUDA(h, cudaGetLastError());
    h->last_stream = s;
    return TA_OK;
}

int ta_set_curvature(ta_handle *h, const float *lambda_max_host)
{
    if (!h || !lambda_max_host) return TA_ERR_ARG;
    TA_CUDA(h, cudaStreamSynchronize(h->last_stream));
    std::vector<ta::LayerState> st(h->L);
    TA_CUDA(h, cudaMemcpy(st.data(), h->d.state, h->L * sizeof(ta::LayerState), cudaMemcpyDeviceToHost));
    for (uint32_t l = 0; l < h->L; ++l) {
        if (!(lambda_max_host[l] >= 0.f)) return fail(h, TA_ERR_ARG, "ta_set_curvature: values must be finite and >= 0");
        st[l].lambda_max = lambda_max_host[l];
    }
    TA_CUDA(h, cudaMemcpy(h->d.state, st.data(), h->L * sizeof(ta::LayerState), cudaMemcpyHostToDevice));
    return TA_OK;
}

int ta_probe(ta_handle *h, uint64_t probe_seed, uint64_t step, uint32_t p, float *z_out, void *stream)
{
    if (!h) return TA_ERR_ARG;
    if (!z_out) return fail(h, TA_ERR_ARG, "ta_probe: z_out must not be NULL");
    if (!aligned16(z_out)) return fail(h, TA_ERR_ALIGN, "ta_probe: z_out must be 16-byte aligned");
    if (p >= h->hp.num_probes) return fail(h, TA_ERR_ARG, "ta_probe: p must be below num_probes");
    if (step >= (1ull << 32)) return fail(h, TA_ERR_ARG, "ta_probe: step must be below 2^32");
    const uint64_t n_vec = h->n_total / 4;
    if (n_vec == 0) return TA_OK;
    const int grid = (int)std::min<uint64_t>((n_vec + ta::kThreads - 1) / ta::kThreads, (uint64_t)h->sm_count * 16);
    ta::k_probe<<<grid, ta::kThreads, 0, static_cast<cudaStream_t>(stream)>>>(z_out, n_vec, probe_seed, (uint32_t)step, p);
    ++h->launches;
    TA_CUDA(h, cudaGetLastError());
    return TA_OK;
}

int ta_stats(ta_handle *h, ta_layer_stats *out_host, ta_step_status *status)
{
    if (!h) return TA_ERR_ARG;
    TA_CUDA(h, cudaStreamSynchronize(h->last_stream));
    if (out_host) {
        std::vector<ta::LayerState> st(h->L);
        TA_CUDA(h, cudaMemcpy(st.data(), h->d.state, h->L * sizeof(ta::LayerState), cudaMemcpyDeviceToHost));
        for (uint32_t l = 0; l < h->L; ++l) {
            ta_layer_stats &o = out_host[l];
            o.grad_mean = (float)st[l].grad_mean;
            o.grad_var = (float)st[l].grad_var;
            o.ema_mean = st[l].ema_mean;
            o.ema_var = st[l].ema_var;
            o.lambda_max = st[l].lambda_max;
            o.topk_threshold = st[l].thr;
            o.topk_mass = (float)st[l].topk_mass;
            o.eta_scale = st[l].eta_scale;
            o.k = h->seg_k[l];
            o.code = st[l].code;
            o.near_threshold = st[l].near;
        }
    }
    if (status) {
        ta::Status s;
        TA_CUDA(h, cudaMemcpy(&s, h->d.status, sizeof(s), cudaMemcpyDeviceToHost));
        status->step = s.step;
        status->nonfinite_count = s.nonfinite;
        status->skipped = s.skipped;
        std::vector<ta::LayerState> st(h->L);
        TA_CUDA(h, cudaMemcpy(st.data(), h->d.state, h->L * sizeof(ta::LayerState), cudaMemcpyDeviceToHost));
        uint32_t near = 0;
        for (uint32_t l = 0; l < h->L; ++l) near += st[l].near ? 1u : 0u;
        status->near_threshold_count = near;       // layers flagged at the last decision
    }
    return check_device_error(h);
}

int ta_precision_codes(ta_handle *h, uint8_t *out_host)
{
    if (!h || !out_host) return TA_ERR_ARG;
    TA_CUDA(h, cudaStreamSynchronize(h->last_stream));
    std::vector<ta::LayerState> st(h->L);
    TA_CUDA(h, cudaMemcpy(st.data(), h->d.state, h->L * sizeof(ta::LayerState), cudaMemcpyDeviceToHost));
    for (uint32_t l = 0; l < h->L; ++l) out_host[l] = (uint8_t)st[l].code;
    return check_device_error(h);
}

int ta_masks(ta_handle *h, const uint32_t **dev_bits, uint64_t *num_words)
{
    if (!h || !dev_bits || !num_words) return TA_ERR_ARG;
    *dev_bits = nullptr;
    *num_words = h->mask_words;
    if (!h->topk) return TA_OK;
    // two buffers take turns; which one holds the mask is decided on the device when a step commits
    TA_CUDA(h, cudaStreamSynchronize(h->last_stream));
    ta::Status st;
    TA_CUDA(h, cudaMemcpy(&st, h->d.status, sizeof(st), cudaMemcpyDeviceToHost));
    *dev_bits = h->d.mask + (size_t)(st.mask_cur & 1u) * h->mask_words;
    return TA_OK;
}

int ta_state_size(ta_handle *h, uint64_t *bytes)
{
    if (!h || !bytes) return TA_ERR_ARG;
    *bytes = sizeof(StateHeader) + h->L * sizeof(ta::LayerState) + sizeof(ta::Status) + h->mask_words * sizeof(uint32_t) +
             (h->d.mom ? h->n_total * sizeof(float) : 0);
    return TA_OK;
}

int ta_state_save(ta_handle *h, void *buf_host, uint64_t bytes)
{
    uint64_t need = 0;
    if (!h || !buf_host) return TA_ERR_ARG;
    ta_state_size(h, &need);
    if (bytes < need) return fail(h, TA_ERR_ARG, "ta_state_save: buffer too small");
    TA_CUDA(h, cudaStreamSynchronize(h->last_stream));
    char *p = static_cast<char *>(buf_host);
    StateHeader hd{};
    hd.magic = kStateMagic; hd.n_total = h->n_total; hd.last_step = h->last_step; hd.mask_words = h->mask_words;
    hd.L = h->L; hd.stepped = h->stepped ? 1u : 0u; hd.hp = h->hp;
    std::memcpy(p, &hd, sizeof(hd));
    p += sizeof(hd);
    TA_CUDA(h, cudaMemcpy(p, h->d.state, h->L * sizeof(ta::LayerState), cudaMemcpyDeviceToHost));
    p += h->L * sizeof(ta::LayerState);
    TA_CUDA(h, cudaMemcpy(p, h->d.status, sizeof(ta::Status), cudaMemcpyDeviceToHost));
    const uint32_t mask_cur = reinterpret_cast<const ta::Status *>(p)->mask_cur & 1u;
    p += sizeof(ta::Status);
    if (h->mask_words) TA_CUDA(h, cudaMemcpy(p, h->d.mask + (size_t)mask_cur * h->mask_words, h->mask_words * sizeof(uint32_t), cudaMemcpyDeviceToHost));
    p += h->mask_words * sizeof(uint32_t);
    if (h->d.mom) TA_CUDA(h, cudaMemcpy(p, h->d.mom, h->n_total * sizeof(float), cudaMemcpyDeviceToHost));
    return TA_OK;
}

int ta_state_load(ta_handle *h, const void *buf_host, uint64_t bytes)
{
    uint64_t need = 0;
    if (!h || !buf_host) return TA_ERR_ARG;
    ta_state_size(h, &need);
    if (bytes < need) return fail(h, TA_ERR_STATE, "ta_state_load: buffer smaller than this handle's state");
    const char *p = static_cast<const char *>(buf_host);
    StateHeader hd;
    std::memcpy(&hd, p, sizeof(hd));
    ta_hparams a = hd.hp, b = h->hp;
    a.eta0 = b.eta0 = 0.f;     // the learning rate may differ: it is restored from the checkpoint
    if (hd.magic != kStateMagic || hd.L != h->L || hd.n_total != h->n_total || hd.mask_words != h->mask_words ||
        std::memcmp(&a, &b, sizeof(a)) != 0)
        return fail(h, TA_ERR_STATE, "ta_state_load: checkpoint was written for another table or other hyper-parameters");
    TA_CUDA(h, cudaStreamSynchronize(h->last_stream));
    p += sizeof(hd);
    TA_CUDA(h, cudaMemcpy(h->d.state, p, h->L * sizeof(ta::LayerState), cudaMemcpyHostToDevice));
    p += h->L * sizeof(ta::LayerState);
    TA_CUDA(h, cudaMemcpy(h->d.status, p, sizeof(ta::Status), cudaMemcpyHostToDevice));
    ta::Status loaded;
    std::memcpy(&loaded, p, sizeof(loaded));
    p += sizeof(ta::Status);
    if (h->mask_words) TA_CUDA(h, cudaMemcpy(h->d.mask + (size_t)(loaded.mask_cur & 1u) * h->mask_words, p, h->mask_words * sizeof(uint32_t), cudaMemcpyHostToDevice));
    p += h->mask_words * sizeof(uint32_t);
    if (h->d.mom) TA_CUDA(h, cudaMemcpy(h->d.mom, p, h->n_total * sizeof(float), cudaMemcpyHostToDevice));
    h->hp.eta0 = hd.hp.eta0;
    h->last_step = hd.last_step;
    h->stepped = hd.stepped != 0;
    return TA_OK;
}

int ta_batch_next(ta_batch_ctrl *bc, int64_t *B_next)
{
    if (!bc || !B_next) return TA_ERR_ARG;
    if (!(bc->rho_low <= bc->rho_high) || bc->B_min > bc->B_max || bc->delta_up < 0 || bc->delta_down < 0) return TA_ERR_ARG;
    uint64_t free_b = 0, total_b = 0;
    ta_mem_reader rd = bc->mem_reader ? bc->mem_reader : default_mem_reader;
    if (rd(bc->user, &free_b, &total_b) != 0 || free_b > total_b) return TA_ERR_CUDA;
    const double usage = (double)(total_b - free_b);
    const double mem_max = bc->mem_budget_bytes ? (double)bc->mem_budget_bytes : (double)total_b;
    int64_t next = bc->B;
    if (usage < bc->rho_low * mem_max) next = bc->B + bc->delta_up;          // Sec. 3.3, first case
    else if (usage > bc->rho_high * mem_max) next = bc->B - bc->delta_down;  // second case
    next = std::max(bc->B_min, std::min(bc->B_max, next));
    bc->B = next;
    *B_next = next;
    return TA_OK;
}

#pragma GCC visibility pop
}  // extern "C"
