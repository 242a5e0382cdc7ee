// The layer-pipelined pass: one persistent launch for large dense models whose caller vouches for finite inputs.
//
// The default pass reads the gradient twice from DRAM: no layer may be updated before every layer has been screened
// for non-finite values.  When the caller takes that screen upon itself (TA_FLAG_INPUTS_FINITE), a layer can be
// updated as soon as its own statistics are complete (Sec. 3.1, 3.2: all decisions are per layer), while its gradient
// is still in the L2 cache.  This kernel runs the whole step as one queue of tasks that its blocks take in order:
//
//   sweep  batch b   statistics of seven items (2048 elements each) of one layer; the block that finishes a layer's last
//                    sweep batch combines the layer's batch sums in a fixed order, takes the layer's decisions
//                    (EMAs, code, promotion, step size: Sec. 3.1, 3.2, 3.4) and publishes them
//   apply  batch b   update + cast of the same items; waits (bounded) until the layer's decisions are published
//   both   batch b   steps without decisions (step % T_ctrl != 0, Sec. 3.4): the step size and code of every layer are
//                    known beforehand, so statistics, update and cast run in a single pass over the data
//
// A step with decisions has two queues, sweep tasks in buffer order and apply tasks layer by layer (within a layer the
// last batch first: the rows swept last are the ones most surely still in L2).  Blocks draw tickets from both; an apply
// task is handed out only once its layer's decisions are published, and until then the block keeps sweeping, so a
// layer is updated as soon as it is decided and nobody ever waits for anybody: a block polls, it never blocks, and the
// launch needs no co-residency.  A step without decisions has only the queue of single-pass tasks.
//
// Seven warps of a block sweep and update; the eighth runs the queues.  It hands tasks to the seven through a ring of
// slots in shared memory and stays a few tasks ahead of them; each of the seven works through the slots at its own
// pace (item `warp` of every task) and never meets a block-wide barrier, so its loads follow one another without gaps.
// Behind them the eighth warp retires the slots in order: it publishes a sweep task's sums (store, fence, counter),
// takes a layer's decisions when the counter says the layer is complete, draws tickets and fetches task records: all
// the dependent trips to L2 that would otherwise sit between two tasks.
#pragma once
#include "kernels.cuh"

namespace ta {

constexpr uint32_t kTaskSweep = 0u, kTaskApply = 1u, kTaskBoth = 2u, kTaskNone = 3u;      // bits 31..30 of seg_type
#ifndef TA_PIPE_APPLY_ROWS
#define TA_PIPE_APPLY_ROWS 8
#endif
#ifndef TA_PIPE_SWEEP_ROWS
#define TA_PIPE_SWEEP_ROWS 0
#endif
#ifndef TA_PIPE_RING
#define TA_PIPE_RING 3
#endif
#ifndef TA_PIPE_MIN_BLOCKS
#define TA_PIPE_MIN_BLOCKS 2
#endif
#ifndef TA_PIPE_ITEM_ELEMS
#define TA_PIPE_ITEM_ELEMS 2048
#endif
constexpr uint32_t kPipeItemElems = TA_PIPE_ITEM_ELEMS;                   // elements per item of this path
constexpr uint32_t kPipeCells = kWarps - 1;                               // items per batch: one per warp but the last
constexpr uint32_t kNoLayer = 0xFFFFFFFFu;

// One task: the batch of up to kPipeCells items that the grid of kPipeItemElems-element cells cuts out of
// [begin, begin + len), all inside layer seg.
struct PipeTask {
    uint64_t begin;
    uint32_t len;
    uint32_t seg_type;                // layer | kind << 30
    uint32_t batch;                   // number of the batch (its slot in the batch sums)
    uint32_t layer_batches;           // batches of the layer
    uint32_t pad0, pad1;
};
static_assert(sizeof(PipeTask) == 32, "task records are read as two 16-byte words");

// Statistics of one batch (kPipeCells items of one layer), sums taken around the batch's first gradient value.
struct __align__(16) BatchSums {
    double s1, s2;
    float piv;
    uint32_t n, amax, amin, bad, pad0, pad1, pad2;
};
static_assert(sizeof(BatchSums) == 48, "batch sums are read as three 16-byte words");

struct PipeControl {
    unsigned long long head_s, head_a; // tickets of the two queues handed out since the counters were last cleared
    uint32_t layers_done, pad;
};

struct PipeArgs {
    const PipeTask *tasks_s, *tasks_a;   // sweep (or single-pass) tasks; apply tasks
    uint32_t n_s, n_a;
    const uint32_t *batch_lo;         // [L + 1] first batch of every layer
    const uint64_t *seg_len;          // [L]
    BatchSums *bsum;                  // [batches]
    uint32_t *layer_done;             // [L] sweep batches of the layer finished in this launch (cleared by the deciding block)
    uint32_t *layer_ready;            // [L] number of the last launch that published the layer's decisions
    PipeControl *ctl;
    unsigned long long base_s, base_a;   // tickets handed out before this launch
    uint32_t epoch;                   // number of this launch (from 1)
    float *w;
    const void *g;
    const float *hz;
    uint16_t *c;
    uint64_t n_total, seed;
    uint32_t step32;
    LayerState *state;
    LayerScratch *scratch;
    Status *status;
    DecideParams dp;
    uint32_t L;
    unsigned long long step;
};

__device__ __forceinline__ uint32_t ld_acquire(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Shared-memory flags between the warps of a block.
__device__ __forceinline__ uint32_t ld_shared_volatile(const uint32_t *p) { return *reinterpret_cast<const volatile uint32_t *>(p); }
__device__ __forceinline__ void st_shared_volatile(uint32_t *p, uint32_t v) { *reinterpret_cast<volatile uint32_t *>(p) = v; }

constexpr uint32_t kRing = TA_PIPE_RING;                          // task slots between the queue warp and the working warps
constexpr uint32_t kWorkerSpinLimit = 1u << 23;        // a working warp gives up after about a second without a task

struct RingSlot {
    PipeTask task;
    ItemSums sums[kPipeCells];
};

// One warp: combines the batch sums of layer `seg` in a fixed order, takes the layer's decisions and publishes them;
// the warp that decides the step's last layer writes the step's status.
__device__ __forceinline__ void pipe_finish_layer(const PipeArgs &A, uint32_t seg, uint32_t lane)
{
    __threadfence();
    const uint32_t lo = A.batch_lo[seg], hi = A.batch_lo[seg + 1];
    const double pivot = (double)__ldcg(&A.bsum[lo].piv);
    double s1 = 0.0, s2 = 0.0, bad = 0.0;
    uint32_t amax = 0u, amin = 0xFFFFFFFFu;
    // the wait for this sum is what separates a layer's sweep from its update: many loads in flight per lane
#pragma unroll 8
    for (uint32_t i = lo + lane; i < hi; i += 32) {
        const uint4 *rec = reinterpret_cast<const uint4 *>(A.bsum + i);
        const uint4 a = __ldcg(rec), b = __ldcg(rec + 1);
        const uint32_t x_bad = __ldcg(&A.bsum[i].bad);
        const double x_s1 = __hiloint2double((int)a.y, (int)a.x), x_s2 = __hiloint2double((int)a.w, (int)a.z);
        const MomentSums m = rebase(x_s1, x_s2, (double)b.y, (double)__uint_as_float(b.x), pivot);
        s1 += m.s1;
        s2 += m.s2;
        bad += (double)x_bad;
        amax = max(amax, b.z);
        amin = min(amin, b.w);
    }
    s1 = warp_sum(s1);
    s2 = warp_sum(s2);
    bad = warp_sum(bad);
    amax = __reduce_max_sync(0xFFFFFFFFu, amax);
    amin = __reduce_min_sync(0xFFFFFFFFu, amin);
    uint32_t last = 0u;
    if (lane == 0) {
        const double n = (double)A.seg_len[seg];
        const double shift = s1 / n;
        double var = s2 / n - shift * shift;
        if (!(var > 0.0)) var = 0.0;
        LayerScratch sc;
        sc.mean = pivot + shift; sc.var = var; sc.sum_abs = 0.0;
        sc.bad = (unsigned long long)bad;
        sc.amax = amax; sc.amin = amin;
        uint32_t near;
        A.state[seg] = decide_layer(A.dp, A.state[seg], sc, near);
        A.scratch[seg] = sc;
        A.layer_done[seg] = 0u;
        __threadfence();
        atomicExch(A.layer_ready + seg, A.epoch);
        last = atomicAdd(&A.ctl->layers_done, 1u) + 1u == A.L ? 1u : 0u;
    }
    last = __shfl_sync(0xFFFFFFFFu, last, 0);
    if (last) {
        // every layer of this step is decided: the step's status
        __threadfence();
        double total = 0.0;
        for (uint32_t j = lane; j < A.L; j += 32) total += (double)__ldcg(&A.scratch[j].bad);
        total = warp_sum(total);
        if (lane == 0) {
            A.status->step = A.step;
            A.status->nonfinite = (unsigned long long)total;
            A.status->skipped = 0u;
            A.ctl->layers_done = 0u;
        }
    }
}

template <int P, bool BF16>
__global__ void __launch_bounds__(kThreads, (P >= 8 ? 1 : TA_PIPE_MIN_BLOCKS)) k_pipe(const PipeArgs A)
{
    __shared__ RingSlot ring[kRing];
    __shared__ uint32_t slot_seq[kRing];          // queue warp -> working warps: slot holds task number slot_seq - 1
    __shared__ uint32_t slot_done[kRing];         // working warps -> queue warp: warps through with the slot's task
    __shared__ Item sh_items[kWarps];
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    if (tid < kRing) { slot_seq[tid] = 0u; slot_done[tid] = 0u; }
    __syncthreads();

    if (warp != kPipeCells) {
        // ---------------------------------------------------------------- a working warp
        SweepArgs S{};
        S.items = sh_items; S.n_items = kPipeCells; S.n_batches = 1u;
        S.g = A.g; S.hz = A.hz; S.n_total = A.n_total; S.seed = A.seed; S.step = A.step32;
        const SinglePass sp{A.w, A.c, A.state, A.dp.eta0};
        const ApplyArgs U{sh_items, kPipeCells, 1u, A.w, A.g, A.c, A.state, A.status, nullptr, 0.f, 0.f};
        // decisions published by another block of this launch: read past L1
        const LayerState *state = A.state;
        auto decision = [state](uint32_t seg, float &eta, uint32_t &code) { eta = __ldcg(&state[seg].eta); code = __ldcg(&state[seg].code); };
        for (uint32_t n = 0;; ++n) {
            const uint32_t s = n % kRing;
            uint32_t ok = 1u;
            if (lane == 0) {
                uint32_t spins = 0;
                while (ld_shared_volatile(slot_seq + s) != n + 1u) {
                    if (++spins > kWorkerSpinLimit) { atomicExch(&A.status->device_error, 1u); ok = 0u; break; }
                    __nanosleep(32);
                }
            }
            ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
            if (!ok) return;
            const PipeTask task = ring[s].task;
            const uint32_t type = task.seg_type >> 30, seg = task.seg_type & 0x3FFFFFFFu;
            if (type == kTaskNone) return;
            // this warp's item: cell `warp` of the batch
            if (lane == 0) {
                const uint64_t end = task.begin + task.len;
                const uint64_t cell = task.begin / kPipeItemElems + warp;
                const uint64_t b = max(task.begin, cell * kPipeItemElems), e = min(end, (cell + 1) * kPipeItemElems);
                sh_items[warp] = Item{e > b ? b : end, e > b ? (uint32_t)(e - b) : 0u, seg};
            }
            __syncwarp();
            if (type == kTaskApply) {
                apply_batch<BF16, false, true, TA_PIPE_APPLY_ROWS>(U, 0u, decision);
            } else {
                ItemSums *sums = ring[s].sums;
                auto store = [sums](uint32_t it, const ItemSums &r) { sums[it] = r; };
                if (type == kTaskSweep) sweep_batch<P, BF16, false, false, (P <= 1 ? TA_PIPE_SWEEP_ROWS : 0)>(S, 0u, nullptr, store);
                else sweep_batch<P, BF16, false, true, (P <= 1 ? TA_PIPE_SWEEP_ROWS : 0)>(S, 0u, nullptr, store, sp);
            }
            __syncwarp();
            if (lane == 0) {
                __threadfence_block();
                atomicAdd(slot_done + s, 1u);
            }
        }
    }

    // -------------------------------------------------------------------- the queue warp
    auto fetch = [&](const PipeTask *tasks, uint32_t n_tasks, unsigned long long ticket) {
        PipeTask t;
        if (ticket < (unsigned long long)n_tasks) {
            const uint4 a = __ldg(reinterpret_cast<const uint4 *>(tasks + ticket));
            const uint4 b = __ldg(reinterpret_cast<const uint4 *>(tasks + ticket) + 1);
            t.begin = (uint64_t)a.x | ((uint64_t)a.y << 32); t.len = a.z; t.seg_type = a.w;
            t.batch = b.x; t.layer_batches = b.y; t.pad0 = 0u; t.pad1 = 0u;
        } else {
            t.begin = 0ull; t.len = 0u; t.seg_type = kTaskNone << 30; t.batch = 0u; t.layer_batches = 0u; t.pad0 = 0u; t.pad1 = 0u;
        }
        return t;
    };
    auto next_sweep = [&]() { return fetch(A.tasks_s, A.n_s, atomicAdd(&A.ctl->head_s, 1ull) - A.base_s); };
    auto next_apply = [&]() { return fetch(A.tasks_a, A.n_a, atomicAdd(&A.ctl->head_a, 1ull) - A.base_a); };
    // lane 0 holds the next task of either queue (kind kTaskNone once a queue has run out: a block draws exactly one
    // ticket past the end of each queue)
    PipeTask rs{}, ra{};
    if (lane == 0) {
        rs = next_sweep();
        ra = next_apply();
    }
    uint32_t n_issue = 0, n_retire = 0, idle = 0;
    uint32_t ready_seg = kNoLayer;                // the last layer whose decisions this warp saw published
    bool more = true;
    while (more || n_retire < n_issue) {
        bool progressed = false;
        // a look at the flag of the layer the next apply task belongs to; the answer is used further down
        uint32_t flag = 0u;
        if (lane == 0 && (ra.seg_type >> 30) == kTaskApply && (ra.seg_type & 0x3FFFFFFFu) != ready_seg)
            flag = *reinterpret_cast<const volatile uint32_t *>(A.layer_ready + (ra.seg_type & 0x3FFFFFFFu));
        // retire finished slots in order: publish a sweep task's sums, count the batch, decide the layer if it is complete
        while (n_retire < n_issue) {
            const uint32_t s = n_retire % kRing;
            uint32_t done = 0u;
            if (lane == 0) done = ld_shared_volatile(slot_done + s);
            done = __shfl_sync(0xFFFFFFFFu, done, 0);
            if (done != kPipeCells) break;
            uint32_t finish = kNoLayer;
            if (lane == 0) {
                __threadfence_block();
                const PipeTask t = ring[s].task;
                if ((t.seg_type >> 30) != kTaskApply) {
                    // the batch's items in order, around the first item's pivot
                    const ItemSums *sums = ring[s].sums;
                    BatchSums b{0.0, 0.0, sums[0].piv, 0u, 0u, 0xFFFFFFFFu, 0u, 0u, 0u, 0u};
                    for (uint32_t k = 0; k < kPipeCells; ++k) {
                        const ItemSums x = sums[k];
                        const MomentSums m = rebase(x.s1, x.s2, (double)x.n, (double)x.piv, (double)b.piv);
                        b.s1 += m.s1; b.s2 += m.s2; b.n += x.n;
                        b.amax = max(b.amax, x.amax); b.amin = min(b.amin, x.amin);
                        b.bad += x.bad;
                    }
                    A.bsum[t.batch] = b;
                    __threadfence();
                    const uint32_t seg = t.seg_type & 0x3FFFFFFFu;
                    if (atomicAdd(A.layer_done + seg, 1u) + 1u == t.layer_batches) finish = seg;      // the layer's last batch
                }
                st_shared_volatile(slot_done + s, 0u);
            }
            finish = __shfl_sync(0xFFFFFFFFu, finish, 0);
            ++n_retire;
            progressed = true;
            if (finish != kNoLayer) pipe_finish_layer(A, finish, lane);
        }
        // hand out the next task: an apply task if its layer is decided, else a sweep task
        if (more && n_issue - n_retire < kRing) {
            uint32_t pick = 0u;       // 0: nothing can be handed out now, 1: apply, 2: sweep, 3: both queues are empty
            if (lane == 0) {
                const uint32_t a_kind = ra.seg_type >> 30, s_kind = rs.seg_type >> 30, a_seg = ra.seg_type & 0x3FFFFFFFu;
                if (a_kind == kTaskApply && a_seg != ready_seg && flag == A.epoch) {
                    __threadfence();              // what the deciding block wrote before the flag is visible from here on
                    ready_seg = a_seg;
                }
                if (a_kind == kTaskApply && a_seg == ready_seg) pick = 1u;
                else if (s_kind != kTaskNone) pick = 2u;
                else if (a_kind == kTaskNone) pick = 3u;
                if (pick != 0u) {
                    const uint32_t s = n_issue % kRing;
                    ring[s].task = pick == 1u ? ra : rs;          // with pick 3 rs is the "no task" record
                    __threadfence_block();
                    st_shared_volatile(slot_seq + s, n_issue + 1u);
                    if (pick == 1u) ra = next_apply();
                    else if (pick == 2u) rs = next_sweep();
                }
            }
            pick = __shfl_sync(0xFFFFFFFFu, pick, 0);
            if (pick == 3u) more = false;                 // the working warps leave when they reach this slot
            else if (pick != 0u) ++n_issue;
            if (pick != 0u) progressed = true;
        }
        if (progressed) {
            idle = 0;
        } else {
            // nothing to retire and nothing to hand out: the other warps are busy, or the layer of the next apply task is
            // being decided elsewhere
            if (++idle > kWorkerSpinLimit) { if (lane == 0) atomicExch(&A.status->device_error, 1u); more = false; }
            __nanosleep(32);
        }
    }
}

}  // namespace ta
