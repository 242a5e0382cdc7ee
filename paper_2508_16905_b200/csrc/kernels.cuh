// Device code of the Tri-Accel optimizer pass for sm_100a.
//
// The flat parameter buffer is cut into "rows" of 128 consecutive elements on a global grid
// (row r covers flat indices [128 r, 128 r + 128)).  A warp reads one row per instruction:
// lane j owns the four elements 128 r + 4 j .. + 3, i.e. one 16-byte vector of a float buffer.
// 32 rows make a 4096-element block; the Rademacher bits of lane j for a whole block come from
// one Philox call, so a lane pays one generator call per 128 elements it touches.
//
// Work is described by "items": a contiguous piece of ONE layer, handled by one warp.  Items are
// cut on the global row grid, so only the first and last row of a layer can be partial; partial
// rows take a scalar path with per-element bounds checks.  Gaps between layers are never touched.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

// Tuning constants (rows of 128 elements a lane keeps in flight).
#ifndef TA_SWEEP_ROWS_P1
#define TA_SWEEP_ROWS_P1 8
#endif
#ifndef TA_SWEEP_ROWS_P1_BF16
#define TA_SWEEP_ROWS_P1_BF16 8
#endif
#ifndef TA_SWEEP_ROWS_P2
#define TA_SWEEP_ROWS_P2 4
#endif
#ifndef TA_SWEEP_ROWS_P4
#define TA_SWEEP_ROWS_P4 2
#endif
#ifndef TA_SWEEP_MIN_BLOCKS_P4
#define TA_SWEEP_MIN_BLOCKS_P4 2
#endif
#ifndef TA_APPLY_ROWS
#define TA_APPLY_ROWS 8
#endif
#ifndef TA_APPLY_ROWS_BF16
#define TA_APPLY_ROWS_BF16 16
#endif
#ifndef TA_APPLY_STREAM_W_STORE
#define TA_APPLY_STREAM_W_STORE 0
#endif
// One-launch path: blocks per SM the compiler must leave room for (with one probe or none; two blocks with two or four
// probes, one with eight, whose rows need more registers), slots in flight in the sweep (P <= 1) and in the update.
#ifndef TA_FUSED_MIN_BLOCKS
#define TA_FUSED_MIN_BLOCKS 3
#endif
#ifndef TA_FUSED_SWEEP_SLOTS
#define TA_FUSED_SWEEP_SLOTS 4
#endif
#ifndef TA_FUSED_UPDATE_SLOTS
#define TA_FUSED_UPDATE_SLOTS 4
#endif

namespace ta {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr uint32_t kNonFiniteBits = 0x7F800000u;   // |x| bit patterns at or above this are inf / NaN
constexpr int kHistBins = 2048;                    // radix-select levels: 11 + 11 + 9 bits of |S|

struct Item {
    uint64_t begin;   // first flat element
    uint32_t len;     // elements, all inside layer `seg`
    uint32_t seg;
};

// Per-layer state kept on the device between steps.
struct LayerState {
    double grad_mean, grad_var, topk_mass;
    float ema_mean, ema_var;        // m_l, v_l                     (Sec. 3.1)
    float lambda_max, thr;          // max|S|/P, k-th largest |S|   (Sec. 3.2)
    float eta_scale, eta;           // s_l, eta_l = eta0 * s_l      (Sec. 3.2)
    uint32_t code, near;            // precision code               (Sec. 3.1)
};

// Per-layer results of one sweep, before the decision to commit or skip the step.
struct LayerScratch {
    double mean, var, sum_abs;
    unsigned long long bad;
    uint32_t amax, amin;
};

struct Status {
    unsigned long long step, nonfinite;
    uint32_t skipped, near_count;
    uint32_t done_counter, device_error;   // device_error: a bounded wait inside a kernel ran out
    uint32_t mask_cur;                     // top-k: which of the two mask buffers holds the current mask
    uint32_t redo_layers;                  // top-k: layers of this step whose guessed selection window missed
};

// Per-layer bookkeeping of the radix select.
struct SelectState {
    uint32_t prefix;      // level-1 bin (bits 30..20 of |S|) of the layer's k-th largest |S|
    uint32_t remaining;   // how many elements are still to be taken inside that bin
    uint32_t thr_bits;    // final threshold bit pattern
    uint32_t take_equal;  // how many elements equal to the threshold belong to the mask
    uint32_t surplus;     // 1: more elements equal the threshold than are taken (index tie-break needed)
    uint32_t valid;       // 1: the window the sweep collected candidates in contains the bin
    uint32_t lo_bin;      // lowest bin the layer's candidate list holds
    uint32_t pad;
};

// What one rank of a sharded pass knows about a layer after its sweep: the sums over the elements it holds, taken
// around its first gradient value of the layer.  Ranks exchange these records and every rank combines them in rank order.
struct LayerRecord {
    double s1, s2;        // sums of (g - pivot) and (g - pivot)^2
    double n;             // elements of the layer on this rank (0: none, the other fields are then ignored)
    float pivot;
    uint32_t amax, amin;  // largest / smallest |S| as bit patterns
    uint32_t bad;         // non-finite inputs
};
static_assert(sizeof(LayerRecord) == 40, "the record is part of the C ABI (ta_layer_record)");

struct Hyper {
    float beta, tau_low, tau_high, tau_curv, alpha;
    uint32_t num_probes, t_ctrl, topk_ppm;
};

// ------------------------------------------------------------------ Philox-4x32-10

// Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3" (SC'11).
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t (&out)[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Bits of lane `slot` for the 4096-element block `block`: 128 bits, bit 4*row + comp.
__device__ __forceinline__ void probe_bits(uint64_t block, uint32_t slot, uint64_t seed, uint32_t step,
                                           uint32_t p, uint32_t (&out)[4])
{
    const uint64_t q = block * 32ull + slot;
    philox4x32_10((uint32_t)q, (uint32_t)(q >> 32), step, p, (uint32_t)seed, (uint32_t)(seed >> 32), out);
}

__device__ __forceinline__ uint32_t pick_word(const uint32_t (&x)[4], uint32_t j)
{
    uint32_t lo = (j & 1u) ? x[1] : x[0];
    uint32_t hi = (j & 1u) ? x[3] : x[2];
    return (j & 2u) ? hi : lo;
}

// ------------------------------------------------------------------ small helpers

// Dependencies between consecutive launches of one stream that the hardware resolves (no spinning): a launch may
// start while its predecessor still runs, and waits here until the predecessor is complete and its writes are visible.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// From here on the next launch of the stream may start.
__device__ __forceinline__ void grid_dependency_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }


__device__ __forceinline__ float4 ld_stream(const float *p)
{
    return __ldcs(reinterpret_cast<const float4 *>(p));
}
__device__ __forceinline__ float4 ld_keep(const float *p)
{
    return __ldg(reinterpret_cast<const float4 *>(p));
}

// Loads that take no line of the L1 cache: for kernels that give most of the SM's memory to shared memory, where
// the few lines left to L1 would otherwise bound the number of loads in flight.
__device__ __forceinline__ float4 ld_no_l1(const float *p)
{
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ld_no_l1(const uint2 *p)
{
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}

// Asynchronous copies to shared memory (no register is held while the data travels).
__device__ __forceinline__ void cp_async16_stream(void *smem, const void *gmem)
{
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async8_stream(void *smem, const void *gmem)
{
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(s), "l"(gmem) : "memory");
}
// The same with a say in what L2 keeps: `policy` from createpolicy (evict_first for data that is read once,
// evict_last for data that a later kernel of the step reads again).
__device__ __forceinline__ void cp_async16_hint(void *smem, const void *gmem, uint64_t policy)
{
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(s), "l"(gmem), "l"(policy) : "memory");
}
__device__ __forceinline__ void cp_async8_hint(void *smem, const void *gmem, uint64_t policy)
{
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.ca.shared.global.L2::cache_hint [%0], [%1], 8, %2;" ::"r"(s), "l"(gmem), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t l2_evict_first_policy()
{
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}
__device__ __forceinline__ uint64_t l2_evict_last_policy()
{
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}
__device__ __forceinline__ void cp_async_commit_group() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <bool BF16> struct GradVec;
template <> struct GradVec<false> {
    static __device__ __forceinline__ float4 load4(const void *g, uint64_t i, bool stream)
    {
        const float *p = static_cast<const float *>(g) + i;
        return stream ? ld_stream(p) : ld_keep(p);
    }
    static __device__ __forceinline__ float load1(const void *g, uint64_t i)
    {
        return __ldg(static_cast<const float *>(g) + i);
    }
    static __device__ __forceinline__ float4 load4_no_l1(const void *g, uint64_t i)
    {
        return ld_no_l1(static_cast<const float *>(g) + i);
    }
};
template <> struct GradVec<true> {
    static __device__ __forceinline__ float4 load4(const void *g, uint64_t i, bool stream)
    {
        const uint2 *p = reinterpret_cast<const uint2 *>(static_cast<const uint16_t *>(g) + i);
        const uint2 v = stream ? __ldcs(p) : __ldg(p);
        float4 r;
        r.x = __uint_as_float(v.x << 16);
        r.y = __uint_as_float(v.x & 0xFFFF0000u);
        r.z = __uint_as_float(v.y << 16);
        r.w = __uint_as_float(v.y & 0xFFFF0000u);
        return r;
    }
    static __device__ __forceinline__ float load1(const void *g, uint64_t i)
    {
        return __uint_as_float((uint32_t)__ldg(static_cast<const uint16_t *>(g) + i) << 16);
    }
    static __device__ __forceinline__ float4 load4_no_l1(const void *g, uint64_t i)
    {
        const uint2 v = ld_no_l1(reinterpret_cast<const uint2 *>(static_cast<const uint16_t *>(g) + i));
        float4 r;
        r.x = __uint_as_float(v.x << 16);
        r.y = __uint_as_float(v.x & 0xFFFF0000u);
        r.z = __uint_as_float(v.y << 16);
        r.w = __uint_as_float(v.y & 0xFFFF0000u);
        return r;
    }
};

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Sum over a 256-thread block in a fixed order; result valid in every thread.
__device__ __forceinline__ double block_sum(double v, double *smem /*[kWarps]*/)
{
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) smem[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) t += smem[w];
    return t;
}

// ------------------------------------------------------------------ phase A: the sweep

struct SweepArgs {
    const Item *items;
    uint32_t n_items, n_batches;
    const void *g;
    const float *hz;          // [P][n_total] or unused when P == 0
    uint64_t n_total;
    uint64_t seed;
    uint32_t step;
    // per-item partial results; p_s1 / p_s2 are sums of (x - pivot) and (x - pivot)^2, the pivot being the item's
    // first gradient value (p_piv): the variance of a layer whose mean is far larger than its spread then comes out
    // of numbers of the size of the spread instead of the difference of two nearly equal sums
    double *p_s1, *p_s2, *p_sa;
    float *p_piv;
    uint32_t *p_amax, *p_amin, *p_bad;
    // top-k only.  The sweep selects as it goes: from the last step with curvature it knows, per layer, a window of
    // level-1 bins (bits 30..20 of |S|) in which the k-th largest |S| should fall again.  Elements above the window get
    // their mask bit at once, elements inside it are listed as candidates, and the level-1 histogram tells afterwards
    // whether the window held.  Where it did not (or there was none: the first step), a second launch with redo = 1
    // repeats the layer with the exact bin.  All of it goes to the mask buffer that is not current; the buffers swap
    // roles when the step commits.
    uint32_t *hist;           // [L][kHistBins], level-1 histogram of |S| bit patterns
    const uint32_t *batch_seg; // [n_batches] layer of a batch whose items all lie in one layer, else kMixedBatch
    uint32_t *mask2;          // two buffers of mask_words words
    uint64_t mask_words;
    const uint2 *window;      // [L] lowest and highest bin of the window (lowest > highest: no guess)
    const SelectState *sel;   // [L] redo: the exact bin and whether the layer needs the second pass
    uint32_t *cand_count;     // [L]
    uint32_t *cand_val;       // [n_total], candidates of layer l at seg_off[l] ...
    uint32_t *cand_idx;       // [n_total]
    const uint64_t *seg_off;  // [L]
    double *p_mass;           // per item: sum of |S| above the window
    const Status *status;
    uint32_t redo;
};

constexpr uint32_t kMixedBatch = 0xFFFFFFFFu;

constexpr uint32_t kStageCap = 384;      // candidates a warp collects in shared memory before it reserves list slots

// Stages this lane's candidates (bit e of `cand` = element e of its vector) in the warp's shared-memory buffer.
// A lane with candidates reserves its places on the warp's counter `count` (a shared-memory word); `bound` is a
// warp-uniform upper bound of that counter, which is all the caller needs to know when to empty the buffer.
// Whole warp; returns whether anything was staged.  The order of the staged candidates is arbitrary (so is the order
// of the layer's list).
__device__ __forceinline__ bool stage_candidates(uint32_t cand, const uint32_t (&ab)[4], uint32_t local0,
                                                 uint32_t &bound, uint32_t *count, uint32_t *sval, uint32_t *sidx)
{
    const uint32_t who = __ballot_sync(0xFFFFFFFFu, cand != 0u);
    if (who == 0u) return false;
    bound += 4u * (uint32_t)__popc(who);
    if (cand != 0u) {
        uint32_t pos = atomicAdd(count, (uint32_t)__popc(cand));
#pragma unroll
        for (uint32_t e = 0; e < 4; ++e)
            if ((cand >> e) & 1u) {
                sval[pos] = ab[e];
                sidx[pos] = local0 + e;
                ++pos;
            }
    }
    return true;
}

// 8 lanes make one 32-bit mask word out of their 4-bit pieces.
__device__ __forceinline__ uint32_t gather_word(uint32_t nib, uint32_t lane)
{
    uint32_t word = nib << ((lane & 7u) * 4u);
    word |= __shfl_xor_sync(0xFFFFFFFFu, word, 1);
    word |= __shfl_xor_sync(0xFFFFFFFFu, word, 2);
    word |= __shfl_xor_sync(0xFFFFFFFFu, word, 4);
    return word;
}

template <int P> struct RowData {
    float4 g;
    float4 hz[P > 0 ? P : 1];
    float4 w;                 // only used by the single-pass variant of the sweep
};

// w <- fl32(w - eta g) for one 16-byte vector, stored together with its 16-bit cast when the layer keeps a copy
// (code 0: binary16, 1: bfloat16, 2: none).  Sec. 3.2 step, Sec. 2 master copy and cast.
template <bool STREAM_W>
__device__ __forceinline__ void update_store4(float *w, uint16_t *c, uint64_t i0, float4 wv, const float4 gv, float neg_eta, uint32_t code)
{
    wv.x = fmaf(neg_eta, gv.x, wv.x);
    wv.y = fmaf(neg_eta, gv.y, wv.y);
    wv.z = fmaf(neg_eta, gv.z, wv.z);
    wv.w = fmaf(neg_eta, gv.w, wv.w);
    if (STREAM_W) __stcs(reinterpret_cast<float4 *>(w + i0), wv);
    else *reinterpret_cast<float4 *>(w + i0) = wv;
    if (code == 0u) {
        const __half2 a = __floats2half2_rn(wv.x, wv.y), b = __floats2half2_rn(wv.z, wv.w);
        uint2 o;
        o.x = *reinterpret_cast<const uint32_t *>(&a);
        o.y = *reinterpret_cast<const uint32_t *>(&b);
        __stcs(reinterpret_cast<uint2 *>(c + i0), o);
    } else if (code == 1u) {
        const __nv_bfloat162 a = __floats2bfloat162_rn(wv.x, wv.y), b = __floats2bfloat162_rn(wv.z, wv.w);
        uint2 o;
        o.x = *reinterpret_cast<const uint32_t *>(&a);
        o.y = *reinterpret_cast<const uint32_t *>(&b);
        __stcs(reinterpret_cast<uint2 *>(c + i0), o);
    }
}

__device__ __forceinline__ uint16_t cast16(float x, uint32_t code)
{
    return code == 0u ? __half_as_ushort(__float2half_rn(x)) : __bfloat16_as_ushort(__float2bfloat16_rn(x));
}

// What the single-pass variant of the sweep needs besides the sweep's own arguments: on a step without decisions the
// step size and the precision code of every layer are known beforehand (Sec. 3.4: decisions only every T_ctrl steps),
// so the update can be applied in the pass that gathers the statistics.
struct SinglePass {
    float *w;
    uint16_t *c;
    const LayerState *state;
    float eta0;
};

// Balanced pairwise sum: adjacent pairs, level by level.
template <int P> __device__ __forceinline__ float pairwise(const float (&t)[P > 0 ? P : 1])
{
    if constexpr (P == 2) {
        return __fadd_rn(t[0], t[1]);
    } else if constexpr (P == 4) {
        return __fadd_rn(__fadd_rn(t[0], t[1]), __fadd_rn(t[2], t[3]));
    } else if constexpr (P == 8) {
        return __fadd_rn(__fadd_rn(__fadd_rn(t[0], t[1]), __fadd_rn(t[2], t[3])),
                         __fadd_rn(__fadd_rn(t[4], t[5]), __fadd_rn(t[6], t[7])));
    } else {
        return t[0];
    }
}

template <int P, bool TOPK> struct SweepAcc {
    double pivot = 0.0;     // subtracted from every gradient value before it is summed
    double s1 = 0.0, s2 = 0.0, sa = 0.0;
    float sa_row = 0.f;     // |S| of the current row (four values), folded into sa by end_row()
    uint32_t amax = 0u, amin = 0xFFFFFFFFu;   // amin is kept only without top-k (it is the dense threshold)

    __device__ __forceinline__ void end_row() { sa += (double)sa_row; sa_row = 0.f; }

    // A non-finite gradient value (or pivot) makes s2 non-finite, and finite values cannot: |x| < 2^129, so
    // the sum of 2^64 squares still fits a double.  That is the screen of the gradients; no maximum is kept.
    static __device__ __forceinline__ bool gradients_suspect(double s2_total) { return !(s2_total < (double)INFINITY); }

    // one element: gradient value gv, probe products hv[p], sign words of the row sel[p] with the sign bit of the
    // lane's element 0 moved to bit 28 (element e: bit 28 + e), e = 0..3
    __device__ __forceinline__ uint32_t element(float gv, const float (&hv)[P > 0 ? P : 1],
                                                const uint32_t (&sel)[P > 0 ? P : 1], uint32_t e)
    {
        const double x = (double)gv - pivot;
        s1 += x;
        s2 = fma(x, x, s2);
        uint32_t ab = 0u;
        if (P == 1) {
            ab = __float_as_uint(hv[0]) & 0x7FFFFFFFu;       // |z h| = |h|
        } else if (P > 1) {
            float t[P > 0 ? P : 1];
#pragma unroll
            for (int p = 0; p < P; ++p) {
                const uint32_t hb = __float_as_uint(hv[p]);
                t[p] = __uint_as_float(hb ^ ((sel[p] << (3u - e)) & 0x80000000u));
            }
            ab = __float_as_uint(pairwise<P>(t)) & 0x7FFFFFFFu;
        }
        if (P > 0) {
            amax = max(amax, ab);
            if (!TOPK) amin = min(amin, ab);
            if (TOPK) sa_row += __uint_as_float(ab);
        }
        return ab;
    }
};

// What one item contributes to its layer's statistics (valid in lane 0 of the warp that swept it).
struct ItemSums {
    double s1, s2, sa;           // sums of (g - piv), (g - piv)^2 and |S|
    float piv;
    uint32_t n, amax, amin, bad;
};

// One batch (eight items, one per warp) of the sweep.  Called by the whole block.  `store(it, sums)` is called by
// lane 0 of each warp with the results of item `it`.  APPLY: the single-pass variant, which also updates the weights
// of the rows it sweeps (with the step size and code the layers had before this step) and writes their 16-bit copies.
// RING > 0: full rows travel through a ring of RING rows per warp in shared memory (sh_ring, [kWarps][RING][1 + P] rows
// of 32 x 16 bytes), filled by asynchronous copies that run ahead of the arithmetic: a warp then has loads in flight
// all the time, not only between two bursts, which is what the multi-probe sweeps (many instructions per byte) need.
// HIST (top-k) says at compile time where the batch counts its level-1 histogram, which spares the row loop the
// tests: 0 nowhere (the second sweep), 1 in shared memory (all items in one layer), 2 in the layers' own histograms.
template <int P, bool BF16, bool TOPK, bool APPLY, int ROWS = 0, int RING = 0, int HIST = 1, typename Store>
__device__ __forceinline__ void sweep_batch(const SweepArgs &A, uint32_t batch, uint32_t *sh_hist, const Store &store,
                                            const SinglePass &sp = SinglePass{nullptr, nullptr, nullptr, 0.f},
                                            uint32_t *sh_stage = nullptr /* TOPK: [kWarps][2][kStageCap], then [kWarps] counters */,
                                            float4 *sh_ring = nullptr)
{
    static_assert(!(RING > 0 && (APPLY || P == 0)), "the ring is for sweeps with probe products");
    static_assert(!(APPLY && TOPK), "the single-pass variant is for dense curvature");
    constexpr int PP = P > 0 ? P : 1;
    constexpr int U = RING > 0 ? 1 : ROWS > 0 ? ROWS : (P <= 1) ? (BF16 ? TA_SWEEP_ROWS_P1_BF16 : TA_SWEEP_ROWS_P1)
                               : (P == 2 ? TA_SWEEP_ROWS_P2 : TA_SWEEP_ROWS_P4);     // rows in flight per lane
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    {
        const uint32_t it = batch * kWarps + warp;
        // a batch whose items share one layer counts its histogram in shared memory and flushes it once
        constexpr bool uniform = TOPK && HIST == 1, redo = TOPK && HIST == 0;
        uint32_t batch_layer = 0;
        if (TOPK && !redo) {          // (the second sweep counts nothing)
            batch_layer = A.batch_seg[batch];
            if (uniform)
                for (uint32_t b = threadIdx.x; b < (uint32_t)kHistBins; b += kThreads) sh_hist[b] = 0u;
            __syncthreads();
        }
        Item item = it < A.n_items ? A.items[it] : Item{0, 0, 0};
        if (it < A.n_items && item.len == 0u && lane == 0) {   // padding item: neutral partials
            store(it, ItemSums{0.0, 0.0, 0.0, 0.f, 0u, 0u, 0xFFFFFFFFu, 0u});
            if (TOPK) A.p_mass[it] = 0.0;
        }
        // top-k: the window of level-1 bins this pass works with, and whether it touches the mask at all
        uint32_t win_lo = 1u, win_hi = 0u;
        if (TOPK && item.len != 0u) {
            if (redo) {
                const SelectState ss = A.sel[item.seg];
                if (ss.valid) item.len = 0u;                   // the first pass got this layer right
                win_lo = win_hi = ss.prefix;
            } else {
                const uint2 win = A.window[item.seg];
                win_lo = win.x; win_hi = win.y;
            }
        }
        const bool masking = TOPK && win_lo <= win_hi;
        // the same window on the bit patterns: above it from thr_hi on (2^31 when the window ends at the last bin: no
        // pattern of a magnitude reaches that), inside it from thr_lo on
        const uint32_t thr_lo = win_lo << 20, thr_hi = (win_hi + 1u) << 20;
        if (item.len != 0u) {
        const uint64_t begin = item.begin, end = begin + item.len;
        const uint64_t row_first = begin >> 7, row_last = (end - 1) >> 7;
        SweepAcc<P, TOPK> acc;
        const float piv = GradVec<BF16>::load1(A.g, begin);
        acc.pivot = (double)piv;
        float neg_eta = 0.f;
        uint32_t code = 2u;
        if (APPLY) {
            neg_eta = -__fmul_rn(sp.eta0, sp.state[item.seg].eta_scale);
            code = sp.state[item.seg].code;
        }
        auto hist_add = [&](uint32_t ab) {
            if (redo) return;
            if (uniform) atomicAdd(&sh_hist[ab >> 20], 1u);
            else atomicAdd(A.hist + (uint64_t)item.seg * kHistBins + (ab >> 20), 1u);
        };
        // top-k: mask bits above the window, candidates inside it
        const uint64_t seg_b = TOPK ? A.seg_off[item.seg] : 0ull;
        uint32_t *mask = TOPK ? A.mask2 + (size_t)(redo ? A.status->mask_cur : 1u - A.status->mask_cur) * A.mask_words : nullptr;
        uint32_t *sval = TOPK ? sh_stage + (size_t)warp * 2u * kStageCap : nullptr, *sidx = TOPK ? sval + kStageCap : nullptr;
        uint32_t *scount = TOPK ? sh_stage + (size_t)kWarps * 2u * kStageCap + warp : nullptr;      // candidates staged by this warp
        uint32_t staged = 0u;                                   // upper bound of *scount, warp-uniform
        double mass = 0.0;
        if (TOPK) {
            if (lane == 0) *scount = 0u;
            __syncwarp();
        }
        // moves the staged candidates to the layer's list: one slot reservation for all of them
        auto flush = [&]() {
            if (staged == 0u) return;
            __syncwarp();
            const uint32_t n = *scount;
            uint32_t base = 0;
            if (lane == 0) base = atomicAdd(A.cand_count + item.seg, n);
            base = __shfl_sync(0xFFFFFFFFu, base, 0);
            for (uint32_t j = lane; j < n; j += 32) {
                A.cand_val[seg_b + base + j] = sval[j];
                A.cand_idx[seg_b + base + j] = sidx[j];
            }
            __syncwarp();
            if (lane == 0) *scount = 0u;
            __syncwarp();
            staged = 0u;
        };
        // one row: ab = |S| patterns of this lane's four elements, inside = which of them belong to the item
        auto mask_row = [&](uint64_t row, const uint32_t (&ab)[4], uint32_t inside, bool whole) {
            uint32_t nib = 0u, cand = 0u;
            float above = 0.f;
#pragma unroll
            for (uint32_t e = 0; e < 4; ++e) {
                const bool over = ab[e] >= thr_hi, reach = ab[e] >= thr_lo;       // selects, no branches
                nib |= over ? 1u << e : 0u;
                cand |= reach ? 1u << e : 0u;
                above += over ? __uint_as_float(ab[e]) : 0.f;
            }
            nib &= inside;
            cand &= inside & ~nib;
            if (!whole) {         // elements outside the item carry no value, but say so where it costs nothing
                above = 0.f;
#pragma unroll
                for (uint32_t e = 0; e < 4; ++e) above += (nib >> e) & 1u ? __uint_as_float(ab[e]) : 0.f;
            }
            mass += (double)above;
            if (staged + 128u > kStageCap) flush();
            stage_candidates(cand, ab, (uint32_t)(row * 128ull - seg_b) + lane * 4u, staged, scount, sval, sidx);
            if (whole) {
                // two lanes make one byte of the row's 16 mask bytes (little-endian words: byte j = bits 8j .. 8j+7)
                const uint32_t pair = nib | (__shfl_xor_sync(0xFFFFFFFFu, nib, 1) << 4);
                if ((lane & 1u) == 0u) reinterpret_cast<uint8_t *>(mask)[row * 16ull + (lane >> 1)] = (uint8_t)pair;
                return;
            }
            const uint32_t word = gather_word(nib, lane);
            if ((lane & 7u) == 0u) {
                const uint64_t w0 = row * 128ull + (lane >> 3) * 32ull;     // first element of this word
                uint32_t *dst = mask + (w0 >> 5);
                if (whole || (w0 >= begin && w0 + 32u <= end)) {
                    *dst = word;
                } else if (w0 + 32u > begin && w0 < end) {
                    // the other bits of this word belong to a neighbouring layer or a gap: replace only ours
                    const uint32_t lo_bit = begin > w0 ? (uint32_t)(begin - w0) : 0u;
                    const uint32_t hi_bit = end < w0 + 32u ? (uint32_t)(end - w0) : 32u;     // exclusive
                    const uint32_t ours = (hi_bit == 32u ? 0xFFFFFFFFu : ((1u << hi_bit) - 1u)) & ~((1u << lo_bit) - 1u);
                    atomicAnd(dst, ~ours);
                    if (word) atomicOr(dst, word);
                }
            }
        };
        uint32_t X[PP][4];
        uint64_t have_block = ~0ull;

        auto refresh = [&](uint64_t row) {
            if (P > 1) {
                const uint64_t blk = row >> 5;
                if (blk != have_block) {
#pragma unroll
                    for (int p = 0; p < PP; ++p) probe_bits(blk, lane, A.seed, A.step, (uint32_t)p, X[p]);
                    have_block = blk;
                }
            }
        };

        // scalar path for a row that is not entirely inside [begin, end)
        auto partial_row = [&](uint64_t row) {
            refresh(row);
            const uint32_t k = (uint32_t)(row & 31u);
            uint32_t sel[PP];
#pragma unroll
            for (int p = 0; p < PP; ++p) sel[p] = (P > 1) ? pick_word(X[p], k >> 3) << (28u - (k & 7u) * 4u) : 0u;
            const uint64_t i0 = row * 128ull + lane * 4u;
            uint32_t abs4[4] = {0u, 0u, 0u, 0u}, inside = 0u;
#pragma unroll
            for (uint32_t e = 0; e < 4; ++e) {
                const uint64_t i = i0 + e;
                if (i >= begin && i < end) {
                    float hv[PP];
#pragma unroll
                    for (int p = 0; p < PP; ++p) hv[p] = (P > 0) ? __ldcs(A.hz + (uint64_t)p * A.n_total + i) : 0.f;
                    const float gv = GradVec<BF16>::load1(A.g, i);
                    const uint32_t ab = acc.element(gv, hv, sel, e);
                    abs4[e] = ab;
                    inside |= 1u << e;
                    if (APPLY) {
                        const float wn = fmaf(neg_eta, gv, sp.w[i]);
                        sp.w[i] = wn;
                        if (code < 2u) sp.c[i] = cast16(wn, code);
                    }
                    if (TOPK) hist_add(ab);
                }
            }
            if (TOPK) {
                acc.end_row();
                if (masking) mask_row(row, abs4, inside, false);
            }
        };

        // top-k bookkeeping of one full row: level-1 histogram, mask bits, candidates
        auto count_row = [&](const uint32_t (&abs4)[4]) {
            // exact zeros (pruned or untouched weights) would all hit one counter: the warp counts them together
            uint32_t zeros = 0u;
#pragma unroll
            for (uint32_t e = 0; e < 4; ++e) {
                zeros += (uint32_t)__popc(__ballot_sync(0xFFFFFFFFu, abs4[e] == 0u));
                if (abs4[e] != 0u) hist_add(abs4[e]);
            }
            if (lane == 0 && !redo) {
                if (uniform) atomicAdd(&sh_hist[0], zeros);
                else atomicAdd(A.hist + (uint64_t)item.seg * kHistBins, zeros);
            }
        };
        auto book_row = [&](uint64_t row, const uint32_t (&abs4)[4]) {
            const uint32_t least = min(min(abs4[0], abs4[1]), min(abs4[2], abs4[3]));
            if (__any_sync(0xFFFFFFFFu, least == 0u)) {
                count_row(abs4);
            } else {
#pragma unroll
                for (uint32_t e = 0; e < 4; ++e) hist_add(abs4[e]);
            }
            if (masking) mask_row(row, abs4, 0xFu, true);
        };
        auto full_rows = [&](uint64_t row, RowData<P> (&rd)[U], int count) {
            uint32_t abs_all[U][4];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (u < count) {
                    const uint32_t k = (uint32_t)((row + u) & 31u);
                    uint32_t sel[PP];
#pragma unroll
                    for (int p = 0; p < PP; ++p) sel[p] = (P > 1) ? pick_word(X[p], k >> 3) << (28u - (k & 7u) * 4u) : 0u;
                    const float gv[4] = {rd[u].g.x, rd[u].g.y, rd[u].g.z, rd[u].g.w};
#pragma unroll
                    for (uint32_t e = 0; e < 4; ++e) {
                        float hv[PP];
#pragma unroll
                        for (int p = 0; p < PP; ++p) {
                            const float4 h = rd[u].hz[p];
                            hv[p] = e == 0 ? h.x : (e == 1 ? h.y : (e == 2 ? h.z : h.w));
                        }
                        abs_all[u][e] = acc.element(gv[e], hv, sel, e);
                    }
                    if (TOPK) acc.end_row();
                    if (APPLY) update_store4<true>(sp.w, sp.c, (row + u) * 128ull + lane * 4u, rd[u].w, rd[u].g, neg_eta, code);
                }
            }
            if constexpr (TOPK) {
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (u < count) book_row(row + u, abs_all[u]);
            }
        };

        auto load_rows = [&](uint64_t row, RowData<P> (&rd)[U], int count) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (u < count) {
                    const uint64_t i0 = (row + u) * 128ull + lane * 4u;
                    rd[u].g = GradVec<BF16>::load4(A.g, i0, APPLY);       // read once when the update rides along
#pragma unroll
                    for (int p = 0; p < PP; ++p)
                        if (P > 0) rd[u].hz[p] = ld_stream(A.hz + (uint64_t)p * A.n_total + i0);
                    if (APPLY) rd[u].w = ld_stream(sp.w + i0);
                }
            }
        };

        // rows [full_lo, full_hi) lie entirely inside the item; at most one partial row at each end
        const uint64_t full_lo = (begin + 127) >> 7, full_hi = end >> 7;
        const bool head_partial = (begin & 127u) != 0u;
        const bool tail_partial = (end & 127u) != 0u && !(head_partial && row_last == row_first);
        if (head_partial) partial_row(row_first);
        if constexpr (RING > 0) {
            if (full_hi > full_lo) {
            // this lane's 16-byte pieces of RING rows are on their way while it works on the oldest one; a lane reads
            // back only what it copied itself, so the wait for its own copies is all the ordering needed
            float4 *mine = sh_ring + (size_t)warp * RING * (1 + PP) * 32u + lane;
            const uint64_t keep = l2_evict_last_policy(), once = l2_evict_first_policy();
            auto issue = [&](uint64_t row, int slot) {
                if (row < full_hi) {
                    const uint64_t i0 = row * 128ull + lane * 4u;
                    float4 *dst = mine + (size_t)slot * (1 + PP) * 32u;
                    // the update reads the gradient again, nothing reads the probe products again
                    if (BF16) cp_async8_hint(dst, static_cast<const uint16_t *>(A.g) + i0, keep);
                    else cp_async16_hint(dst, static_cast<const float *>(A.g) + i0, keep);
#pragma unroll
                    for (int p = 0; p < PP; ++p) cp_async16_hint(dst + (size_t)(1 + p) * 32u, A.hz + (uint64_t)p * A.n_total + i0, once);
                }
                cp_async_commit_group();          // one group per row, empty behind the last row, so that the count below holds
            };
#pragma unroll
            for (int r = 0; r < RING; ++r) issue(full_lo + r, r);
            int slot = 0;
            auto take = [&](int sl, RowData<P> &r) {
                const float4 *src = mine + (size_t)sl * (1 + PP) * 32u;
                if (BF16) {
                    const uint2 v = *reinterpret_cast<const uint2 *>(src);
                    r.g = make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u),
                                      __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xFFFF0000u));
                } else {
                    r.g = src[0];
                }
#pragma unroll
                for (int p = 0; p < PP; ++p) r.hz[p] = src[(size_t)(1 + p) * 32u];
            };
            for (uint64_t row = full_lo; row < full_hi; ++row) {
                RowData<P> rd[U];
                cp_async_wait_group<RING - 1>();
                refresh(row);
                take(slot, rd[0]);
                issue(row + RING, slot);          // the slot is free again: the values are in registers
                full_rows(row, rd, 1);
                slot = slot + 1 == RING ? 0 : slot + 1;
            }
            cp_async_wait_group<0>();
            }
        } else if (full_hi > full_lo) {
            uint64_t row = full_lo;
            RowData<P> rd[U];
            // single rows up to the next multiple of U, so that an unrolled group never crosses a 32-row block
            while (row < full_hi && (row & (U - 1))) {
                refresh(row);
                load_rows(row, rd, 1);
                full_rows(row, rd, 1);
                ++row;
            }
            while (row + U <= full_hi) {
                refresh(row);
                load_rows(row, rd, U);
                full_rows(row, rd, U);
                row += U;
            }
            while (row < full_hi) {
                refresh(row);
                load_rows(row, rd, 1);
                full_rows(row, rd, 1);
                ++row;
            }
        }
        if (tail_partial) partial_row(row_last);

        // warp reduction
        const double s1 = warp_sum(acc.s1), s2 = warp_sum(acc.s2);
        const double sa = TOPK ? warp_sum(acc.sa) : 0.0;
        const uint32_t amax = __reduce_max_sync(0xFFFFFFFFu, acc.amax);
        const uint32_t amin = __reduce_min_sync(0xFFFFFFFFu, acc.amin);
        // a non-finite Hz value always makes its probe sum non-finite, so max|S| flags it (a sum of finite values
        // that overflows also lands here; the exact recount below then finds nothing)
        const uint32_t hmax = amax;
        uint32_t bad = 0;
        if (SweepAcc<P, TOPK>::gradients_suspect(s2) || (P > 0 && hmax >= kNonFiniteBits)) {
            // rare: count the non-finite inputs of this item exactly
            for (uint64_t i = begin + lane; i < end; i += 32) {
                if ((__float_as_uint(GradVec<BF16>::load1(A.g, i)) & 0x7FFFFFFFu) >= kNonFiniteBits) ++bad;
                for (int p = 0; p < P; ++p)
                    if ((__float_as_uint(A.hz[(uint64_t)p * A.n_total + i]) & 0x7FFFFFFFu) >= kNonFiniteBits) ++bad;
            }
            bad = __reduce_add_sync(0xFFFFFFFFu, bad);
        }
        if (lane == 0) store(it, ItemSums{s1, s2, sa, piv, item.len, amax, amin, bad});
        if (masking) {
            flush();
            mass = warp_sum(mass);
            if (lane == 0) A.p_mass[it] = mass;
        }
        }   // item.len != 0
        if (TOPK && !redo) {
            __syncthreads();
            if (uniform)
                for (uint32_t b = threadIdx.x; b < (uint32_t)kHistBins; b += kThreads) {
                    const uint32_t v = sh_hist[b];
                    if (v) atomicAdd(A.hist + (uint64_t)batch_layer * kHistBins + b, v);
                }
            __syncthreads();
        }
    }
}

// Rows per warp in the shared-memory ring of the top-k sweeps: two blocks per SM must fit with their 32 KB of
// histogram and candidate staging (3 rows of 2.5 KB with four probes: 61 KB per block).
__host__ __device__ constexpr int sweep_ring_rows(int P) { return P >= 8 ? 2 : (P >= 4 ? 3 : (P == 2 ? 4 : 6)); }
__host__ __device__ constexpr size_t sweep_ring_bytes(int P) { return (size_t)kWarps * sweep_ring_rows(P) * (1 + P) * 512u; }

template <int P, bool BF16, bool TOPK>
__global__ void __launch_bounds__(kThreads, ((P == 4 || TOPK) && P <= 4 ? 2 : 1)) k_sweep(const SweepArgs A)
{
    __shared__ uint32_t sh_hist[TOPK ? kHistBins : 1];
    __shared__ uint32_t sh_stage[TOPK ? kWarps * 2 * kStageCap + kWarps : 1];     // + one counter per warp
    extern __shared__ __align__(16) float4 sh_ring[];          // TOPK: kWarps * kSweepRing<P> rows of (1 + P) x 512 bytes
    grid_dependency_wait();         // launched ahead of time: the kernel before this one is complete from here on
    grid_dependency_release();
    if (TOPK && A.redo && (A.status->skipped || A.status->redo_layers == 0u)) return;      // nothing to repeat
    auto store = [&A](uint32_t it, const ItemSums &r) {
        A.p_s1[it] = r.s1;
        A.p_s2[it] = r.s2;
        A.p_piv[it] = r.piv;
        A.p_bad[it] = r.bad;
        if (P > 0) { A.p_amax[it] = r.amax; A.p_amin[it] = r.amin; }
        if (TOPK) A.p_sa[it] = r.sa;
    };
    constexpr int R = TOPK ? sweep_ring_rows(P) : 0;
    const SinglePass none{nullptr, nullptr, nullptr, 0.f};
    for (uint32_t batch = blockIdx.x; batch < A.n_batches; batch += gridDim.x) {
        if (!TOPK) sweep_batch<P, BF16, TOPK, false, 0, R>(A, batch, sh_hist, store, none, sh_stage, sh_ring);
        else if (A.redo) sweep_batch<P, BF16, TOPK, false, 0, R, 0>(A, batch, sh_hist, store, none, sh_stage, sh_ring);
        else if (A.batch_seg[batch] != kMixedBatch) sweep_batch<P, BF16, TOPK, false, 0, R, 1>(A, batch, sh_hist, store, none, sh_stage, sh_ring);
        else sweep_batch<P, BF16, TOPK, false, 0, R, 2>(A, batch, sh_hist, store, none, sh_stage, sh_ring);
    }
}

// ------------------------------------------------------------------ decisions

// Sums of (x - p) and (x - p)^2 over n values, moved from pivot p to pivot q:  with d = p - q,
//   sum (x - q) = s1 + n d,   sum (x - q)^2 = s2 + d (2 s1 + n d).
struct MomentSums { double s1, s2; };
__device__ __forceinline__ MomentSums rebase(double s1, double s2, double n, double p, double q)
{
    const double d = p - q;
    return MomentSums{fma(n, d, s1), fma(d, fma(n, d, 2.0 * s1), s2)};
}

// Whole block: the bin in which the `need`-th element falls when bins are walked from the top
// (DESC) or from the bottom, and how many elements lie in the bins walked before it.
template <bool DESC>
__device__ __forceinline__ void block_find_bin(const uint32_t *h, int bins, uint32_t need, uint32_t *scan /*[kThreads]*/,
                                               uint32_t *out /*[2]*/)
{
    const int tid = threadIdx.x, per = bins / kThreads;
    uint32_t mine = 0;
    for (int j = 0; j < per; ++j) {
        const int pos = per * tid + j;
        mine += h[DESC ? bins - 1 - pos : pos];
    }
    scan[tid] = mine;
    __syncthreads();
    for (int o = 1; o < kThreads; o <<= 1) {
        const uint32_t add = tid >= o ? scan[tid - o] : 0u;
        __syncthreads();
        scan[tid] += add;
        __syncthreads();
    }
    const uint32_t incl = scan[tid], before_me = incl - mine;
    if (before_me < need && need <= incl) {
        uint32_t cum = before_me;
        for (int j = 0; j < per; ++j) {
            const int pos = per * tid + j;
            const int b = DESC ? bins - 1 - pos : pos;
            const uint32_t cnt = h[b];
            if (cum < need && need <= cum + cnt) { out[0] = (uint32_t)b; out[1] = cum; }
            cum += cnt;
        }
    }
    __syncthreads();
}


struct DecideArgs {
    const uint32_t *item_lo;        // [L + 1] first item of each layer
    const uint64_t *seg_len;        // [L]
    const Item *items;
    const double *p_s1, *p_s2, *p_sa;
    const float *p_piv;
    const uint32_t *p_amax, *p_amin, *p_bad;
    LayerScratch *scratch;          // [L]
    LayerState *state;              // [L]
    Status *status;
    Hyper hp;
    float eta0;
    uint32_t L;
    uint32_t has_hz, control, topk;
    unsigned long long step;
    // top-k only: level-1 histogram [L][kHistBins], selection bookkeeping, candidate counters, mask population
    uint32_t *hist;
    SelectState *sel;
    uint32_t *cand_count;
    const uint64_t *seg_k;
    uint2 *window;                  // [L] the bins the sweep collected candidates in; rewritten for the next step
    LayerRecord *record_out;        // sharded pass: [L] this rank's sums per layer are written here and nothing is decided
};

// Reads another block's results past the L1 cache (they were published with a fence).
__device__ __forceinline__ LayerScratch load_scratch(const LayerScratch *p)
{
    LayerScratch sc;
    sc.mean = __ldcg(&p->mean);
    sc.var = __ldcg(&p->var);
    sc.sum_abs = __ldcg(&p->sum_abs);
    sc.bad = __ldcg(&p->bad);
    sc.amax = __ldcg(&p->amax);
    sc.amin = __ldcg(&p->amin);
    return sc;
}

struct DecideParams {
    Hyper hp;
    float eta0;
    uint32_t has_hz, control, topk;
};

// Sec. 3.1 (EMAs, code cases), Sec. 3.2 (step size, promotion), Sec. 3.4 (control interval):
// the new state of one layer from its old state and this step's statistics.
__device__ __forceinline__ LayerState decide_layer(const DecideParams &P, LayerState st, const LayerScratch &sc, uint32_t &near)
{
    const double beta = (double)P.hp.beta;
    st.grad_mean = sc.mean;
    st.grad_var = sc.var;
    st.ema_mean = (float)(beta * (double)st.ema_mean + (1.0 - beta) * sc.mean);
    st.ema_var = (float)(beta * (double)st.ema_var + (1.0 - beta) * sc.var);
    if (P.has_hz) {
        st.lambda_max = __fdiv_rn(__uint_as_float(sc.amax), (float)P.hp.num_probes);
        if (!P.topk) { st.thr = __uint_as_float(sc.amin); st.topk_mass = 1.0; }
    }
    near = 0;
    if (P.control) {
        const float v = st.ema_var;
        uint32_t code = v < P.hp.tau_low ? 0u : (v < P.hp.tau_high ? 1u : 2u);
        if (st.lambda_max > P.hp.tau_curv && code < 2u) code += 1u;
        st.code = code;
        st.eta_scale = __fdiv_rn(1.0f, __fadd_rn(1.0f, __fmul_rn(P.hp.alpha, st.lambda_max)));
        if (fabs((double)v - (double)P.hp.tau_low) <= 1e-5 * fabs((double)P.hp.tau_low)) near = 1;
        if (fabs((double)v - (double)P.hp.tau_high) <= 1e-5 * fabs((double)P.hp.tau_high)) near = 1;
        if (fabs((double)st.lambda_max - (double)P.hp.tau_curv) <= 1e-5 * fabs((double)P.hp.tau_curv)) near = 1;
        st.near = near;
    }
    st.eta = __fmul_rn(P.eta0, st.eta_scale);
    return st;
}

__device__ __forceinline__ uint32_t commit_layer(const DecideArgs &A, uint32_t l)
{
    DecideParams P;
    P.hp = A.hp; P.eta0 = A.eta0; P.has_hz = A.has_hz; P.control = A.control; P.topk = A.topk;
    uint32_t near;
    A.state[l] = decide_layer(P, A.state[l], load_scratch(A.scratch + l), near);
    return near;
}

// Whole block: screens the step for non-finite input over all layers and, if it is clean, commits every layer
// (EMAs, codes, step sizes); writes the step's status.
__device__ __forceinline__ void commit_step(const DecideArgs &A, double *red)
{
    const uint32_t tid = threadIdx.x;
    double total_bad = 0.0;
    for (uint32_t j = tid; j < A.L; j += kThreads)
        total_bad += (double)__ldcg(&A.scratch[j].bad);
    total_bad = block_sum(total_bad, red);
    double near = 0.0;
    if (total_bad == 0.0)
        for (uint32_t j = tid; j < A.L; j += kThreads) near += (double)commit_layer(A, j);
    near = block_sum(near, red);
    if (A.topk && total_bad != 0.0)          // a skipped step: what the sweep listed is of no use
        for (uint32_t j = tid; j < A.L; j += kThreads) A.cand_count[j] = 0u;
    if (tid == 0) {
        A.status->step = A.step;
        A.status->nonfinite = (unsigned long long)total_bad;
        A.status->skipped = total_bad != 0.0 ? 1u : 0u;
        if (A.control && total_bad == 0.0) A.status->near_count = (uint32_t)near;
        if (A.topk && total_bad == 0.0) A.status->mask_cur ^= 1u;       // the buffer the sweep wrote becomes the mask
        A.status->done_counter = 0u;
    }
}

// One block per layer combines the layer's item partials in a fixed order; the block that
// finishes last screens the whole step for non-finite input and commits every layer.
__global__ void __launch_bounds__(kThreads) k_decide(const DecideArgs A)
{
    __shared__ double red[kWarps];
    __shared__ uint32_t red_u[2][kWarps];
    __shared__ uint32_t is_last;
    __shared__ uint32_t h[kHistBins];
    __shared__ uint32_t scan[kThreads];
    __shared__ uint32_t found[2];
    const uint32_t l = blockIdx.x, tid = threadIdx.x;
    grid_dependency_wait();
    grid_dependency_release();
    const uint32_t lo = A.item_lo[l], hi = A.item_lo[l + 1];
    if (A.topk) {
        // level-1 digit (bits 30..20) of the layer's k-th largest |S|; the histogram is cleared for the next
        // step.  These are scratch results: harmless when the step turns out to be skipped.
        uint32_t *gh = A.hist + (uint64_t)l * kHistBins;
        uint32_t bins[kHistBins / kThreads];
#pragma unroll
        for (int j = 0; j < kHistBins / kThreads; ++j) bins[j] = gh[j * kThreads + tid];      // all loads in flight at once
#pragma unroll
        for (int j = 0; j < kHistBins / kThreads; ++j) { h[j * kThreads + tid] = bins[j]; gh[j * kThreads + tid] = 0u; }
        __syncthreads();
        const uint32_t k = (uint32_t)A.seg_k[l];
        block_find_bin<true>(h, kHistBins, k, scan, found);
        if (tid == 0) {
            // did the window the sweep worked with contain the bin?  If not, its candidates are dropped and the layer
            // is repeated with the exact bin.  Either way the next step starts from a window around this bin.
            const uint2 win = A.window[l];
            SelectState s;
            s.prefix = found[0];
            s.remaining = k - found[1];
            s.thr_bits = 0u; s.take_equal = 0u; s.surplus = 0u; s.pad = 0u;
            s.valid = (win.x <= win.y && win.x <= found[0] && found[0] <= win.y) ? 1u : 0u;
            s.lo_bin = s.valid ? win.x : found[0];
            A.sel[l] = s;
            if (!s.valid) {
                A.cand_count[l] = 0u;
                atomicAdd(&A.status->redo_layers, 1u);
            }
            // how far the bin moves from one step to the next is a matter of the layer's size: the k-th largest of a few
            // thousand values wanders over several bins (an eighth of an octave each), that of millions stays put.  A wide
            // window costs candidates, so only small layers get one; their second sweep would be cheap anyway.
            const uint64_t n_l = A.seg_len[l];
            const uint32_t half = n_l >= (1ull << 19) ? 0u : (n_l >= (1ull << 13) ? 3u : 8u);
            A.window[l] = make_uint2(found[0] > half ? found[0] - half : 0u, min(found[0] + half, (uint32_t)kHistBins - 1u));
        }
    }
    double s1 = 0.0, s2 = 0.0, sa = 0.0, bad = 0.0;
    uint32_t amax = 0u, amin = 0xFFFFFFFFu;
    // every item summed around its own pivot; here the sums are moved to the pivot of the layer's first item
    const float pivot_f = lo < hi ? A.p_piv[lo] : 0.f;
    const double pivot = (double)pivot_f;
    double n_local = 0.0;
    // Eight items per thread and trip, all their loads issued before the first is used (a layer of thousands of
    // items is otherwise a chain of dependent trips to memory); each thread still adds its items in ascending order.
    constexpr int kTrip = 8;
    for (uint32_t i0 = lo + tid; i0 < hi; i0 += kThreads * kTrip) {
        double x_s1[kTrip], x_s2[kTrip], x_sa[kTrip];
        float x_piv[kTrip];
        uint32_t x_len[kTrip], x_bad[kTrip], x_amax[kTrip], x_amin[kTrip];
#pragma unroll
        for (int k = 0; k < kTrip; ++k) {
            const uint32_t i = i0 + (uint32_t)k * kThreads;
            const bool in = i < hi;
            x_s1[k] = in ? A.p_s1[i] : 0.0;
            x_s2[k] = in ? A.p_s2[i] : 0.0;
            x_piv[k] = in ? A.p_piv[i] : pivot_f;
            x_len[k] = in ? A.items[i].len : 0u;
            x_bad[k] = in ? A.p_bad[i] : 0u;
            x_amax[k] = in && A.has_hz ? A.p_amax[i] : 0u;
            x_amin[k] = in && A.has_hz ? A.p_amin[i] : 0xFFFFFFFFu;
            x_sa[k] = in && A.has_hz && A.topk ? A.p_sa[i] : 0.0;
        }
#pragma unroll
        for (int k = 0; k < kTrip; ++k) {
            if (i0 + (uint32_t)k * kThreads < hi) {
                const MomentSums m = rebase(x_s1[k], x_s2[k], (double)x_len[k], (double)x_piv[k], pivot);
                s1 += m.s1;
                s2 += m.s2;
                n_local += (double)x_len[k];
                bad += (double)x_bad[k];
                amax = max(amax, x_amax[k]);
                amin = min(amin, x_amin[k]);
                sa += x_sa[k];
            }
        }
    }
    s1 = block_sum(s1, red);
    s2 = block_sum(s2, red);
    sa = block_sum(sa, red);
    bad = block_sum(bad, red);
    if (A.record_out) n_local = block_sum(n_local, red);
    amax = __reduce_max_sync(0xFFFFFFFFu, amax);
    amin = __reduce_min_sync(0xFFFFFFFFu, amin);
    if ((tid & 31) == 0) { red_u[0][tid >> 5] = amax; red_u[1][tid >> 5] = amin; }
    __syncthreads();
    if (A.record_out) {
        if (tid == 0) {
            for (int w = 1; w < kWarps; ++w) { amax = max(amax, red_u[0][w]); amin = min(amin, red_u[1][w]); }
            A.record_out[l] = LayerRecord{s1, s2, n_local, pivot_f, amax, amin, (uint32_t)min(bad, 4294967295.0)};
        }
        return;
    }
    if (tid == 0) {
        for (int w = 1; w < kWarps; ++w) { amax = max(amax, red_u[0][w]); amin = min(amin, red_u[1][w]); }
        const double n = (double)A.seg_len[l];
        const double shift = s1 / n;
        double var = s2 / n - shift * shift;
        if (!(var > 0.0)) var = 0.0;
        LayerScratch sc;
        sc.mean = pivot + shift; sc.var = var; sc.sum_abs = sa;
        sc.bad = (unsigned long long)bad;
        sc.amax = amax; sc.amin = amin;
        A.scratch[l] = sc;
        __threadfence();
        const uint32_t ticket = atomicAdd(&A.status->done_counter, 1u);
        is_last = (ticket == A.L - 1) ? 1u : 0u;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    commit_step(A, red);
}

// Sharded pass: the records of all ranks for every layer, [world][L], combined in rank order (so that every rank
// arrives at the same numbers), give the layer's statistics.  One thread per layer.
__global__ void __launch_bounds__(kThreads) k_merge_records(const LayerRecord *all, uint32_t world, uint32_t L, LayerScratch *scratch)
{
    const uint32_t l = blockIdx.x * kThreads + threadIdx.x;
    if (l >= L) return;
    double pivot = 0.0, s1 = 0.0, s2 = 0.0, n = 0.0, bad = 0.0;
    uint32_t amax = 0u, amin = 0xFFFFFFFFu;
    bool have = false;
    for (uint32_t r = 0; r < world; ++r) {
        const LayerRecord x = all[(size_t)r * L + l];
        if (!(x.n > 0.0)) continue;
        if (!have) { pivot = (double)x.pivot; have = true; }
        const MomentSums m = rebase(x.s1, x.s2, x.n, (double)x.pivot, pivot);
        s1 += m.s1; s2 += m.s2; n += x.n; bad += (double)x.bad;
        amax = max(amax, x.amax); amin = min(amin, x.amin);
    }
    const double shift = n > 0.0 ? s1 / n : 0.0;
    double var = n > 0.0 ? s2 / n - shift * shift : 0.0;
    if (!(var > 0.0)) var = 0.0;
    LayerScratch sc;
    sc.mean = pivot + shift; sc.var = var; sc.sum_abs = 0.0;
    sc.bad = (unsigned long long)bad;
    sc.amax = amax; sc.amin = amin;
    scratch[l] = sc;
}

__global__ void __launch_bounds__(kThreads) k_commit(const DecideArgs A)
{
    __shared__ double red[kWarps];
    commit_step(A, red);
}

// ------------------------------------------------------------------ phase B: update + cast

struct ApplyArgs {
    const Item *items;
    uint32_t n_items, n_batches;
    float *w;
    const void *g;
    uint16_t *c;
    const LayerState *state;
    const Status *status;
    float *mom;                  // momentum buffer [n_total] or NULL
    float momentum, weight_decay;
};

// Direction of the SGD update (Sec. 4.1): d = g + wd w, then b = mu b + d with the buffer updated in place.
// One float rounding each.
__device__ __forceinline__ float sgd_direction(float g, float w, float *buf, float momentum, float weight_decay)
{
    float d = weight_decay != 0.f ? fmaf(weight_decay, w, g) : g;
    if (buf) { d = fmaf(momentum, *buf, d); *buf = d; }
    return d;
}

// w <- fl32(w - eta_l g) (Sec. 3.2, Sec. 4.1); c <- RNE cast of the new w for FP16 / BF16 layers (Sec. 2).
// One batch of the update.  `decision(seg, eta, code)` supplies the layer's step size and precision code.
// MOM: the launch has a momentum buffer; its rows are loaded together with the weights and gradients, and fewer rows
// are kept in flight.
// STREAM_W: the new weights are stored with the streaming hint (first to leave L2), for callers that keep other data
// in L2 on purpose.
// ROWS: rows of loads a lane keeps in flight (0: the default for the gradient type).
template <bool BF16, bool MOM, bool STREAM_W, int ROWS = 0, typename Decision>
__device__ __forceinline__ void apply_batch(const ApplyArgs &A, uint32_t batch, const Decision &decision)
{
    constexpr int U0 = ROWS > 0 ? ROWS : (BF16 ? TA_APPLY_ROWS_BF16 : TA_APPLY_ROWS);
    constexpr int U = MOM ? U0 / 2 : U0;
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    {
        const uint32_t it = batch * kWarps + warp;
        if (it >= A.n_items) return;
        const Item item = A.items[it];
        if (item.len == 0u) return;
        const uint64_t begin = item.begin, end = begin + item.len;
        float eta;
        uint32_t code;
        decision(item.seg, eta, code);
        const float neg_eta = -eta;

        auto partial_row = [&](uint64_t row) {
            const uint64_t i0 = row * 128ull + lane * 4u;
            for (uint32_t e = 0; e < 4; ++e) {
                const uint64_t i = i0 + e;
                if (i >= begin && i < end) {
                    const float w_old = A.w[i];
                    const float dir = sgd_direction(GradVec<BF16>::load1(A.g, i), w_old, A.mom ? A.mom + i : nullptr, A.momentum, A.weight_decay);
                    const float wn = fmaf(neg_eta, dir, w_old);
                    A.w[i] = wn;
                    if (code < 2u) A.c[i] = cast16(wn, code);
                }
            }
        };
        auto store_row = [&](uint64_t i0, float4 wv, float4 gv, float4 mv) {
            if (A.mom || A.weight_decay != 0.f) {      // uniform over the launch
                gv.x = sgd_direction(gv.x, wv.x, A.mom ? &mv.x : nullptr, A.momentum, A.weight_decay);
                gv.y = sgd_direction(gv.y, wv.y, A.mom ? &mv.y : nullptr, A.momentum, A.weight_decay);
                gv.z = sgd_direction(gv.z, wv.z, A.mom ? &mv.z : nullptr, A.momentum, A.weight_decay);
                gv.w = sgd_direction(gv.w, wv.w, A.mom ? &mv.w : nullptr, A.momentum, A.weight_decay);
                if (A.mom) *reinterpret_cast<float4 *>(A.mom + i0) = mv;
            }
            update_store4<STREAM_W>(A.w, A.c, i0, wv, gv, neg_eta, code);
        };

        const uint64_t row_first = begin >> 7, row_last = (end - 1) >> 7;
        const uint64_t full_lo = (begin + 127) >> 7, full_hi = end >> 7;
        const bool head_partial = (begin & 127u) != 0u;
        const bool tail_partial = (end & 127u) != 0u && !(head_partial && row_last == row_first);
        if (head_partial) partial_row(row_first);
        if (full_hi > full_lo) {
            uint64_t row = full_lo;
            while (row + U <= full_hi) {
                float4 wv[U], gv[U], mv[MOM ? U : 1];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const uint64_t i0 = (row + u) * 128ull + lane * 4u;
                    wv[u] = ld_stream(A.w + i0);
                    gv[u] = GradVec<BF16>::load4(A.g, i0, true);
                    if (MOM) mv[u] = __ldcs(reinterpret_cast<const float4 *>(A.mom + i0));
                }
#pragma unroll
                for (int u = 0; u < U; ++u)
                    store_row((row + u) * 128ull + lane * 4u, wv[u], gv[u], MOM ? mv[u] : make_float4(0.f, 0.f, 0.f, 0.f));
                row += U;
            }
            while (row < full_hi) {
                const uint64_t i0 = row * 128ull + lane * 4u;
                store_row(i0, ld_stream(A.w + i0), GradVec<BF16>::load4(A.g, i0, true),
                          MOM ? __ldcs(reinterpret_cast<const float4 *>(A.mom + i0)) : make_float4(0.f, 0.f, 0.f, 0.f));
                ++row;
            }
        }
        if (tail_partial) partial_row(row_last);
    }
}

template <bool BF16, bool MOM>
__global__ void __launch_bounds__(kThreads) k_apply(const ApplyArgs A)
{
    grid_dependency_wait();
    grid_dependency_release();
    if (A.status->skipped) return;
    const LayerState *state = A.state;
    auto decision = [state](uint32_t seg, float &eta, uint32_t &code) { eta = state[seg].eta; code = state[seg].code; };
    // from the end of the buffer to its start: the gradient rows the sweep read last are the ones still in L2
    for (uint32_t batch = blockIdx.x; batch < A.n_batches; batch += gridDim.x)
        apply_batch<BF16, MOM, TA_APPLY_STREAM_W_STORE != 0>(A, A.n_batches - 1u - batch, decision);
}

// ------------------------------------------------------------------ one launch for small models
//
// When the whole model is small, three launches cost more than the data movement.  k_fused runs the
// sweep, the decisions and the update in ONE cooperative launch (every block resident) around one
// grid-wide barrier.
//
// The plan gives every warp a list of "runs" (contiguous pieces of layers, the items of this path) of
// equal total cost, cut on the global row grid.  A warp walks the rows of all its runs as one stream of
// "slots" (a row plus the range of its elements that belong to the run; only the first and last row of
// a layer are partial), several slots in flight, so a warp that owns a dozen tiny tensors waits for
// memory as often as a warp that owns one long piece.  Before the barrier the warp accumulates the
// statistics of its runs and parks as many of its gradient rows as fit in shared memory; its weights
// travel to shared memory (cp.async, no registers held) while the grid waits at the barrier.  The block
// folds the results of its runs into one partial per layer it touches.  After the barrier every block
// combines, in a fixed order, the block partials of just the layers its own runs touch, takes their
// decisions (every block arrives at identical values), and updates its slots from shared memory: nothing
// is read from DRAM after the barrier except rows that did not fit.  The block holding a layer's first
// run writes the layer's new state; old states were copied to shared memory before the barrier, so no
// block can see a state of this step.  The wait is bounded: a block that gives up sets
// status->device_error and returns, so a lost block cannot hang the GPU.

// Statistics of one run, and of all runs of one layer inside one block.
struct FusedPartial {
    double s1, s2;               // sums of (g - pivot) and (g - pivot)^2
    uint32_t amax, amin;         // largest / smallest |S| as bit patterns
    uint32_t bad;                // non-finite inputs
    float pivot;                 // the first gradient value of the run (of the block's first run of the layer)
    uint32_t n, pad;             // gradient values summed
};

// One slot: row `row` of the flat buffer, of which elements [lo, hi) (0..128 inside the row, packed as
// lo | hi << 16) belong to run `run` (counted inside the warp) of layer `seg`.
struct FusedSlot {
    uint32_t row, lo_hi, run, seg;
};

// What the plan tells a warp and a block of the one-launch grid, and a block about each layer it touches.
struct FusedWarpHead {
    uint32_t run_lo, n_slots;        // first run of the warp, slots it walks
    uint32_t pad0, pad1;
};
struct FusedBlockHead {
    uint32_t run_lo, run_hi;         // runs of the block
    uint32_t layer_lo, n_layers;     // layers they touch
    uint32_t part_lo;                // first block partial (and first FusedBlockLayer) of the block
    uint32_t pad0, pad1, pad2;
};
struct FusedBlockLayer {
    double n;                        // length of the layer
    uint32_t part_lo, part_hi;       // the layer's block partials
    uint32_t own;                    // 1: this block holds the layer's first run and writes its state
    uint32_t run_lo, run_hi;         // the layer's runs inside the block
    uint32_t pad;
};

struct FusedArgs {
    const Item *runs;
    uint32_t n_runs;
    const void *g;
    const float *hz;                    // [P][n_total] or unused when P == 0
    uint64_t n_total;
    uint64_t seed;
    uint32_t step32;
    float *w;
    uint16_t *c;
    const FusedWarpHead *warp_head;     // [warps]
    const FusedBlockHead *block_head;   // [blocks]
    const FusedBlockLayer *block_layer; // [n_part] one per (block, layer it touches), grouped by layer
    const FusedSlot *slot_table;        // [warps][max_slots] the rows every warp walks
    FusedPartial *part;                 // block partials, grouped by layer
    uint32_t n_part;
    LayerState *state;                  // [L]
    Status *status;
    DecideParams dp;
    uint32_t L;
    uint32_t cap_w, cap_g;              // slots per warp whose weights / gradients stay in shared memory
    uint32_t max_slots;                 // slots of the longest warp
    uint32_t max_block_runs;            // runs of the block with most runs
    uint32_t max_block_layers;          // layers of the block that touches most layers
    uint32_t early_weights;             // 1: the weight copies start with the first loads of the sweep, 0: after the sweep
    unsigned long long step;
    unsigned long long *barrier;        // [0] arrivals, only ever incremented
    unsigned long long *flag;           // number of the last launch that saw non-finite input
    unsigned long long barrier_base;    // arrivals before this launch
    unsigned long long epoch;           // number of this launch (from 1)
};

constexpr uint32_t kBarrierSpinLimit = 1u << 20;     // with a 64 ns back-off: gives up after a few hundred milliseconds

__device__ __forceinline__ void cp_async16(void *smem, const void *gmem)
{
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async16_once(void *smem, const void *gmem, uint64_t policy)
{
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(s), "l"(gmem), "l"(policy) : "memory");
}
__device__ __forceinline__ void cp_async8(void *smem, const void *gmem)
{
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
// All groups of copies but the newest one have arrived.
__device__ __forceinline__ void cp_async_wait_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

__device__ __forceinline__ uint4 ld_plan(const void *p, uint64_t policy)
{
    uint4 v;
    asm volatile("ld.global.nc.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(policy));
    return v;
}

// Grid-wide barrier on a monotonic arrival counter.  Returns false when the wait ran out.
__device__ __forceinline__ bool grid_barrier(unsigned long long *counter, unsigned long long target, Status *status)
{
    __shared__ uint32_t ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(counter, 1ull);
        uint32_t spins = 0;
        bool arrived = true;
        while (*reinterpret_cast<volatile unsigned long long *>(counter) < target) {
            if (++spins > kBarrierSpinLimit) { arrived = false; break; }
            __nanosleep(64);
        }
        if (!arrived) atomicExch(&status->device_error, 1u);
        __threadfence();
        ok = arrived ? 1u : 0u;
    }
    __syncthreads();
    return ok != 0u;
}

// MODE 0: the whole step in one cooperative launch.  The same step as two dependent launches over the same plan, with
// nothing kept in shared memory between them: MODE 1 is the sweep (statistics and block partials), MODE 2 the decisions
// and the update.  The sweep of step t + 1 needs nothing from the update of step t, so it may run beside it; it only
// ends after it (so that "the update of step t + 1 has waited for its sweep" also means "... and for the update of
// step t").  Partials and the non-finite flag alternate between two buffers for that reason.
constexpr int kWholeStep = 0, kSweepHalf = 1, kUpdateHalf = 2;

template <int P, bool BF16, int MODE>
__global__ void __launch_bounds__(kThreads, (P <= 1 ? TA_FUSED_MIN_BLOCKS : (P <= 4 ? 2 : 1))) k_fused(const FusedArgs A)
{
    constexpr int PP = P > 0 ? P : 1;
    if (MODE == kSweepHalf) grid_dependency_release();      // the update half may take its places and read its plan
    constexpr int U = (P <= 1) ? TA_FUSED_SWEEP_SLOTS : (P == 2 ? 4 : 2);     // slots in flight per lane during the sweep
    constexpr int UA = TA_FUSED_UPDATE_SLOTS;                                  // slots per group of the update
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const unsigned long long G = gridDim.x;
    // dynamic shared memory: weight slots, gradient slots, slot descriptors (one slice per warp each), then the
    // block's tables: what the plan says about its layers, results of its runs, old states and decisions
    unsigned char *ptr = dyn_smem;
    float4 *sh_w = reinterpret_cast<float4 *>(ptr) + (size_t)warp * A.cap_w * 32u;
    ptr += (size_t)kWarps * A.cap_w * 512u;
    float4 *sh_g = reinterpret_cast<float4 *>(ptr) + (size_t)warp * A.cap_g * 32u;
    ptr += (size_t)kWarps * A.cap_g * 512u;
    FusedSlot *sh_slot = reinterpret_cast<FusedSlot *>(ptr) + (size_t)warp * A.max_slots;
    ptr += (size_t)kWarps * A.max_slots * sizeof(FusedSlot);
    FusedBlockLayer *sh_bl = reinterpret_cast<FusedBlockLayer *>(ptr);
    ptr += (size_t)A.max_block_layers * sizeof(FusedBlockLayer);
    FusedPartial *sh_run = reinterpret_cast<FusedPartial *>(ptr);
    ptr += (size_t)A.max_block_runs * sizeof(FusedPartial);
    unsigned long long *sh_old = reinterpret_cast<unsigned long long *>(ptr);                          // LayerState each
    ptr += (size_t)A.max_block_layers * sizeof(LayerState);
    float *sh_eta = reinterpret_cast<float *>(ptr);
    uint32_t *sh_code = reinterpret_cast<uint32_t *>(sh_eta + A.max_block_layers);
    static_assert(sizeof(LayerState) % 8 == 0, "LayerState is copied as 64-bit words");
    static_assert(sizeof(FusedSlot) == 16 && sizeof(FusedPartial) == 40, "shared-memory layout");
    static_assert(sizeof(FusedWarpHead) == 16 && sizeof(FusedBlockHead) == 32 && sizeof(FusedBlockLayer) == 32, "plan records");
    constexpr uint32_t kStateWords = sizeof(LayerState) / 8;

    const uint64_t once = l2_evict_first_policy();       // the weights pass through L2 once on their way to shared memory
    const uint64_t keep = l2_evict_last_policy();
    // the plan of this warp and block: independent loads, one trip to L2
    const uint32_t gw = blockIdx.x * kWarps + warp;
    const uint4 wh = ld_plan(A.warp_head + gw, keep);
    const uint4 bh0 = ld_plan(A.block_head + blockIdx.x, keep);
    const uint4 bh1 = ld_plan(reinterpret_cast<const uint4 *>(A.block_head + blockIdx.x) + 1, keep);
    for (uint32_t s = lane; s < A.max_slots; s += 32) {
        const uint4 v = ld_plan(A.slot_table + (size_t)gw * A.max_slots + s, keep);
        sh_slot[s] = FusedSlot{v.x, v.y, v.z, v.w};
    }
    const uint32_t run_lo = wh.x, n_slots = wh.y;
    const uint32_t brun_lo = bh0.x, lf = bh0.z, nl = bh0.w, bpart_lo = bh1.x;
    // the block's tables: its layers as the plan sees them, and the states the decisions start from, copied before
    // anybody can have written a new one
    for (uint32_t i = tid; i < nl * 2u; i += kThreads)
        cp_async16(reinterpret_cast<uint4 *>(sh_bl) + i, reinterpret_cast<const uint4 *>(A.block_layer + bpart_lo) + i);
    if (MODE == kUpdateHalf) {
        // everything above is the plan, which no launch writes; what follows needs the sweep of this step (and, through
        // it, the update of the step before) complete.  Then the sweep of the next step may start.
        grid_dependency_wait();
        grid_dependency_release();
    }
    if (MODE != kSweepHalf)
        for (uint32_t i = tid; i < nl * kStateWords; i += kThreads)
            cp_async8(sh_old + i, reinterpret_cast<const unsigned long long *>(A.state + lf) + i);
    cp_async_commit();
    __syncwarp();

    // element range of this lane inside a slot: elements e of its vector with e_lo <= e < e_hi belong to the run
    auto lane_range = [lane](const FusedSlot &sl, uint32_t &e_lo, uint32_t &e_hi) {
        const uint32_t lo = sl.lo_hi & 0xFFFFu, hi = sl.lo_hi >> 16, l0 = lane * 4u;
        e_lo = lo > l0 ? min(lo - l0, 4u) : 0u;
        e_hi = hi < l0 + 4u ? (hi > l0 ? hi - l0 : 0u) : 4u;
    };

    // phase 1: statistics of this warp's runs (Sec. 3.1 moments; Sec. 3.2 probe sums)
    if constexpr (MODE != kUpdateHalf) {
        SweepAcc<P, false> acc;
        uint32_t X[PP][4];
        uint64_t have_block = ~0ull;
        uint32_t cur_run = 0xFFFFFFFFu, run_n = 0u;
        float run_pivot = 0.f;
        bool bad_seen = false;
        auto flush = [&](uint32_t run) {
            const double s1 = warp_sum(acc.s1), s2 = warp_sum(acc.s2);
            const uint32_t amax = __reduce_max_sync(0xFFFFFFFFu, acc.amax);
            const uint32_t amin = __reduce_min_sync(0xFFFFFFFFu, acc.amin);
            uint32_t bad = 0u;
            // a non-finite Hz value always makes its probe sum non-finite, so max|S| flags it
            if (SweepAcc<P, false>::gradients_suspect(s2) || (P > 0 && amax >= kNonFiniteBits)) {
                // rare: count the non-finite inputs of this run exactly
                const Item item = A.runs[run_lo + run];
                for (uint64_t i = item.begin + lane; i < item.begin + item.len; i += 32) {
                    if ((__float_as_uint(GradVec<BF16>::load1(A.g, i)) & 0x7FFFFFFFu) >= kNonFiniteBits) ++bad;
                    for (int p = 0; p < P; ++p)
                        if ((__float_as_uint(A.hz[(uint64_t)p * A.n_total + i]) & 0x7FFFFFFFu) >= kNonFiniteBits) ++bad;
                }
                bad = __reduce_add_sync(0xFFFFFFFFu, bad);
                bad_seen = bad_seen || bad != 0u;
            }
            if (lane == 0) sh_run[run_lo - brun_lo + run] = FusedPartial{s1, s2, amax, amin, bad, run_pivot, run_n, 0u};
            acc = SweepAcc<P, false>();
            run_n = 0u;
        };
        auto start_weight_copies = [&]() {
            const uint32_t n = min(n_slots, A.cap_w);
            for (uint32_t s = 0; s < n; ++s) {
                const FusedSlot sl = sh_slot[s];
                uint32_t e_lo, e_hi;
                lane_range(sl, e_lo, e_hi);
                if (e_hi > e_lo) cp_async16_once(sh_w + s * 32u + lane, A.w + (uint64_t)sl.row * 128ull + lane * 4u, once);
            }
            cp_async_commit();
        };
        for (uint32_t s0 = 0; s0 < n_slots; s0 += U) {
            RowData<P> rd[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (s0 + u < n_slots) {
                    const FusedSlot sl = sh_slot[s0 + u];
                    uint32_t e_lo, e_hi;
                    lane_range(sl, e_lo, e_hi);
                    if (e_hi > e_lo) {
                        const uint64_t i0 = (uint64_t)sl.row * 128ull + lane * 4u;
                        // a gradient row that will wait in shared memory needs no place in L1 or L2; one that the
                        // update reads again stays in L2 (a load without an L1 line is also among the first to
                        // leave L2); probe products are read once
                        rd[u].g = s0 + u < A.cap_g ? GradVec<BF16>::load4_no_l1(A.g, i0) : GradVec<BF16>::load4(A.g, i0, false);
#pragma unroll
                        for (int p = 0; p < PP; ++p)
                            if (P > 0) rd[u].hz[p] = ld_stream(A.hz + (uint64_t)p * A.n_total + i0);
                    }
                }
            }
            if (s0 == 0 && A.early_weights) start_weight_copies();
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (s0 + u < n_slots) {
                    const FusedSlot sl = sh_slot[s0 + u];
                    const float gv[4] = {rd[u].g.x, rd[u].g.y, rd[u].g.z, rd[u].g.w};
                    if (sl.run != cur_run) {
                        // a new run: its first gradient value, held by one lane of this row, becomes the pivot of its sums
                        if (cur_run != 0xFFFFFFFFu) flush(cur_run);
                        cur_run = sl.run;
                        const uint32_t first = sl.lo_hi & 0xFFFFu, comp = first & 3u;
                        const float mine = comp == 0u ? gv[0] : (comp == 1u ? gv[1] : (comp == 2u ? gv[2] : gv[3]));
                        run_pivot = __shfl_sync(0xFFFFFFFFu, mine, first >> 2);
                        acc.pivot = (double)run_pivot;
                    }
                    run_n += (sl.lo_hi >> 16) - (sl.lo_hi & 0xFFFFu);
                    uint32_t e_lo, e_hi;
                    lane_range(sl, e_lo, e_hi);
                    uint32_t sel[PP];
                    const uint32_t k = sl.row & 31u;
                    if (P > 1) {
                        const uint64_t blk = sl.row >> 5;
                        if (blk != have_block) {
#pragma unroll
                            for (int p = 0; p < PP; ++p) probe_bits(blk, lane, A.seed, A.step32, (uint32_t)p, X[p]);
                            have_block = blk;
                        }
                    }
#pragma unroll
                    for (int p = 0; p < PP; ++p) sel[p] = (P > 1) ? pick_word(X[p], k >> 3) << (28u - (k & 7u) * 4u) : 0u;
#pragma unroll
                    for (uint32_t e = 0; e < 4; ++e) {
                        if (e >= e_lo && e < e_hi) {
                            float hv[PP];
#pragma unroll
                            for (int p = 0; p < PP; ++p) {
                                const float4 h = rd[u].hz[p];
                                hv[p] = e == 0 ? h.x : (e == 1 ? h.y : (e == 2 ? h.z : h.w));
                            }
                            acc.element(gv[e], hv, sel, e);
                        }
                    }
                    if (s0 + u < A.cap_g && e_hi > e_lo) sh_g[(s0 + u) * 32u + lane] = rd[u].g;
                }
            }
        }
        if (n_slots) flush(cur_run);
        if (MODE == kSweepHalf) {
            // nothing to start: the update half reads the weights itself
        } else if (!A.early_weights || n_slots == 0) {
            start_weight_copies();      // the weights arrive while the grid waits at the barrier and takes the decisions
        }
        if (bad_seen && lane == 0) atomicMax(A.flag, A.epoch);
    }
    // decisions of one layer of this block, from the layer's sums over all blocks (Sec. 3.1 - 3.4).  The new state
    // replaces the old one in shared memory; the block that holds the layer's first run writes it out once the step
    // is known to be committed.
    auto decide = [&](uint32_t q, double pivot, double s1, double s2, uint32_t amax, uint32_t amin) {
        LayerState st;
        unsigned long long *words = reinterpret_cast<unsigned long long *>(&st);
#pragma unroll
        for (uint32_t i = 0; i < kStateWords; ++i) words[i] = sh_old[q * kStateWords + i];
        const double n = sh_bl[q].n;
        const double shift = s1 / n;
        double var = s2 / n - shift * shift;
        if (!(var > 0.0)) var = 0.0;
        LayerScratch sc;
        sc.mean = pivot + shift; sc.var = var; sc.sum_abs = 0.0; sc.bad = 0ull; sc.amax = amax; sc.amin = amin;
        uint32_t near;
        st = decide_layer(A.dp, st, sc, near);
        sh_eta[q] = st.eta;
        sh_code[q] = st.code;
#pragma unroll
        for (uint32_t i = 0; i < kStateWords; ++i) sh_old[q * kStateWords + i] = words[i];
    };
    // a layer's sums over the blocks lo .. hi that share it, in block order, read past L1
    auto combine_serial = [&](uint32_t q, uint32_t lo, uint32_t hi) {
        double s1 = 0.0, s2 = 0.0;
        uint32_t amax = 0u, amin = 0xFFFFFFFFu;
        const double pivot = (double)__ldcg(&A.part[lo].pivot);
        for (uint32_t i = lo; i < hi; ++i) {
            const MomentSums m = rebase(__ldcg(&A.part[i].s1), __ldcg(&A.part[i].s2), (double)__ldcg(&A.part[i].n),
                                        (double)__ldcg(&A.part[i].pivot), pivot);
            s1 += m.s1;
            s2 += m.s2;
            amax = max(amax, __ldcg(&A.part[i].amax));
            amin = min(amin, __ldcg(&A.part[i].amin));
        }
        decide(q, pivot, s1, s2, amax, amin);
    };
    auto combine_warp = [&](uint32_t q, uint32_t lo, uint32_t hi) {
        double s1 = 0.0, s2 = 0.0;
        uint32_t amax = 0u, amin = 0xFFFFFFFFu;
        const double pivot = (double)__ldcg(&A.part[lo].pivot);
        for (uint32_t i = lo + lane; i < hi; i += 32) {
            const MomentSums m = rebase(__ldcg(&A.part[i].s1), __ldcg(&A.part[i].s2), (double)__ldcg(&A.part[i].n),
                                        (double)__ldcg(&A.part[i].pivot), pivot);
            s1 += m.s1;
            s2 += m.s2;
            amax = max(amax, __ldcg(&A.part[i].amax));
            amin = min(amin, __ldcg(&A.part[i].amin));
        }
        s1 = warp_sum(s1);
        s2 = warp_sum(s2);
        amax = __reduce_max_sync(0xFFFFFFFFu, amax);
        amin = __reduce_min_sync(0xFFFFFFFFu, amin);
        if (lane == 0) decide(q, pivot, s1, s2, amax, amin);
    };
    constexpr uint32_t kThreadCombine = 4;       // layers with at most this many block partials: one thread each

    // update + cast of this warp's slots (Sec. 3.2 step, Sec. 2 master copy and cast)
    auto walk = [&]() {
        for (uint32_t s0 = 0; s0 < n_slots; s0 += UA) {
            float4 wv[UA], gv[UA];
#pragma unroll
            for (int u = 0; u < UA; ++u) {
                const uint32_t s = s0 + u;
                if (s < n_slots) {
                    const FusedSlot sl = sh_slot[s];
                    uint32_t e_lo, e_hi;
                    lane_range(sl, e_lo, e_hi);
                    if (e_hi > e_lo) {
                        const uint64_t i0 = (uint64_t)sl.row * 128ull + lane * 4u;
                        wv[u] = s < A.cap_w ? sh_w[s * 32u + lane] : ld_stream(A.w + i0);
                        gv[u] = s < A.cap_g ? sh_g[s * 32u + lane] : GradVec<BF16>::load4(A.g, i0, true);
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < UA; ++u) {
                const uint32_t s = s0 + u;
                if (s < n_slots) {
                    const FusedSlot sl = sh_slot[s];
                    uint32_t e_lo, e_hi;
                    lane_range(sl, e_lo, e_hi);
                    if (e_hi > e_lo) {
                        const uint64_t i0 = (uint64_t)sl.row * 128ull + lane * 4u;
                        const uint32_t code = sh_code[sl.seg - lf];
                        float4 x = wv[u];
                        const float neg_eta = -sh_eta[sl.seg - lf];
                        x.x = fmaf(neg_eta, gv[u].x, x.x);
                        x.y = fmaf(neg_eta, gv[u].y, x.y);
                        x.z = fmaf(neg_eta, gv[u].z, x.z);
                        x.w = fmaf(neg_eta, gv[u].w, x.w);
                        if (e_lo == 0u && e_hi == 4u) {
                            __stcs(reinterpret_cast<float4 *>(A.w + i0), x);
                            {
                                if (code == 0u) {
                                    const __half2 a = __floats2half2_rn(x.x, x.y), b = __floats2half2_rn(x.z, x.w);
                                    uint2 o;
                                    o.x = *reinterpret_cast<const uint32_t *>(&a);
                                    o.y = *reinterpret_cast<const uint32_t *>(&b);
                                    __stcs(reinterpret_cast<uint2 *>(A.c + i0), o);
                                } else if (code == 1u) {
                                    const __nv_bfloat162 a = __floats2bfloat162_rn(x.x, x.y), b = __floats2bfloat162_rn(x.z, x.w);
                                    uint2 o;
                                    o.x = *reinterpret_cast<const uint32_t *>(&a);
                                    o.y = *reinterpret_cast<const uint32_t *>(&b);
                                    __stcs(reinterpret_cast<uint2 *>(A.c + i0), o);
                                }
                            }
                        } else {
                            // a vector on the edge of the layer: only the elements of this run are written
                            const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                            for (uint32_t e = 0; e < 4; ++e) {
                                if (e >= e_lo && e < e_hi) {
                                    A.w[i0 + e] = xs[e];
                                    if (code < 2u) A.c[i0 + e] = cast16(xs[e], code);
                                }
                            }
                        }
                    }
                }
            }
        }
    };
    // the step's status; a skipped step changes nothing and block 0 sums the exact count of non-finite values
    auto write_status = [&](bool skip) {
        if (blockIdx.x == 0 && tid == 0) {
            A.status->step = A.step;
            A.status->skipped = skip ? 1u : 0u;
            if (!skip) A.status->nonfinite = 0ull;
        }
        if (skip && blockIdx.x == 0) {
            __shared__ double red[kWarps];
            double total = 0.0;
            for (uint32_t i = tid; i < A.n_part; i += kThreads) total += (double)__ldcg(&A.part[i].bad);
            total = block_sum(total, red);
            if (tid == 0) A.status->nonfinite = (unsigned long long)total;
        }
    };
    auto commit_states = [&]() {
        for (uint32_t q = tid; q < nl; q += kThreads) {
            if (!sh_bl[q].own) continue;
            unsigned long long *dst = reinterpret_cast<unsigned long long *>(A.state + lf + q);
#pragma unroll
            for (uint32_t i = 0; i < kStateWords; ++i) dst[i] = sh_old[q * kStateWords + i];
        }
    };

    // the block's runs folded into one partial per layer it touches, in run order
    if (MODE == kUpdateHalf) cp_async_wait_all();
    else cp_async_wait_but_one();   // the block's tables have arrived (the weight copies may still be under way)
    __syncthreads();
    if constexpr (MODE != kUpdateHalf) {
        for (uint32_t q = tid; q < nl; q += kThreads) {
            const uint32_t lo = sh_bl[q].run_lo, hi = sh_bl[q].run_hi;
            FusedPartial t{0.0, 0.0, 0u, 0xFFFFFFFFu, 0u, sh_run[lo - brun_lo].pivot, 0u, 0u};
            for (uint32_t r = lo; r < hi; ++r) {
                const FusedPartial x = sh_run[r - brun_lo];
                const MomentSums m = rebase(x.s1, x.s2, (double)x.n, (double)x.pivot, (double)t.pivot);
                t.s1 += m.s1; t.s2 += m.s2;
                t.n += x.n;
                t.amax = max(t.amax, x.amax); t.amin = min(t.amin, x.amin);
                t.bad += x.bad;
            }
            A.part[bpart_lo + q] = t;
        }
    }
    if (MODE == kSweepHalf) {
        // this launch is complete only when the update of the step before is (see kSweepHalf above)
        grid_dependency_wait();
        return;
    }

    if (MODE == kWholeStep && !grid_barrier(A.barrier, A.barrier_base + G, A.status)) {
        cp_async_wait_all();
        return;
    }

    // did any warp of the grid see a non-finite input?  The answer is needed only when results are committed, so
    // the decisions below are taken while it is on its way; those of a skipped step are thrown away
    const bool skip = __ldcg(A.flag) == A.epoch || __ldcg(&A.status->device_error) != 0u;
    for (uint32_t q = tid; q < nl; q += kThreads) {
        const uint32_t lo = sh_bl[q].part_lo, hi = sh_bl[q].part_hi;
        if (hi - lo <= kThreadCombine) combine_serial(q, lo, hi);
    }
    for (uint32_t q = warp; q < nl; q += kWarps) {      // layers spread over many blocks: one warp each
        const uint32_t lo = sh_bl[q].part_lo, hi = sh_bl[q].part_hi;
        if (hi - lo > kThreadCombine) combine_warp(q, lo, hi);
    }
    cp_async_wait_all();
    write_status(skip);
    if (skip) return;
    __syncthreads();
    commit_states();
    walk();
}

// ------------------------------------------------------------------ power iteration support (Sec. 3.2)
//
// u <- H_l u / ||H_l u||,  lambda ~ (u^T H_l u) / (u^T u), per layer, with the products H_l u supplied by the
// caller.  Eigenvectors found earlier (V, with eigenvalues lambda_V) are deflated:
//   t = Hu - sum_j a_j v_j,   a_j = lambda_j (v_j . u)   per layer.
// Three sweeps over the same items as the optimizer pass: projections v_j . u, then the dots of u and t, then
// the normalised write.  All sums are double and combined in a fixed order.

constexpr int kMaxEigs = 8;

struct PowerArgs {
    const Item *items;
    uint32_t n_items, n_batches;
    const float *u, *hu, *v;       // v: [m][n_total]
    uint64_t n_total;
    uint32_t m, L;
    double *part;                  // [max(3, m)][n_items] per-item partial sums
    const float *coef;             // [kMaxEigs][L] a_j per layer
    const float *norm;             // [L]
    float *u_next;
};

__device__ __forceinline__ float4 load_row4(const float *p, uint64_t i0, bool full, uint64_t begin, uint64_t end)
{
    if (full) return __ldg(reinterpret_cast<const float4 *>(p + i0));
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i0 + 0 >= begin && i0 + 0 < end) r.x = __ldg(p + i0 + 0);
    if (i0 + 1 >= begin && i0 + 1 < end) r.y = __ldg(p + i0 + 1);
    if (i0 + 2 >= begin && i0 + 2 < end) r.z = __ldg(p + i0 + 2);
    if (i0 + 3 >= begin && i0 + 3 < end) r.w = __ldg(p + i0 + 3);
    return r;
}

// MODE 0: projections v_j . u;  MODE 1: u.u, u.t, t.t;  MODE 2: u_next = t / ||t||
template <int MODE>
__global__ void __launch_bounds__(kThreads) k_power(const PowerArgs A)
{
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    for (uint32_t batch = blockIdx.x; batch < A.n_batches; batch += gridDim.x) {
        const uint32_t it = batch * kWarps + warp;
        if (it >= A.n_items) continue;
        const Item item = A.items[it];
        double acc[kMaxEigs];
#pragma unroll
        for (int j = 0; j < kMaxEigs; ++j) acc[j] = 0.0;
        if (item.len != 0u) {
            const uint64_t begin = item.begin, end = begin + item.len;
            float a[kMaxEigs];
#pragma unroll
            for (int j = 0; j < kMaxEigs; ++j) a[j] = (MODE != 0 && j < (int)A.m) ? A.coef[(uint64_t)j * A.L + item.seg] : 0.f;
            const float nrm = MODE == 2 ? A.norm[item.seg] : 1.f;
            const uint64_t row_first = begin >> 7, row_last = (end - 1) >> 7;
            constexpr int UR = 4;                          // rows whose loads are issued together
            uint64_t row = row_first;
            while (row <= row_last) {
                const bool group = row * 128ull >= begin && (row + UR) * 128ull <= end;
                const int cnt = group ? UR : 1;
                const bool full = group || (row * 128ull >= begin && row * 128ull + 128u <= end);
                float4 uu[UR], t[UR];
#pragma unroll
                for (int r = 0; r < UR; ++r) {
                    if (r < cnt) {
                        const uint64_t i0 = (row + r) * 128ull + lane * 4u;
                        if (MODE != 2) uu[r] = load_row4(A.u, i0, full, begin, end);
                        if (MODE != 0) t[r] = load_row4(A.hu, i0, full, begin, end);
                    }
                }
#pragma unroll
                for (int j = 0; j < kMaxEigs; ++j) {
                    if (j < (int)A.m) {
                        float4 vv[UR];
#pragma unroll
                        for (int r = 0; r < UR; ++r)
                            if (r < cnt) vv[r] = load_row4(A.v + (uint64_t)j * A.n_total, (row + r) * 128ull + lane * 4u, full, begin, end);
#pragma unroll
                        for (int r = 0; r < UR; ++r) {
                            if (r < cnt) {
                                if (MODE == 0) {
                                    acc[j] += (double)vv[r].x * (double)uu[r].x + (double)vv[r].y * (double)uu[r].y +
                                              (double)vv[r].z * (double)uu[r].z + (double)vv[r].w * (double)uu[r].w;
                                } else {
                                    t[r].x = fmaf(-a[j], vv[r].x, t[r].x); t[r].y = fmaf(-a[j], vv[r].y, t[r].y);
                                    t[r].z = fmaf(-a[j], vv[r].z, t[r].z); t[r].w = fmaf(-a[j], vv[r].w, t[r].w);
                                }
                            }
                        }
                    }
                }
#pragma unroll
                for (int r = 0; r < UR; ++r) {
                    if (r < cnt) {
                        const uint64_t i0 = (row + r) * 128ull + lane * 4u;
                        if (MODE == 1) {
                            const float4 q = uu[r], p = t[r];
                            acc[0] += (double)q.x * (double)q.x + (double)q.y * (double)q.y + (double)q.z * (double)q.z + (double)q.w * (double)q.w;
                            acc[1] += (double)q.x * (double)p.x + (double)q.y * (double)p.y + (double)q.z * (double)p.z + (double)q.w * (double)p.w;
                            acc[2] += (double)p.x * (double)p.x + (double)p.y * (double)p.y + (double)p.z * (double)p.z + (double)p.w * (double)p.w;
                        } else if (MODE == 2) {
                            float4 o;
                            o.x = nrm > 0.f ? __fdiv_rn(t[r].x, nrm) : 0.f; o.y = nrm > 0.f ? __fdiv_rn(t[r].y, nrm) : 0.f;
                            o.z = nrm > 0.f ? __fdiv_rn(t[r].z, nrm) : 0.f; o.w = nrm > 0.f ? __fdiv_rn(t[r].w, nrm) : 0.f;
                            if (full) {
                                *reinterpret_cast<float4 *>(A.u_next + i0) = o;
                            } else {
                                if (i0 + 0 >= begin && i0 + 0 < end) A.u_next[i0 + 0] = o.x;
                                if (i0 + 1 >= begin && i0 + 1 < end) A.u_next[i0 + 1] = o.y;
                                if (i0 + 2 >= begin && i0 + 2 < end) A.u_next[i0 + 2] = o.z;
                                if (i0 + 3 >= begin && i0 + 3 < end) A.u_next[i0 + 3] = o.w;
                            }
                        }
                    }
                }
                row += cnt;
            }
        }
        if (MODE != 2) {
            const int n_acc = MODE == 0 ? (int)A.m : 3;
#pragma unroll
            for (int j = 0; j < kMaxEigs; ++j) {
                if (j < n_acc) {
                    const double v = warp_sum(acc[j]);
                    if (lane == 0) A.part[(uint64_t)j * A.n_items + it] = v;
                }
            }
        }
    }
}

struct PowerLayerArgs {
    const uint32_t *item_lo;
    uint32_t n_items, m, L;
    const double *part;
    const float *lambda_v;         // [m][L] eigenvalues of the deflated vectors
    float *coef;                   // [kMaxEigs][L]
    float *lambda_out, *norm_out;  // [L]
};

// One block per layer.  STAGE 0: a_j = lambda_j * (v_j . u).  STAGE 1: lambda = u.t / u.u, norm = sqrt(t.t).
template <int STAGE>
__global__ void __launch_bounds__(kThreads) k_power_layer(const PowerLayerArgs A)
{
    __shared__ double red[kWarps];
    const uint32_t l = blockIdx.x, tid = threadIdx.x;
    const uint32_t lo = A.item_lo[l], hi = A.item_lo[l + 1];
    const int n_acc = STAGE == 0 ? (int)A.m : 3;
    double tot[3] = {0.0, 0.0, 0.0};
    for (int j = 0; j < n_acc; ++j) {
        double sum = 0.0;
#pragma unroll 4
        for (uint32_t i = lo + tid; i < hi; i += kThreads) sum += A.part[(uint64_t)j * A.n_items + i];
        sum = block_sum(sum, red);
        if (STAGE == 0) {
            if (tid == 0) A.coef[(uint64_t)j * A.L + l] = (float)((double)A.lambda_v[(uint64_t)j * A.L + l] * sum);
        } else {
            tot[j] = sum;
        }
    }
    if (STAGE == 1 && tid == 0) {
        A.lambda_out[l] = tot[0] > 0.0 ? (float)(tot[1] / tot[0]) : 0.f;
        A.norm_out[l] = (float)sqrt(tot[2]);
    }
}

// ------------------------------------------------------------------ probe writer

__global__ void __launch_bounds__(kThreads) k_probe(float *z, uint64_t n_vec, uint64_t seed, uint32_t step, uint32_t p)
{
    for (uint64_t v = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; v < n_vec; v += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t i0 = v * 4ull;
        const uint64_t row = i0 >> 7;
        const uint32_t k = (uint32_t)(row & 31u), slot = (uint32_t)(v & 31u);
        uint32_t x[4];
        probe_bits(row >> 5, slot, seed, step, p, x);
        const uint32_t bits = pick_word(x, k >> 3) >> ((k & 7u) * 4u);
        float4 o;
        o.x = (bits & 1u) ? -1.f : 1.f;
        o.y = (bits & 2u) ? -1.f : 1.f;
        o.z = (bits & 4u) ? -1.f : 1.f;
        o.w = (bits & 8u) ? -1.f : 1.f;
        *reinterpret_cast<float4 *>(z + i0) = o;
    }
}

// ------------------------------------------------------------------ top-k: radix select on |S| bit patterns
//
// |S| >= 0, so the order of the values is the order of their 31-bit patterns.  Level 1 (bits 30..20) is counted
// during the sweep, which also sets the mask bits of every element above a window of bins around the bin that held
// the k-th largest value at the last step, and lists the elements inside the window as candidates (value, index in
// layer).  k_decide finds, per layer, the bin b1 that holds the k-th largest value now, and whether the window
// contains it; layers where it does not are swept once more with the window [b1, b1].  k_apply_resolve then finishes
// the selection on the candidates alone: those in bins above b1 are taken, those in b1 go through two more value
// digits and, if more of them equal the threshold than are to be taken, three digits of the index (lower index
// first).  The result does not depend on the order in which candidates were listed.

struct ResolveArgs {
    const uint32_t *item_lo;
    const uint64_t *seg_off, *seg_len;
    const uint32_t *cand_count, *cand_val, *cand_idx;
    uint32_t *cand_count_out;      // cleared for the next step once the layer is resolved
    uint32_t *mask2;               // the two mask buffers
    uint64_t mask_words;
    const double *p_mass;
    const LayerScratch *scratch;
    SelectState *sel;
    LayerState *state;
    const Status *status;
};

// Candidate values a thread keeps in flight per pass: one block works on a whole layer, so the passes of a long
// candidate list are bound by round trips to memory, not by bandwidth.
#ifndef TA_RESOLVE_LOADS
#define TA_RESOLVE_LOADS 32
#endif
constexpr int kResolveLoads = TA_RESOLVE_LOADS;

// One block per layer: finishes the selection among the layer's candidates.
__device__ __forceinline__ void resolve_layer(const ResolveArgs &A, const uint32_t l)
{
    __shared__ uint32_t h[kHistBins];
    __shared__ uint32_t scan[kThreads];
    __shared__ uint32_t found[2];
    __shared__ double red[kWarps];
    __shared__ unsigned long long acc_u64;
    const uint32_t tid = threadIdx.x;
    const uint64_t off = A.seg_off[l];
    SelectState s = A.sel[l];
    const uint32_t b1 = s.prefix;
    uint32_t *mask = A.mask2 + (size_t)A.status->mask_cur * A.mask_words;

    auto clear = [&](int bins) { for (int b = tid; b < bins; b += kThreads) h[b] = 0u; __syncthreads(); };

    const uint32_t m = A.cand_count[l];
    const uint32_t *cv = A.cand_val + off, *ci = A.cand_idx + off;

    // value digits of the candidates in bin b1: bits 19..9, then bits 8..0
    clear(kHistBins);
    for (uint32_t j0 = 0; j0 < m; j0 += kThreads * kResolveLoads) {
        uint32_t v[kResolveLoads];
#pragma unroll
        for (int u = 0; u < kResolveLoads; ++u) { const uint32_t j = j0 + u * kThreads + tid; v[u] = j < m ? __ldg(cv + j) : 0xFFFFFFFFu; }
#pragma unroll
        for (int u = 0; u < kResolveLoads; ++u) if ((v[u] >> 20) == b1) atomicAdd(&h[(v[u] >> 9) & 2047u], 1u);
    }
    __syncthreads();
    block_find_bin<true>(h, kHistBins, s.remaining, scan, found);
    const uint32_t b2 = found[0], r2 = s.remaining - found[1];
    const uint32_t pre22 = (b1 << 11) | b2;
    __syncthreads();
    clear(512);
    for (uint32_t j0 = 0; j0 < m; j0 += kThreads * kResolveLoads) {
        uint32_t v[kResolveLoads];
#pragma unroll
        for (int u = 0; u < kResolveLoads; ++u) { const uint32_t j = j0 + u * kThreads + tid; v[u] = j < m ? __ldg(cv + j) : 0xFFFFFFFFu; }
#pragma unroll
        for (int u = 0; u < kResolveLoads; ++u) if ((v[u] >> 9) == pre22) atomicAdd(&h[v[u] & 511u], 1u);
    }
    __syncthreads();
    block_find_bin<true>(h, 512, r2, scan, found);
    const uint32_t thr = (pre22 << 9) | found[0];
    const uint32_t take_equal = r2 - found[1];
    const uint32_t n_equal = h[found[0]];
    __syncthreads();

    // index digits (only when ties at the threshold exceed what is taken): bits 31..21, 20..10, 9..0
    uint32_t idx_limit = 0xFFFFFFFFu;           // equal-valued candidates with index <= idx_limit are taken
    if (n_equal > take_equal) {
        uint32_t need = take_equal, prefix = 0u;
        const int shifts[3] = {21, 10, 0};
        const int widths[3] = {11, 11, 10};
        for (int lev = 0; lev < 3; ++lev) {
            const int bins = 1 << widths[lev];
            clear(kHistBins);
            for (uint32_t j = tid; j < m; j += kThreads) {
                if (cv[j] != thr) continue;
                const uint32_t ix = ci[j];
                const bool match = lev == 0 ? true : (ix >> (shifts[lev] + widths[lev])) == prefix;
                if (match) atomicAdd(&h[(ix >> shifts[lev]) & (uint32_t)(bins - 1)], 1u);
            }
            __syncthreads();
            block_find_bin<false>(h, lev == 2 ? 1024 : kHistBins, need, scan, found);
            prefix = (prefix << widths[lev]) | found[0];
            need -= found[1];
            __syncthreads();
        }
        idx_limit = prefix;
    }

    // set the bits of the taken candidates.  Their sum is exact: the window spans a few binary exponents at most
    // (seventeen bins of an eighth of an octave), so every value is an integer multiple of the smallest exponent's unit,
    // and the integers are added.
    const uint32_t e_lo = (s.lo_bin >> 3) & 0xFFu, e_unit = e_lo ? e_lo : 1u;      // exponent field 0 (subnormal) counts as 1
    unsigned long long units = 0ull;
    for (uint32_t j0 = 0; j0 < m; j0 += kThreads * (kResolveLoads / 2)) {
        uint32_t v[kResolveLoads / 2], ix[kResolveLoads / 2];
#pragma unroll
        for (int u = 0; u < kResolveLoads / 2; ++u) {
            const uint32_t j = j0 + u * kThreads + tid;
            v[u] = j < m ? __ldg(cv + j) : 0u;          // 0 is never taken: thr > 0 here or handled by the index rule
            ix[u] = j < m ? __ldg(ci + j) : 0xFFFFFFFFu;
        }
#pragma unroll
        for (int u = 0; u < kResolveLoads / 2; ++u) {
            const uint32_t j = j0 + u * kThreads + tid;
            if (j < m && (v[u] > thr || (v[u] == thr && ix[u] <= idx_limit))) {
                const uint64_t i = off + ix[u];
                atomicOr(mask + (i >> 5), 1u << (i & 31u));
                const uint32_t e = v[u] >> 23;
                const unsigned long long sig = e ? ((v[u] & 0x007FFFFFu) | 0x00800000u) : (v[u] & 0x007FFFFFu);
                units += sig << ((e ? e : 1u) - e_unit);
            }
        }
    }
    if (tid == 0) acc_u64 = 0ull;
    __syncthreads();
    atomicAdd(&acc_u64, units);
    double mass = 0.0;
    for (uint32_t i = A.item_lo[l] + tid; i < A.item_lo[l + 1]; i += kThreads) mass += A.p_mass[i];
    mass = block_sum(mass, red);
    if (tid == 0) {
        const double cand_sum = (double)acc_u64 * ldexp(1.0, (int)e_unit - 127 - 23);
        const double all = A.scratch[l].sum_abs;
        s.thr_bits = thr; s.take_equal = take_equal; s.surplus = n_equal > take_equal ? 1u : 0u;
        A.sel[l] = s;
        A.state[l].thr = __uint_as_float(thr);
        A.state[l].topk_mass = all > 0.0 ? (mass + cand_sum) / all : 1.0;
        A.cand_count_out[l] = 0u;          // the list is used up; the next sweep starts a new one
    }
}

// Top-k steps: the update needs nothing from the resolve step, so both run in ONE launch.  The first
// n_layers blocks finish the selection of one layer each; the other blocks stride over the update batches.
template <bool BF16, bool MOM>
__global__ void __launch_bounds__(kThreads) k_apply_resolve(const ApplyArgs A, const ResolveArgs R, const uint32_t n_layers)
{
    grid_dependency_wait();
    grid_dependency_release();
    if (A.status->skipped) return;
    if (blockIdx.x < n_layers) {
        resolve_layer(R, blockIdx.x);
        return;
    }
    const LayerState *state = A.state;
    // eta and code were fixed by k_decide; resolve blocks write other fields (threshold, mass) of the same records
    auto decision = [state](uint32_t seg, float &eta, uint32_t &code) { eta = state[seg].eta; code = state[seg].code; };
    // the new weights are stored with the streaming hint: what is worth keeping in L2 is the gradient that the sweep
    // has just read (measured on the ResNet-50 mix: update 49.6 -> 45.9 us; walking the batches from the end, as
    // k_apply does, was slower here)
    for (uint32_t batch = blockIdx.x - n_layers; batch < A.n_batches; batch += gridDim.x - n_layers)
        apply_batch<BF16, MOM, true>(A, batch, decision);
}

}  // namespace ta
