// ta_grad_moments_static: per-layer gradient mean and variance with no allocation of any kind.
//
// It is the statistics part of the sweep kernel (the moments of Sec. 3.1), re-cut so that every
// byte of scratch it needs sits in one file-scope device array of fixed size instead of buffers
// that ta_create allocates.  See include/triaccel.h for who needs this and for the limits.
#include "../../include/triaccel.h"

#include <cuda_runtime.h>

#include <atomic>
#include <cstdio>

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr uint32_t kNonFiniteBits = 0x7F800000u;   // |x| bit patterns at or above this are inf / NaN

template <bool BF16> __device__ __forceinline__ float load1(const void *g, uint64_t i)
{
    if (BF16) return __uint_as_float((uint32_t)__ldg(static_cast<const uint16_t *>(g) + i) << 16);
    return __ldg(static_cast<const float *>(g) + i);
}

template <bool BF16> __device__ __forceinline__ float4 load4(const void *g, uint64_t i)
{
    if (BF16) {
        const uint2 v = __ldcs(reinterpret_cast<const uint2 *>(static_cast<const uint16_t *>(g) + i));
        return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u),
                           __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xFFFF0000u));
    }
    return __ldcs(reinterpret_cast<const float4 *>(static_cast<const float *>(g) + i));
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Sum over the block in a fixed order; valid in every thread.
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

constexpr uint32_t kTileElems = TA_STATIC_TILE_ELEMS;     // elements one warp reduces into one partial
constexpr uint32_t kMaxTiles = TA_STATIC_MAX_TILES;
constexpr uint32_t kMaxLayers = TA_STATIC_MAX_LAYERS;

// One partial per tile: sums of (x - pivot) and (x - pivot)^2 with the tile's first value as pivot (so that a
// layer whose mean dwarfs its spread loses no digits), that pivot, and the count of non-finite values.
struct StaticScratch {
    double s1[kMaxTiles];
    double s2[kMaxTiles];
    float pivot[kMaxTiles];
    uint32_t bad[kMaxTiles];
};

// The scratch itself.  A GPU holds these bytes from the moment the CUDA runtime loads this file's device code on
// it (with the runtime's default lazy loading: at the first call on that device) until the process exits.
// In host code the name below is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

// The layer table travels as a kernel argument, so it needs no device buffer either.
struct StaticTable {
    uint64_t offset[kMaxLayers];
    uint32_t length[kMaxLayers];
    uint32_t tile_lo[kMaxLayers + 1];   // first tile of each layer; tiles are cut on a global grid of kTileElems
    uint32_t L;
};

constexpr int kMaxDevices = 64;
std::atomic<StaticScratch *> g_scratch_addr[kMaxDevices];  // device address of the array, per device (looked up once)
thread_local char g_error[256] = "";

template <bool BF16>
__global__ void __launch_bounds__(kThreads) k_moments_static_tiles(const StaticTable T, const void *g, StaticScratch *scr)
{
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t n_tiles = T.tile_lo[T.L];
    for (uint32_t tile = blockIdx.x * kWarps + (threadIdx.x >> 5); tile < n_tiles; tile += gridDim.x * kWarps) {
        // layer of this tile: the last l with tile_lo[l] <= tile
        uint32_t lo = 0, hi = T.L;
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (T.tile_lo[mid] <= tile) lo = mid; else hi = mid;
        }
        const uint64_t seg_b = T.offset[lo], seg_e = seg_b + T.length[lo];
        const uint64_t first_cell = seg_b / kTileElems;
        const uint64_t cell = first_cell + (tile - T.tile_lo[lo]);
        const uint64_t begin = cell * kTileElems > seg_b ? cell * kTileElems : seg_b;
        const uint64_t end = (cell + 1) * kTileElems < seg_e ? (cell + 1) * kTileElems : seg_e;
        double s1 = 0.0, s2 = 0.0;
        uint32_t bad = 0;
        const float pivot = load1<BF16>(g, begin);
        auto one = [&](float v) {
            if ((__float_as_uint(v) & 0x7FFFFFFFu) >= kNonFiniteBits) ++bad;
            const double x = (double)v - (double)pivot;
            s1 += x;
            s2 = fma(x, x, s2);
        };
        // rows of 128 elements on the global grid; partial rows at the ends take the scalar path
        const uint64_t full_lo = (begin + 127) >> 7, full_hi = end >> 7;
        if (full_hi > full_lo) {
            for (uint64_t i = begin + lane; i < full_lo * 128ull; i += 32) one(load1<BF16>(g, i));
            for (uint64_t row = full_lo; row < full_hi; ++row) {
                const float4 v = load4<BF16>(g, row * 128ull + lane * 4u);
                one(v.x); one(v.y); one(v.z); one(v.w);
            }
            for (uint64_t i = full_hi * 128ull + lane; i < end; i += 32) one(load1<BF16>(g, i));
        } else {
            for (uint64_t i = begin + lane; i < end; i += 32) one(load1<BF16>(g, i));
        }
        s1 = warp_sum(s1);
        s2 = warp_sum(s2);
        bad = __reduce_add_sync(0xFFFFFFFFu, bad);
        if (lane == 0) { scr->s1[tile] = s1; scr->s2[tile] = s2; scr->pivot[tile] = pivot; scr->bad[tile] = bad; }
    }
}

// One block per layer adds the layer's tile partials in a fixed order.
__global__ void __launch_bounds__(kThreads) k_moments_static_layers(const StaticTable T, const StaticScratch *scr,
                                                                        double *mean_var, uint32_t *nonfinite)
{
    __shared__ double red[kWarps];
    const uint32_t l = blockIdx.x;
    double s1 = 0.0, s2 = 0.0, bad = 0.0;
    // the tiles summed around their own pivots; move every tile's sums to the pivot of the layer's first tile:
    // with d = p_tile - p_layer, sum (x - p_layer) = s1 + n d and sum (x - p_layer)^2 = s2 + d (2 s1 + n d)
    const uint64_t seg_b = T.offset[l], seg_e = seg_b + T.length[l];
    const double p_layer = (double)scr->pivot[T.tile_lo[l]];
    for (uint32_t t = T.tile_lo[l] + threadIdx.x; t < T.tile_lo[l + 1]; t += kThreads) {
        const uint64_t cell = seg_b / kTileElems + (t - T.tile_lo[l]);
        const uint64_t begin = cell * kTileElems > seg_b ? cell * kTileElems : seg_b;
        const uint64_t end = (cell + 1) * kTileElems < seg_e ? (cell + 1) * kTileElems : seg_e;
        const double n = (double)(end - begin), d = (double)scr->pivot[t] - p_layer;
        const double a = scr->s1[t];
        s1 += fma(n, d, a);
        s2 += fma(d, fma(n, d, 2.0 * a), scr->s2[t]);
        bad += (double)scr->bad[t];
    }
    s1 = block_sum(s1, red);
    s2 = block_sum(s2, red);
    bad = block_sum(bad, red);
    if (threadIdx.x == 0) {
        const double n = (double)T.length[l];
        const double shift = s1 / n;
        double var = s2 / n - shift * shift;
        if (!(var > 0.0)) var = 0.0;
        mean_var[2 * l] = p_layer + shift;
        mean_var[2 * l + 1] = var;
        if (nonfinite) nonfinite[l] = (uint32_t)(bad > 4294967295.0 ? 4294967295.0 : bad);
    }
}

int fail(int code, const char *msg)
{
    snprintf(g_error, sizeof(g_error), "%s", msg);
    return code;
}

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

const char *ta_static_last_error(void) { return g_error; }

int ta_grad_moments_static(const ta_segment *table, uint32_t L, const void *g, uint32_t grad_dtype,
                           double *mean_var, uint32_t *nonfinite, void *stream)
{
    g_error[0] = 0;
    if (!table || !g || !mean_var || L == 0) return fail(TA_ERR_ARG, "ta_grad_moments_static: NULL argument or empty table");
    if (L > kMaxLayers) return fail(TA_ERR_ARG, "ta_grad_moments_static: more than TA_STATIC_MAX_LAYERS layers");
    if (grad_dtype != TA_GRAD_F32 && grad_dtype != TA_GRAD_BF16) return fail(TA_ERR_ARG, "ta_grad_moments_static: unknown grad_dtype");
    if ((reinterpret_cast<uintptr_t>(g) & 15u) || (reinterpret_cast<uintptr_t>(mean_var) & 7u) ||
        (reinterpret_cast<uintptr_t>(nonfinite) & 3u))
        return fail(TA_ERR_ALIGN, "ta_grad_moments_static: g must be 16-byte aligned, mean_var 8-byte, nonfinite 4-byte aligned");
    StaticTable T;
    uint64_t end = 0, tiles = 0;
    for (uint32_t l = 0; l < L; ++l) {
        if (table[l].length == 0 || table[l].length > 0xFFFFFFFEull || table[l].offset < end)
            return fail(TA_ERR_ARG, "ta_grad_moments_static: segments must be non-empty, ascending and non-overlapping");
        end = table[l].offset + table[l].length;
        T.offset[l] = table[l].offset;
        T.length[l] = (uint32_t)table[l].length;
        T.tile_lo[l] = (uint32_t)tiles;
        tiles += (end - 1) / kTileElems - table[l].offset / kTileElems + 1;
        if (tiles > kMaxTiles)
            return fail(TA_ERR_ARG, "ta_grad_moments_static: table needs more than TA_STATIC_MAX_TILES tiles of "
                                    "TA_STATIC_TILE_ELEMS elements; the static scratch cannot hold it");
    }
    T.tile_lo[L] = (uint32_t)tiles;
    T.L = L;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
        return fail(TA_ERR_CUDA, "ta_grad_moments_static: no current CUDA device");
    StaticScratch *scr = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!scr) {
        // first call on this device: ask the runtime where this device's copy of the array lives (this is also the
        // moment the runtime loads this file's device code onto the device).  Threads that race here all get the
        // same answer, so whichever store lands last changes nothing.
        void *p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) {
            snprintf(g_error, sizeof(g_error), "ta_grad_moments_static: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
            return TA_ERR_CUDA;
        }
        scr = static_cast<StaticScratch *>(p);
        g_scratch_addr[dev].store(scr, std::memory_order_release);
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
    const uint32_t want = (uint32_t)((tiles + kWarps - 1) / kWarps);
    const uint32_t grid = want < (uint32_t)sms * 8u ? want : (uint32_t)sms * 8u;
    // every partial slot that the second kernel reads is written by the first one in this call, so
    // nothing left over from an earlier call is ever read and nothing has to be cleared
    if (grad_dtype == TA_GRAD_BF16) k_moments_static_tiles<true><<<grid, kThreads, 0, s>>>(T, g, scr);
    else k_moments_static_tiles<false><<<grid, kThreads, 0, s>>>(T, g, scr);
    k_moments_static_layers<<<L, kThreads, 0, s>>>(T, scr, mean_var, nonfinite);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        snprintf(g_error, sizeof(g_error), "ta_grad_moments_static: launch failed: %s", cudaGetErrorString(e));
        return TA_ERR_CUDA;
    }
    return TA_OK;
}

#pragma GCC visibility pop
}  // extern "C"
