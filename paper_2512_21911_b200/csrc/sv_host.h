// Host-side helpers shared by the entry points: argument checks and launch-error mapping.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "sv.h"

namespace svh {

constexpr int kHeadDim = 128;
constexpr int kMaxRows = 128;      // query rows (G * draft tokens) packed into one M = 128 tile
constexpr int kMaxRowTiles = 8;    // row tiles per (sequence, KV head): G * T <= 1024 at most
constexpr int kMaxDraft = 64;      // ancestor masks are 64-bit; the draft tokens form one 64-key unit
constexpr int kMaxBlocksSelect = 32768;

inline bool aligned(const void *p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// Draft tokens whose G query rows fit one M = 128 row tile, and the number of such tiles.
inline int tokens_per_tile(const sv_geom *g)
{
    const int G = g->n_q_heads / g->n_kv_heads;
    return G * g->n_draft <= kMaxRows ? g->n_draft : (kMaxRows / G > 0 ? kMaxRows / G : 1);
}
inline int row_tiles(const sv_geom *g)
{
    const int tt = tokens_per_tile(g);
    return (g->n_draft + tt - 1) / tt;
}


inline sv_status check_geom(const sv_geom *g)
{
    if (!g) return SV_ERR_NULL;
    if (g->n_seq < 1 || g->n_q_heads < 1 || g->n_kv_heads < 1 || g->max_blocks < 1 || g->n_draft < 1)
        return SV_ERR_SHAPE;
    if (g->n_q_heads % g->n_kv_heads) return SV_ERR_SHAPE;
    if (g->head_dim != kHeadDim) return SV_ERR_UNSUPPORTED;
    if (g->block_size != 64 && g->block_size != 128) return SV_ERR_UNSUPPORTED;
    if (g->n_draft > kMaxDraft) return SV_ERR_UNSUPPORTED;
    if (g->n_q_heads / g->n_kv_heads > kMaxRows || row_tiles(g) > kMaxRowTiles) return SV_ERR_UNSUPPORTED;
    if (g->n_seq > 65535 || g->n_kv_heads > 65535) return SV_ERR_SHAPE;
    return SV_OK;
}

inline sv_status check_kv(const sv_geom *g, const sv_kv *kv, bool need_v)
{
    if (!kv || !kv->k_pool || !kv->block_table || !kv->seq_lens || (need_v && !kv->v_pool)) return SV_ERR_NULL;
    if (kv->n_pages < 1) return SV_ERR_SHAPE;
    if ((int64_t)kv->n_pages * g->n_kv_heads * g->block_size >= (int64_t)1 << 31) return SV_ERR_SHAPE;
    if (!aligned(kv->k_pool, 128) || (need_v && !aligned(kv->v_pool, 128))) return SV_ERR_ALIGN;
    if (!aligned(kv->block_table, 4) || !aligned(kv->seq_lens, 4)) return SV_ERR_ALIGN;
    return SV_OK;
}

// Launch attribute for programmatic dependent launch: the kernel may be scheduled while its
// predecessor in the stream drains; every kernel of the library executes griddepcontrol.wait before it
// reads anything the predecessor wrote.
inline void pdl_attribute(cudaLaunchAttribute *attr)
{
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
}

// Per-device state.  One process may drive several GPUs, and function attributes and SM counts belong to
// a device, so both are kept per device index (devices beyond the table are handled uncached).
constexpr int kMaxDevices = 64;

inline int current_device()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        dev = 0;
    }
    return dev;
}

// Runs `configure` (a callable returning cudaError_t, e.g. a cudaFuncSetAttribute call) once per device
// for the call site that owns this object.
struct OncePerDevice {
    std::atomic<uint64_t> done{0};
    template <class F>
    cudaError_t run(F configure)
    {
        const int dev = current_device();
        const bool cached = dev >= 0 && dev < kMaxDevices;
        if (cached && ((done.load(std::memory_order_acquire) >> dev) & 1ull)) return cudaSuccess;
        const cudaError_t e = configure();
        if (e == cudaSuccess && cached) done.fetch_or(1ull << dev, std::memory_order_release);
        return e;
    }
};

// SMs of the current device (148 when there is no device to ask).
inline int sm_count()
{
    static std::atomic<int> count[kMaxDevices];
    const int dev = current_device();
    const bool cached = dev >= 0 && dev < kMaxDevices;
    int v = cached ? count[dev].load(std::memory_order_relaxed) : 0;
    if (v > 0) return v;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) {
        cudaGetLastError();
        return 148;
    }
    if (cached) count[dev].store(v, std::memory_order_relaxed);
    return v;
}

// CTAs per (sequence, KV head, split): one per row tile, or one per pair of row tiles (a CTA then serves both tiles
// from one gather, each softmax warpgroup taking every unit for its own tile).  One per tile is the default: the CTAs
// that share a slice of the blocks sit next to each other in the grid, request the same K/V tiles at about the same
// time, and all but the first find them in L2 (240 rows, one sequence: 29.6 MB from DRAM for 29.8 MB algorithmic), and
// the finer CTAs fill the SMs better.  A paired CTA takes 1.93 times as long as a single-tile one (batches of 240-row
// trees: 99.5 against 51.6 us per wave of CTAs), so pairs are used where they save enough waves to pay for that -- in
// practice when the row-tile CTAs just miss fitting the SMs once or twice (10 to 16 such sequences of 8 KV heads:
// 99 against 103 us).
inline bool pair_row_tiles(const sv_geom *g)
{
    const int t = row_tiles(g);
    if (t < 2) return false;
    const long long pairs = (long long)g->n_seq * g->n_kv_heads, sms = sm_count();
    const long long waves_tile = (pairs * t + sms - 1) / sms, waves_pair = (pairs * ((t + 1) / 2) + sms - 1) / sms;
    return 29 * waves_pair < 15 * waves_tile;
}
inline int row_groups(const sv_geom *g)
{
    const int t = row_tiles(g);
    return pair_row_tiles(g) ? (t + 1) / 2 : t;
}

inline sv_status launch_status()
{
    return cudaGetLastError() == cudaSuccess ? SV_OK : SV_ERR_CUDA;
}

}  // namespace svh
