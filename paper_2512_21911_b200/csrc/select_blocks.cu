// sv_select_blocks: importance scores (Eq. 5) of every block of a (sequence, KV head) against the
// first draft token's query, then the top-N blocks with the first/last few kept (Section 3.1), in one
// launch.  reuse_prev copies the previous layer's set (Section 3.3, Eq. 9).
//
// One thread-block cluster (up to 8 CTAs; 16 for a few very long block lists) per (sequence, KV head).  Each CTA of
// the cluster scores a contiguous slice of the blocks (a GEMV over the representatives: one warp per block row, 128-bit loads,
// several rows in flight per warp), turns the scores into order-preserving 32-bit keys and pushes them
// straight into CTA 0's shared memory with st.async stores that count their bytes on an mbarrier there;
// the senders then exit.  CTA 0 waits (bounded) for the expected byte count and selects exactly: the
// scores are mapped linearly onto 16-bit codes, a 256-bin histogram of the upper byte (and, for a crowded
// bin, of the lower byte) finds the boundary, the few keys left at the boundary are ranked by their exact
// keys (ties: smaller block index), and an ascending ballot compaction writes the list.  More than 2048
// blocks, equal scores everywhere or a still crowded boundary take the general radix select on the key
// bits (8-bit digits from the highest differing bit).  No global scratch.  If the bounded wait for the
// keys ever gives up, the count of that (sequence, KV head) is written as -1 (see sv.h).
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include "select_core.cuh"
#include "sv_host.h"
#include "sv_ptx.cuh"

namespace cg = cooperative_groups;

namespace {

// Threads per CTA: 512 while the CTAs of a launch are resident together (two per SM: the selection's barriers are
// the critical path, sixteen warps finish the passes between them soonest, and the attention kernel behind waits for
// the last CTA), 256 for launches of several waves (four CTAs per SM overlap one CTA's latencies with another's work:
// 128 sequences 31 -> 24 us per call and 216 -> 208 us with the attention behind it; with one wave the smaller CTAs
// finish a stand-alone call sooner too, but the attention behind them starts later -- 4 x 128K: 31.0 against 29.8 us).
constexpr int kThreadsFew = 512, kThreadsMany = 256;
constexpr int kRowsPerIter = 4;   // consecutive representative rows a warp scores per pass (one 16-byte store of keys)

using svsel::kForcedKey;
using svsel::order_key;

struct SelectParams {
    const __nv_bfloat16 *q;   // [S][T][Hq][128]
    const void *reps;         // [S][Hkv][NBmax][128], float or bfloat16
    const int32_t *seq_lens;
    const int32_t *budget;
    int32_t *out_idx;
    int32_t *out_cnt;
    float *out_scores;
    int T, Hq, Hkv, B, NBmax, n_sink, n_local, max_sel, chunk;
};

// Cluster of CL CTAs per (sequence, KV head).  Every CTA scores a slice of the blocks and writes the
// keys straight into CTA 0's shared memory (distributed shared memory) with stores that count their bytes
// on an mbarrier there, and exits; CTA 0 waits for the expected number of bytes and selects.  The only cluster-wide barrier is split (arrive early, wait late) so that
// its latency hides behind the loads.
// kBf16: the representatives are stored in bfloat16 (storage variant); scores are fp32 either way.
// kDepth: passes whose rows a warp loads together (1, or 2 for slices of more than 64 blocks: eight rows in flight per
// warp, half as many trips to DRAM; more would cost the second CTA per SM its registers).
template <bool kBf16, int kDepth, int kThreads>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads) select_kernel(const SelectParams p)
{
    constexpr int kWarps = kThreads / 32;
    constexpr int kStride = kWarps * kRowsPerIter;   // blocks the CTA covers per pass
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int CL = (int)cluster.num_blocks();
    const int h = blockIdx.y, s = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    extern __shared__ __align__(16) uint32_t keys_all[];         // [CL*chunk] keys of all blocks (used in CTA 0)
    __shared__ float qbar[128];
    __shared__ svsel::Scratch scratch;
    __shared__ uint64_t keys_ready;                // mbarrier in CTA 0: the bytes of all keys (one arrival: CTA 0 itself)

    // While the kernel that precedes this one in the stream drains: pull this warp's first batch of
    // representative rows and the query row towards L2 (a prefetch consumes no data, so it is safe even if
    // that kernel is still writing them), set up the barrier, zero the histograms.
    if (tid == 0) {
        svk::mbar_init(svk::smem_u32(&keys_ready), 1);
        svk::mbar_fence_init();
    }
    scratch.init(tid, kThreads);
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");   // before any global request is in flight
    const int b0 = rank * p.chunk;
    constexpr int kRowBytes = kBf16 ? 256 : 512, kLaneBytes = kRowBytes / 32;
    const char *rbase = static_cast<const char *>(p.reps) + ((size_t)s * p.Hkv + h) * p.NBmax * kRowBytes;
    auto row_ptr = [&](int row) { return rbase + (size_t)row * kRowBytes + lane * kLaneBytes; };
    auto load_row = [&](int row) {
        if constexpr (kBf16) {
            const uint2 raw = __ldg(reinterpret_cast<const uint2 *>(row_ptr(row)));
            const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&raw.x));
            const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&raw.y));
            return make_float4(lo.x, lo.y, hi.x, hi.y);
        } else {
            return __ldg(reinterpret_cast<const float4 *>(row_ptr(row)));
        }
    };
    int b = b0 + warp * kRowsPerIter;
#pragma unroll
    for (int d = 0; d < kDepth; ++d)
#pragma unroll
        for (int i = 0; i < kRowsPerIter; ++i)
            if (b + d * kStride + i < min(b0 + p.chunk, p.NBmax)) svk::prefetch_l2(row_ptr(b + d * kStride + i));
    const int G = p.Hq / p.Hkv;
    const __nv_bfloat16 *q0 = p.q + ((size_t)s * p.T * p.Hq + (size_t)h * G) * 128;
    if (tid < G * 2) svk::prefetch_l2(q0 + tid * 64);
    svk::grid_dependency_wait();
    svk::grid_launch_dependents();

    // every load below is issued before the first use
    const int L = p.seq_lens[s];
    const int budget = p.budget[s];
    float4 r[kDepth][kRowsPerIter];
    auto load_rows = [&](int bb, int hi) {
#pragma unroll
        for (int d = 0; d < kDepth; ++d)
#pragma unroll
            for (int i = 0; i < kRowsPerIter; ++i)
                r[d][i] = (bb + d * kStride + i < hi) ? load_row(bb + d * kStride + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    };
    load_rows(b, min(b0 + p.chunk, p.NBmax));
    float qsum = 0.f;
    if (tid < 128)
        for (int g = 0; g < G; ++g) qsum += __bfloat162float(q0[(size_t)g * 128 + tid]);
    // CTA 0's barrier is initialised (every CTA arrived before its first global request); the wait costs a few hundred
    // cycles even then, so it sits here, behind the loads it can overlap with
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");

    const int nb = min((L + p.B - 1) / p.B, p.NBmax);
    const int forced = min(nb, p.n_sink + p.n_local);
    int N = min(max(budget, forced), p.max_sel);
    const bool keep_all = N >= nb;
    if (keep_all) N = nb;
    const bool need_scores = !keep_all || p.out_scores;
    const int b1 = min(b0 + p.chunk, nb);

    // retrieval query: mean of the first draft token's query over the GQA group
    if (tid < 128) qbar[tid] = qsum / (float)G;
    __syncthreads();

    const uint32_t keys0 = svk::cluster_map_shared(svk::smem_u32(keys_all), 0);
    const uint32_t ready0 = svk::cluster_map_shared(svk::smem_u32(&keys_ready), 0);
    if (rank == 0 && tid == 0) {
        // what the cluster is about to send: one 16-byte store per four keys of every CTA's slice; the slices are
        // multiples of four blocks long and only the last one in use can be ragged, so that is ceil(nb / 4) stores
        const uint32_t quads = keep_all ? 0u : (uint32_t)(nb + 3) >> 2;
        svk::mbar_arrive_expect_tx(svk::smem_u32(&keys_ready), 16u * quads);
    }
    if (need_scores) {
        const float4 qv = reinterpret_cast<const float4 *>(qbar)[lane];
        for (; b < b1; b += kDepth * kStride) {
#pragma unroll
            for (int d = 0; d < kDepth; ++d) {
                const int bd = b + d * kStride;
                if (bd >= b1) break;   // (warp-uniform)
                uint32_t kk[kRowsPerIter];
#pragma unroll
                for (int i = 0; i < kRowsPerIter; ++i) {
                    float dot = r[d][i].x * qv.x + r[d][i].y * qv.y + r[d][i].z * qv.z + r[d][i].w * qv.w;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                    const int bb = bd + i;
                    const bool is_forced = bb < p.n_sink || bb >= nb - p.n_local;
                    kk[i] = is_forced ? kForcedKey : order_key(dot);
                    if (p.out_scores && lane == 0 && bb < b1) p.out_scores[((size_t)s * p.Hkv + h) * p.NBmax + bb] = dot;
                }
                // rows bd .. bd+3 are 4 consecutive keys: one 16-byte store into CTA 0 (entries past nb are never read)
                if (lane == 0 && !keep_all)
                    svk::st_async_cluster_v4(keys0 + 4u * (uint32_t)bd, make_uint4(kk[0], kk[1], kk[2], kk[3]), ready0);
            }
            if (b + kDepth * kStride < b1) load_rows(b + kDepth * kStride, b1);
        }
    }
    if (rank != 0) return;

    int32_t *out = p.out_idx + ((size_t)s * p.Hkv + h) * p.max_sel;
    int cnt_out;
    if (keep_all) {
        for (int bb = tid; bb < nb; bb += kThreads) out[bb] = bb;
        cnt_out = nb;
    } else if (!__syncthreads_and(svk::mbar_wait_cluster_bounded(svk::smem_u32(&keys_ready), 0))) {
        cnt_out = -1;   // gave up: mark the list invalid (sv_verify_attn then attends over the draft tokens only and reports it)
    } else {
        svsel::select_top<kThreads>(
            keys_all, nb, N, forced, scratch, tid, [] { __syncthreads(); }, [&](int pos, int block) { out[pos] = block; });
        cnt_out = N;
    }
    __syncthreads();   // every thread's entries of the list are written
    if (tid == 0) {
        p.out_cnt[(size_t)s * p.Hkv + h] = cnt_out;
    }
}

__global__ void copy_selection_kernel(const int32_t *__restrict__ prev_idx, const int32_t *__restrict__ prev_cnt,
                                      int32_t *__restrict__ out_idx, int32_t *__restrict__ out_cnt, int n_idx,
                                      int n_cnt)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n_idx) out_idx[i] = prev_idx[i];
    if (i < n_cnt) out_cnt[i] = prev_cnt[i];
}

}  // namespace

template <int kThreads>
static const void *select_fn(bool reps_bf16, bool deep)
{
    return reps_bf16 ? (deep ? reinterpret_cast<const void *>(select_kernel<true, 2, kThreads>)
                             : reinterpret_cast<const void *>(select_kernel<true, 1, kThreads>))
                     : (deep ? reinterpret_cast<const void *>(select_kernel<false, 2, kThreads>)
                             : reinterpret_cast<const void *>(select_kernel<false, 1, kThreads>));
}

// Whether this device can hold clusters of 16 CTAs of the select kernel (asked once per device and instantiation).
static bool clusters_of_16_fit(bool reps_bf16)
{
    static std::atomic<int> state[2][svh::kMaxDevices];   // 0: not asked, 1: yes, 2: no
    const int dev = svh::current_device();
    if (dev < 0 || dev >= svh::kMaxDevices) return false;
    int v = state[reps_bf16][dev].load(std::memory_order_acquire);
    if (v == 0) {
        const void *fn = select_fn<kThreadsFew>(reps_bf16, true);   // (slices of 128 blocks)
        v = 2;
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(16, 8, 1);
            cfg.blockDim = dim3(kThreadsFew);
            cfg.dynamicSmemBytes = 16 * 128 * sizeof(uint32_t);
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 16;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, fn, &cfg) == cudaSuccess && n >= 8) v = 1;
        }
        (void)cudaGetLastError();   // a refusal is an answer, not an error of the call that asked
        state[reps_bf16][dev].store(v, std::memory_order_release);
    }
    return v == 1;
}

static sv_status select_impl(const sv_geom *geom, const void *q, const void *reps, bool reps_bf16, const int32_t *seq_lens,
                             const int32_t *budget_blocks, int32_t n_sink, int32_t n_local, int32_t reuse_prev,
                             const int32_t *prev_idx, const int32_t *prev_cnt, int32_t *out_idx, int32_t *out_cnt,
                             int32_t max_sel, float *out_scores, void *stream)
{
    sv_status st = svh::check_geom(geom);
    if (st != SV_OK) return st;
    if (!out_idx || !out_cnt) return SV_ERR_NULL;
    if (max_sel < 1) return SV_ERR_SHAPE;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (reuse_prev) {
        if (!prev_idx || !prev_cnt) return SV_ERR_NULL;
        const long long n_cnt = (long long)geom->n_seq * geom->n_kv_heads;
        const long long n_idx = n_cnt * max_sel;
        if (n_idx >= (1ll << 31)) return SV_ERR_SHAPE;
        if (prev_idx == out_idx && prev_cnt == out_cnt) return SV_OK;   // already in place
        copy_selection_kernel<<<(unsigned)((n_idx + 255) / 256), 256, 0, cs>>>(prev_idx, prev_cnt, out_idx, out_cnt,
                                                                              (int)n_idx, (int)n_cnt);
        return svh::launch_status();
    }
    if (!q || !reps || !seq_lens || !budget_blocks) return SV_ERR_NULL;
    if (!svh::aligned(q, 16) || !svh::aligned(reps, 16)) return SV_ERR_ALIGN;
    if (n_sink < 0 || n_local < 0) return SV_ERR_SHAPE;
    if (n_sink + n_local > max_sel) return SV_ERR_BUDGET;
    if (geom->max_blocks > svh::kMaxBlocksSelect) return SV_ERR_UNSUPPORTED;

    // CTAs per (sequence, KV head): at least 32 blocks each, and no more CTAs than two per SM (a second wave costs more
    // than the shorter slices save)
    const int pairs = geom->n_seq * geom->n_kv_heads;
    int CL = 1;
    while (CL < 8 && geom->max_blocks / (CL * 2) >= 32 && pairs * CL * 2 <= 2 * svh::sm_count()) CL *= 2;
    // Few pairs with very long block lists (one sequence of 128K tokens: 8 pairs x 2048 blocks) leave most SMs idle at
    // 8 CTAs per pair, and reading the representatives (128 KB per CTA) is what the kernel then waits for: clusters of
    // 16 (beyond the portable size, so the device is asked first whether it can hold them)
    if (CL == 8 && geom->max_blocks >= 2048 && pairs * 16 <= svh::sm_count() && clusters_of_16_fit(reps_bf16)) CL = 16;
    const int per = (geom->max_blocks + CL - 1) / CL;
    const bool many = (long long)pairs * CL > 2 * svh::sm_count();   // more CTAs than fit at once: smaller CTAs, four per SM
    const int threads = many ? kThreadsMany : kThreadsFew;
    const int stride = threads / 32 * kRowsPerIter;              // blocks a CTA covers per pass
    const int chunk = (per + stride - 1) / stride * stride;

    SelectParams p;
    p.q = static_cast<const __nv_bfloat16 *>(q);
    p.reps = reps;
    p.seq_lens = seq_lens;
    p.budget = budget_blocks;
    p.out_idx = out_idx;
    p.out_cnt = out_cnt;
    p.out_scores = out_scores;
    p.T = geom->n_draft, p.Hq = geom->n_q_heads, p.Hkv = geom->n_kv_heads, p.B = geom->block_size;
    p.NBmax = geom->max_blocks, p.n_sink = n_sink, p.n_local = n_local, p.max_sel = max_sel, p.chunk = chunk;

    const size_t smem = (size_t)CL * chunk * sizeof(uint32_t);
    const bool deep = chunk > stride;   // more than one pass per warp: load two passes' rows together
    const void *fn = many ? select_fn<kThreadsMany>(reps_bf16, deep) : select_fn<kThreadsFew>(reps_bf16, deep);
    if (smem > 48 * 1024 && cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return SV_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(CL, geom->n_kv_heads, geom->n_seq);
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = cs;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CL;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    svh::pdl_attribute(attr + 1);
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    void *args[] = {&p};
    if (cudaLaunchKernelExC(&cfg, fn, args) != cudaSuccess) return SV_ERR_CUDA;
    return svh::launch_status();
}

extern "C" sv_status sv_select_blocks(const sv_geom *geom, const void *q, const float *reps, const int32_t *seq_lens,
                                      const int32_t *budget_blocks, int32_t n_sink, int32_t n_local,
                                      int32_t reuse_prev, const int32_t *prev_idx, const int32_t *prev_cnt,
                                      int32_t *out_idx, int32_t *out_cnt, int32_t max_sel, float *out_scores,
                                      void *stream)
{
    return select_impl(geom, q, reps, false, seq_lens, budget_blocks, n_sink, n_local, reuse_prev, prev_idx, prev_cnt,
                       out_idx, out_cnt, max_sel, out_scores, stream);
}

extern "C" sv_status sv_select_blocks_bf16reps(const sv_geom *geom, const void *q, const void *reps_bf16,
                                               const int32_t *seq_lens, const int32_t *budget_blocks, int32_t n_sink,
                                               int32_t n_local, int32_t reuse_prev, const int32_t *prev_idx,
                                               const int32_t *prev_cnt, int32_t *out_idx, int32_t *out_cnt,
                                               int32_t max_sel, float *out_scores, void *stream)
{
    return select_impl(geom, q, reps_bf16, true, seq_lens, budget_blocks, n_sink, n_local, reuse_prev, prev_idx, prev_cnt,
                       out_idx, out_cnt, max_sel, out_scores, stream);
}
