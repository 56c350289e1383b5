// sv_select_blocks: importance scores (Eq. 5) of every block of a (sequence, KV head) against the
// first draft token's query, then the top-N blocks with the first/last few kept (Section 3.1), in one
// launch.  reuse_prev copies the previous layer's set (Section 3.3, Eq. 9).
//
// One thread-block cluster per (sequence, KV head).  Each CTA of the cluster scores a contiguous
// slice of the blocks (a GEMV over fp32 representatives: one warp per block row, 128-bit loads,
// several rows in flight per warp) into its own shared memory as order-preserving 32-bit keys.  After a
// cluster barrier CTA 0 pulls the slices through distributed shared memory and runs an exact
// radix select (4 passes of 8 bits) for the N-th largest key, then compacts the kept block indices in
// ascending order with a block-wide scan; equal keys are taken smallest index first.  No global
// scratch, no spin-waits (hardware cluster barriers only).
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include "sv_host.h"
#include "sv_ptx.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kRowsPerIter = 4;   // independent representative rows a warp has in flight

__device__ __forceinline__ uint32_t order_key(float x)
{
    const uint32_t u = __float_as_uint(x + 0.0f);   // -0 -> +0
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct SelectParams {
    const __nv_bfloat16 *q;   // [S][T][Hq][128]
    const float *reps;        // [S][Hkv][NBmax][128]
    const int32_t *seq_lens;
    const int32_t *budget;
    int32_t *out_idx;
    int32_t *out_cnt;
    float *out_scores;
    int T, Hq, Hkv, B, NBmax, n_sink, n_local, max_sel, chunk;
};

__global__ void __launch_bounds__(kThreads) select_kernel(const SelectParams p)
{
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int CL = (int)cluster.num_blocks();
    const int h = blockIdx.y, s = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    extern __shared__ uint32_t smem_keys[];
    uint32_t *keys_local = smem_keys;              // [chunk]   this CTA's slice
    uint32_t *keys_all = smem_keys + p.chunk;      // [CL*chunk] gathered by CTA 0
    __shared__ float qbar[128];
    __shared__ uint32_t hist[256];
    __shared__ uint32_t sh_bin, sh_remaining;
    __shared__ uint32_t warp_sel[kWarps], warp_eq[kWarps];

    const int L = p.seq_lens[s];
    const int nb = min((L + p.B - 1) / p.B, p.NBmax);
    const int forced = min(nb, p.n_sink + p.n_local);
    int N = min(max(p.budget[s], forced), p.max_sel);
    const bool keep_all = N >= nb;
    if (keep_all) N = nb;

    // While the kernel that precedes this one in the stream drains, pull this warp's first batch of
    // representative rows towards L2 (a prefetch consumes no data, so it is safe even if that kernel
    // is still writing them); all real loads come after the dependency wait.
    const bool need_scores = !keep_all || p.out_scores;
    const int b0 = rank * p.chunk;
    const int b1 = min(b0 + p.chunk, nb);
    const float4 *rbase = reinterpret_cast<const float4 *>(p.reps + ((size_t)s * p.Hkv + h) * p.NBmax * 128);
    float4 r[kRowsPerIter];
    int b = b0 + warp * kRowsPerIter;
    auto load_rows = [&](int bb) {
#pragma unroll
        for (int i = 0; i < kRowsPerIter; ++i)
            r[i] = (bb + i < b1) ? __ldg(rbase + (size_t)(bb + i) * 32 + lane) : make_float4(0.f, 0.f, 0.f, 0.f);
    };
    if (need_scores) {
#pragma unroll
        for (int i = 0; i < kRowsPerIter; ++i)
            if (b + i < b1) svk::prefetch_l2(rbase + (size_t)(b + i) * 32 + lane);
    }
    svk::grid_dependency_wait();
    svk::grid_launch_dependents();
    if (need_scores && b < b1) load_rows(b);

    // retrieval query: mean of the first draft token's query over the GQA group
    const int G = p.Hq / p.Hkv;
    if (tid < 128) {
        const __nv_bfloat16 *q0 = p.q + ((size_t)s * p.T * p.Hq + (size_t)h * G) * 128 + tid;
        float sum = 0.f;
        for (int g = 0; g < G; ++g) sum += __bfloat162float(q0[(size_t)g * 128]);
        qbar[tid] = sum / (float)G;
    }
    __syncthreads();

    if (need_scores) {
        const float4 qv = reinterpret_cast<const float4 *>(qbar)[lane];
        for (; b < b1; b += kWarps * kRowsPerIter) {
#pragma unroll
            for (int i = 0; i < kRowsPerIter; ++i) {
                float d = r[i].x * qv.x + r[i].y * qv.y + r[i].z * qv.z + r[i].w * qv.w;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
                if (lane == 0 && b + i < b1) {
                    const int bb = b + i;
                    const bool is_forced = bb < p.n_sink || bb >= nb - p.n_local;
                    keys_local[bb - b0] = is_forced ? 0xFFFFFFFFu : order_key(d);
                    if (p.out_scores) p.out_scores[((size_t)s * p.Hkv + h) * p.NBmax + bb] = d;
                }
            }
            if (b + kWarps * kRowsPerIter < b1) load_rows(b + kWarps * kRowsPerIter);
        }
    }
    cluster.sync();
    if (rank == 0 && !keep_all) {
        for (int b = tid; b < nb; b += kThreads) {
            const uint32_t *remote = cluster.map_shared_rank(keys_local, b / p.chunk);
            keys_all[b] = remote[b % p.chunk];
        }
    }
    cluster.sync();   // no CTA may exit while CTA 0 still reads its shared memory
    if (rank != 0) return;

    int32_t *out = p.out_idx + ((size_t)s * p.Hkv + h) * p.max_sel;
    if (keep_all) {
        for (int b = tid; b < nb; b += kThreads) out[b] = b;
        if (tid == 0) p.out_cnt[(size_t)s * p.Hkv + h] = nb;
        return;
    }

    // exact radix select of the N-th largest key
    uint32_t prefix = 0, mask = 0, remaining = (uint32_t)N;
#pragma unroll 1
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        for (int b = tid; b < nb; b += kThreads) {
            const uint32_t k = keys_all[b];
            if ((k & mask) == prefix) atomicAdd(&hist[(k >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (warp == 0) {
            // lane j owns bins 255-8j .. 248-8j (descending)
            uint32_t c[8], tot = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                c[i] = hist[255 - 8 * lane - i];
                tot += c[i];
            }
            uint32_t incl = tot;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            const uint32_t excl = incl - tot;
            if (excl < remaining && remaining <= incl) {   // exactly one lane
                uint32_t above = excl;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (above < remaining && remaining <= above + c[i]) {
                        sh_bin = 255 - 8 * lane - i;
                        sh_remaining = remaining - above;
                    }
                    above += c[i];
                }
            }
        }
        __syncthreads();
        prefix |= sh_bin << shift;
        mask |= 0xFFu << shift;
        remaining = sh_remaining;
        __syncthreads();
    }
    const uint32_t thr = prefix;          // N-th largest key
    const uint32_t take_eq = remaining;   // how many keys equal to thr are kept (smallest indices first)

    // ascending compaction
    uint32_t base_sel = 0, base_eq = 0;
    for (int c0 = 0; c0 < nb; c0 += kThreads) {
        const int b = c0 + tid;
        const uint32_t k = b < nb ? keys_all[b] : 0u;
        const bool gt = b < nb && k > thr;
        const bool eq = b < nb && k == thr;
        const uint32_t eq_ballot = __ballot_sync(0xffffffffu, eq);
        if (lane == 0) warp_eq[warp] = __popc(eq_ballot);
        __syncthreads();
        uint32_t eq_before = base_eq, eq_total = 0;
        for (int w = 0; w < kWarps; ++w) {
            if (w < warp) eq_before += warp_eq[w];
            eq_total += warp_eq[w];
        }
        const uint32_t eq_rank = eq_before + __popc(eq_ballot & ((1u << lane) - 1u));
        const bool sel = gt || (eq && eq_rank < take_eq);
        const uint32_t sel_ballot = __ballot_sync(0xffffffffu, sel);
        if (lane == 0) warp_sel[warp] = __popc(sel_ballot);
        __syncthreads();
        uint32_t sel_before = base_sel, sel_total = 0;
        for (int w = 0; w < kWarps; ++w) {
            if (w < warp) sel_before += warp_sel[w];
            sel_total += warp_sel[w];
        }
        if (sel) out[sel_before + __popc(sel_ballot & ((1u << lane) - 1u))] = b;
        base_sel += sel_total;
        base_eq += eq_total;
        __syncthreads();
    }
    if (tid == 0) p.out_cnt[(size_t)s * p.Hkv + h] = N;
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

extern "C" sv_status sv_select_blocks(const sv_geom *geom, const void *q, const float *reps, const int32_t *seq_lens,
                                      const int32_t *budget_blocks, int32_t n_sink, int32_t n_local,
                                      int32_t reuse_prev, const int32_t *prev_idx, const int32_t *prev_cnt,
                                      int32_t *out_idx, int32_t *out_cnt, int32_t max_sel, float *out_scores,
                                      void *stream)
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

    int CL = 1;
    while (CL < 8 && geom->max_blocks / (CL * 2) >= 32) CL *= 2;
    const int per = (geom->max_blocks + CL - 1) / CL;
    const int chunk = (per + kWarps * kRowsPerIter - 1) / (kWarps * kRowsPerIter) * (kWarps * kRowsPerIter);

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

    const size_t smem = (size_t)(CL + 1) * chunk * sizeof(uint32_t);
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return SV_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(CL, geom->n_kv_heads, geom->n_seq);
    cfg.blockDim = dim3(kThreads);
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
    if (cudaLaunchKernelEx(&cfg, select_kernel, p) != cudaSuccess) return SV_ERR_CUDA;
    return svh::launch_status();
}
