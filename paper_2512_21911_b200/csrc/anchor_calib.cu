// Anchor-layer calibration (Section 3.3, Eq. 7-8): Jaccard similarity between the block masks that adjacent
// layers kept, and the choice of the K least similar layers as anchors.
//
// sv_anchor_jaccard: one CTA per (sample, layer).  Per KV head the previous layer's list is scattered into a
// shared-memory bitmap (one bit per block) and the current layer's list is tested against it:
// |A n B| = hits, |A u B| = |A| + |B| - hits.  Integer set arithmetic, exact.  sv_pick_anchors runs on the
// host (a few dozen numbers).
#include <cuda_runtime.h>

#include "sv_host.h"
#include "sv_ptx.cuh"

namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads) anchor_jaccard_kernel(const int32_t *__restrict__ idx,
                                                                  const int32_t *__restrict__ cnt, int32_t *__restrict__ inter,
                                                                  int32_t *__restrict__ uni, int S, int Hkv, int NBmax,
                                                                  int max_sel)
{
    extern __shared__ uint32_t bitmap[];   // [(NBmax + 31) / 32]
    __shared__ int s_inter, s_union;
    const int s = blockIdx.x, l = blockIdx.y;
    svk::grid_dependency_wait();
    svk::grid_launch_dependents();
    if (threadIdx.x == 0) s_inter = 0, s_union = 0;
    const int words = (NBmax + 31) >> 5;
    if (l > 0) {
        for (int h = 0; h < Hkv; ++h) {
            for (int i = threadIdx.x; i < words; i += kThreads) bitmap[i] = 0u;
            __syncthreads();
            const size_t cur = ((size_t)l * S + s) * Hkv + h, prev = ((size_t)(l - 1) * S + s) * Hkv + h;
            const int na = min(max(cnt[cur], 0), max_sel), nb = min(max(cnt[prev], 0), max_sel);
            for (int i = threadIdx.x; i < nb; i += kThreads) {
                const int b = idx[prev * max_sel + i];
                if (b >= 0 && b < NBmax) atomicOr(&bitmap[b >> 5], 1u << (b & 31));
            }
            __syncthreads();
            int hits = 0;
            for (int i = threadIdx.x; i < na; i += kThreads) {
                const int b = idx[cur * max_sel + i];
                if (b >= 0 && b < NBmax) hits += (bitmap[b >> 5] >> (b & 31)) & 1u;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) hits += __shfl_xor_sync(0xffffffffu, hits, o);
            if ((threadIdx.x & 31) == 0 && hits) atomicAdd(&s_inter, hits);
            if (threadIdx.x == 0) atomicAdd(&s_union, na + nb);
            __syncthreads();
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        inter[(size_t)l * S + s] = s_inter;
        uni[(size_t)l * S + s] = s_union - s_inter;
    }
}

}  // namespace

extern "C" sv_status sv_anchor_jaccard(const sv_geom *geom, int32_t n_layers, const int32_t *sel_idx_all,
                                       const int32_t *sel_cnt_all, int32_t max_sel, int32_t *inter, int32_t *uni,
                                       void *stream)
{
    sv_status st = svh::check_geom(geom);
    if (st != SV_OK) return st;
    if (!sel_idx_all || !sel_cnt_all || !inter || !uni) return SV_ERR_NULL;
    if (n_layers < 1 || n_layers > 65535 || max_sel < 1) return SV_ERR_SHAPE;
    const size_t smem = (size_t)((geom->max_blocks + 31) / 32) * 4;
    if (smem > 48 * 1024) return SV_ERR_UNSUPPORTED;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(geom->n_seq, n_layers);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    svh::pdl_attribute(attr);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, anchor_jaccard_kernel, sel_idx_all, sel_cnt_all, inter, uni, (int)geom->n_seq,
                           (int)geom->n_kv_heads, (int)geom->max_blocks, (int)max_sel) != cudaSuccess)
        return SV_ERR_CUDA;
    return svh::launch_status();
}

extern "C" sv_status sv_pick_anchors(const int32_t *inter, const int32_t *uni, int32_t n_layers, int32_t n_samples,
                                     int32_t n_anchors, uint8_t *anchors, double *jaccard)
{
    if (!inter || !uni || !anchors) return SV_ERR_NULL;
    if (n_layers < 1 || n_samples < 1 || n_anchors < 1 || n_anchors > n_layers) return SV_ERR_SHAPE;
    double local[256];
    double *J = jaccard ? jaccard : local;
    if (!jaccard && n_layers > 256) return SV_ERR_UNSUPPORTED;
    for (int l = 0; l < n_layers; ++l) {
        double sum = 0.0;
        for (int s = 0; s < n_samples; ++s) {
            const int u = uni[(size_t)l * n_samples + s];
            sum += u > 0 ? (double)inter[(size_t)l * n_samples + s] / (double)u : 1.0;
        }
        J[l] = l > 0 ? sum / (double)n_samples : 0.0;   // J(M_1, M_0) = 0 by definition
        anchors[l] = 0;
    }
    for (int k = 0; k < n_anchors; ++k) {
        int best = -1;
        for (int l = 0; l < n_layers; ++l)
            if (!anchors[l] && (best < 0 || 1.0 - J[l] > 1.0 - J[best])) best = l;   // ties: the earlier layer
        anchors[best] = 1;
    }
    return SV_OK;
}
