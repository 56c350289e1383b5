// sv_block_reps: mean key of every KV block (the block representative implied by Eq. 5).
//
// Pure streaming reduction, bound by HBM bandwidth: one CTA per (block, KV head,
// sequence) reads the contiguous B x 128 bf16 tile of the block with 128-bit loads
// (all of a thread's loads are issued before the first use), accumulates in fp32 in a
// fixed order and writes 128 fp32 values.  Algorithmic traffic: B*256 bytes read +
// 512 bytes written per block.
#include <cuda_bf16.h>

#include "sv_host.h"
#include "sv_ptx.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kRowGroups = kThreads / 16;   // 16 threads cover one 256-byte key row

// OutT: float (the default representatives) or __nv_bfloat16 (storage variant: the fp32 mean rounded once).
template <int B, typename OutT>
__global__ void __launch_bounds__(kThreads) block_reps_kernel(const uint4 *__restrict__ k_pool,
                                                              const int32_t *__restrict__ block_table,
                                                              const int32_t *__restrict__ seq_lens,
                                                              OutT *__restrict__ reps, int Hkv, int NBmax,
                                                              int block_begin, int block_end)
{
    const int s = blockIdx.z, h = blockIdx.y;
    svk::grid_dependency_wait();      // the keys may come from the kernel just before (a cache append)
    svk::grid_launch_dependents();
    const int L = seq_lens[s];
    const int nb = min((L + B - 1) / B, NBmax);
    const int b = block_begin < 0 ? nb - 1 : block_begin + blockIdx.x;   // block_begin < 0: the tail block
    if (b < 0 || b >= nb || (block_begin >= 0 && block_end >= 0 && b >= block_end)) return;
    const int cnt = min(B, L - b * B);
    const int page = block_table[(size_t)s * NBmax + b];
    const uint4 *tile = k_pool + ((size_t)page * Hkv + h) * (B * 16);

    const int chunk = threadIdx.x & 15;     // 8 dims = one 16-byte chunk of the row
    const int rg = threadIdx.x >> 4;
    constexpr int kIter = B / kRowGroups;
    uint4 v[kIter];
#pragma unroll
    for (int i = 0; i < kIter; ++i) {
        const int row = rg + i * kRowGroups;
        v[i] = row < cnt ? __ldg(tile + row * 16 + chunk) : make_uint4(0u, 0u, 0u, 0u);
    }
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int i = 0; i < kIter; ++i) {
        const __nv_bfloat162 *p = reinterpret_cast<const __nv_bfloat162 *>(&v[i]);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 f = __bfloat1622float2(p[j]);
            acc[2 * j] += f.x;
            acc[2 * j + 1] += f.y;
        }
    }
    __shared__ float part[kRowGroups][128];
#pragma unroll
    for (int j = 0; j < 8; ++j) part[rg][chunk * 8 + j] = acc[j];
    __syncthreads();
    if (threadIdx.x < 128) {
        float sum = 0.f;
#pragma unroll
        for (int g = 0; g < kRowGroups; ++g) sum += part[g][threadIdx.x];
        reps[(((size_t)s * Hkv + h) * NBmax + b) * 128 + threadIdx.x] = static_cast<OutT>(sum / (float)cnt);
    }
}

}  // namespace

template <typename OutT>
static sv_status launch_block_reps(const sv_geom *geom, const sv_kv *kv, int32_t block_begin, int32_t block_end,
                                   OutT *reps, void *stream)
{
    sv_status st = svh::check_geom(geom);
    if (st != SV_OK) return st;
    st = svh::check_kv(geom, kv, false);
    if (st != SV_OK) return st;
    if (!reps) return SV_ERR_NULL;
    if (!svh::aligned(reps, 16)) return SV_ERR_ALIGN;
    if (block_begin < 0 && block_begin != SV_TAIL_BLOCK) return SV_ERR_SHAPE;
    const int hi = (block_end < 0 || block_end > geom->max_blocks) ? geom->max_blocks : block_end;
    if (block_begin >= 0 && hi <= block_begin) return SV_OK;   // empty range: nothing to do
    dim3 grid(block_begin < 0 ? 1 : hi - block_begin, geom->n_kv_heads, geom->n_seq);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    svh::pdl_attribute(attr);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const uint4 *pool = static_cast<const uint4 *>(kv->k_pool);
    const cudaError_t e =
        geom->block_size == 64
            ? cudaLaunchKernelEx(&cfg, block_reps_kernel<64, OutT>, pool, kv->block_table, kv->seq_lens, reps,
                                 (int)geom->n_kv_heads, (int)geom->max_blocks, (int)block_begin, (int)block_end)
            : cudaLaunchKernelEx(&cfg, block_reps_kernel<128, OutT>, pool, kv->block_table, kv->seq_lens, reps,
                                 (int)geom->n_kv_heads, (int)geom->max_blocks, (int)block_begin, (int)block_end);
    return e == cudaSuccess ? svh::launch_status() : SV_ERR_CUDA;
}

extern "C" sv_status sv_block_reps(const sv_geom *geom, const sv_kv *kv, int32_t block_begin, int32_t block_end,
                                   float *reps, void *stream)
{
    return launch_block_reps<float>(geom, kv, block_begin, block_end, reps, stream);
}

extern "C" sv_status sv_block_reps_bf16(const sv_geom *geom, const sv_kv *kv, int32_t block_begin, int32_t block_end,
                                        void *reps_bf16, void *stream)
{
    return launch_block_reps<__nv_bfloat16>(geom, kv, block_begin, block_end, static_cast<__nv_bfloat16 *>(reps_bf16), stream);
}
