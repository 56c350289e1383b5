// sv_kv_append: commit the accepted draft tokens of a verification step to the paged KV cache and refresh
// the representatives (block means, Eq. 5) of the blocks that grew -- the step on either side of the
// verification attention (Section 2.1: the accepted prefix of the draft is kept; Section 3.1: blocks are cut
// from the current cache).
//
// One CTA per (KV head, sequence).  At most 64 tokens are appended per sequence, so at most two blocks are
// touched: the rows are copied with 128-bit loads/stores (K and V), then the one or two affected block
// means are recomputed from the pool exactly as sv_block_reps does (fp32 sums in a fixed order), which keeps
// them bit-identical to a full rebuild.  Page ids are checked against the pool size before anything is
// written: a table entry that is not a page of the pool ends the table (the rows are dropped).  Traffic: n*512 bytes copied + at most 2*B*256 bytes re-read per
// (sequence, KV head): latency-bound, not bandwidth-bound.
#include <cuda_bf16.h>

#include "sv_host.h"
#include "sv_ptx.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kRowGroups = kThreads / 16;

template <int B>
__global__ void __launch_bounds__(kThreads) kv_append_kernel(uint4 *__restrict__ k_pool, uint4 *__restrict__ v_pool,
                                                             const int32_t *__restrict__ block_table,
                                                             const int32_t *__restrict__ seq_lens,
                                                             const uint4 *__restrict__ draft_k,
                                                             const uint4 *__restrict__ draft_v,
                                                             const int32_t *__restrict__ accept_idx,
                                                             const int32_t *__restrict__ n_accept, int max_accept,
                                                             int32_t *__restrict__ seq_lens_out, float *__restrict__ reps,
                                                             int T, int Hkv, int NBmax, int n_pages)
{
    const int h = blockIdx.x, s = blockIdx.y;
    svk::grid_dependency_wait();
    svk::grid_launch_dependents();
    const int L = seq_lens[s];
    int n = min(max(n_accept[s], 0), max_accept);
    n = L < 0 ? 0 : max(0, min(n, NBmax * B - L));   // never past the last page of the table (nothing if L is already there)
    // A block whose table entry is not a page of the pool (not assigned yet: -1, or stale) ends the table: no row
    // enters it.  n <= 64 <= B, so the rows touch at most the blocks L / B and L / B + 1.
    for (int b = L / B; n > 0 && b <= (L + n - 1) / B; ++b) {
        const int page = block_table[(size_t)s * NBmax + b];
        if (page < 0 || page >= n_pages) n = max(0, min(n, b * B - L));
    }
    const int Ln = L + n;
    if (h == 0 && threadIdx.x == 0) seq_lens_out[s] = Ln;
    if (n <= 0) return;

    // copy the accepted rows: 16 threads per 256-byte row, K and V
    for (int idx = threadIdx.x; idx < n * 32; idx += kThreads) {
        const int a = idx >> 5, which = (idx >> 4) & 1, c = idx & 15;
        const int j = min(max(accept_idx[(size_t)s * max_accept + a], 0), T - 1);
        const int t = L + a;
        const int page = block_table[(size_t)s * NBmax + t / B];
        const size_t dst = (((size_t)page * Hkv + h) * B + (t % B)) * 16 + c;
        const size_t src = (((size_t)s * T + j) * Hkv + h) * 16 + c;
        if (which)
            v_pool[dst] = __ldg(draft_v + src);
        else
            k_pool[dst] = __ldg(draft_k + src);
    }
    if (!reps) return;
    __syncthreads();   // the rows written above are read back below by other threads of this CTA

    __shared__ float part[kRowGroups][128];
    const int chunk = threadIdx.x & 15, rg = threadIdx.x >> 4;
    for (int b = L / B; b <= (Ln - 1) / B; ++b) {
        const int cnt = min(B, Ln - b * B);
        const int page = block_table[(size_t)s * NBmax + b];
        const uint4 *tile = k_pool + ((size_t)page * Hkv + h) * (B * 16);
        constexpr int kIter = B / kRowGroups;
        uint4 v[kIter];
#pragma unroll
        for (int i = 0; i < kIter; ++i) {
            const int row = rg + i * kRowGroups;
            v[i] = row < cnt ? tile[row * 16 + chunk] : make_uint4(0u, 0u, 0u, 0u);   // plain loads: some rows were just written
        }
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int i = 0; i < kIter; ++i) {
            const __nv_bfloat162 *p2 = reinterpret_cast<const __nv_bfloat162 *>(&v[i]);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 f = __bfloat1622float2(p2[j]);
                acc[2 * j] += f.x;
                acc[2 * j + 1] += f.y;
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) part[rg][chunk * 8 + j] = acc[j];
        __syncthreads();
        if (threadIdx.x < 128) {
            float sum = 0.f;
#pragma unroll
            for (int g = 0; g < kRowGroups; ++g) sum += part[g][threadIdx.x];
            reps[(((size_t)s * Hkv + h) * NBmax + b) * 128 + threadIdx.x] = sum / (float)cnt;
        }
        __syncthreads();
    }
}

}  // namespace

extern "C" sv_status sv_kv_append(const sv_geom *geom, void *k_pool, void *v_pool, int32_t n_pages,
                                  const int32_t *block_table, const int32_t *seq_lens, const void *draft_k,
                                  const void *draft_v, const int32_t *accept_idx, const int32_t *n_accept,
                                  int32_t max_accept, int32_t *seq_lens_out, float *reps, void *stream)
{
    sv_status st = svh::check_geom(geom);
    if (st != SV_OK) return st;
    if (!k_pool || !v_pool || !block_table || !seq_lens || !draft_k || !draft_v || !accept_idx || !n_accept || !seq_lens_out)
        return SV_ERR_NULL;
    if (n_pages < 1 || max_accept < 1 || max_accept > geom->n_draft) return SV_ERR_SHAPE;
    if (seq_lens_out == seq_lens) return SV_ERR_SHAPE;   // CTAs of the other KV heads still read the old length
    if (!svh::aligned(k_pool, 128) || !svh::aligned(v_pool, 128) || !svh::aligned(draft_k, 16) ||
        !svh::aligned(draft_v, 16) || (reps && !svh::aligned(reps, 16)))
        return SV_ERR_ALIGN;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(geom->n_kv_heads, geom->n_seq);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    svh::pdl_attribute(attr);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    uint4 *kp = static_cast<uint4 *>(k_pool), *vp = static_cast<uint4 *>(v_pool);
    const uint4 *dk = static_cast<const uint4 *>(draft_k), *dv = static_cast<const uint4 *>(draft_v);
    const cudaError_t e =
        geom->block_size == 64
            ? cudaLaunchKernelEx(&cfg, kv_append_kernel<64>, kp, vp, block_table, seq_lens, dk, dv, accept_idx, n_accept,
                                 (int)max_accept, seq_lens_out, reps, (int)geom->n_draft, (int)geom->n_kv_heads,
                                 (int)geom->max_blocks, (int)n_pages)
            : cudaLaunchKernelEx(&cfg, kv_append_kernel<128>, kp, vp, block_table, seq_lens, dk, dv, accept_idx, n_accept,
                                 (int)max_accept, seq_lens_out, reps, (int)geom->n_draft, (int)geom->n_kv_heads,
                                 (int)geom->max_blocks, (int)n_pages);
    return e == cudaSuccess ? svh::launch_status() : SV_ERR_CUDA;
}
