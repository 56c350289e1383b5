// Acceptance of the draft tokens after verification (Section 2.1, Eq. 2-3), chains and trees.
//
// One thread-block cluster per sequence; the vocabulary is split into contiguous ranges, one per CTA, and
// inside a CTA into contiguous segments, one per thread.  Every CTA runs the same walk from the root (row 0):
// a child c of the current row with token x is accepted when u_accept[c] < min(1, p(x) / q(x)) (Eq. 2); a
// rejected child replaces p by norm(max(0, p - q)) (Eq. 3), which is never materialised: after k rejections at
// a row, p_k(y) follows from p_target(y), q(y) and the k normalisers Z_1..Z_k by k subtract-clamp-scale steps.
// Each normaliser is one pass over the vocabulary: per-thread segment sums, a block reduction in fixed order,
// CTA totals exchanged through distributed shared memory, one hardware cluster barrier.  All CTAs add the
// totals in the same order, so every CTA takes the same decisions.  The next token is drawn by inverting the
// cumulative sum of the final p in vocabulary order: CTA totals -> the CTA that holds the target, block scan
// of its thread sums -> the thread, a sequential walk of that thread's segment -> the token.
// fp32 throughout; no spin-waits (cluster barriers only).
#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <math.h>

#include "sv_host.h"
#include "sv_ptx.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxRows = 64;     // draft rows per step (the ancestor masks of the attention kernel are 64 bits)
constexpr int kMaxCluster = 8;

struct AcceptParams {
    const float *p_target;   // [S][T][V]
    const float *p_draft;    // [S][T][V]
    const int32_t *tokens;   // [S][T]
    const int32_t *parent;   // [S][T] or nullptr (chain)
    const float *u_accept;   // [S][T]
    const float *u_next;     // [S]
    int32_t *path;           // [S][T]
    int32_t *n_path;         // [S]
    int32_t *next_token;     // [S]
    float *alpha;            // [S][T] or nullptr
    int T, V, chunk, seg;    // chunk: vocabulary entries per CTA, seg: per thread (multiples of 4)
};

// p after `r` rejections at the current row, at one vocabulary entry
__device__ __forceinline__ float adjusted(float pt, float q, int r, const float *inv_z)
{
    float v = pt;
    for (int k = 0; k < r; ++k) v = fmaxf(v - q, 0.f) * inv_z[k];
    return v;
}

// Weight of entry y in the current pass: kResidual ? max(0, p_r - q) : p_r
template <bool kResidual>
__device__ __forceinline__ float weight(float pt, float q, int r, const float *inv_z)
{
    const float v = adjusted(pt, q, r, inv_z);
    return kResidual ? fmaxf(v - q, 0.f) : v;
}

// Sum of this thread's segment [y0, y1) in vocabulary order.
template <bool kResidual>
__device__ __forceinline__ float segment_sum(const float *pt, const float *q, int y0, int y1, int r, const float *inv_z)
{
    float acc = 0.f;
    for (int y = y0; y < y1; y += 4) {
        const float4 a = __ldg(reinterpret_cast<const float4 *>(pt + y));
        const float4 b = __ldg(reinterpret_cast<const float4 *>(q + y));
        acc += weight<kResidual>(a.x, b.x, r, inv_z);
        acc += weight<kResidual>(a.y, b.y, r, inv_z);
        acc += weight<kResidual>(a.z, b.z, r, inv_z);
        acc += weight<kResidual>(a.w, b.w, r, inv_z);
    }
    return acc;
}

// Inclusive prefix of `v` over the CTA in thread order (fixed association); total returned through `total`.
__device__ __forceinline__ float block_inclusive_scan(float v, float *warp_tot, float &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();   // warp_tot of the previous scan has been consumed
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    float before = 0.f, tot = 0.f;
    for (int w = 0; w < kWarps; ++w) {
        if (w == warp) before = tot;
        tot += warp_tot[w];
    }
    total = tot;
    return before + inc;
}

__global__ void __launch_bounds__(kThreads) accept_kernel(const AcceptParams p)
{
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank(), CL = (int)cluster.num_blocks();
    const int s = blockIdx.y, tid = threadIdx.x;
    __shared__ int tok[kMaxRows], par[kMaxRows];
    __shared__ float u[kMaxRows];
    __shared__ float inv_z[kMaxRows];
    __shared__ float warp_tot[kWarps];
    __shared__ float cta_tot[2][kMaxCluster];   // totals of all CTAs, written by their owners; two buffers in turn
    __shared__ int s_first, s_last;

    svk::grid_dependency_wait();
    svk::grid_launch_dependents();
    if (tid < p.T) {
        tok[tid] = p.tokens[(size_t)s * p.T + tid];
        par[tid] = p.parent ? p.parent[(size_t)s * p.T + tid] : tid - 1;
        u[tid] = p.u_accept[(size_t)s * p.T + tid];
    }
    const float u_next = p.u_next[s];
    __syncthreads();
    cluster.sync();   // every CTA of the cluster is running: its shared memory may be written from here on

    const int lo = min(p.V, rank * p.chunk), hi = min(p.V, lo + p.chunk);
    const int y0 = min(hi, lo + tid * p.seg), y1 = min(hi, y0 + p.seg);
    const bool writer = rank == 0 && tid == 0;
    int n_red = 0;

    // total over the cluster of the CTAs' sums; leaves the per-CTA sums in cta_tot[buf]
    auto cluster_total = [&](float cta_sum, int &buf) {
        buf = n_red & 1;
        ++n_red;
        if (tid < CL) *cluster.map_shared_rank(&cta_tot[buf][rank], tid) = cta_sum;
        cluster.sync();
        float t = 0.f;
        for (int c = 0; c < CL; ++c) t += cta_tot[buf][c];
        return t;
    };

    int cur = 0, n = 1, r = 0, buf = 0;
    if (writer) p.path[(size_t)s * p.T] = 0;
    const float *pt = nullptr, *q = nullptr;
    for (;;) {
        pt = p.p_target + ((size_t)s * p.T + cur) * p.V;
        q = p.p_draft + ((size_t)s * p.T + cur) * p.V;
        r = 0;
        bool moved = false;
        for (int c = cur + 1; c < p.T; ++c) {
            if (par[c] != cur) continue;
            const int x = min(max(tok[c], 0), p.V - 1);
            const float qx = __ldg(q + x);
            const float px = adjusted(__ldg(pt + x), qx, r, inv_z);
            const float a = (qx <= 0.f || px >= qx) ? 1.f : __fdiv_rn(px, qx);   // Eq. 2
            if (writer && p.alpha) p.alpha[(size_t)s * p.T + c] = a;
            if (u[c] < a) {
                if (writer) p.path[(size_t)s * p.T + n] = c;
                ++n;
                cur = c;
                moved = true;
                break;
            }
            // rejected: Z = sum_y max(0, p - q) (Eq. 3); p itself is never stored
            float tot;
            block_inclusive_scan(segment_sum<true>(pt, q, y0, y1, r, inv_z), warp_tot, tot);
            const float z = cluster_total(tot, buf);
            if (z > 0.f) {   // a residual without mass (p == q) leaves p as it is
                if (tid == 0) inv_z[r] = __frcp_rn(z);
                ++r;
                __syncthreads();
            }
        }
        if (!moved) break;
    }
    if (writer) {
        p.n_path[s] = n;
        for (int i = n; i < p.T; ++i) p.path[(size_t)s * p.T + i] = -1;
    }

    // next token: the smallest x with  sum_{y <= x} p(y) >= u_next * sum_y p(y)  and p(x) > 0
    float tot;
    const float mine = segment_sum<false>(pt, q, y0, y1, r, inv_z);
    const float inc = block_inclusive_scan(mine, warp_tot, tot);
    const float W = cluster_total(tot, buf);
    const float target = u_next * W;
    int owner = -1, last_pos = -1;
    float before = 0.f, before_last = 0.f, run = 0.f;
    for (int c = 0; c < CL; ++c) {
        const float t = cta_tot[buf][c];
        if (t > 0.f) {
            if (owner < 0 && run + t >= target) owner = c, before = run;
            last_pos = c, before_last = run;
        }
        run += t;
    }
    if (owner < 0) owner = last_pos, before = before_last;   // rounding left the target just above the total
    if (owner < 0) {                                         // no mass anywhere
        if (writer) p.next_token[s] = p.V - 1;
        return;
    }
    if (rank != owner) return;
    const float local = target - before;
    if (tid == 0) s_first = kThreads, s_last = -1;
    __syncthreads();
    if (mine > 0.f) {
        if (inc >= local) atomicMin(&s_first, tid);
        atomicMax(&s_last, tid);
    }
    __syncthreads();
    const int chosen = s_first < kThreads ? s_first : s_last;
    if (tid != chosen) return;
    float acc = inc - mine;
    int pick = -1, last_y = -1;
    for (int y = y0; y < y1 && pick < 0; ++y) {
        const float w = weight<false>(__ldg(pt + y), __ldg(q + y), r, inv_z);
        acc += w;
        if (w > 0.f) {
            last_y = y;
            if (acc >= local) pick = y;
        }
    }
    p.next_token[s] = pick >= 0 ? pick : last_y;
}

}  // namespace

extern "C" sv_status sv_accept(int32_t n_seq, int32_t n_draft, int32_t vocab, const float *p_target, const float *p_draft,
                               const int32_t *tokens, const int32_t *parent, const float *u_accept, const float *u_next,
                               int32_t *path, int32_t *n_path, int32_t *next_token, float *alpha, void *stream)
{
    if (!p_target || !p_draft || !tokens || !u_accept || !u_next || !path || !n_path || !next_token) return SV_ERR_NULL;
    if (n_seq < 1 || n_seq > 65535 || vocab < 1) return SV_ERR_SHAPE;
    if (n_draft < 1) return SV_ERR_SHAPE;
    if (n_draft > kMaxRows) return SV_ERR_UNSUPPORTED;
    if (vocab % 4 != 0 || !svh::aligned(p_target, 16) || !svh::aligned(p_draft, 16)) return SV_ERR_ALIGN;
    int CL = 1;
    while (CL < kMaxCluster && vocab / (CL * 2) >= 4096) CL *= 2;   // at least 4096 entries per CTA
    AcceptParams p;
    p.p_target = p_target, p.p_draft = p_draft, p.tokens = tokens, p.parent = parent, p.u_accept = u_accept;
    p.u_next = u_next, p.path = path, p.n_path = n_path, p.next_token = next_token, p.alpha = alpha;
    p.T = n_draft, p.V = vocab;
    p.chunk = ((vocab / 4 + CL - 1) / CL) * 4;
    p.seg = ((p.chunk / 4 + kThreads - 1) / kThreads) * 4;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(CL, n_seq);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CL;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    svh::pdl_attribute(attr + 1);
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, accept_kernel, p) != cudaSuccess) return SV_ERR_CUDA;
    return svh::launch_status();
}
