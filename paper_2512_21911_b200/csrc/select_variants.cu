// Retrieval variants the paper discusses but does not adopt (Section 2.2 and Eq. 6), for comparison with the
// adopted strategy (first draft token retrieves, one budget per KV head):
//
//   sv_select_blocks_tokens  every draft token retrieves with its own query: the per-head selection kernel
//                            run once per token row
//   sv_token_overlap         |Sel_i n Sel_j| for every pair of draft tokens (the block-overlap statistic of
//                            Section 2.2): shared-memory bitmaps, AND + popcount.  Integer, exact.
//   sv_select_blocks_global  one budget of budget * Hkv blocks per sequence shared by the KV heads (Eq. 6 counts
//                            blocks over all heads): scores from the per-head kernel, then an exact radix
//                            select over all (head, block) pairs of the sequence and an ordered compaction.
#include <cuda_runtime.h>

#include "sv_host.h"
#include "sv_ptx.cuh"

namespace {

constexpr int kOverlapThreads = 256;
constexpr int kGlobalThreads = 512;   // block barriers dominate this kernel: 1024 threads 32.7 us per cold call, 512 24.6, 256 26.6
constexpr int kGlobalWarps = kGlobalThreads / 32;
constexpr int kMaxParts = 128;          // parts of the ordered compaction (heads x warps per head)
constexpr int kMaxGlobalKeys = 49152;   // (head, block) pairs of one sequence held in shared memory (192 KB)

// One CTA per (sequence, KV head): bitmap of every token's set, then all pairs.
__global__ void __launch_bounds__(kOverlapThreads) token_overlap_kernel(const int32_t *__restrict__ idx,
                                                                        const int32_t *__restrict__ cnt,
                                                                        int32_t *__restrict__ inter, int T, int S, int Hkv,
                                                                        int NBmax, int max_sel)
{
    extern __shared__ uint32_t bitmap[];   // [T][words]
    const int h = blockIdx.x, s = blockIdx.y;
    const int words = (NBmax + 31) >> 5;
    svk::grid_dependency_wait();
    svk::grid_launch_dependents();
    __shared__ int n_of[64];
    for (int i = threadIdx.x; i < T * words; i += kOverlapThreads) bitmap[i] = 0u;
    if (threadIdx.x < T) n_of[threadIdx.x] = min(max(cnt[((size_t)threadIdx.x * S + s) * Hkv + h], 0), max_sel);
    __syncthreads();
    // all tokens' lists in one sweep, so that the kernel pays one memory round trip, not one per token
    for (int e = threadIdx.x; e < T * max_sel; e += kOverlapThreads) {
        const int i = e / max_sel, x = e - i * max_sel;
        if (x < n_of[i]) {
            const int b = idx[(((size_t)i * S + s) * Hkv + h) * max_sel + x];
            if (b >= 0 && b < NBmax) atomicOr(&bitmap[i * words + (b >> 5)], 1u << (b & 31));
        }
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int pair = warp; pair < T * T; pair += kOverlapThreads / 32) {
        const int i = pair / T, j = pair - i * T;
        int c = 0;
        for (int w = lane; w < words; w += 32) c += __popc(bitmap[i * words + w] & bitmap[j * words + w]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
        if (lane == 0) inter[(((size_t)s * Hkv + h) * T + i) * T + j] = c;
    }
}

__device__ __forceinline__ uint32_t order_key(float x)
{
    const uint32_t u = __float_as_uint(x + 0.0f);   // -0 -> +0
    const uint32_t k = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return min(max(k, 1u), 0xFFFFFFFEu);            // 0 = no block, 0xFFFFFFFF = kept without eviction
}

// Exclusive prefix of a per-thread flag over the CTA (thread order) and the CTA total.
__device__ __forceinline__ int block_scan_flag(bool flag, uint32_t *warp_tot, int &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ball = __ballot_sync(0xffffffffu, flag);
    __syncthreads();   // warp_tot of the previous scan has been read by everyone
    if (lane == 0) warp_tot[warp] = __popc(ball);
    __syncthreads();
    int before = 0, tot = 0;
    for (int w = 0; w < kGlobalWarps; ++w) {
        const int v = (int)warp_tot[w];
        if (w < warp) before += v;
        tot += v;
    }
    total = tot;
    return before + __popc(ball & ((1u << lane) - 1u));
}

// One CTA per sequence.
__global__ void __launch_bounds__(kGlobalThreads) select_global_kernel(const float *__restrict__ scores,
                                                                       const int32_t *__restrict__ seq_lens,
                                                                       const int32_t *__restrict__ budget,
                                                                       int32_t *__restrict__ out_idx,
                                                                       int32_t *__restrict__ out_cnt, int Hkv, int B, int NBmax,
                                                                       int n_sink, int n_local, int max_sel)
{
    extern __shared__ uint32_t keys[];   // [Hkv][NBmax]
    __shared__ uint32_t hist[256];
    __shared__ uint32_t warp_tot[kGlobalWarps];
    __shared__ uint32_t s_prefix, s_need, s_and, s_or;
    __shared__ int part_gt[kMaxParts], part_eq[kMaxParts];   // per part: blocks kept for sure / ties; later: start position / ties before
    const int s = blockIdx.x, tid = threadIdx.x;
    svk::grid_dependency_wait();   // the scores come from the kernel just before
    svk::grid_launch_dependents();
    const int L = seq_lens[s];
    const int nb = min((L + B - 1) / B, NBmax);
    const int N = budget[s];
    if (N >= nb) {   // no eviction
        for (int e = tid; e < Hkv * nb; e += kGlobalThreads) {
            const int h = e / nb, b = e - h * nb;
            if (b < max_sel) out_idx[((size_t)s * Hkv + h) * max_sel + b] = b;
        }
        if (tid < Hkv) out_cnt[(size_t)s * Hkv + tid] = min(nb, max_sel);
        return;
    }
    const int forced_per_head = min(nb, n_sink + n_local);
    const int n = Hkv * NBmax;
    for (int e = tid; e < n; e += kGlobalThreads) {
        const int h = e / NBmax, b = e - h * NBmax;
        uint32_t k = 0u;
        if (b < nb) k = (b < n_sink || b >= nb - n_local) ? 0xFFFFFFFFu : order_key(scores[((size_t)s * Hkv + h) * NBmax + b]);
        keys[e] = k;
    }
    // K-th largest key among the evictable blocks: passes of up to 8 bits, most significant first.  The keys of one
    // sequence share their leading bits (same sign, neighbouring exponents), so the digits start at the highest bit in
    // which any two evictable keys differ: the first pass then spreads the keys over the bins instead of piling
    // them into a few (shared-memory atomics on one address serialise).
    uint32_t k_and = 0xFFFFFFFFu, k_or = 0u;
    for (int e = tid; e < n; e += kGlobalThreads) {
        const uint32_t k = keys[e];
        if (k != 0u && k != 0xFFFFFFFFu) k_and &= k, k_or |= k;
    }
    k_and = __reduce_and_sync(0xffffffffu, k_and);
    k_or = __reduce_or_sync(0xffffffffu, k_or);
    if (tid == 0) {
        s_prefix = 0u;
        s_need = (uint32_t)max(0, N * Hkv - forced_per_head * Hkv);
        s_and = 0xFFFFFFFFu, s_or = 0u;
    }
    __syncthreads();
    if ((tid & 31) == 0) {
        atomicAnd(&s_and, k_and);
        atomicOr(&s_or, k_or);
    }
    __syncthreads();
    const bool take_none = s_need == 0u;
    const uint32_t diff = s_and ^ s_or;               // 0: every evictable key is the same (or there is none)
    int top = diff ? 32 - __clz(diff) : 0;           // bits [0, top) still undecided
    uint32_t mask = top >= 32 ? 0u : ~((1u << top) - 1u);
    if (tid == 0) s_prefix = s_or & mask;             // the common leading bits
    __syncthreads();
    while (top > 0 && !take_none) {
        const int w = min(8, top), shift = top - w;
        if (tid < 256) hist[tid] = 0u;
        __syncthreads();
        const uint32_t prefix = s_prefix;
        for (int e = tid; e < n; e += kGlobalThreads) {
            const uint32_t k = keys[e];
            if (k != 0u && k != 0xFFFFFFFFu && (k & mask) == prefix) atomicAdd(&hist[(k >> shift) & ((1u << w) - 1u)], 1u);
        }
        __syncthreads();
        if (tid < 32) {
            // bins from 255 downwards, 8 per lane: the digit d with  #(digit > d) < need <= #(digit >= d)
            const uint32_t need = s_need;
            uint32_t c[8], tot = 0u;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                c[k] = hist[255 - (tid * 8 + k)];
                tot += c[k];
            }
            uint32_t inc = tot;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t v = __shfl_up_sync(0xffffffffu, inc, o);
                if (tid >= o) inc += v;
            }
            uint32_t above = inc - tot;
            const bool here = (above < need && inc >= need) || (tid == 31 && inc < need);
            __syncwarp();
            if (here) {
                int d = 255 - tid * 8;
#pragma unroll
                for (int k = 0; k < 7; ++k) {
                    if (above + c[k] >= need) break;
                    above += c[k];
                    --d;
                }
                s_need = need - min(above, need - 1u);   // how many to take among the keys that share the longer prefix
                s_prefix = prefix | ((uint32_t)d << shift);
            }
        }
        mask |= ((1u << w) - 1u) << shift;
        top = shift;
        __syncthreads();
    }
    const uint32_t thr = take_none ? 0xFFFFFFFFu : s_prefix;   // keys above thr are taken, equal keys in (head, block) order
    const int need_eq = take_none ? 0 : (int)s_need;
    const int lane = tid & 31, warp = tid >> 5;
    if (Hkv <= kMaxParts) {
        // Ordered compaction without block-wide scans: every head's blocks are cut into parts (a multiple of 32 blocks,
        // one warp each, in (head, block) order); pass A counts per part, one warp turns the counts into start
        // positions, pass B writes.
        const int wph = max(1, kGlobalWarps / Hkv);                         // parts per head
        const int part_len = (((nb + wph - 1) / wph) + 31) & ~31;
        const int n_parts = Hkv * wph;                                      // <= max(kGlobalWarps, kMaxParts)
        for (int part = warp; part < n_parts; part += kGlobalWarps) {
            const int h = part / wph, sub = part - h * wph;
            const int b_end = min(nb, (sub + 1) * part_len);
            int n_gt = 0, n_eq = 0;
            for (int b = sub * part_len + lane; b - lane < b_end; b += 32) {
                const uint32_t k = b < b_end ? keys[h * NBmax + b] : 0u;
                n_gt += __popc(__ballot_sync(0xffffffffu, k == 0xFFFFFFFFu || (k > thr && k != 0u)));
                n_eq += __popc(__ballot_sync(0xffffffffu, k == thr && k != 0xFFFFFFFFu && k != 0u));
            }
            if (lane == 0) part_gt[part] = n_gt, part_eq[part] = n_eq;
        }
        __syncthreads();
        if (warp == 0) {
            // serial over the parts in order (at most kMaxParts + kGlobalWarps of them), 32 at a time
            int eq_before = 0, head_pos = 0, cur_head = 0;
            for (int p0 = 0; p0 < n_parts; p0 += 32) {
                const int part = p0 + lane;
                const int g = part < n_parts ? part_gt[part] : 0, e = part < n_parts ? part_eq[part] : 0;
                int e_inc = e;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int v = __shfl_up_sync(0xffffffffu, e_inc, o);
                    if (lane >= o) e_inc += v;
                }
                const int my_eq_before = eq_before + e_inc - e;               // ties in earlier parts
                const int take = g + max(0, min(e, need_eq - my_eq_before));  // blocks this part keeps
                // start position inside the head: sum of `take` over the earlier parts of the same head
                const int h = part < n_parts ? part / wph : -1;
                int t_inc = take;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int v = __shfl_up_sync(0xffffffffu, t_inc, o);
                    const int hv = __shfl_up_sync(0xffffffffu, h, o);
                    if (lane >= o && hv == h) t_inc += v;   // parts of one head are contiguous: a segmented scan
                }
                int start = t_inc - take + (h == cur_head ? head_pos : 0);
                if (part < n_parts) {
                    part_eq[part] = my_eq_before;
                    part_gt[part] = start;
                    const bool last_of_head = part == n_parts - 1 || (part + 1) / wph != h;
                    if (last_of_head) out_cnt[(size_t)s * Hkv + h] = min(start + take, max_sel);
                }
                // carry into the next 32 parts
                eq_before += __shfl_sync(0xffffffffu, e_inc, 31);
                const int last_h = __shfl_sync(0xffffffffu, h, 31), last_end = __shfl_sync(0xffffffffu, start + take, 31);
                cur_head = last_h, head_pos = last_end;
            }
        }
        __syncthreads();
        for (int part = warp; part < n_parts; part += kGlobalWarps) {
            const int h = part / wph, sub = part - h * wph;
            const int b_end = min(nb, (sub + 1) * part_len);
            int pos = part_gt[part], eq_rank = part_eq[part];
            for (int b = sub * part_len + lane; b - lane < b_end; b += 32) {
                const uint32_t k = b < b_end ? keys[h * NBmax + b] : 0u;
                const bool eq = k == thr && k != 0xFFFFFFFFu && k != 0u;
                const uint32_t eq_ball = __ballot_sync(0xffffffffu, eq);
                const int my_rank = eq_rank + __popc(eq_ball & ((1u << lane) - 1u));
                const bool take = k == 0xFFFFFFFFu || (k > thr && k != 0u) || (eq && my_rank < need_eq);
                const uint32_t take_ball = __ballot_sync(0xffffffffu, take);
                const int my_pos = pos + __popc(take_ball & ((1u << lane) - 1u));
                if (take && my_pos < max_sel) out_idx[((size_t)s * Hkv + h) * max_sel + my_pos] = b;
                pos += __popc(take_ball);
                eq_rank += __popc(eq_ball);
            }
        }
        return;
    }
    // more heads than the part tables hold: block-wide scans, head by head
    int eq_seen = 0;
    for (int h = 0; h < Hkv; ++h) {
        int taken = 0;
        for (int b0 = 0; b0 < nb; b0 += kGlobalThreads) {
            const int b = b0 + tid;
            const uint32_t k = b < nb ? keys[h * NBmax + b] : 0u;
            const bool eq = k == thr && k != 0xFFFFFFFFu && k != 0u;
            int eq_total, take_total;
            const int eq_rank = eq_seen + block_scan_flag(eq, warp_tot, eq_total);
            const bool take = k == 0xFFFFFFFFu || (k > thr && k != 0u) || (eq && eq_rank < need_eq);
            const int pos = taken + block_scan_flag(take, warp_tot, take_total);
            if (take && pos < max_sel) out_idx[((size_t)s * Hkv + h) * max_sel + pos] = b;
            eq_seen += eq_total;
            taken += take_total;
        }
        if (tid == 0) out_cnt[(size_t)s * Hkv + h] = min(taken, max_sel);
    }
}

}  // namespace

extern "C" sv_status sv_select_blocks_tokens(const sv_geom *geom, const void *q, const float *reps,
                                             const int32_t *seq_lens, const int32_t *budget_blocks, int32_t n_sink,
                                             int32_t n_local, int32_t *out_idx, int32_t *out_cnt, int32_t max_sel,
                                             void *stream)
{
    sv_status st = svh::check_geom(geom);
    if (st != SV_OK) return st;
    if (!q || !out_idx || !out_cnt) return SV_ERR_NULL;
    if (max_sel < 1) return SV_ERR_SHAPE;
    const size_t row_elems = (size_t)geom->n_q_heads * geom->head_dim;   // one token row of q, bf16 elements
    const size_t pairs = (size_t)geom->n_seq * geom->n_kv_heads;
    for (int i = 0; i < geom->n_draft; ++i) {
        // the selection kernel retrieves with "row 0" of every sequence: shift the base so that row i is that row
        const void *qi = static_cast<const char *>(q) + (size_t)i * row_elems * 2;
        st = sv_select_blocks(geom, qi, reps, seq_lens, budget_blocks, n_sink, n_local, 0, nullptr, nullptr,
                              out_idx + (size_t)i * pairs * max_sel, out_cnt + (size_t)i * pairs, max_sel, nullptr, stream);
        if (st != SV_OK) return st;
    }
    return SV_OK;
}

extern "C" sv_status sv_token_overlap(const sv_geom *geom, const int32_t *sel_idx_all, const int32_t *sel_cnt_all,
                                      int32_t max_sel, int32_t *inter, void *stream)
{
    sv_status st = svh::check_geom(geom);
    if (st != SV_OK) return st;
    if (!sel_idx_all || !sel_cnt_all || !inter) return SV_ERR_NULL;
    if (max_sel < 1) return SV_ERR_SHAPE;
    const size_t smem = (size_t)geom->n_draft * ((geom->max_blocks + 31) / 32) * 4;
    if (smem > 48 * 1024) return SV_ERR_UNSUPPORTED;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(geom->n_kv_heads, geom->n_seq);
    cfg.blockDim = dim3(kOverlapThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    svh::pdl_attribute(attr);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, token_overlap_kernel, sel_idx_all, sel_cnt_all, inter, (int)geom->n_draft,
                           (int)geom->n_seq, (int)geom->n_kv_heads, (int)geom->max_blocks, (int)max_sel) != cudaSuccess)
        return SV_ERR_CUDA;
    return svh::launch_status();
}

extern "C" sv_status sv_select_blocks_global(const sv_geom *geom, const void *q, const float *reps,
                                             const int32_t *seq_lens, const int32_t *budget_blocks, int32_t n_sink,
                                             int32_t n_local, int32_t *out_idx, int32_t *out_cnt, int32_t max_sel,
                                             float *scores, void *stream)
{
    sv_status st = svh::check_geom(geom);
    if (st != SV_OK) return st;
    if (!scores) return SV_ERR_NULL;
    if (max_sel < geom->max_blocks) return SV_ERR_SHAPE;   // one head may end up with every block of the sequence
    const size_t n_keys = (size_t)geom->n_kv_heads * geom->max_blocks;
    if (n_keys > (size_t)kMaxGlobalKeys) return SV_ERR_UNSUPPORTED;
    // scores of every (head, block): the per-head kernel (its own selection is overwritten below)
    st = sv_select_blocks(geom, q, reps, seq_lens, budget_blocks, n_sink, n_local, 0, nullptr, nullptr, out_idx, out_cnt,
                          max_sel, scores, stream);
    if (st != SV_OK) return st;
    const size_t smem = n_keys * sizeof(uint32_t);
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(select_global_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return SV_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(geom->n_seq);
    cfg.blockDim = dim3(kGlobalThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    svh::pdl_attribute(attr);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, select_global_kernel, (const float *)scores, seq_lens, budget_blocks, out_idx, out_cnt,
                           (int)geom->n_kv_heads, (int)geom->block_size, (int)geom->max_blocks, (int)n_sink, (int)n_local,
                           (int)max_sel) != cudaSuccess)
        return SV_ERR_CUDA;
    return svh::launch_status();
}
