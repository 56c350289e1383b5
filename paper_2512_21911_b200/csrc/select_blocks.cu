// sv_select_blocks: importance scores (Eq. 5) of every block of a (sequence, KV head) against the
// first draft token's query, then the top-N blocks with the first/last few kept (Section 3.1), in one
// launch.  reuse_prev copies the previous layer's set (Section 3.3, Eq. 9).
//
// One thread-block cluster (up to 8 CTAs) per (sequence, KV head).  Each CTA of the cluster scores a
// contiguous slice of the blocks (a GEMV over the representatives: one warp per block row, 128-bit loads,
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

#include <type_traits>

#include "sv_host.h"
#include "sv_ptx.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kRowsPerIter = 4;   // independent representative rows a warp has in flight

// Histogram bin -> shared-memory slot: one pad word per 32 bins, so that a warp whose lane j reads bins
// 8j .. 8j+7 (the scan below) touches 32 different banks with every load.
constexpr int kHistSlots = 256 + 8;
constexpr int kFastCap = 32;     // ... and at most this many keys left at the boundary after the histogram levels
__device__ __forceinline__ uint32_t hist_slot(uint32_t bin) { return bin + (bin >> 5); }

// inverse of order_key (defined below): the score a key was made from
__device__ __forceinline__ float key_score(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k ^ 0x80000000u) : ~k);
}

__device__ __forceinline__ uint32_t order_key(float x)
{
    const uint32_t u = __float_as_uint(x + 0.0f);   // -0 -> +0
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

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

__device__ __forceinline__ uint32_t cluster_map_shared(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// 16-byte store into another CTA's shared memory that reports its bytes to an mbarrier there when it has landed: the
// receiver needs no fence and no separate arrival from the sender
__device__ __forceinline__ void st_async_cluster_v4(uint32_t addr, uint4 v, uint32_t remote_bar)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(addr),
                 "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(remote_bar)
                 : "memory");
}
__device__ __forceinline__ bool mbar_wait_cluster_bounded(uint32_t bar, uint32_t parity, uint32_t limit = (1u << 19))
{
    for (uint32_t i = 0; i < limit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
    }
    return false;
}

// Cluster of CL CTAs per (sequence, KV head).  Every CTA scores a slice of the blocks and writes the
// keys straight into CTA 0's shared memory (distributed shared memory) with stores that count their bytes
// on an mbarrier there, and exits; CTA 0 waits for the expected number of bytes and selects.  The only cluster-wide barrier is split (arrive early, wait late) so that
// its latency hides behind the loads.
// kBf16: the representatives are stored in bfloat16 (storage variant); scores are fp32 either way.
template <bool kBf16>
__global__ void __launch_bounds__(kThreads) select_kernel(const SelectParams p)
{
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int CL = (int)cluster.num_blocks();
    const int h = blockIdx.y, s = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    extern __shared__ __align__(16) uint32_t keys_all[];         // [CL*chunk] keys of all blocks (used in CTA 0)
    __shared__ float qbar[128];
    __shared__ uint32_t hist[4][kHistSlots];
    __shared__ unsigned long long cand[kFastCap];   // (key, ~block index) of the keys at the boundary (fast path)
    __shared__ uint32_t cand_n;
    __shared__ uint32_t pass_bin[3];               // boundary bin of a radix pass: index, keys still to take in it, its size
    __shared__ uint32_t warp_sel[kWarps], warp_eq[kWarps];
    __shared__ uint32_t key_min, key_max;          // smallest / largest evictable key (fast path)
    __shared__ uint64_t keys_ready;                // mbarrier in CTA 0: the bytes of all keys (one arrival: CTA 0 itself)

    // While the kernel that precedes this one in the stream drains: pull this warp's first batch of
    // representative rows and the query row towards L2 (a prefetch consumes no data, so it is safe even if
    // that kernel is still writing them), set up the barrier, zero the histograms.
    if (tid == 0) {
        key_min = 0xFFFFFFFFu, key_max = 0u, cand_n = 0;
        svk::mbar_init(svk::smem_u32(&keys_ready), 1);
        svk::mbar_fence_init();
    }
    for (int i = tid; i < 4 * kHistSlots; i += kThreads) (&hist[0][0])[i] = 0;
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
    for (int i = 0; i < kRowsPerIter; ++i)
        if (b + i < min(b0 + p.chunk, p.NBmax)) svk::prefetch_l2(row_ptr(b + i));
    const int G = p.Hq / p.Hkv;
    const __nv_bfloat16 *q0 = p.q + ((size_t)s * p.T * p.Hq + (size_t)h * G) * 128;
    if (tid < G * 2) svk::prefetch_l2(q0 + tid * 64);
    svk::grid_dependency_wait();
    svk::grid_launch_dependents();

    // every load below is issued before the first use
    const int L = p.seq_lens[s];
    const int budget = p.budget[s];
    float4 r[kRowsPerIter];
    auto load_rows = [&](int bb, int hi) {
#pragma unroll
        for (int i = 0; i < kRowsPerIter; ++i)
            r[i] = (bb + i < hi) ? load_row(bb + i) : make_float4(0.f, 0.f, 0.f, 0.f);
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

    const uint32_t keys0 = cluster_map_shared(svk::smem_u32(keys_all), 0);
    const uint32_t ready0 = cluster_map_shared(svk::smem_u32(&keys_ready), 0);
    if (rank == 0 && tid == 0) {
        // what the cluster is about to send: one 16-byte store per four keys of every CTA's slice; the slices are
        // multiples of four blocks long and only the last one in use can be ragged, so that is ceil(nb / 4) stores
        const uint32_t quads = keep_all ? 0u : (uint32_t)(nb + 3) >> 2;
        svk::mbar_arrive_expect_tx(svk::smem_u32(&keys_ready), 16u * quads);
    }
    if (need_scores) {
        const float4 qv = reinterpret_cast<const float4 *>(qbar)[lane];
        for (; b < b1; b += kWarps * kRowsPerIter) {
            uint32_t kk[kRowsPerIter];
#pragma unroll
            for (int i = 0; i < kRowsPerIter; ++i) {
                float d = r[i].x * qv.x + r[i].y * qv.y + r[i].z * qv.z + r[i].w * qv.w;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
                const int bb = b + i;
                const bool is_forced = bb < p.n_sink || bb >= nb - p.n_local;
                kk[i] = is_forced ? 0xFFFFFFFFu : order_key(d);
                if (p.out_scores && lane == 0 && bb < b1) p.out_scores[((size_t)s * p.Hkv + h) * p.NBmax + bb] = d;
            }
            // rows b .. b+3 are 4 consecutive keys: one 16-byte store into CTA 0 (entries past nb are never read)
            if (lane == 0 && !keep_all) st_async_cluster_v4(keys0 + 4u * (uint32_t)b, make_uint4(kk[0], kk[1], kk[2], kk[3]), ready0);
            if (b + kWarps * kRowsPerIter < b1) load_rows(b + kWarps * kRowsPerIter, b1);
        }
    }
    if (rank != 0) return;

    int32_t *out = p.out_idx + ((size_t)s * p.Hkv + h) * p.max_sel;
    if (keep_all) {
        for (int bb = tid; bb < nb; bb += kThreads) out[bb] = bb;
        if (tid == 0) p.out_cnt[(size_t)s * p.Hkv + h] = nb;
        return;
    }
    if (!mbar_wait_cluster_bounded(svk::smem_u32(&keys_ready), 0)) {
        // gave up: mark the list invalid (sv_verify_attn then attends over the draft tokens only and reports it)
        if (tid == 0) p.out_cnt[(size_t)s * p.Hkv + h] = -1;
        return;
    }

    // ---- fast path (up to 2048 blocks = 4 keys per thread, scores not all equal) -----------------------------------
    // The scores of one (sequence, KV head) are mapped linearly onto 0..65535 (monotone in the score, so the
    // order is kept; equal codes are possible, equal scores are not split).  One histogram pass over the upper
    // 8 bits of the code finds the boundary bin: unlike the raw float bits, the codes spread over all 256 bins,
    // so plain shared-memory atomics rarely collide and the boundary bin holds only a few keys.  Those few are
    // ranked against one another by their exact keys (ties: smaller block index first), which settles the
    // selection exactly.  A boundary bin with more than kFastCap keys (outliers stretching the range) falls
    // through to the general radix select below.
    // NC = keys per thread (1, 2 or 4); returns true when the selection has been written
    const auto fast_select = [&](auto nc_tag) -> bool {
        constexpr int NC = decltype(nc_tag)::value;
        uint32_t kk[NC], kmin = 0xFFFFFFFFu, kmax = 0u;
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const int bb = c * kThreads + tid;
            kk[c] = bb < nb ? keys_all[bb] : 0xFFFFFFFFu;
            if (kk[c] != 0xFFFFFFFFu) kmin = min(kmin, kk[c]), kmax = max(kmax, kk[c]);
        }
        kmin = __reduce_min_sync(0xffffffffu, kmin);
        kmax = __reduce_max_sync(0xffffffffu, kmax);
        if (lane == 0) {
            atomicMin(&key_min, kmin);
            atomicMax(&key_max, kmax);
        }
        __syncthreads();
        kmin = key_min, kmax = key_max;
        const float xmin = key_score(kmin), xmax = key_score(kmax);
        const float scale = 65535.f / (xmax - xmin);
        const uint32_t R = (uint32_t)(N - forced);   // evictable blocks to keep: 0 <= R < number of evictable blocks
        if (kmin < kmax && scale > 0.f && scale < 3.0e38f) {   // block-uniform
            uint32_t q[NC];   // 16-bit code of the score; 0x10000 = forced or absent
#pragma unroll
            for (int c = 0; c < NC; ++c)
                q[c] = kk[c] == 0xFFFFFFFFu ? 0x10000u : min(65535u, (uint32_t)((key_score(kk[c]) - xmin) * scale));
            // level 0: upper byte of the code over all evictable keys; level 1 (only when the boundary bin of
            // level 0 is too crowded to rank directly): lower byte over the keys of that bin
            uint32_t bound = 0x100u, need = R, in_bin = 0;   // boundary prefix of the code, keys to keep / present at it
            int shift = 8;
            bool settled = R == 0;   // nothing evictable is kept: every code is below the boundary 0x100
#pragma unroll 1
            for (int lvl = 0; lvl < 2 && !settled; ++lvl) {
                shift = 8 - 8 * lvl;
#pragma unroll
                for (int c = 0; c < NC; ++c)
                    if (q[c] < 0x10000u && (lvl == 0 || (q[c] >> 8) == bound))
                        atomicAdd(&hist[lvl][hist_slot((q[c] >> shift) & 255u)], 1u);
                __syncthreads();
                if (warp == 0) {   // lane j owns bins 255-8j .. 248-8j (descending)
                    uint32_t c8[8], tot = 0;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        c8[i] = hist[lvl][hist_slot(255 - 8 * lane - i)];
                        tot += c8[i];
                    }
                    uint32_t incl = tot;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= o) incl += v;
                    }
                    uint32_t above = incl - tot;
                    if (above < need && need <= incl) {   // exactly one lane
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            if (above < need && need <= above + c8[i]) {
                                pass_bin[0] = 255 - 8 * lane - i;
                                pass_bin[1] = need - above;
                                pass_bin[2] = c8[i];
                            }
                            above += c8[i];
                        }
                    }
                }
                __syncthreads();
                bound = lvl == 0 ? pass_bin[0] : ((bound << 8) | pass_bin[0]);
                need = pass_bin[1];
                in_bin = pass_bin[2];
                settled = need == in_bin || in_bin <= (uint32_t)kFastCap;
                if (!settled) __syncthreads();   // block-uniform; pass_bin is rewritten by the next level
            }
            if (settled) {   // block-uniform
                const bool rank_them = need < in_bin;   // otherwise every key at the boundary prefix is kept
                if (rank_them) {
                    // the few keys at the boundary: order them exactly, by key, ties by smaller block index
#pragma unroll
                    for (int c = 0; c < NC; ++c)
                        if ((q[c] >> shift) == bound) {
                            const uint32_t bb = (uint32_t)(c * kThreads + tid);
                            cand[atomicAdd(&cand_n, 1u)] = ((unsigned long long)kk[c] << 32) | (0xFFFFFFFFu - bb);
                        }
                    __syncthreads();
                }
                bool sel[NC];
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    const uint32_t bb = (uint32_t)(c * kThreads + tid);
                    const uint32_t pc = q[c] >> shift;   // forced / absent: 0x10000 >> shift is above every boundary
                    sel[c] = bb < (uint32_t)nb && pc > bound;
                    if (bb < (uint32_t)nb && pc == bound) {
                        sel[c] = true;
                        if (rank_them) {
                            const unsigned long long mine = ((unsigned long long)kk[c] << 32) | (0xFFFFFFFFu - bb);
                            uint32_t rk = 0;
#pragma unroll 4
                            for (uint32_t t = 0; t < in_bin; ++t) rk += cand[t] > mine ? 1u : 0u;
                            sel[c] = rk < need;
                        }
                    }
                }
                // ascending compaction
                uint32_t base = 0;
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    if (c * kThreads < nb) {   // block-uniform
                        const uint32_t ballot = __ballot_sync(0xffffffffu, sel[c]);
                        if (lane == 0) warp_sel[warp] = __popc(ballot);
                        __syncthreads();
                        uint32_t before = 0, total = 0;
#pragma unroll
                        for (int w = 0; w < kWarps; ++w) {
                            const uint32_t v = warp_sel[w];
                            if (w < warp) before += v;
                            total += v;
                        }
                        if (sel[c]) out[base + before + __popc(ballot & ((1u << lane) - 1u))] = c * kThreads + tid;
                        base += total;
                        if ((c + 1) * kThreads < nb) __syncthreads();   // block-uniform; warp_sel is rewritten by the next round
                    }
                }
                if (tid == 0) p.out_cnt[(size_t)s * p.Hkv + h] = N;
                return true;
            }
            // fall through: the fast path used hist[0] and hist[1]; clear them for the radix passes
            for (int i = tid; i < 2 * kHistSlots; i += kThreads) (&hist[0][0])[i] = 0;
            __syncthreads();
        }
        return false;
    };
    if (nb <= kThreads) {
        if (fast_select(std::integral_constant<int, 1>{})) return;
    } else if (nb <= 2 * kThreads) {
        if (fast_select(std::integral_constant<int, 2>{})) return;
    } else if (nb <= 4 * kThreads) {
        if (fast_select(std::integral_constant<int, 4>{})) return;
    }

    // Exact radix select of the boundary key among the evictable blocks (the forced ones carry 0xFFFFFFFF and
    // are kept without taking part).  The keys of one (sequence, KV head) share their leading bits (same sign,
    // neighbouring exponents), so the digits start at the highest bit in which any two keys differ: the first
    // 8-bit pass then spreads the keys over the bins (shared-memory atomics rarely collide) and usually leaves a
    // boundary bin of a few keys, so that the second pass ends the search.  Every warp scans the histogram itself
    // (one block barrier per pass); the passes stop as soon as the boundary bin is taken whole.
    uint32_t k_and = 0xFFFFFFFFu, k_or = 0u;
    for (int c0 = 0; c0 < nb; c0 += kThreads) {
        const int bb = c0 + tid;
        const uint32_t k = bb < nb ? keys_all[bb] : 0xFFFFFFFFu;
        if (k != 0xFFFFFFFFu) k_and &= k, k_or |= k;
    }
    k_and = __reduce_and_sync(0xffffffffu, k_and);
    k_or = __reduce_or_sync(0xffffffffu, k_or);
    if (lane == 0) warp_sel[warp] = k_and, warp_eq[warp] = k_or;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kWarps; ++w) k_and &= warp_sel[w], k_or |= warp_eq[w];
    __syncthreads();   // warp_sel / warp_eq are reused by the compaction
    const uint32_t diff = k_and ^ k_or;
    uint32_t remaining = (uint32_t)(N - forced);        // evictable blocks to keep (N < nb here, so fewer than there are)
    int lo = diff ? 32 - __clz(diff) : 0;               // undecided low bits
    uint32_t mask = lo == 32 ? 0u : ~((1u << lo) - 1u); // bits decided so far: the common leading bits
    uint32_t prefix = k_and & mask;
#pragma unroll 1
    for (int pass = 0; pass < 4 && lo > 0 && remaining > 0; ++pass) {
        const int width = min(8, lo), shift = lo - width;
        const uint32_t dmask = (1u << width) - 1u;
        for (int c0 = 0; c0 < nb; c0 += kThreads) {
            const int bb = c0 + tid;
            const uint32_t k = bb < nb ? keys_all[bb] : 0xFFFFFFFFu;
            const bool cand = k != 0xFFFFFFFFu && (k & mask) == prefix;
            // one shared-memory atomic per distinct digit per warp: keys of similar magnitude pile onto few bins
            const uint32_t digit = cand ? ((k >> shift) & dmask) : 256u;
            const uint32_t peers = __match_any_sync(0xffffffffu, digit);
            if (cand && lane == __ffs(peers) - 1) atomicAdd(&hist[pass][hist_slot(digit)], (uint32_t)__popc(peers));
        }
        __syncthreads();
        // warp 0 scans the histogram (the other warps would only compete for issue slots) and publishes the
        // boundary bin; lane j owns bins 255-8j .. 248-8j (descending)
        if (warp == 0) {
            uint32_t c[8], tot = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                c[i] = hist[pass][hist_slot(255 - 8 * lane - i)];
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
                        pass_bin[0] = 255 - 8 * lane - i;
                        pass_bin[1] = remaining - above;
                        pass_bin[2] = c[i];
                    }
                    above += c[i];
                }
            }
        }
        __syncthreads();
        const uint32_t bin = pass_bin[0], rem_in_bin = pass_bin[1], bin_count = pass_bin[2];
        // (pass_bin is rewritten only after the next pass's barrier)
        prefix |= bin << shift;
        mask |= dmask << shift;
        remaining = rem_in_bin;
        lo = shift;
        if (remaining == bin_count) break;   // the whole boundary bin is kept: lower bits cannot matter
    }
    // evictable keys whose decided bits exceed the prefix are kept; of those equal to it, the first `remaining`
    // in index order (all of them after an early stop, none when only the forced blocks fit the budget)
    const uint32_t thr = prefix;
    const uint32_t take_eq = remaining;

    // ascending compaction
    uint32_t base_sel = 0, base_eq = 0;
    for (int c0 = 0; c0 < nb; c0 += kThreads) {
        const int bb = c0 + tid;
        const uint32_t key = bb < nb ? keys_all[bb] : 0u;
        const bool is_forced = bb < nb && key == 0xFFFFFFFFu;
        const uint32_t k = key & mask;
        const bool gt = is_forced || (bb < nb && k > thr);
        const bool eq = bb < nb && !is_forced && k == thr;
        const uint32_t eq_ballot = __ballot_sync(0xffffffffu, eq);
        const uint32_t gt_ballot = __ballot_sync(0xffffffffu, gt);
        if (lane == 0) {
            warp_eq[warp] = __popc(eq_ballot);
            warp_sel[warp] = __popc(gt_ballot);
        }
        __syncthreads();
        uint32_t eq_before = base_eq, eq_total = 0, gt_before = 0, gt_total = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const uint32_t e = warp_eq[w], g = warp_sel[w];
            if (w < warp) eq_before += e, gt_before += g;
            eq_total += e, gt_total += g;
        }
        // kept ties are the first take_eq in index order
        const uint32_t lt = (1u << lane) - 1u;
        const uint32_t eq_rank = eq_before + __popc(eq_ballot & lt);
        const bool sel = gt || (eq && eq_rank < take_eq);
        // position = kept entries before this one = greater keys before + kept ties before
        const uint32_t eq_kept_before = min(eq_rank, take_eq) - min(base_eq, take_eq);   // kept ties before, this chunk
        if (sel) out[base_sel + gt_before + __popc(gt_ballot & lt) + eq_kept_before] = bb;
        base_sel += gt_total + min(base_eq + eq_total, take_eq) - min(base_eq, take_eq);
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

    // CTAs per (sequence, KV head): at least 32 blocks each, and no more CTAs than two per SM can hold at once
    // (512 threads x 60 registers: two CTAs per SM) -- a second wave costs more than the shorter slices save
    const int pairs = geom->n_seq * geom->n_kv_heads;
    int CL = 1;
    while (CL < 8 && geom->max_blocks / (CL * 2) >= 32 && pairs * CL * 2 <= 2 * svh::sm_count()) CL *= 2;
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

    const size_t smem = (size_t)CL * chunk * sizeof(uint32_t);
    if (smem > 48 * 1024 &&
        (reps_bf16 ? cudaFuncSetAttribute(select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                   : cudaFuncSetAttribute(select_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) !=
            cudaSuccess)
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
    if ((reps_bf16 ? cudaLaunchKernelEx(&cfg, select_kernel<true>, p) : cudaLaunchKernelEx(&cfg, select_kernel<false>, p)) !=
        cudaSuccess)
        return SV_ERR_CUDA;
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
