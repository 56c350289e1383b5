// Exact top-N selection over the order-preserving keys of one (sequence, KV head), run by kThreads threads of
// one CTA on keys that sit in its shared memory (Section 3.1: the N best-scoring blocks, the first / last few
// always kept).  Used by the stand-alone selection kernel (select_blocks.cu) and by the attention kernel
// that selects for itself (verify_attn_tc.cu).  Device code only.
//
// Fast path (up to 8 keys per thread, scores not all equal): the scores are mapped linearly onto 0..65535
// (monotone in the score, so the order is kept; equal codes are possible, equal scores are not split).  One
// histogram pass over the upper 8 bits of the code finds the boundary bin: unlike the raw float bits, the
// codes spread over all 256 bins, so plain shared-memory atomics rarely collide and the boundary bin holds
// only a few keys.  A crowded bin (outliers stretching the range) is thinned by a second pass over the lower
// byte.  The few keys left at the boundary are ranked against one another by their exact keys (ties: smaller
// block index first), which settles the selection exactly.  Everything else -- more keys, equal scores
// everywhere, a still crowded boundary -- takes the general radix select on the key bits (8-bit digits from
// the highest bit in which any two keys differ, warp-aggregated atomics, early stop).
#pragma once
#include <stdint.h>

#include <type_traits>

namespace svsel {

// Histogram bin -> shared-memory slot: one pad word per 32 bins, so that a warp whose lane j reads bins
// 8j .. 8j+7 (the scan below) touches 32 different banks with every load.
constexpr int kHistSlots = 256 + 8;
constexpr int kFastCap = 64;     // at most this many keys left at the boundary after the histogram levels
constexpr uint32_t kForcedKey = 0xFFFFFFFFu;   // key of a block that is kept whatever its score (sink / local)

__device__ __forceinline__ uint32_t hist_slot(uint32_t bin) { return bin + (bin >> 5); }

// Order-preserving map float -> uint32 (larger score, larger key; -0 and +0 coincide) and its inverse.
__device__ __forceinline__ uint32_t order_key(float x)
{
    const uint32_t u = __float_as_uint(x + 0.0f);   // -0 -> +0
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_score(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k ^ 0x80000000u) : ~k);
}

// Shared-memory scratch of one selection (about 4.6 KB).  init() must have run, and a barrier passed, before
// select_top(); a Scratch serves one selection (the kernels select once per CTA).
struct Scratch {
    uint32_t hist[4][kHistSlots];
    unsigned long long cand[kFastCap];   // (key, ~block index) of the keys at the boundary (fast path)
    uint32_t cand_n;
    uint32_t pass_bin[3];                // boundary bin of a pass: index, keys still to take in it, its size
    uint32_t warp_sel[16], warp_eq[16];

    __device__ __forceinline__ void init(int tid, int n_threads)
    {
        for (int i = tid; i < 4 * kHistSlots; i += n_threads) (&hist[0][0])[i] = 0;
        if (tid == 0) cand_n = 0;
    }
};

// Keeps N of the nb blocks (requires forced <= N < nb; the caller handles "keep everything"): every block
// whose key is kForcedKey (there are `forced` of them) and the N - forced largest other keys, equal keys
// smallest index first.  Calls emit(position, block) once per kept block, positions 0..N-1 in ascending block
// order.  Every one of the kThreads threads must call it; `sync` is a barrier over exactly those threads
// that also orders their shared-memory accesses.
template <int kThreads, class Sync, class Emit>
__device__ __forceinline__ void select_top(const uint32_t *keys_all, int nb, int N, int forced, Scratch &sc, int tid,
                                           Sync sync, Emit emit)
{
    static_assert(kThreads % 32 == 0 && kThreads / 32 <= 16, "warp counters");
    constexpr int kWarps = kThreads / 32;
    const int lane = tid & 31, warp = tid >> 5;

    // NC = keys per thread (thread t owns the consecutive blocks NC t .. NC t + NC - 1, so that the ascending
    // compaction is one prefix sum over the threads); returns true when the selection has been emitted
    const auto fast_select = [&](auto nc_tag) -> bool {
        constexpr int NC = decltype(nc_tag)::value;
        uint32_t kk[NC], kmin = 0xFFFFFFFFu, kmax = 0u;
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const int bb = NC * tid + c;
            kk[c] = bb < nb ? keys_all[bb] : kForcedKey;
            if (kk[c] != kForcedKey) kmin = min(kmin, kk[c]), kmax = max(kmax, kk[c]);
        }
        kmin = __reduce_min_sync(0xffffffffu, kmin);
        kmax = __reduce_max_sync(0xffffffffu, kmax);
        if (lane == 0) sc.warp_sel[warp] = kmin, sc.warp_eq[warp] = kmax;
        sync();
#pragma unroll
        for (int w = 0; w < kWarps; ++w) kmin = min(kmin, sc.warp_sel[w]), kmax = max(kmax, sc.warp_eq[w]);
        const float xmin = key_score(kmin), xmax = key_score(kmax);
        const float scale = 65535.f / (xmax - xmin);
        const uint32_t R = (uint32_t)(N - forced);   // evictable blocks to keep: 0 <= R < number of evictable blocks
        if (kmin < kmax && scale > 0.f && scale < 3.0e38f) {   // uniform over the threads
            uint32_t q[NC];   // 16-bit code of the score; 0x10000 = forced or absent
#pragma unroll
            for (int c = 0; c < NC; ++c)
                q[c] = kk[c] == kForcedKey ? 0x10000u : min(65535u, (uint32_t)((key_score(kk[c]) - xmin) * scale));
            // level 0: upper byte of the code over all evictable keys; level 1 (only when the boundary bin of
            // level 0 is too crowded to rank directly): lower byte over the keys of that bin
            uint32_t bound = 0x100u, need = R, in_bin = 0;   // boundary prefix of the code, keys to keep / present at it
            int shift = 8;
            bool settled = R == 0;   // nothing evictable is kept: every code is below the boundary 0x100
            if (settled) sync();     // (the barrier the levels would have passed: warp_sel / warp_eq are reused below)
#pragma unroll 1
            for (int lvl = 0; lvl < 2 && !settled; ++lvl) {
                shift = 8 - 8 * lvl;
#pragma unroll
                for (int c = 0; c < NC; ++c)
                    if (q[c] < 0x10000u && (lvl == 0 || (q[c] >> 8) == bound))
                        atomicAdd(&sc.hist[lvl][hist_slot((q[c] >> shift) & 255u)], 1u);
                sync();   // (also: every thread has read warp_sel / warp_eq, which the compaction reuses)
                if (warp == 0) {   // lane j owns bins 255-8j .. 248-8j (descending)
                    uint32_t c8[8], tot = 0;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        c8[i] = sc.hist[lvl][hist_slot(255 - 8 * lane - i)];
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
                                sc.pass_bin[0] = 255 - 8 * lane - i;
                                sc.pass_bin[1] = need - above;
                                sc.pass_bin[2] = c8[i];
                            }
                            above += c8[i];
                        }
                    }
                }
                sync();
                bound = lvl == 0 ? sc.pass_bin[0] : ((bound << 8) | sc.pass_bin[0]);
                need = sc.pass_bin[1];
                in_bin = sc.pass_bin[2];
                settled = need == in_bin || in_bin <= (uint32_t)kFastCap;
                if (!settled) sync();   // uniform; pass_bin is rewritten by the next level
            }
            if (settled) {   // uniform
                const bool rank_them = need < in_bin;   // otherwise every key at the boundary prefix is kept
                uint32_t my_slot[NC];
                if (rank_them) {
                    // the few keys at the boundary: order them exactly, by key, ties by smaller block index.  Their
                    // owners list them; then kThreads / kFastCap threads per listed key count the larger ones (a slice
                    // of the list each, summed with shuffles) and leave its rank in shared memory.
#pragma unroll
                    for (int c = 0; c < NC; ++c) {
                        my_slot[c] = 0xFFFFFFFFu;
                        if ((q[c] >> shift) == bound) {
                            const uint32_t bb = (uint32_t)(NC * tid + c);
                            my_slot[c] = atomicAdd(&sc.cand_n, 1u);
                            sc.cand[my_slot[c]] = ((unsigned long long)kk[c] << 32) | (0xFFFFFFFFu - bb);
                        }
                    }
                    sync();
                    constexpr int TPC = kThreads / kFastCap;   // threads per listed key (a power of two <= 32)
                    static_assert(TPC >= 1 && TPC <= 32 && (TPC & (TPC - 1)) == 0 && kThreads % kFastCap == 0, "rank layout");
                    const uint32_t ci = (uint32_t)tid / TPC, part = (uint32_t)tid % TPC;
                    const unsigned long long mine = ci < in_bin ? sc.cand[ci] : ~0ull;
                    uint32_t rk = 0;
                    for (uint32_t t = part; t < in_bin; t += TPC) rk += sc.cand[t] > mine ? 1u : 0u;
#pragma unroll
                    for (int o = TPC / 2; o > 0; o >>= 1) rk += __shfl_xor_sync(0xffffffffu, rk, o);
                    if (part == 0) sc.hist[2][ci] = rk;   // (hist[2] serves the radix path only, which is not taken from here)
                    sync();
                }
                uint32_t n_mine = 0, sel_bits = 0;
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    const uint32_t bb = (uint32_t)(NC * tid + c);
                    const uint32_t pc = q[c] >> shift;   // forced / absent: 0x10000 >> shift is above every boundary
                    bool sel = bb < (uint32_t)nb && pc > bound;
                    if (bb < (uint32_t)nb && pc == bound) sel = rank_them ? sc.hist[2][my_slot[c]] < need : true;
                    if (sel) sel_bits |= 1u << c, ++n_mine;
                }
                // ascending compaction: exclusive prefix sum of the per-thread counts (warp scan, then the warps' totals)
                uint32_t incl = n_mine;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += v;
                }
                if (lane == 31) sc.warp_sel[warp] = incl;
                sync();
                uint32_t pos = incl - n_mine;
#pragma unroll
                for (int w = 0; w < kWarps; ++w)
                    if (w < warp) pos += sc.warp_sel[w];
#pragma unroll
                for (int c = 0; c < NC; ++c)
                    if ((sel_bits >> c) & 1u) emit((int)pos++, NC * tid + c);
                return true;
            }
            // fall through: the fast path used hist[0] and hist[1]; clear them for the radix passes
            for (int i = tid; i < 2 * kHistSlots; i += kThreads) (&sc.hist[0][0])[i] = 0;
        }
        sync();   // hist is clean and everybody has read warp_sel / warp_eq, which the radix path reuses
        return false;
    };
    if (nb <= kThreads) {
        if (fast_select(std::integral_constant<int, 1>{})) return;
    } else if (nb <= 2 * kThreads) {
        if (fast_select(std::integral_constant<int, 2>{})) return;
    } else if (nb <= 4 * kThreads) {
        if (fast_select(std::integral_constant<int, 4>{})) return;
    } else if (nb <= 8 * kThreads && 8 * kThreads <= 2048) {
        if (fast_select(std::integral_constant<int, 8>{})) return;
    }

    // Exact radix select of the boundary key among the evictable blocks (the forced ones carry kForcedKey and
    // are kept without taking part).  The keys of one (sequence, KV head) share their leading bits (same sign,
    // neighbouring exponents), so the digits start at the highest bit in which any two keys differ: the first
    // 8-bit pass then spreads the keys over the bins (shared-memory atomics rarely collide) and usually leaves a
    // boundary bin of a few keys, so that the second pass ends the search.  The passes stop as soon as the
    // boundary bin is taken whole.
    uint32_t k_and = 0xFFFFFFFFu, k_or = 0u;
    for (int c0 = 0; c0 < nb; c0 += kThreads) {
        const int bb = c0 + tid;
        const uint32_t k = bb < nb ? keys_all[bb] : kForcedKey;
        if (k != kForcedKey) k_and &= k, k_or |= k;
    }
    k_and = __reduce_and_sync(0xffffffffu, k_and);
    k_or = __reduce_or_sync(0xffffffffu, k_or);
    if (lane == 0) sc.warp_sel[warp] = k_and, sc.warp_eq[warp] = k_or;
    sync();
#pragma unroll
    for (int w = 0; w < kWarps; ++w) k_and &= sc.warp_sel[w], k_or |= sc.warp_eq[w];
    sync();   // warp_sel / warp_eq are reused by the compaction
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
            const uint32_t k = bb < nb ? keys_all[bb] : kForcedKey;
            const bool cand = k != kForcedKey && (k & mask) == prefix;
            // one shared-memory atomic per distinct digit per warp: keys of similar magnitude pile onto few bins
            const uint32_t digit = cand ? ((k >> shift) & dmask) : 256u;
            const uint32_t peers = __match_any_sync(0xffffffffu, digit);
            if (cand && lane == __ffs(peers) - 1) atomicAdd(&sc.hist[pass][hist_slot(digit)], (uint32_t)__popc(peers));
        }
        sync();
        // warp 0 scans the histogram (the other warps would only compete for issue slots) and publishes the
        // boundary bin; lane j owns bins 255-8j .. 248-8j (descending)
        if (warp == 0) {
            uint32_t c[8], tot = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                c[i] = sc.hist[pass][hist_slot(255 - 8 * lane - i)];
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
                        sc.pass_bin[0] = 255 - 8 * lane - i;
                        sc.pass_bin[1] = remaining - above;
                        sc.pass_bin[2] = c[i];
                    }
                    above += c[i];
                }
            }
        }
        sync();
        const uint32_t bin = sc.pass_bin[0], rem_in_bin = sc.pass_bin[1], bin_count = sc.pass_bin[2];
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
        const bool is_forced = bb < nb && key == kForcedKey;
        const uint32_t k = key & mask;
        const bool gt = is_forced || (bb < nb && k > thr);
        const bool eq = bb < nb && !is_forced && k == thr;
        const uint32_t eq_ballot = __ballot_sync(0xffffffffu, eq);
        const uint32_t gt_ballot = __ballot_sync(0xffffffffu, gt);
        if (lane == 0) {
            sc.warp_eq[warp] = __popc(eq_ballot);
            sc.warp_sel[warp] = __popc(gt_ballot);
        }
        sync();
        uint32_t eq_before = base_eq, eq_total = 0, gt_before = 0, gt_total = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const uint32_t e = sc.warp_eq[w], g = sc.warp_sel[w];
            if (w < warp) eq_before += e, gt_before += g;
            eq_total += e, gt_total += g;
        }
        // kept ties are the first take_eq in index order
        const uint32_t lt = (1u << lane) - 1u;
        const uint32_t eq_rank = eq_before + __popc(eq_ballot & lt);
        const bool sel = gt || (eq && eq_rank < take_eq);
        // position = kept entries before this one = greater keys before + kept ties before
        const uint32_t eq_kept_before = min(eq_rank, take_eq) - min(base_eq, take_eq);   // kept ties before, this chunk
        if (sel) emit((int)(base_sel + gt_before + __popc(gt_ballot & lt) + eq_kept_before), bb);
        base_sel += gt_total + min(base_eq + eq_total, take_eq) - min(base_eq, take_eq);
        base_eq += eq_total;
        sync();
    }
}

}  // namespace svsel
