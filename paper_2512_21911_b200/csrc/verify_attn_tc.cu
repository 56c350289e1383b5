// Sparse verification attention on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// Grid (split [x row tile], KV head, sequence); a CTA owns
// a contiguous slice of the ascending block list of its (sequence, KV head) and all G*T query rows of
// that KV head, padded to one M = 64 (up to 64 rows) or M = 128 tile.  Per 64-key unit (32 KB of K and V gathered
// by TMA), with M = 128:
//
//   S[128 x 64]  = Q[128 x 128] . K^T     8 x tcgen05.mma (M128 N64 K16), K from shared memory (K-major, 128-byte
//                                         swizzle), Q from shared memory (same layout) or, for 128-row tiles,
//                                         from tensor memory; accumulator in TMEM
//   softmax      up to 64 query rows: four threads per row (tcgen05.ld 16x256b, the mma.sync accumulator
//                fragment layout, rows spread over all four lane quadrants): mask, running max / sum in
//                fp32 with quad shuffles; 65-128 rows: one thread per row (tcgen05.ld 32x32b), no shuffles.
//                P rounded to bf16 into shared memory (K-major, 128-byte swizzle) or, for a single 128-row
//                tile, into tensor memory (two keys per 32-bit column)
//   O[128x128]  += P[128 x 64] . V        4 x tcgen05.mma (M128 N128 K16), V read MN-major from the
//                                         tile exactly as TMA stored it; O stays in TMEM for the whole
//                                         kernel.  The exponentials use a reference maximum that is only
//                                         moved -- with a rescale of O in TMEM -- when the true maximum
//                                         has grown by more than 2^8 (the final O / l does not depend on
//                                         the reference), so most units never touch O.
//
// Warp roles (384 threads): warps 0-3 and 4-7 are two softmax warpgroups that take units alternately,
// each with its own S / P / O buffers; warp 8 is the TMA producer, one thread of warp 9 issues every
// S = Q K^T (and the warp owns the TMEM allocation), one thread of warp 10 issues every O += P V.  The
// third warpgroup gives its registers to the other two (setmaxnreg).  Everything is chained with mbarriers; tcgen05.commit signals MMA completion.
// At the end warpgroup 0 reads both accumulators from TMEM (warp q of either warpgroup owns lane quadrant q),
// merges them in registers and writes the rows (or the fp32 partial of its split) out.
// All waits are bounded; a wait that gives up sets *status and the CTA drains and frees its TMEM.
#include <cuda.h>
#include <cuda_bf16.h>

#include "attn_common.cuh"
#include "sv_host.h"
#include "sv_ptx.cuh"

namespace svk {
namespace {

constexpr int kThreads = 384;
constexpr int kUnit = 64;                        // keys per unit
constexpr int kTile = kUnit * 128;               // bytes of one [64 rows][64 bf16] half tile (8 KB)
constexpr int kStageBytes = 4 * kTile;           // K lo/hi + V lo/hi
constexpr int kStages = 5;                       // ring stages; a CTA that serves two row tiles has two Q tiles and four stages;
                                                 // 128-row tiles keep P in tensor memory and use its 32 KB as one more stage
constexpr int kMaxStages = kStages + 1;
constexpr int kQBytes = 2 * 128 * 128;           // Q of one row tile: two halves [128 rows][64 bf16]
constexpr int kPBytes = 128 * 128;               // P: [128 rows][64 bf16]
constexpr int kOffP = kStages * kStageBytes + kQBytes;   // (= 4 stages + 2 Q tiles)
constexpr int kOffDraft = 0;                     // the draft unit is the first occupant of ring stage 0 (last split only)
constexpr int kOffMisc = kOffP + 2 * kPBytes;
constexpr int kSmemBytes = 1024 + kOffMisc + 1024;
static_assert(kSmemBytes <= 232448, "shared memory budget");
static_assert(2 * kMaxStages + 10 <= 32, "one lane of the producer warp per barrier");
static_assert((kStages - 1) * kStageBytes + 2 * kQBytes == kOffP, "both layouts put P at the same offset");
constexpr int kTmemCols = 512;                   // S: 2 x 64 columns, O: 2 x 128 columns; 128-row tiles also P: 2 x 32 and
                                                 // Q: 64, or (two row tiles per CTA) Q: 2 x 64
constexpr int kTmemP = 384;                      // first column of P: [warpgroup][32 packed columns]
constexpr int kTmemQ = 448;                      // Q of a single row tile: 128 dims = 64 packed columns (two row tiles: 384, 448)

// barrier slots (8 bytes each) inside the misc area
enum Bar {
    kFull = 0,                  // [kMaxStages] TMA landed
    kEmpty = kFull + kMaxStages,   // [kStages] PV of the unit finished reading the stage
    kSReady = kEmpty + kMaxStages, // [2] S of the warpgroup's unit is in TMEM
    kSFree = kSReady + 2,       // [2] the warpgroup has read S
    kPReady = kSFree + 2,       // [2] P is in shared memory
    kOReady = kPReady + 2,      // [2] the warpgroup's latest PV has been added to O in TMEM
    kStaged = kOReady + 2,      // Q (and the draft unit) are staged
    kTmemDone = kStaged + 1,    // all warps are done with TMEM
    kNumBars = kTmemDone + 1
};

// NH = 8-row groups per TMEM lane quadrant that hold real query rows: 1 (rows <= 32), 2 (<= 64), 4 (<= 128).
// kWide: more than one row tile per (sequence, KV head) or more than 32 draft tokens (64-bit ancestor masks).  The
// common case keeps split = blockIdx.x, plain row arithmetic and 32-bit masks: deriving the split from a division
// costs 3 % on long loops, and the wider mask code 7 % at 128 rows.
// kPair (with kWide, NH = 4): the CTA serves two row tiles of its (sequence, KV head) from one gather: warpgroup w owns
// row tile 2 * pair + w -- its own Q tile, S / P / O buffers -- and takes every unit instead of every other one.  The
// host chooses it where it saves enough waves of CTAs (svh::pair_row_tiles).
template <int NH, bool kWide, bool kPair, bool kUnitSlices>
__global__ void __launch_bounds__(kThreads, 1)
    verify_attn_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                          const AttnParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (smem0 - smem_u32(smem_raw));
    uint8_t *misc = smem + kOffMisc;
    const uint32_t bars = smem0 + kOffMisc;                               // kNumBars x 8 bytes
    int *meta = reinterpret_cast<int *>(misc + 256);                      // [kStages] valid keys per stage
    unsigned long long *anc = reinterpret_cast<unsigned long long *>(misc + 512);   // [64] visible-draft masks (kWide)
    uint32_t *anc32 = reinterpret_cast<uint32_t *>(misc + 320);                     // [32] the same, up to 32 draft tokens
    volatile int *abort_flag = reinterpret_cast<volatile int *>(misc + 448);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(misc + 456);
    auto bar = [&](int slot) { return bars + 8u * slot; };

    static_assert(!kPair || (kWide && NH == 4), "row-tile pairs exist only where one tile is full (more than 64 rows)");
    // 128-row tiles are bound by the tensor pipe when every MMA fetches both operands from shared memory (S = Q K^T: eight
    // 128 x 64 x 16 MMAs, each re-reading 4 KB of Q), so their Q lives in tensor memory (A operand from TMEM), and with a
    // single row tile P does too (one tile per warpgroup), which frees 32 KB for a sixth ring stage.
    constexpr bool kQTmem = NH == 4;
    // Up to 64 query rows run as M = 64 MMAs (half the Q and P bytes of the zero-padded M = 128 tile): matrix row m is
    // TMEM lane (m / 16) * 32 + m % 16, the 16 lanes per quadrant that the NH <= 2 softmax layout uses anyway.
    constexpr int MT = NH == 4 ? 128 : 64;                   // rows of the Q and P tiles and of the MMAs
    constexpr int QR = NH == 4 ? 32 : 16;                    // tile rows per TMEM lane quadrant
    constexpr bool kPTmem = NH == 4 && !kPair;
    constexpr int NS = kPair ? kStages - 1 : kPTmem ? kStages + 1 : kStages;   // ring stages
    constexpr int OFFQ = NS * kStageBytes;                   // the Q tile (kPair: of warpgroup 0; warpgroup 1's follows)
    // blockIdx.x = split * groups + group: the CTAs that gather the same slice of the blocks are neighbours in the grid
    // (they share those K/V tiles through L2; 1-2 % faster than group-major order).  A group is a row tile (kWide), or
    // a pair of row tiles (kPair) of which softmax warpgroup w owns tile 2 * group + w; `tile`, `i0`, `Tq`, `rows` are
    // those of the executing warpgroup (the query rows of draft tokens i0 .. i0 + Tq - 1).
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_groups = kPair ? (p.tiles + 1) / 2 : p.tiles;
    const int split = kWide ? blockIdx.x / n_groups : blockIdx.x, h = blockIdx.y, s = blockIdx.z;
    const int group = kWide ? blockIdx.x - split * n_groups : 0;
    const int tile = kPair ? 2 * group + ((warp >> 2) & 1) : group;
    const int i0 = kWide ? tile * p.Tt : 0, Tq = kWide ? max(0, min(p.Tt, p.T - i0)) : p.T;
    const int upb = p.B / kUnit;
    const bool has_draft = split == p.splits - 1;
    const int rows = p.G * Tq;                               // query rows of this tile (0: the pair's second tile does not exist)
    constexpr int RPQ = 8 * NH;                              // query rows per TMEM lane quadrant
    const int n_active = min(4, (rows + RPQ - 1) / RPQ);     // warps of this softmax warpgroup that own real rows
    // the same for either warpgroup, for the roles that serve both
    const int rows_w1 = kPair ? p.G * max(0, min(p.Tt, p.T - (2 * group + 1) * p.Tt)) : 0;
    const int rows_w0 = kPair ? p.G * min(p.Tt, p.T - 2 * group * p.Tt) : rows;
    const int na0 = min(4, (rows_w0 + RPQ - 1) / RPQ), na1 = kPair ? min(4, (rows_w1 + RPQ - 1) / RPQ) : na0;
    const int n_wg = (kPair && rows_w1 == 0) ? 1 : 2;        // warpgroups that take part

    // r / G for the small row indices of this kernel (0 <= r < 8192, 1 <= G <= 128) without an integer division:
    // (r + 0.5) / G is at least 0.5 / G >= 2^-8 away from the next integer, far more than the fp32 rounding error
    // First block of split k's slice of a list of n blocks.  With 65-128 rows the draft tokens' unit of the last split
    // costs about as much as three ordinary units (masking 64 columns per thread, a first pass through that code), so
    // there the list is cut as if it were that much longer and the last slice comes out shorter.
    // kUnitSlices (128 rows, blocks of 128 tokens): the slices are cut at 64-key units instead, so that two neighbouring
    // splits may share a block (32 blocks over 4 splits: 17 / 17 / 17 / 13 + draft units instead of 16 / 18 / 16 / 14 +
    // draft); slice_begin then returns a unit.  A compile-time variant because the extra index arithmetic costs the
    // other shapes 2-4 %.
    // (Up to 64 rows: 32-bit products -- k <= 148 splits, n <= 32768 blocks -- because a 64-bit division here costs every
    // CTA of a short launch 0.3 us before its first load; the 128-row instantiation measured faster with the 64-bit form.)
    auto slice_begin = [&](int k, int n) {
        if constexpr (kUnitSlices) {
            return min(2 * n, (int)((long long)k * (2 * n + 3) / p.splits));
        } else if constexpr (NH == 4) {
            const int w_draft = (3 + upb - 1) / upb;
            return min(n, (int)((long long)k * (n + w_draft) / p.splits));
        } else {
            return (int)((uint32_t)k * (uint32_t)n / (uint32_t)p.splits);
        }
    };
    // units of split k's slice
    auto slice_units = [&](int k, int n) {
        return kUnitSlices ? slice_begin(k + 1, n) - slice_begin(k, n) : (slice_begin(k + 1, n) - slice_begin(k, n)) * upb;
    };
    const float inv_g = 1.f / (float)p.G;
    auto div_g = [&](int r) { return (int)(((float)r + 0.5f) * inv_g); };
    // The TMA producer warp initialises the barriers and runs ahead; everybody else meets it at a named
    // barrier (the producer only arrives), with the TMEM allocation done by warp 9 on the way.
    if (warp == 8) {
        if (lane < kNumBars) {
            uint32_t count = 1;
            if (lane == kSFree || lane == kPReady) count = na0;
            if (lane == kSFree + 1 || lane == kPReady + 1) count = max(1, na1);
            if (lane == kStaged) count = 8;
            if (lane == kTmemDone) count = na0 + (n_wg == 2 ? na1 : 0);
            mbar_init(bar(lane), count);
            mbar_fence_init();
        }
        if (lane == 0) *abort_flag = 0;
        __syncwarp();
        named_bar_arrive(3, kThreads);
    } else {
        if (warp == 9) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
        tc_fence_before_sync();
        named_bar_sync(3, kThreads);
        tc_fence_after_sync();
    }
    const uint32_t tmem_base = warp == 8 ? 0u : *tmem_slot;

    if (warp >= 8) {
        reg_dealloc<40>();   // hand registers to the softmax warpgroups
        if (warp == 8) {
            // ---------------------------------------------------------- TMA producer
            if (lane == 0) {
                tma_prefetch_desc(&tm_k);
                tma_prefetch_desc(&tm_v);
            }
            const uint64_t policy = policy_evict_first();
            // pull this sequence's block-table row towards L2 while the previous kernel drains
            for (int i = lane * 32; i < p.NBmax; i += 32 * 32) prefetch_l2(p.block_table + (size_t)s * p.NBmax + i);
            // The block list is normally written by the kernel just before.  When the caller vouches that neither the
            // list nor the tables, lengths and pools come from that kernel (a layer that reuses an earlier layer's
            // list), the gather starts at once, while that kernel drains: the tiles are in shared memory by the time
            // the queries, which do come from it, may be read.
            if (!p.early_gather) grid_dependency_wait();
            // First batch of block indices speculatively, assuming the list is full (cnt == max_sel): its
            // load then overlaps the loads of the count and the length instead of following them.
            const int j0_spec = kUnitSlices ? slice_begin(split, p.max_sel) >> 1 : slice_begin(split, p.max_sel);
            int blk_spec = 0;
            if (p.sel_idx && j0_spec + lane < p.max_sel)
                blk_spec = p.sel_idx[((size_t)s * p.Hkv + h) * p.max_sel + j0_spec + lane];
            const int L = p.seq_lens[s];
            const int nb = min(p.B == 128 ? (L + 127) >> 7 : (L + 63) >> 6, p.NBmax);
            const int cnt_in = p.sel_idx ? p.sel_cnt[(size_t)s * p.Hkv + h] : nb;
            // a negative count marks a list that block selection could not produce: attend over the draft tokens
            // only, and say so
            if (cnt_in < 0 && lane == 0 && p.status) atomicOr(p.status, kStatusNoList);
            const int n_sel = p.sel_idx ? max(0, min(cnt_in, p.max_sel)) : nb;
            // blocks j0 .. j1 - 1 of the list; kUnitSlices: units u0 .. u1 - 1 of the list, which those blocks hold
            const int u0 = slice_begin(split, n_sel), u1 = slice_begin(split + 1, n_sel);
            const int j0 = kUnitSlices ? u0 >> 1 : u0, j1 = kUnitSlices ? (u1 + 1) >> 1 : u1;
            const int off = has_draft ? 1 : 0;
            bool dead = false;
            for (int base = j0; base < j1; base += 32) {
                const int j = base + lane;
                int row0 = 0, tok0 = 0;
                if (j < j1) {
                    int blk = j;
                    if (p.sel_idx)
                        blk = (base == j0 && j0 == j0_spec) ? blk_spec : p.sel_idx[((size_t)s * p.Hkv + h) * p.max_sel + j];
                    // indices are clamped into their tables before any address is formed; a clamp that fires is reported
                    const int blk_in = blk;
                    blk = max(0, min(blk, p.NBmax - 1));
                    const int page_in = p.block_table[(size_t)s * p.NBmax + blk];
                    const int page = max(0, min(page_in, p.n_pages - 1));
                    if ((blk != blk_in || page != page_in) && p.status) atomicOr(p.status, kStatusIndex);
                    row0 = (page * p.Hkv + h) * p.B;
                    tok0 = blk * p.B;
                }
                const int n_here = min(32, j1 - base);
                for (int i = 0; i < n_here; ++i) {
                    const int r0 = __shfl_sync(0xffffffffu, row0, i);
                    const int t0 = __shfl_sync(0xffffffffu, tok0, i);
                    if (lane == 0 && !dead) {
                        const int ub = 2 * (base + i);   // (kUnitSlices) first unit of the block
                        for (int uo = kUnitSlices ? max(0, u0 - ub) : 0; uo < (kUnitSlices ? min(2, u1 - ub) : upb); ++uo) {
                            // ring unit; the draft unit (if any) came first
                            const int u = kUnitSlices ? ub + uo - u0 : (base - j0 + i) * upb + uo;
                            const int stage = (u + off) % NS, it = (u + off) / NS;
                            if (it > 0 && (*abort_flag || !mbar_wait_bounded(bar(kEmpty + stage), (it - 1) & 1))) {
                                dead = true;
                                *abort_flag = 1;
                                if (p.status) atomicOr(p.status, 1);
                                break;
                            }
                            const int nvalid = max(0, min(kUnit, L - (t0 + uo * kUnit)));
                            meta[stage] = nvalid;
                            const uint32_t fb = bar(kFull + stage);
                            const uint32_t dst = smem0 + stage * kStageBytes;
                            const int y = r0 + uo * kUnit;
                            // an empty unit (block 128, tail of at most 64 tokens) is still loaded:
                            // it keeps the unit sequence uniform and is fully masked downstream
                            mbar_arrive_expect_tx(fb, kStageBytes);
                            // one copy per operand: the box spans both 64-column halves (third coordinate), which
                            // land as two consecutive [64 rows][128 bytes] swizzled tiles
                            tma_load_3d(dst, &tm_k, 0, y, 0, fb, policy);
                            tma_load_3d(dst + 2 * kTile, &tm_v, 0, y, 0, fb, policy);
                        }
                    }
                }
            }
        } else if (warp == 9 || warp == 10) {
            // ---------------------------------------------------------- MMA issuers (one thread each)
            // warp 9 issues every S = Q K^T and owns the TMEM allocation; warp 10 issues every Ou = P V.
            // Descriptors are built once; per instruction only the 14-bit address field moves.
            if (lane == 0) {
                grid_dependency_wait();   // the lengths may come from the kernel just before (a cache commit)
                const int L = p.seq_lens[s];
                const int nb = min(p.B == 128 ? (L + 127) >> 7 : (L + 63) >> 6, p.NBmax);
                const int n_sel = p.sel_idx ? max(0, min(p.sel_cnt[(size_t)s * p.Hkv + h], p.max_sel)) : nb;
                const int off = has_draft ? 1 : 0;
                const int n_total = slice_units(split, n_sel) + off;
                bool dead = !mbar_wait_bounded(bar(kStaged), 0);
                if (warp == 9) {
                    constexpr uint32_t idesc_s = umma_idesc_bf16(MT, kUnit, false);
                    const uint64_t dq = umma_desc_sw128(smem0 + OFFQ, 16, 1024);
                    const uint64_t dk = umma_desc_sw128(smem0, 16, 1024);
                    const uint32_t dq_lo = (uint32_t)dq, dk_lo = (uint32_t)dk;
                    const uint64_t d_hi = dq & 0xFFFFFFFF00000000ull;
                    // one S per (unit, warpgroup that takes it): the warpgroups alternate units, or (kPair) each takes all
                    const int n_issue = kPair ? n_total * n_wg : n_total;
                    for (int x = 0; x < n_issue && !dead; ++x) {
                        const int u = kPair ? (n_wg == 2 ? x >> 1 : x) : x;
                        const int g = kPair ? (n_wg == 2 ? (x & 1) : 0) : (u & 1), k = kPair ? u : (u >> 1);
                        const int stage = u % NS, it = u / NS;
                        if (*abort_flag || !mbar_wait_bounded(bar(kFull + stage), it & 1) ||
                            (k > 0 && !mbar_wait_bounded(bar(kSFree + g), (k - 1) & 1))) {
                            dead = true;
                            *abort_flag = 1;
                            if (p.status) atomicOr(p.status, 8);
                            break;
                        }
                        tc_fence_after_sync();
                        const uint32_t k_lo = dk_lo + (uint32_t)((stage * kStageBytes) >> 4);
                        const uint32_t d = tmem_base + g * kUnit;
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            const uint32_t qo = (uint32_t)(((kPair ? g * kQBytes : 0) + (ks >> 2) * (kQBytes / 2) + (ks & 3) * 32) >> 4);
                            const uint32_t ko = (uint32_t)(((ks >> 2) * kTile + (ks & 3) * 32) >> 4);
                            if constexpr (kQTmem)   // 16 dims = 8 packed columns of Q per instruction
                                tc_mma_bf16_ta(d, tmem_base + (kPair ? kTmemP + g * 64 : kTmemQ) + ks * 8, d_hi | (k_lo + ko), idesc_s, ks > 0);
                            else
                                tc_mma_bf16(d, d_hi | (dq_lo + qo), d_hi | (k_lo + ko), idesc_s, ks > 0);
                        }
                        tc_commit(bar(kSReady + g));
                    }
                    // free TMEM only after every softmax warp has finished reading it
                    if (!mbar_wait_bounded(bar(kTmemDone), 0) && p.status) atomicOr(p.status, 16);
                } else {
                    constexpr uint32_t idesc_pv = umma_idesc_bf16(MT, 128, true);
                    const uint64_t dp = umma_desc_sw128(smem0 + kOffP, 16, 1024);
                    const uint64_t dv = umma_desc_sw128(smem0 + 2 * kTile, kTile, 1024);
                    const uint32_t dp_lo = (uint32_t)dp, dv_lo = (uint32_t)dv;
                    const uint64_t dp_hi = dp & 0xFFFFFFFF00000000ull, dv_hi = dv & 0xFFFFFFFF00000000ull;
                    const int n_issue = kPair ? n_total * n_wg : n_total;
                    for (int x = 0; x < n_issue && !dead; ++x) {
                        const int u = kPair ? (n_wg == 2 ? x >> 1 : x) : x;
                        const int g = kPair ? (n_wg == 2 ? (x & 1) : 0) : (u & 1), k = kPair ? u : (u >> 1);
                        const int stage = u % NS;
                        if (*abort_flag || !mbar_wait_bounded(bar(kPReady + g), k & 1)) {
                            dead = true;
                            *abort_flag = 1;
                            if (p.status) atomicOr(p.status, 32);
                            break;
                        }
                        tc_fence_after_sync();
                        const uint32_t v_lo = dv_lo + (uint32_t)((stage * kStageBytes) >> 4);
                        const uint32_t p_lo = dp_lo + (uint32_t)((g * kPBytes) >> 4);
                        const uint32_t d = tmem_base + 128 + g * 128;
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) {   // (the warpgroup's first unit starts O)
                            if constexpr (kPTmem)   // A = P from tensor memory: 16 keys = 8 packed columns per instruction
                                tc_mma_bf16_ta(d, tmem_base + kTmemP + g * 32 + kk * 8,
                                               dv_hi | (v_lo + (uint32_t)((kk * 2048) >> 4)), idesc_pv, (k > 0 || kk > 0) ? 1u : 0u);
                            else
                                tc_mma_bf16(d, dp_hi | (p_lo + (uint32_t)((kk * 32) >> 4)), dv_hi | (v_lo + (uint32_t)((kk * 2048) >> 4)),
                                            idesc_pv, (k > 0 || kk > 0) ? 1u : 0u);
                        }
                        tc_commit(bar(kOReady + g));
                        if (!kPair || g == n_wg - 1) tc_commit(bar(kEmpty + stage));   // the last reader of the stage
                    }
                }
            }
            if (warp == 9) {
                __syncwarp();
                tc_fence_after_sync();
                tmem_dealloc(tmem_base, kTmemCols);
            }
        }
        return;
    }

    // ------------------------------------------------------------------ softmax warpgroups
    reg_alloc<232>();
    // Stage Q and, in the last split, the draft tokens' K/V as one more unit; both in the swizzled layout
    // the tensor cores read.  Query row r = i*G + g (q[s][i][h*G + g][:]) goes to tile row
    // (r / RPQ)*32 + r % RPQ: RPQ rows per TMEM lane quadrant, so that all four warps of a warpgroup
    // share the softmax work even when only a few of the 128 tile rows are real.
    // The zero padding needs no input and is written while the previous kernel in the stream drains.
    // kPair: each warpgroup stages the Q tile of its own row tile (128 threads each); otherwise all 256 threads share one
    constexpr int kQThreads = kPair ? 128 : 256;
    const int qtid = kPair ? (tid & 127) : tid;
    uint8_t *q_tile = smem + OFFQ + (kPair ? ((warp >> 2) & 1) * kQBytes : 0);
    for (int idx = qtid; idx < MT * 16; idx += kQThreads) {
        const int tr = idx >> 4, c = idx & 15;
        const int r = (tr / QR) * RPQ + (tr % QR);
        if (!((tr % QR) < RPQ && r < rows))
            *reinterpret_cast<uint4 *>(q_tile + (c >> 3) * (kQBytes / 2) + swz128(tr, c & 7)) = make_uint4(0u, 0u, 0u, 0u);
    }
    if (has_draft) {
        for (int idx = tid; idx < 2 * kUnit * 16; idx += 256) {
            const int which = idx / (kUnit * 16);   // 0: K, 1: V
            const int r = (idx >> 4) % kUnit, c = idx & 15;
            if (r >= p.T)
                *reinterpret_cast<uint4 *>(smem + kOffDraft + which * (2 * kTile) + (c >> 3) * kTile + swz128(r, c & 7)) =
                    make_uint4(0u, 0u, 0u, 0u);
        }
    }
    grid_dependency_wait();
    {
        // real rows: all loads of a thread are in flight together (16-byte chunks: Q up to 128 rows x 16, draft K and
        // V up to 64 tokens x 16 each)
        constexpr int kQB = (NH == 4 ? 8 : 4) * (kPair ? 2 : 1), kDB = kWide ? 8 : 4;
        const int n_q = rows * 16, n_d = has_draft ? 2 * p.T * 16 : 0;
        uint4 v[kQB];
#pragma unroll
        for (int x = 0; x < kQB; ++x) {
            const int idx = qtid + x * kQThreads;
            if (idx < n_q) {
                const int r = idx >> 4, c = idx & 15;
                const int i = div_g(r), g = r - i * p.G;
                v[x] = __ldg(reinterpret_cast<const uint4 *>(p.q + (((size_t)s * p.T + i0 + i) * p.Hq + h * p.G + g) * 128) + c);
            }
        }
        uint4 w[kDB];
#pragma unroll
        for (int x = 0; x < kDB; ++x) {
            const int idx = tid + x * 256;
            if (idx < n_d) {
                const int which = (idx >> 4) >= p.T, r = (idx >> 4) - which * p.T, c = idx & 15;   // K rows, then V rows
                const __nv_bfloat16 *src = (which ? p.draft_v : p.draft_k) + (((size_t)s * p.T + r) * p.Hkv + h) * 128;
                w[x] = __ldg(reinterpret_cast<const uint4 *>(src) + c);
            }
        }
        if (!kWide && has_draft && tid < 32) {
            uint32_t mask = 0;
            if (tid < p.T) {
                if (p.parent) {
                    int a = tid;
                    for (int step = 0; step < p.T && a >= 0; ++step) {
                        mask |= 1u << a;
                        const int nxt = p.parent[(size_t)s * p.T + a];
                        a = nxt < a ? nxt : -1;   // parents must precede their children
                    }
                } else {
                    mask = (tid == 31) ? 0xFFFFFFFFu : ((1u << (tid + 1)) - 1u);
                }
            }
            anc32[tid] = mask;
        }
        if (kWide && has_draft && tid < 64) {
            unsigned long long mask = 0;
            if (tid < p.T) {
                if (p.parent) {
                    int a = tid;
                    for (int step = 0; step < p.T && a >= 0; ++step) {
                        mask |= 1ull << a;
                        const int nxt = p.parent[(size_t)s * p.T + a];
                        a = nxt < a ? nxt : -1;   // parents must precede their children
                    }
                } else {
                    mask = (tid == 63) ? ~0ull : ((1ull << (tid + 1)) - 1ull);
                }
            }
            anc[tid] = mask;
        }
#pragma unroll
        for (int x = 0; x < kQB; ++x) {
            const int idx = qtid + x * kQThreads;
            if (idx < n_q) {
                const int r = idx >> 4, c = idx & 15;
                const int tr = (r / RPQ) * QR + (r % RPQ);
                *reinterpret_cast<uint4 *>(q_tile + (c >> 3) * (kQBytes / 2) + swz128(tr, c & 7)) = v[x];
            }
        }
#pragma unroll
        for (int x = 0; x < kDB; ++x) {
            const int idx = tid + x * 256;
            if (idx < n_d) {
                const int which = (idx >> 4) >= p.T, r = (idx >> 4) - which * p.T, c = idx & 15;
                *reinterpret_cast<uint4 *>(smem + kOffDraft + which * (2 * kTile) + (c >> 3) * kTile + swz128(r, c & 7)) = w[x];
            }
        }
    }
    fence_proxy_async();   // the tensor cores read these tiles through the async proxy
    named_bar_sync(2, 256);
    if constexpr (kQTmem) {
        // Q goes on to tensor memory (thread = tile row = TMEM lane; the 64 32-bit words of the row are the 64 packed
        // columns): every S = Q K^T then reads only the K tile from shared memory, which is what bounds a
        // 128 x 64 x 16 MMA whose two operands both come from there.
        if (kPair || warp < 4) {   // (two row tiles: either warpgroup copies its own)
            const int tr = (warp & 3) * 32 + lane;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t w[32];
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint4 v = *reinterpret_cast<const uint4 *>(q_tile + half * (kQBytes / 2) + swz128(tr, c));
                    w[4 * c] = v.x, w[4 * c + 1] = v.y, w[4 * c + 2] = v.z, w[4 * c + 3] = v.w;
                }
                tmem_st_x32(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (kPair ? kTmemP + (warp >> 2) * 64 : kTmemQ) + half * 32, w);
            }
            tmem_st_wait();
            tc_fence_before_sync();
        }
    }
    if (lane == 0) mbar_arrive(bar(kStaged));
    if (has_draft && tid == 0) mbar_arrive(bar(kFull + 0));   // the draft unit fills stage 0 in place of a TMA load

    const int wg = warp >> 2, quad = warp & 3;
    if (quad >= n_active) return;                                 // this warp's TMEM lanes hold padding only
    const int qd = lane & 3, lr = lane >> 2;
    const uint32_t t_lane = (uint32_t)(quad * 32) << 16;
    const uint32_t t_s = tmem_base + t_lane + wg * kUnit;
    const uint32_t t_o = tmem_base + t_lane + 128 + wg * 128;
    const int wg_threads = n_active * 32;
    // per slot, the draft tokens the row may see: kWide: bit 2j + e <-> this thread's column 8j + 2qd + e; else bit = token
    uint32_t vis[NH];
    int trow[NH], lrow[NH];
    unsigned long long row_vis = ~0ull;   // NH == 4: the draft tokens row quad * 32 + lane may see
    if constexpr (NH == 4) {
        const int r = quad * 32 + lane;
        if (has_draft && r < rows) row_vis = kWide ? anc[i0 + div_g(r)] : (unsigned long long)anc32[div_g(r)];
    }
#pragma unroll
    for (int i = 0; i < NH; ++i) {
        lrow[i] = quad * RPQ + 8 * i + lr;
        trow[i] = quad * QR + 8 * i + lr;
        if constexpr (kWide) {
            const unsigned long long all_t = (p.T == 64) ? ~0ull : ((1ull << p.T) - 1ull);
            const unsigned long long row_vis = (has_draft && lrow[i] < rows) ? anc[i0 + div_g(lrow[i])] : all_t;
            uint32_t mine = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) mine |= (uint32_t)((row_vis >> (8 * j + 2 * qd)) & 3ull) << (2 * j);
            vis[i] = mine;
        } else {
            const uint32_t all_t = (p.T == 32) ? 0xFFFFFFFFu : ((1u << p.T) - 1u);
            vis[i] = (has_draft && lrow[i] < rows) ? anc32[div_g(lrow[i])] : all_t;
        }
    }

    const int L = p.seq_lens[s];
    const int nb = min(p.B == 128 ? (L + 127) >> 7 : (L + 63) >> 6, p.NBmax);
    const int n_sel = p.sel_idx ? max(0, min(p.sel_cnt[(size_t)s * p.Hkv + h], p.max_sel)) : nb;
    const int off = has_draft ? 1 : 0;
    const int n_total = slice_units(split, n_sel) + off;

    // per slot (row): reference maximum of the exponentials (log2 units) and partial row sum
    float m[NH], l[NH];
#pragma unroll
    for (int i = 0; i < NH; ++i) {
        m[i] = -INFINITY;
        l[i] = 0.f;
    }
    bool dead = false;
    constexpr float kLazy = 8.f;   // the reference maximum may trail the true one by up to 2^8

    // wait until the warpgroup's k-th PV has been added to O (warp-uniform outcome)
    auto wait_pv = [&](int k) {
        if (!dead && __any_sync(0xffffffffu, *abort_flag || !mbar_wait_bounded(bar(kOReady + wg), k & 1))) {
            dead = true;
            *abort_flag = 1;
            if (p.status && lane == 0) atomicOr(p.status, 4);
        }
        if (!dead) tc_fence_after_sync();
    };

    int k = 0;
    for (int u = kPair ? 0 : wg; u < n_total; u += kPair ? 1 : 2, ++k) {   // kPair: every unit, for this warpgroup's row tile
        if (!dead && __any_sync(0xffffffffu, *abort_flag || !mbar_wait_bounded(bar(kSReady + wg), k & 1))) {
            dead = true;
            *abort_flag = 1;
            if (p.status && lane == 0) atomicOr(p.status, 2);
        }
        if (dead) break;
        tc_fence_after_sync();
        const bool is_draft = u < off;
        const int stage = u % NS;
        const int nvalid = is_draft ? p.T : min(meta[stage], kUnit);
        uint8_t *pbuf = smem + kOffP + wg * kPBytes;
        if constexpr (NH == 4) {
        // 128 query rows: one thread per row (tcgen05.ld 32x32b), no shuffles, 16-byte P stores; m[0] / l[0] hold
        // the row's state until the loop ends
        uint32_t sr[2][32];
        tmem_ld_x32(t_s, sr[0]);
        tmem_ld_x32(t_s + 32, sr[1]);
        tmem_ld_wait();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kSFree + wg));   // the next S of this warpgroup may be issued
        float sc[64];
#pragma unroll
        for (int c = 0; c < 64; ++c) sc[c] = __uint_as_float(sr[c >> 5][c & 31]);
        if (is_draft || nvalid < kUnit) {
            unsigned long long allowed = nvalid >= 64 ? ~0ull : ((1ull << nvalid) - 1ull);
            if (is_draft) allowed &= row_vis;
            const uint32_t a_lo = (uint32_t)allowed, a_hi = (uint32_t)(allowed >> 32);
#pragma unroll
            for (int c = 0; c < 32; ++c) {
                if (!((a_lo >> c) & 1u)) sc[c] = -INFINITY;
                if (!((a_hi >> c) & 1u)) sc[32 + c] = -INFINITY;
            }
        }
        float mx4[4];
#pragma unroll
        for (int a = 0; a < 4; ++a) mx4[a] = max3f(sc[16 * a], sc[16 * a + 1], sc[16 * a + 2]);
#pragma unroll
        for (int a = 0; a < 4; ++a) {
#pragma unroll
            for (int c = 3; c < 15; c += 2) mx4[a] = max3f(mx4[a], sc[16 * a + c], sc[16 * a + c + 1]);
            mx4[a] = fmaxf(mx4[a], sc[16 * a + 15]);
        }
        const float um = fmaxf(max3f(mx4[0], mx4[1], mx4[2]), mx4[3]) * p.scale_log2;
        float factor = 1.f;
        bool move = false;
        if (um > m[0] + kLazy || (m[0] == -INFINITY && um > -INFINITY)) {
            factor = fast_exp2(m[0] - um);   // 0 when there was no reference
            m[0] = um;
            l[0] *= factor;
            move = true;
        }
        if (k > 0) {
            wait_pv(k - 1);
            if (dead) break;
        }
        if (k > 0 && __any_sync(0xffffffffu, move)) {
            // rare: rescale this thread's row of O in TMEM
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t r[32];
                tmem_ld_x32(t_o + c * 32, r);
                tmem_ld_wait();
#pragma unroll
                for (int x = 0; x < 32; ++x) r[x] = __float_as_uint(__uint_as_float(r[x]) * factor);
                tmem_st_x32(t_o + c * 32, r);
            }
            tmem_st_wait();
            tc_fence_before_sync();
        }
        {
            const float m_use = (m[0] == -INFINITY) ? 0.f : m[0];
            const unsigned long long scale2 = f2_pack(p.scale_log2, p.scale_log2), neg_m2 = f2_pack(-m_use, -m_use);
            unsigned long long lsum2[2] = {f2_pack(0.f, 0.f), f2_pack(0.f, 0.f)};
            if constexpr (kPTmem) {
                uint32_t pk[32];   // this row of P: keys 2c, 2c + 1 are packed column c
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    float x0, x1;
                    f2_unpack(f2_fma(f2_pack(sc[2 * c], sc[2 * c + 1]), scale2, neg_m2), x0, x1);
                    const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                    lsum2[c & 1] = f2_add(lsum2[c & 1], f2_pack(p0, p1));
                    pk[c] = pack_bf16(p0, p1);
                }
                tmem_st_x32(tmem_base + t_lane + kTmemP + wg * 32, pk);
                tmem_st_wait();   // P is in tensor memory
                tc_fence_before_sync();
            } else {
                const uint32_t row = (uint32_t)(quad * 32 + lane);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    uint32_t pk[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float x0, x1;
                        f2_unpack(f2_fma(f2_pack(sc[8 * j + 2 * e], sc[8 * j + 2 * e + 1]), scale2, neg_m2), x0, x1);
                        const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                        lsum2[e & 1] = f2_add(lsum2[e & 1], f2_pack(p0, p1));
                        pk[e] = pack_bf16(p0, p1);
                    }
                    *reinterpret_cast<uint4 *>(pbuf + swz128(row, j)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
            }
            float ls0, ls1;
            f2_unpack(f2_add(lsum2[0], lsum2[1]), ls0, ls1);
            l[0] += ls0 + ls1;
        }
        } else {
        uint32_t sr[1][32];
        tmem_ld_16x256b_x8(t_s, sr[0]);
        tmem_ld_wait();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kSFree + wg));   // the next S of this warpgroup may be issued

        float sc[NH][16], factor[NH];
        bool move = false;
#pragma unroll
        for (int i = 0; i < NH; ++i) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
#pragma unroll
                for (int e = 0; e < 2; ++e) sc[i][2 * j + e] = __uint_as_float(sr[i >> 1][4 * j + 2 * (i & 1) + e]);
            if (is_draft || nvalid < kUnit) {
#pragma unroll
                for (int j = 0; j < 8; ++j)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int col = 8 * j + 2 * qd + e;
                        bool ok = col < nvalid;
                        if constexpr (kWide) {
                            if (is_draft) ok = ok && ((vis[i] >> (2 * j + e)) & 1u);
                        } else {
                            if (is_draft) ok = ok && col < 32 && ((vis[i] >> (col & 31)) & 1u);
                        }
                        if (!ok) sc[i][2 * j + e] = -INFINITY;
                    }
            }
            // 16 columns with 3-input maxima: 8 instructions instead of 15
            const float x0 = max3f(sc[i][0], sc[i][1], sc[i][2]), x1 = max3f(sc[i][3], sc[i][4], sc[i][5]);
            const float x2 = max3f(sc[i][6], sc[i][7], sc[i][8]), x3 = max3f(sc[i][9], sc[i][10], sc[i][11]);
            const float x4 = max3f(sc[i][12], sc[i][13], sc[i][14]);
            float mx = fmaxf(max3f(x0, x1, x2), max3f(x3, x4, sc[i][15]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float um = mx * p.scale_log2;
            // move the reference only when this unit's maximum exceeds it by more than 2^kLazy (or there is none yet)
            factor[i] = 1.f;
            if (um > m[i] + kLazy || (m[i] == -INFINITY && um > -INFINITY)) {
                factor[i] = fast_exp2(m[i] - um);   // 0 when there was no reference
                m[i] = um;
                l[i] *= factor[i];
                move = true;
            }
        }
        // Every completion of the warpgroup's PV barrier is observed, in order (a parity wait cannot tell phase
        // n from phase n - 2); by now the previous PV has normally landed, so this does not stall.
        if (k > 0) {
            wait_pv(k - 1);
            if (dead) break;
        }
        if (k > 0 && __any_sync(0xffffffffu, move)) {
            // rare: rescale this warp's rows of O in TMEM (the previous PV has landed, the next one is not issued
            // before this warp reports P ready)
#pragma unroll
            for (int lo = 0; lo < (NH == 4 ? 2 : 1); ++lo)
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t r[32];
                    const uint32_t addr = t_o + ((uint32_t)(lo * 16) << 16) + c * 64;
                    tmem_ld_16x256b_x8(addr, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int hh = 0; hh < (NH == 1 ? 1 : 2); ++hh)
#pragma unroll
                        for (int j = 0; j < 8; ++j)
#pragma unroll
                            for (int e = 0; e < 2; ++e)
                                r[4 * j + 2 * hh + e] = __float_as_uint(__uint_as_float(r[4 * j + 2 * hh + e]) * factor[lo * 2 + hh]);
                    tmem_st_16x256b_x8(addr, r);
                }
            tmem_st_wait();
            tc_fence_before_sync();
        }
#pragma unroll
        for (int i = 0; i < NH; ++i) {
            const float m_use = (m[i] == -INFINITY) ? 0.f : m[i];
            // two columns per instruction: x = s * scale - m and the running sums as packed fp32 pairs
            const unsigned long long scale2 = f2_pack(p.scale_log2, p.scale_log2), neg_m2 = f2_pack(-m_use, -m_use);
            unsigned long long lsum2 = f2_pack(0.f, 0.f);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                float x0, x1;
                f2_unpack(f2_fma(f2_pack(sc[i][2 * j], sc[i][2 * j + 1]), scale2, neg_m2), x0, x1);
                const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                lsum2 = f2_add(lsum2, f2_pack(p0, p1));
                *reinterpret_cast<uint32_t *>(pbuf + swz128(trow[i], j) + 4 * qd) = pack_bf16(p0, p1);
            }
            float ls0, ls1;
            f2_unpack(lsum2, ls0, ls1);
            l[i] += ls0 + ls1;
        }
        }
        if (!is_draft && nvalid < kUnit) {
            // zero the value rows past the end of the sequence (0 * junk must stay 0)
            const int t = quad * 32 + lane;
            for (int idx = t; idx < (kUnit - nvalid) * 16; idx += wg_threads) {
                const int r = nvalid + (idx >> 4), c = idx & 15;
                *reinterpret_cast<uint4 *>(smem + stage * kStageBytes + 2 * kTile + (c >> 3) * kTile + swz128(r, c & 7)) =
                    make_uint4(0u, 0u, 0u, 0u);
            }
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kPReady + wg));
    }
    if constexpr (NH == 4) {
        // back to the four-threads-per-row slots the read-out uses: slot i of this thread is row 8 i + lane / 4 of the warp
        const float m_row = m[0], l_row = l[0];
#pragma unroll
        for (int i = 0; i < NH; ++i) {
            m[i] = __shfl_sync(0xffffffffu, m_row, 8 * i + lr);
            const float lv = __shfl_sync(0xffffffffu, l_row, 8 * i + lr);
            l[i] = qd == 0 ? lv : 0.f;   // the read-out sums l over the four threads of a row
        }
    }
    // ------------------------------------------------------------------ combine the two warpgroups, write out
    // Warp q of either warpgroup owns TMEM lane quadrant q, so each warpgroup can read the other's accumulator straight
    // from TMEM: both wait for their last PV, exchange (m, l) through their own (now idle) P tiles, and then each merges
    // and writes one half of the 128 output columns of every row.  (kPair: the warpgroups hold different row tiles;
    // each writes both halves of its own rows and nothing is exchanged.)
    const int n_sm = 2 * wg_threads;
    const int t = quad * 32 + lane;
    float *ml_mine = reinterpret_cast<float *>(smem + kOffP + wg * kPBytes);          // [2 * NH][128]: m, l per slot
    float *ml_other = reinterpret_cast<float *>(smem + kOffP + (wg ^ 1) * kPBytes);
    // Only now may the dependent kernel (the split merge) be scheduled: released at the start, its small CTAs would all
    // become resident on the few SMs this grid leaves idle and later do the whole merge from there; released here,
    // they spread over the SMs that the attention CTAs are about to vacate.
    grid_launch_dependents();
    if (k > 0) wait_pv(k - 1);   // this warpgroup's accumulator is complete
    uint32_t ml_theirs[8] = {};   // (kPTmem) the other warpgroup's m, l of this thread's slots
    if constexpr (!kPair && kPTmem) {
        // no P tiles in shared memory: the exchange goes through the warpgroup's own (now idle) S columns, thread for
        // thread (this thread's slots live on TMEM lane quad * 32 + lane in either warpgroup)
        uint32_t ml_ours[8];
#pragma unroll
        for (int i = 0; i < NH; ++i) ml_ours[2 * i] = __float_as_uint(m[i]), ml_ours[2 * i + 1] = __float_as_uint(l[i]);
        tmem_st_x8(tmem_base + t_lane + wg * kUnit, ml_ours);
        tmem_st_wait();
        tc_fence_before_sync();
        named_bar_sync(1, n_sm);
        tc_fence_after_sync();
        tmem_ld_x8(tmem_base + t_lane + (wg ^ 1) * kUnit, ml_theirs);
        tmem_ld_wait();
    } else if constexpr (!kPair) {
#pragma unroll
        for (int i = 0; i < NH; ++i) {
            ml_mine[(2 * i) * 128 + t] = m[i];
            ml_mine[(2 * i + 1) * 128 + t] = l[i];
        }
        tc_fence_before_sync();
        named_bar_sync(1, n_sm);
        tc_fence_after_sync();
    }
    // a warpgroup without units never wrote its accumulator
    const bool have_mine = k > 0 && !dead, have_other = !kPair && n_total >= (wg == 0 ? 2 : 1);
    const uint32_t t_o_other = tmem_base + t_lane + 128 + (wg ^ 1) * 128;
    for (int ch = kPair ? 0 : wg; ch < (kPair ? 2 : wg + 1); ++ch) {   // column half: 64 output dims
        // this warp's rows of O, 16 output dims 64 ch + 8 j + 2 qd + e (index 2 j + e)
        float o[NH][16], row_m[NH], row_l[NH];
#pragma unroll
        for (int lo = 0; lo < (NH == 4 ? 2 : 1); ++lo) {
            uint32_t r0[32], r1[32];
            if (have_mine) tmem_ld_16x256b_x8(t_o + ((uint32_t)(lo * 16) << 16) + ch * 64, r0);
            if (have_other) tmem_ld_16x256b_x8(t_o_other + ((uint32_t)(lo * 16) << 16) + ch * 64, r1);
#pragma unroll
            for (int hh = 0; hh < (NH == 1 ? 1 : 2); ++hh) {
                const int i = lo * 2 + hh;
                const float m1 = kPair ? -INFINITY : kPTmem ? __uint_as_float(ml_theirs[2 * i]) : ml_other[(2 * i) * 128 + t];
                const float l1 = kPair ? 0.f : kPTmem ? __uint_as_float(ml_theirs[2 * i + 1]) : ml_other[(2 * i + 1) * 128 + t];
                const float M = fmaxf(m[i], m1);
                const float M_use = (M == -INFINITY) ? 0.f : M;
                const float w0 = fast_exp2(m[i] - M_use), w1 = fast_exp2(m1 - M_use);
                float lsum = w0 * l[i] + w1 * l1;
                lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
                lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
                row_m[i] = M, row_l[i] = lsum;
                if (hh == 0) tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 8; ++j)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int x = 4 * j + 2 * hh + e;
                        const float a = have_mine ? w0 * __uint_as_float(r0[x]) : 0.f;
                        const float b = have_other ? w1 * __uint_as_float(r1[x]) : 0.f;
                        o[i][2 * j + e] = a + b;
                    }
            }
        }
        if (!kPair || ch == 1) {
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kTmemDone));   // this warp reads TMEM no more
        }
#pragma unroll
        for (int i = 0; i < NH; ++i) {
            const float M = row_m[i], lsum = row_l[i];
            const int row = lrow[i];
            if (row >= rows) continue;
            if (p.splits == 1) {
                const int ii = div_g(row), g = row - ii * p.G;
                const size_t orow = ((size_t)s * p.T + i0 + ii) * p.Hq + h * p.G + g;
                const float inv = 1.f / lsum;
                uint32_t *dst = reinterpret_cast<uint32_t *>(p.out + orow * 128) + ch * 32 + qd;
#pragma unroll
                for (int j = 0; j < 8; ++j) dst[4 * j] = pack_bf16(o[i][2 * j] * inv, o[i][2 * j + 1] * inv);
                if (p.lse && ch == 0 && qd == 0) p.lse[orow] = (M + log2f(lsum)) * 0.69314718055994531f;
            } else {
                const size_t prow = (((size_t)s * p.Hkv + h) * p.splits + split) * (p.G * p.T) + i0 * p.G + row;
                float2 *dst = reinterpret_cast<float2 *>(p.ws_o + prow * 128) + ch * 32 + qd;
#pragma unroll
                for (int j = 0; j < 8; ++j) dst[4 * j] = make_float2(o[i][2 * j], o[i][2 * j + 1]);
                if (ch == 0 && qd == 0) *reinterpret_cast<float2 *>(p.ws_ml + prow * 2) = make_float2(M, lsum);
            }
        }
    }
}

}  // namespace

template <int NH, bool kWide, bool kPair, bool kUnitSlices = false>
static cudaError_t launch_tc(const CUtensorMap &tm_k, const CUtensorMap &tm_v, const AttnParams &p, dim3 grid,
                             cudaStream_t stream)
{
    static svh::OncePerDevice once;   // function attributes belong to a device
    const cudaError_t ce = once.run([] {
        return cudaFuncSetAttribute(verify_attn_tc_kernel<NH, kWide, kPair, kUnitSlices>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    kSmemBytes);
    });
    if (ce != cudaSuccess) return ce;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    svh::pdl_attribute(attr);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, verify_attn_tc_kernel<NH, kWide, kPair, kUnitSlices>, tm_k, tm_v, p);
}

// grid.x = splits x groups, where a group is a row tile or (p.pair) a pair of row tiles
cudaError_t launch_attn_tc(const CUtensorMap &tm_k, const CUtensorMap &tm_v, const AttnParams &p, dim3 grid,
                           cudaStream_t stream)
{
    const int rows = p.G * p.Tt;   // rows of a full row tile
    const bool units = p.B == 128;   // 128-row tiles over blocks of 128 tokens: slices cut at 64-key units
    if (p.pair) {   // (a full tile has more than 64 rows)
        return units ? launch_tc<4, true, true, true>(tm_k, tm_v, p, grid, stream)
                     : launch_tc<4, true, true>(tm_k, tm_v, p, grid, stream);
    }
    if (p.tiles > 1 || p.T > 32) {
        if (rows <= 32) return launch_tc<1, true, false>(tm_k, tm_v, p, grid, stream);
        if (rows <= 64) return launch_tc<2, true, false>(tm_k, tm_v, p, grid, stream);
        return units ? launch_tc<4, true, false, true>(tm_k, tm_v, p, grid, stream)
                     : launch_tc<4, true, false>(tm_k, tm_v, p, grid, stream);
    }
    if (rows <= 32) return launch_tc<1, false, false>(tm_k, tm_v, p, grid, stream);
    if (rows <= 64) return launch_tc<2, false, false>(tm_k, tm_v, p, grid, stream);
    return units ? launch_tc<4, false, false, true>(tm_k, tm_v, p, grid, stream)
                 : launch_tc<4, false, false>(tm_k, tm_v, p, grid, stream);
}

}  // namespace svk
