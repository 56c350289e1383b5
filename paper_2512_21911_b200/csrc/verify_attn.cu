// sv_verify_attn: attention of all draft tokens of a sequence over the kept KV blocks plus the draft
// tokens' own K/V (Fig. 1), split-KV with a log-sum-exp merge.
//
// Grid (split, KV head, sequence).  A CTA owns a contiguous slice of the ascending block list of its
// (sequence, KV head) and the G*T query rows of that KV head (GQA group x draft tokens packed as the
// M dimension of the tensor-core tiles).  One producer warp walks the block list and gathers 64-token
// K and V tiles from the paged pools with TMA (2-D tiled loads, 128-byte swizzle, completion on
// mbarriers, L2 evict-first) into a ring of 32 KB stages (it belongs to a warpgroup that gives its
// registers to the others with setmaxnreg); eight consumer warps take stages in turn
// (warp groups of WM warps, each warp MT 16-row tiles), compute S = QK^T and O += PV with bf16
// mma.sync, fp32 online softmax, and are merged across warp groups in shared memory at the end.  With
// one split the CTA writes bf16 output directly; otherwise fp32 partials (m, l, o) go to the workspace
// and a small merge kernel combines them.  The kernel is bound by HBM bandwidth (512 bytes of K/V per
// cached token and KV head); tensor cores only keep the arithmetic (4*rows*128 flop per token) off
// the critical path.
//
// The partially filled last block is loaded whole (the page exists) and masked: its key columns
// beyond the sequence length get -inf and its value rows are zeroed in shared memory.  The draft
// tokens' K/V (at most 32 rows) are staged by the CTA of the last split with ordinary loads and
// masked with per-row ancestor bit masks (tree) or j <= i (chain).
//
// All waits are bounded: a wait that gives up sets *status_word and the CTA drains without hanging.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdlib>
#include <mutex>

#include "attn_common.cuh"
#include "sv_host.h"
#include "sv_ptx.cuh"

#ifdef SV_TRACE
// Development aid (never compiled into the library): per-CTA cycle stamps of the attention kernel.
__device__ long long g_sv_trace[256 * 16];
extern "C" __attribute__((visibility("default"))) long long *sv_trace_buffer()
{
    long long *p = nullptr;
    cudaGetSymbolAddress(reinterpret_cast<void **>(&p), g_sv_trace);
    return p;
}
#define SV_STAMP(slot)                                                                      \
    do {                                                                                    \
        const int cta_ = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);    \
        if (cta_ < 256) g_sv_trace[cta_ * 16 + (slot)] = clock64();                         \
    } while (0)
#else
#define SV_STAMP(slot) \
    do {               \
    } while (0)
#endif

namespace {

using namespace svk;

constexpr int kMathWarps = 8;                      // warps 0..7: two warpgroups that get the registers
constexpr int kMathThreads = kMathWarps * 32;
constexpr int kThreads = kMathThreads + 128;       // + one producer warpgroup (one warp of it works)
constexpr int kUnit = 64;                          // keys per pipeline stage
constexpr int kStageBytes = 4 * kUnit * 128;       // K lo/hi + V lo/hi halves, 8 KB each
constexpr int kDraftRows = 32;
constexpr int kDraftBytes = 4 * kDraftRows * 128;
constexpr int kSmemLimit = 232448;                 // 227 KB per CTA
constexpr int kMiscBytes = 1024;


// Warp layout: WM x KS consumer warps.  Warp (wm, ks) owns MT 16-row tiles of the query rows and the
// keys [ks*64/KS, (ks+1)*64/KS) of every 64-key stage, so all warps work on a stage as soon as it lands
// and every warp consumes every stage in order.
template <int WM, int MT, int KS>
struct Cfg {
    static constexpr int kRowsPad = WM * MT * 16;
    static constexpr int kKeysPerWarp = kUnit / KS;
    static constexpr int kConsumerWarps = WM * KS;
    static constexpr int kConsumerThreads = kConsumerWarps * 32;
    static constexpr int kQBytes = kRowsPad * 256;
    static constexpr int kMaxStages = (kSmemLimit - 1024 - kQBytes - kDraftBytes - kMiscBytes) / kStageBytes;
    static constexpr int kStages = kMaxStages > 6 ? 6 : kMaxStages;
    static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kQBytes + kDraftBytes + kMiscBytes;
    static_assert(kConsumerWarps <= kMathWarps, "too many consumer warps");
    static_assert(kStages >= 3, "pipeline too shallow");
    static_assert(kKeysPerWarp == 16 || kKeysPerWarp == 32, "a warp takes 16 or 32 keys of a stage");
    // the cross-warp merge at the end reuses the ring and, behind it, the Q tile
    static_assert(KS * kRowsPad * (128 + 2) * 4 <= kStages * kStageBytes + kQBytes, "merge area does not fit");
};

// NK keys (16 or 32) starting at key0 of a tile: S = Q K^T, masked online softmax, O += P V.
// HALF = bytes between the dim 0-63 and dim 64-127 halves of the tile (rows * 128).
template <int MT, int NK, uint32_t HALF, bool DRAFT>
__device__ __forceinline__ void process_keys(uint32_t kbase, uint32_t vbase, uint32_t qbase, uint32_t q_half_stride,
                                             int row_base, const uint32_t (&qf)[8][4], float (&o)[MT][16][4],
                                             float (&m)[MT][2], float (&l)[MT][2], float scale_log2, int key0,
                                             int nvalid, const uint32_t (&vis)[MT][2], int lane)
{
    float sacc[MT][NK / 8][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NK / 8; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) sacc[mt][nt][e] = 0.f;

#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        uint32_t qa[MT][4];
        if constexpr (MT == 1) {
#pragma unroll
            for (int e = 0; e < 4; ++e) qa[0][e] = qf[ks][e];
        } else {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                const uint32_t row = row_base + mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                const uint32_t chunk = ks * 2 + (lane >> 4);
                ldsm_x4(qa[mt], qbase + (chunk >> 3) * q_half_stride + swz128(row, chunk & 7));
            }
        }
#pragma unroll
        for (int np = 0; np < NK / 16; ++np) {
            const uint32_t key = key0 + np * 16 + (lane >> 4) * 8 + (lane & 7);
            const uint32_t chunk = ks * 2 + ((lane >> 3) & 1);
            uint32_t kb[4];
            ldsm_x4(kb, kbase + (chunk >> 3) * HALF + swz128(key, chunk & 7));
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                mma_bf16_16816(sacc[mt][2 * np], qa[mt], kb[0], kb[1]);
                mma_bf16_16816(sacc[mt][2 * np + 1], qa[mt], kb[2], kb[3]);
            }
        }
    }

    if (DRAFT || nvalid < key0 + NK) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < NK / 8; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int col = key0 + nt * 8 + 2 * (lane & 3) + (e & 1);
                    bool ok = col < nvalid;
                    if (DRAFT) ok = ok && ((vis[mt][e >> 1] >> col) & 1u);
                    if (!ok) sacc[mt][nt][e] = -INFINITY;
                }
    }

    uint32_t pa[MT][NK / 16][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            float mx = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < NK / 8; ++nt) mx = fmaxf(mx, fmaxf(sacc[mt][nt][2 * r], sacc[mt][nt][2 * r + 1]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m[mt][r], mx * scale_log2);
            const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
            const float corr = fast_exp2(m[mt][r] - m_use);
            m[mt][r] = m_new;
            float lsum = 0.f;
#pragma unroll
            for (int nt = 0; nt < NK / 8; ++nt) {
                const float p0 = fast_exp2(fmaf(sacc[mt][nt][2 * r], scale_log2, -m_use));
                const float p1 = fast_exp2(fmaf(sacc[mt][nt][2 * r + 1], scale_log2, -m_use));
                sacc[mt][nt][2 * r] = p0;
                sacc[mt][nt][2 * r + 1] = p1;
                lsum += p0 + p1;
            }
            l[mt][r] = l[mt][r] * corr + lsum;
            if (corr != 1.f) {   // the running maximum moved: rescale the accumulator rows of this thread
#pragma unroll
                for (int nt = 0; nt < 16; ++nt) {
                    o[mt][nt][2 * r] *= corr;
                    o[mt][nt][2 * r + 1] *= corr;
                }
            }
        }
#pragma unroll
        for (int kk = 0; kk < NK / 16; ++kk) {
            pa[mt][kk][0] = pack_bf16(sacc[mt][2 * kk][0], sacc[mt][2 * kk][1]);
            pa[mt][kk][1] = pack_bf16(sacc[mt][2 * kk][2], sacc[mt][2 * kk][3]);
            pa[mt][kk][2] = pack_bf16(sacc[mt][2 * kk + 1][0], sacc[mt][2 * kk + 1][1]);
            pa[mt][kk][3] = pack_bf16(sacc[mt][2 * kk + 1][2], sacc[mt][2 * kk + 1][3]);
        }
    }

#pragma unroll
    for (int kk = 0; kk < NK / 16; ++kk) {
        const uint32_t key = key0 + kk * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
        for (int dp = 0; dp < 8; ++dp) {
            const uint32_t chunk = dp * 2 + (lane >> 4);
            uint32_t vb[4];
            ldsm_x4_trans(vb, vbase + (chunk >> 3) * HALF + swz128(key, chunk & 7));
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                mma_bf16_16816(o[mt][2 * dp], pa[mt][kk], vb[0], vb[1]);
                mma_bf16_16816(o[mt][2 * dp + 1], pa[mt][kk], vb[2], vb[3]);
            }
        }
    }
}

template <int WM, int MT, int KS>
__global__ void __launch_bounds__(kThreads, 1)
    verify_attn_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                       const AttnParams p)
{
    using C = Cfg<WM, MT, KS>;
    constexpr int ROWS_PAD = C::kRowsPad, STAGES = C::kStages, KW = C::kKeysPerWarp;
    constexpr int kConsumerWarps = C::kConsumerWarps, kConsumerThreads = C::kConsumerThreads;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (smem0 - smem_u32(smem_raw));
    const uint32_t stage_base = smem0;
    const uint32_t q_base = stage_base + STAGES * kStageBytes;
    const uint32_t draft_base = q_base + C::kQBytes;
    uint8_t *misc = smem + STAGES * kStageBytes + C::kQBytes + kDraftBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(misc);                 // full[STAGES], empty[STAGES]
    int *meta = reinterpret_cast<int *>(misc + 256);                     // valid keys of the unit in each stage
    uint32_t *anc = reinterpret_cast<uint32_t *>(misc + 256 + 64);       // [32] visible-draft masks
    volatile int *abort_flag = reinterpret_cast<volatile int *>(misc + 256 + 64 + 128);
    const uint32_t full_bar = smem_u32(bars), empty_bar = smem_u32(bars + STAGES);

    const int split = blockIdx.x, h = blockIdx.y, s = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int upb = p.B / kUnit;
    const bool has_draft = split == p.splits - 1;
    const int rows = p.G * p.T;

    if (tid == 0) {
        SV_STAMP(0);
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(full_bar + 8 * i, 1);
            mbar_init(empty_bar + 8 * i, kConsumerWarps);
        }
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    if (tid == 0) SV_STAMP(1);

    if (warp >= kMathWarps) {
        // -------------------------------------------------------------- producer warpgroup
        reg_dealloc<40>();   // hand registers to the math warpgroups
        if (warp != kMathWarps) return;
        if (lane == 0) {
            tma_prefetch_desc(&tm_k);
            tma_prefetch_desc(&tm_v);
        }
        // The block list is written by the kernel that precedes this one in the stream.
        grid_dependency_wait();
        if (lane == 0) SV_STAMP(2);
        const int L = p.seq_lens[s];
        const int nb = min((L + p.B - 1) / p.B, p.NBmax);
        const int n_sel = p.sel_idx ? max(0, min(p.sel_cnt[(size_t)s * p.Hkv + h], p.max_sel)) : nb;
        const int j0 = (int)((long long)split * n_sel / p.splits);
        const int j1 = (int)((long long)(split + 1) * n_sel / p.splits);
        const uint64_t policy = policy_evict_first();
        bool dead = false;
        for (int base = j0; base < j1; base += 32) {
            const int j = base + lane;
            int row0 = 0, tok0 = 0;
            if (j < j1) {
                int blk = p.sel_idx ? p.sel_idx[((size_t)s * p.Hkv + h) * p.max_sel + j] : j;
                blk = max(0, min(blk, p.NBmax - 1));
                const int page = p.block_table[(size_t)s * p.NBmax + blk];
                row0 = (page * p.Hkv + h) * p.B;
                tok0 = blk * p.B;
            }
            const int n_here = min(32, j1 - base);
            for (int i = 0; i < n_here; ++i) {
                const int r0 = __shfl_sync(0xffffffffu, row0, i);
                const int t0 = __shfl_sync(0xffffffffu, tok0, i);
                if (lane == 0 && i == 0 && base == j0) SV_STAMP(3);
                if (lane == 0 && !dead) {
                    for (int uo = 0; uo < upb; ++uo) {
                        const int u = (base - j0 + i) * upb + uo;
                        const int stage = u % STAGES, it = u / STAGES;
                        if (it > 0 && !mbar_wait_bounded(empty_bar + 8 * stage, (it - 1) & 1)) {
                            dead = true;
                            *abort_flag = 1;
                            if (p.status) atomicOr(p.status, 1);
                            break;
                        }
                        const int nvalid = max(0, min(kUnit, L - (t0 + uo * kUnit)));
                        meta[stage] = nvalid;
                        const uint32_t fb = full_bar + 8 * stage;
                        if (nvalid > 0) {
                            const uint32_t dst = stage_base + stage * kStageBytes;
                            const int y = r0 + uo * kUnit;
                            mbar_arrive_expect_tx(fb, kStageBytes);
                            tma_load_2d(dst, &tm_k, 0, y, fb, policy);
                            tma_load_2d(dst + 8192, &tm_k, 64, y, fb, policy);
                            tma_load_2d(dst + 16384, &tm_v, 0, y, fb, policy);
                            tma_load_2d(dst + 24576, &tm_v, 64, y, fb, policy);
                            if (u == 0) SV_STAMP(4);
                        } else {
                            mbar_arrive(fb);
                        }
                    }
                }
            }
        }
        return;
    }

    // ------------------------------------------------------------------ math warpgroups
    reg_alloc<232>();
    grid_dependency_wait();
    grid_launch_dependents();   // the next kernel may be scheduled; it waits for this grid before reading
    // Stage Q (and, in the last split, the draft tokens' K/V) while the producer chases the block list.
    // Q rows r = i*G + g  ->  q[s][i][h*G + g][:], zero padded to ROWS_PAD, stored swizzled
    for (int idx = tid; idx < ROWS_PAD * 16; idx += kMathThreads) {
        const int r = idx >> 4, c = idx & 15;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (r < rows) {
            const int i = r / p.G, g = r - i * p.G;
            v = __ldg(reinterpret_cast<const uint4 *>(p.q + (((size_t)s * p.T + i) * p.Hq + h * p.G + g) * 128) + c);
        }
        *reinterpret_cast<uint4 *>(smem + (q_base - smem0) + (c >> 3) * (ROWS_PAD * 128) + swz128(r, c & 7)) = v;
    }
    if (has_draft) {
        for (int idx = tid; idx < 2 * kDraftRows * 16; idx += kMathThreads) {
            const int which = idx / (kDraftRows * 16);   // 0: K, 1: V
            const int r = (idx >> 4) % kDraftRows, c = idx & 15;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (r < p.T) {
                const __nv_bfloat16 *src = (which ? p.draft_v : p.draft_k) + (((size_t)s * p.T + r) * p.Hkv + h) * 128;
                v = __ldg(reinterpret_cast<const uint4 *>(src) + c);
            }
            *reinterpret_cast<uint4 *>(smem + (draft_base - smem0) + which * (2 * kDraftRows * 128) +
                                       (c >> 3) * (kDraftRows * 128) + swz128(r, c & 7)) = v;
        }
        if (tid < kDraftRows) {
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
            anc[tid] = mask;
        }
    }
    named_bar_sync(2, kMathThreads);
    if (tid == 0) SV_STAMP(5);
    if (warp >= kConsumerWarps) return;   // math warps this shape does not use

    const int wm = warp % WM, kq = warp / WM;
    const int row_base = wm * MT * 16;
    const int key0 = kq * KW;
    uint32_t qf[8][4];
    if constexpr (MT == 1) {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const uint32_t row = row_base + (lane & 7) + ((lane >> 3) & 1) * 8;
            const uint32_t chunk = ks * 2 + (lane >> 4);
            ldsm_x4(qf[ks], q_base + (chunk >> 3) * (ROWS_PAD * 128) + swz128(row, chunk & 7));
        }
    }
    float o[MT][16][4], m[MT][2], l[MT][2];
    uint32_t vis[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
        for (int nt = 0; nt < 16; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) o[mt][nt][e] = 0.f;
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            m[mt][r] = -INFINITY;
            l[mt][r] = 0.f;
            vis[mt][r] = 0xFFFFFFFFu;
        }
    }

    // the draft tokens first: their tile is already in shared memory (warps kq == 0 take all 32 keys)
    if (has_draft && kq == 0) {
        const uint32_t all = (p.T == 32) ? 0xFFFFFFFFu : ((1u << p.T) - 1u);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const int row = row_base + mt * 16 + (lane >> 2) + 8 * r;
                vis[mt][r] = row < rows ? anc[row / p.G] : all;
            }
        process_keys<MT, kDraftRows, kDraftRows * 128, true>(draft_base, draft_base + 2 * kDraftRows * 128, q_base,
                                                             ROWS_PAD * 128, row_base, qf, o, m, l, p.scale_log2, 0,
                                                             p.T, vis, lane);
    }

    if (tid == 0) SV_STAMP(6);
    const int L = p.seq_lens[s];
    const int nb = min((L + p.B - 1) / p.B, p.NBmax);
    const int n_sel = p.sel_idx ? max(0, min(p.sel_cnt[(size_t)s * p.Hkv + h], p.max_sel)) : nb;
    const int j0 = (int)((long long)split * n_sel / p.splits);
    const int j1 = (int)((long long)(split + 1) * n_sel / p.splits);
    const int n_units = (j1 - j0) * upb;
    bool dead = false;
    for (int u = 0; u < n_units; ++u) {
        const int stage = u % STAGES, it = u / STAGES;
        if (!dead && (*abort_flag || !mbar_wait_bounded(full_bar + 8 * stage, it & 1))) {
            dead = true;
            *abort_flag = 1;
            if (p.status && lane == 0) atomicOr(p.status, 2);
        }
        if (dead) continue;
        if (tid == 0 && u == 0) SV_STAMP(7);
        if (tid == 0 && u == n_units - 1) SV_STAMP(8);
        const int nvalid = min(meta[stage], kUnit);
        if (nvalid > key0) {
            const uint32_t kb = stage_base + stage * kStageBytes, vb = kb + 16384;
            if (nvalid < key0 + KW) {
                // zero this warp's value rows past the end of the sequence (0 * junk must stay 0)
                for (int idx = lane; idx < (key0 + KW - nvalid) * 16; idx += 32) {
                    const int r = nvalid + (idx >> 4), c = idx & 15;
                    *reinterpret_cast<uint4 *>(smem + (vb - smem0) + (c >> 3) * 8192 + swz128(r, c & 7)) =
                        make_uint4(0u, 0u, 0u, 0u);
                }
                fence_proxy_async();   // order these generic writes before the next TMA fill of the stage
                __syncwarp();
            }
            process_keys<MT, KW, kUnit * 128, false>(kb, vb, q_base, ROWS_PAD * 128, row_base, qf, o, m, l, p.scale_log2,
                                                     key0, nvalid, vis, lane);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar + 8 * stage);
    }

    // ------------------------------------------------------------------ merge the key splits of the CTA
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            l[mt][r] += __shfl_xor_sync(0xffffffffu, l[mt][r], 1);
            l[mt][r] += __shfl_xor_sync(0xffffffffu, l[mt][r], 2);
        }
    if (tid == 0) SV_STAMP(9);
    named_bar_sync(1, kConsumerThreads);   // every stage has been consumed: the ring is free
    float *part_o = reinterpret_cast<float *>(smem);                 // [KS][ROWS_PAD][128]
    float *part_m = part_o + KS * ROWS_PAD * 128;                    // [KS][ROWS_PAD]
    float *part_l = part_m + KS * ROWS_PAD;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int row = row_base + mt * 16 + (lane >> 2) + 8 * r;
            float *dst = part_o + ((size_t)kq * ROWS_PAD + row) * 128 + 2 * (lane & 3);
#pragma unroll
            for (int nt = 0; nt < 16; ++nt)
                *reinterpret_cast<float2 *>(dst + nt * 8) = make_float2(o[mt][nt][2 * r], o[mt][nt][2 * r + 1]);
            if ((lane & 3) == 0) {
                part_m[kq * ROWS_PAD + row] = m[mt][r];
                part_l[kq * ROWS_PAD + row] = l[mt][r];
            }
        }
    named_bar_sync(1, kConsumerThreads);

    const size_t sh = (size_t)s * p.Hkv + h;
    for (int idx = tid; idx < rows * 32; idx += kConsumerThreads) {
        const int row = idx >> 5, c4 = idx & 31;
        float M = -INFINITY;
#pragma unroll
        for (int g = 0; g < KS; ++g) M = fmaxf(M, part_m[g * ROWS_PAD + row]);
        const float M_use = (M == -INFINITY) ? 0.f : M;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float lsum = 0.f;
#pragma unroll
        for (int g = 0; g < KS; ++g) {
            const float w = fast_exp2(part_m[g * ROWS_PAD + row] - M_use);
            const float4 v = *reinterpret_cast<const float4 *>(part_o + ((size_t)g * ROWS_PAD + row) * 128 + c4 * 4);
            acc.x += w * v.x, acc.y += w * v.y, acc.z += w * v.z, acc.w += w * v.w;
            lsum += w * part_l[g * ROWS_PAD + row];
        }
        if (p.splits == 1) {
            const int i = row / p.G, g = row - i * p.G;
            const size_t orow = ((size_t)s * p.T + i) * p.Hq + h * p.G + g;
            const float inv = 1.f / lsum;
            uint2 pk;
            pk.x = pack_bf16(acc.x * inv, acc.y * inv);
            pk.y = pack_bf16(acc.z * inv, acc.w * inv);
            *reinterpret_cast<uint2 *>(p.out + orow * 128 + c4 * 4) = pk;
            if (p.lse && c4 == 0) p.lse[orow] = (M + log2f(lsum)) * 0.69314718055994531f;
        } else {
            const size_t prow = (sh * p.splits + split) * rows + row;
            *reinterpret_cast<float4 *>(p.ws_o + prow * 128 + c4 * 4) = acc;
            if (c4 == 0) *reinterpret_cast<float2 *>(p.ws_ml + prow * 2) = make_float2(M, lsum);
        }
    }
    if (tid == 0) SV_STAMP(10);
}

// Small CTAs: the reads of one launch (all partials, ~2 MB for the 32K-context case) spread over every SM.
constexpr int kMergeThreads = 64;

// Combine the per-split partials: o = sum_j 2^(m_j - m) o_j / sum_j 2^(m_j - m) l_j.
// One thread per (row, 4 output dims).  The partials sit in L2; all loads of up to U splits are
// issued before the first use so that the kernel costs one memory round trip, not one per split.
// U = 20: 148 SMs / 8 KV heads = 18 splits still fit one batch; U = 4 for launches with few splits and many rows
// (a batch of long sequences, 128 rows per KV head): 34 registers instead of 145, so that all their CTAs are
// resident at once (an 8-split instantiation measured 1 % slower than U = 20 on its shapes).
template <int U>
__global__ void __launch_bounds__(kMergeThreads) merge_splits_kernel(const AttnParams p)
{
    const int h = blockIdx.y, s = blockIdx.z;
    const int rows = p.G * p.T;
    const int idx = blockIdx.x * kMergeThreads + threadIdx.x;
    grid_dependency_wait();     // the partials come from the attention kernel just before
    grid_launch_dependents();
    if (idx >= rows * 32) return;
    const int row = idx >> 5, c4 = idx & 31;
    const size_t sh = (size_t)s * p.Hkv + h;
    const float2 *ml = reinterpret_cast<const float2 *>(p.ws_ml) + sh * p.splits * rows + row;
    const float4 *po = reinterpret_cast<const float4 *>(p.ws_o) + (sh * p.splits * rows + row) * 32 + c4;
    float M = -INFINITY, lsum = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int j0 = 0; j0 < p.splits; j0 += U) {
        float2 mlv[U];
        float4 ov[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const bool in = j0 + u < p.splits;
            mlv[u] = in ? ml[(size_t)(j0 + u) * rows] : make_float2(-INFINITY, 0.f);
            ov[u] = in ? po[(size_t)(j0 + u) * rows * 32] : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        float Mb = M;
#pragma unroll
        for (int u = 0; u < U; ++u) Mb = fmaxf(Mb, mlv[u].x);
        const float M_use = (Mb == -INFINITY) ? 0.f : Mb;
        const float c = fast_exp2(M - M_use);   // rescale what earlier batches accumulated
        acc.x *= c, acc.y *= c, acc.z *= c, acc.w *= c;
        lsum *= c;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const float w = fast_exp2(mlv[u].x - M_use);
            acc.x += w * ov[u].x, acc.y += w * ov[u].y, acc.z += w * ov[u].z, acc.w += w * ov[u].w;
            lsum += w * mlv[u].y;
        }
        M = Mb;
    }
    const int i = row / p.G, g = row - i * p.G;
    const size_t orow = ((size_t)s * p.T + i) * p.Hq + h * p.G + g;
    const float inv = 1.f / lsum;
    uint2 pk;
    pk.x = pack_bf16(acc.x * inv, acc.y * inv);
    pk.y = pack_bf16(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2 *>(p.out + orow * 128 + c4 * 4) = pk;
    if (p.lse && c4 == 0) p.lse[orow] = (M + log2f(lsum)) * 0.69314718055994531f;
}

// ---------------------------------------------------------------------- host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = [] {
        void *f = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            f = nullptr;
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

// Tensor map over a pool viewed as a 2-D bf16 matrix [n_pages*Hkv*B rows][128 cols]; box = 64 rows x 64 cols
// (128 bytes wide, 128-byte swizzle).  Encoding costs microseconds of host time, so maps are kept in a
// small fixed table keyed by (pool, rows) (no heap use; a full table is overwritten round-robin).
bool pool_tensor_map(const void *pool, int64_t n_rows, CUtensorMap *out)
{
    struct Entry {
        const void *pool;
        int64_t rows;
        CUtensorMap map;
    };
    constexpr int kEntries = 256;
    static Entry table[kEntries];
    static int used = 0, next = 0;
    static std::mutex mu;
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < used; ++i)
        if (table[i].pool == pool && table[i].rows == n_rows) {
            *out = table[i].map;
            return true;
        }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {128, (cuuint64_t)n_rows};
    const cuuint64_t strides[1] = {256};
    const cuuint32_t box[2] = {64, kUnit};
    const cuuint32_t estr[2] = {1, 1};
    CUtensorMap tm;
    if (fn(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(pool), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    const int slot = used < kEntries ? used++ : (next++ % kEntries);
    table[slot].pool = pool;
    table[slot].rows = n_rows;
    table[slot].map = tm;
    *out = tm;
    return true;
}

using svh::sm_count;

// The tcgen05 kernel is the product path.  Setting SV_ATTN_IMPL=mma in the environment (read once)
// selects the older mma.sync kernel, kept for A/B comparisons of the two tensor-core paths.
bool use_tensor_memory_path()
{
    static const bool tc = [] {
        const char *v = getenv("SV_ATTN_IMPL");
        return !(v && v[0] == 'm');
    }();
    return tc;
}

// Blocks per CTA are minimised subject to one CTA per SM; then the fewest splits that achieve it.
// With at least one (sequence, KV head, row tile) per SM nothing needs splitting for occupancy, but long lists are
// still cut into pieces of about 64 units when `balance` is set: the sequences of a batch differ in length, one CTA
// per pair makes the longest of them the launch time, and with several CTAs per SM-slot the block scheduler evens
// that out (16 ragged sequences of 4.8-15K tokens, dense: 138 -> 90 us).
int choose_splits(const sv_geom *g, int n_blocks, bool balance = true)
{
    const int pairs = g->n_seq * g->n_kv_heads * (use_tensor_memory_path() ? svh::row_tiles(g) : 1);
    const int per_pair = sm_count() / pairs;
    if (n_blocks <= 1) return 1;
    if (per_pair <= 1) {
        const int units = n_blocks * (g->block_size / 64);
        return (balance && use_tensor_memory_path() && units >= 128) ? (units + 63) / 64 : 1;
    }
    const int blocks_per_cta = (n_blocks + per_pair - 1) / per_pair;
    return (n_blocks + blocks_per_cta - 1) / blocks_per_cta;
}

template <int WM, int MT, int WT>
cudaError_t launch_attn(const CUtensorMap &tk, const CUtensorMap &tv, const AttnParams &p, dim3 grid, cudaStream_t cs)
{
    using C = Cfg<WM, MT, WT>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(verify_attn_kernel<WM, MT, WT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             C::kSmemBytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cfg.stream = cs;
    cudaLaunchAttribute attr[1];
    svh::pdl_attribute(attr);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, verify_attn_kernel<WM, MT, WT>, tk, tv, p);
}

}  // namespace

extern "C" int32_t sv_verify_attn_splits(const sv_geom *geom, int32_t max_sel)
{
    if (svh::check_geom(geom) != SV_OK || max_sel < 1) return 0;
    return choose_splits(geom, max_sel);
}

namespace {

size_t workspace_bytes_for(const sv_geom *geom, int32_t max_sel, bool balance)
{
    const size_t splits = (size_t)choose_splits(geom, max_sel, balance);
    const size_t rows = (size_t)(geom->n_q_heads / geom->n_kv_heads) * geom->n_draft;
    return (size_t)geom->n_seq * geom->n_kv_heads * splits * rows * (128 + 2) * sizeof(float) + 256;
}

}  // namespace

extern "C" size_t sv_workspace_bytes(const sv_geom *geom, int32_t max_sel)
{
    if (svh::check_geom(geom) != SV_OK || max_sel < 1) return 0;
    return workspace_bytes_for(geom, max_sel, true);
}

// `balance`: see choose_splits (the built-in-scratch entry point gives it up when the partials would not fit)
static sv_status verify_attn_impl(const sv_geom *geom, const void *q, const sv_kv *kv, const void *draft_k,
                                  const void *draft_v, const int32_t *parent, const int32_t *sel_idx,
                                  const int32_t *sel_cnt, int32_t max_sel, float softmax_scale, void *out, float *lse,
                                  void *workspace, size_t workspace_bytes, int32_t *status_word, void *stream, bool balance)
{
    sv_status st = svh::check_geom(geom);
    if (st != SV_OK) return st;
    st = svh::check_kv(geom, kv, true);
    if (st != SV_OK) return st;
    if (!q || !draft_k || !draft_v || !out) return SV_ERR_NULL;
    if (sel_idx && !sel_cnt) return SV_ERR_NULL;
    if (!svh::aligned(q, 16) || !svh::aligned(draft_k, 16) || !svh::aligned(draft_v, 16) || !svh::aligned(out, 16))
        return SV_ERR_ALIGN;
    if (!sel_idx) max_sel = geom->max_blocks;
    if (max_sel < 1) return SV_ERR_SHAPE;
    if (!(softmax_scale >= 0.f)) return SV_ERR_SHAPE;

    const int G = geom->n_q_heads / geom->n_kv_heads;
    const int rows = G * geom->n_draft;
    const int splits = choose_splits(geom, max_sel, balance);
    if (splits > 1) {
        if (!workspace) return SV_ERR_NULL;
        if (!svh::aligned(workspace, 16)) return SV_ERR_ALIGN;
        if (workspace_bytes < workspace_bytes_for(geom, max_sel, balance)) return SV_ERR_WORKSPACE;
    }

    CUtensorMap tk, tv;
    const int64_t n_rows = (int64_t)kv->n_pages * geom->n_kv_heads * geom->block_size;
    if (!pool_tensor_map(kv->k_pool, n_rows, &tk) || !pool_tensor_map(kv->v_pool, n_rows, &tv)) return SV_ERR_CUDA;

    AttnParams p;
    p.q = static_cast<const __nv_bfloat16 *>(q);
    p.draft_k = static_cast<const __nv_bfloat16 *>(draft_k);
    p.draft_v = static_cast<const __nv_bfloat16 *>(draft_v);
    p.parent = parent;
    p.block_table = kv->block_table;
    p.seq_lens = kv->seq_lens;
    p.sel_idx = sel_idx;
    p.sel_cnt = sel_cnt;
    p.out = static_cast<__nv_bfloat16 *>(out);
    p.lse = lse;
    const size_t n_part_rows = (size_t)geom->n_seq * geom->n_kv_heads * splits * rows;
    p.ws_o = static_cast<float *>(workspace);
    p.ws_ml = workspace ? static_cast<float *>(workspace) + n_part_rows * 128 : nullptr;
    p.status = status_word;
    p.T = geom->n_draft, p.Hq = geom->n_q_heads, p.Hkv = geom->n_kv_heads, p.G = G, p.B = geom->block_size;
    p.NBmax = geom->max_blocks, p.max_sel = max_sel, p.splits = splits;
    p.Tt = svh::tokens_per_tile(geom), p.tiles = svh::row_tiles(geom);
    const float scale = softmax_scale > 0.f ? softmax_scale : 0.08838834764831845f;   // 1/sqrt(128)
    p.scale_log2 = scale * 1.4426950408889634f;

    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    dim3 grid(splits, geom->n_kv_heads, geom->n_seq);
    cudaError_t e;
    if (!use_tensor_memory_path() && (rows > svh::kMaxRows || geom->n_draft > 32)) return SV_ERR_UNSUPPORTED;
    if (use_tensor_memory_path()) grid.x = splits * p.tiles;   // one CTA per (row tile, split)
    if (use_tensor_memory_path())
        e = launch_attn_tc(tk, tv, p, grid, cs);          // tcgen05 + TMEM, rows padded to one M = 128 tile
    else if (rows <= 16)
        e = launch_attn<1, 1, 4>(tk, tv, p, grid, cs);   // 4 warps: 16 rows x 16 keys of each stage
    else if (rows <= 32)
        e = launch_attn<2, 1, 4>(tk, tv, p, grid, cs);   // 8 warps: 2 row tiles x 4 key quarters
    else if (rows <= 64)
        e = launch_attn<4, 1, 2>(tk, tv, p, grid, cs);   // 8 warps: 4 row tiles x 2 key halves
    else
        e = launch_attn<4, 2, 2>(tk, tv, p, grid, cs);   // 8 warps: 4 x 32 rows x 2 key halves
    if (e != cudaSuccess) return SV_ERR_CUDA;
#ifdef SV_TRACE
    const bool skip_merge = getenv("SV_PROBE_SKIP_MERGE") != nullptr;   // development builds only: time the attention kernel alone
#else
    const bool skip_merge = false;
#endif
    if (splits > 1 && !skip_merge) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((rows * 32 + kMergeThreads - 1) / kMergeThreads, geom->n_kv_heads, geom->n_seq);
        cfg.blockDim = dim3(kMergeThreads);
        cfg.stream = cs;
        cudaLaunchAttribute attr[1];
        svh::pdl_attribute(attr);
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const cudaError_t me = splits <= 4 ? cudaLaunchKernelEx(&cfg, merge_splits_kernel<4>, p)
                                           : cudaLaunchKernelEx(&cfg, merge_splits_kernel<20>, p);
        if (me != cudaSuccess) return SV_ERR_CUDA;
    }
    return SV_OK;
}

extern "C" sv_status sv_verify_attn(const sv_geom *geom, const void *q, const sv_kv *kv, const void *draft_k,
                                    const void *draft_v, const int32_t *parent, const int32_t *sel_idx,
                                    const int32_t *sel_cnt, int32_t max_sel, float softmax_scale, void *out,
                                    float *lse, void *workspace, size_t workspace_bytes, int32_t *status_word,
                                    void *stream)
{
    return verify_attn_impl(geom, q, kv, draft_k, draft_v, parent, sel_idx, sel_cnt, max_sel, softmax_scale, out, lse,
                            workspace, workspace_bytes, status_word, stream, true);
}

// ---------------------------------------------------------------------- sv_verify_attn_noalloc
//
// Built-in scratch for callers that cannot allocate (see sv.h).  The array below is device memory that
// belongs to the library image.  In host code its name is only a handle for the runtime, not an address
// a kernel could use, so the device address is looked up once per device with cudaGetSymbolAddress
// (with that device current) and handed to the ordinary entry point as its workspace.

static __device__ __align__(256) unsigned char g_noalloc_scratch[SV_NOALLOC_SCRATCH_BYTES];

namespace {

// Device address of g_noalloc_scratch on the current device, or nullptr if the look-up fails.
void *noalloc_scratch_address()
{
    constexpr int kMaxDevices = 64;
    static void *addr[kMaxDevices] = {};
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess) {
            cudaGetLastError();   // leave no sticky error behind
            return nullptr;
        }
        addr[dev] = p;
    }
    return addr[dev];
}

}  // namespace

extern "C" sv_status sv_verify_attn_noalloc(const sv_geom *geom, const void *q, const sv_kv *kv, const void *draft_k,
                                            const void *draft_v, const int32_t *parent, const int32_t *sel_idx,
                                            const int32_t *sel_cnt, int32_t max_sel, float softmax_scale, void *out,
                                            float *lse, int32_t *status_word, void *stream)
{
    const sv_status st = svh::check_geom(geom);
    if (st != SV_OK) return st;
    const int32_t eff_sel = sel_idx ? max_sel : geom->max_blocks;
    if (eff_sel < 1) return SV_ERR_SHAPE;
    // a batch that is only split to even out ragged lengths runs unsplit when those partials would not fit
    const bool balance = workspace_bytes_for(geom, eff_sel, true) <= (size_t)SV_NOALLOC_SCRATCH_BYTES;
    if (workspace_bytes_for(geom, eff_sel, balance) > (size_t)SV_NOALLOC_SCRATCH_BYTES) return SV_ERR_SCRATCH_LIMIT;
    void *scratch = noalloc_scratch_address();
    if (!scratch) return SV_ERR_CUDA;
    return verify_attn_impl(geom, q, kv, draft_k, draft_v, parent, sel_idx, sel_cnt, max_sel, softmax_scale, out, lse,
                            scratch, (size_t)SV_NOALLOC_SCRATCH_BYTES, status_word, stream, balance);
}
