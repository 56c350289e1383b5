// sv_verify_attn: attention of all draft tokens of a sequence over the kept KV blocks plus the draft
// tokens' own K/V (Fig. 1), split-KV with a log-sum-exp merge.  This file holds the host side of the
// entry points (argument checks, tensor maps over the paged pools, the split rule, the launches) and the
// merge kernel; the attention kernel itself (tcgen05 tensor cores, TMEM accumulators, TMA gather) is in
// verify_attn_tc.cu.
//
// Grid (split [x row tile], KV head, sequence).  A CTA owns a contiguous slice of the ascending block list
// of its (sequence, KV head) and the G*T query rows of that KV head (GQA group x draft tokens packed as the
// M dimension of the tensor-core tiles).  With one split the CTA writes bf16 output directly; otherwise
// fp32 partials (m, l, o) go to the workspace and the merge kernel below combines them.  The path is bound
// by HBM bandwidth (512 bytes of K/V per cached token and KV head).
//
// All device-side waits are bounded: a wait that gives up sets *status_word and the CTA drains without
// hanging.  Block indices and page ids are clamped into their tables before any address is formed; a
// clamp that fires also sets a bit of *status_word.
#include <cuda.h>
#include <cuda_bf16.h>

#include <mutex>

#include "attn_common.cuh"
#include "sv_host.h"
#include "sv_ptx.cuh"

namespace {

using namespace svk;

constexpr int kUnit = 64;   // keys per pipeline stage of the attention kernel (box rows of the tensor maps)

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

// Tensor map over a pool viewed as a bf16 tensor [2 column halves][n_pages*Hkv*B rows][64 cols] (the halves 128 bytes
// apart inside a 256-byte row); box = 2 halves x 64 rows x 64 cols (128 bytes wide, 128-byte swizzle), so that one copy
// brings a 64-row unit as the two half tiles the tensor cores read.  Encoding costs microseconds of host time, so maps are kept in a
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
    const cuuint64_t dims[3] = {64, (cuuint64_t)n_rows, 2};
    const cuuint64_t strides[2] = {256, 128};
    const cuuint32_t box[3] = {64, kUnit, 2};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUtensorMap tm;
    if (fn(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(pool), dims, strides, box, estr,
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

constexpr int kUnsplitUnits = 4;   // lists of at most this many 64-key units run on one CTA per (sequence, KV head)

// Blocks per CTA are minimised subject to one CTA per SM; then the fewest splits that achieve it.
// With at least one (sequence, KV head, row tile) per SM nothing needs splitting for occupancy, but long lists are
// still cut into pieces of about 64 units when `balance` is set: the sequences of a batch differ in length, one CTA
// per pair makes the longest of them the launch time, and with several CTAs per SM-slot the block scheduler evens
// that out (16 ragged sequences of 4.8-15K tokens, dense: 138 -> 90 us).
int choose_splits(const sv_geom *g, int n_blocks, bool balance = true)
{
    const int pairs = g->n_seq * g->n_kv_heads * svh::row_groups(g);
    const int per_pair = sm_count() / pairs;
    if (n_blocks <= 1) return 1;
    // A list of a few units is not worth a split: partials, the merge kernel and its boundary add 3 us to any split
    // launch, more than one CTA per pair needs for four units in a row (1 MiB gathered: 6.5 -> 5.9 us per call; at
    // eight units the serial chain is already slower: 7.8 against 6.5 us).
    if (n_blocks * (g->block_size / 64) <= kUnsplitUnits) return 1;
    if (per_pair <= 1) {
        const int units = n_blocks * (g->block_size / 64);
        return (balance && units >= 128) ? (units + 63) / 64 : 1;
    }
    const int blocks_per_cta = (n_blocks + per_pair - 1) / per_pair;
    return (n_blocks + blocks_per_cta - 1) / blocks_per_cta;
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
    if (splits <= 1) return 0;   // one CTA per (sequence, KV head) writes the output itself: no partials
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
                                  void *workspace, size_t workspace_bytes, int32_t *status_word, void *stream, bool balance,
                                  bool early_gather = false)
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
    p.pair = svh::pair_row_tiles(geom) ? 1 : 0;
    p.n_pages = kv->n_pages;
    p.early_gather = early_gather ? 1 : 0;
    const float scale = softmax_scale > 0.f ? softmax_scale : 0.08838834764831845f;   // 1/sqrt(128)
    p.scale_log2 = scale * 1.4426950408889634f;

    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    dim3 grid(splits, geom->n_kv_heads, geom->n_seq);
    grid.x = splits * svh::row_groups(geom);   // one CTA per (row tile or pair of row tiles, split)
    if (launch_attn_tc(tk, tv, p, grid, cs) != cudaSuccess) return SV_ERR_CUDA;
    if (splits > 1) {
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

extern "C" sv_status sv_verify_attn_reused(const sv_geom *geom, const void *q, const sv_kv *kv, const void *draft_k,
                                           const void *draft_v, const int32_t *parent, const int32_t *sel_idx,
                                           const int32_t *sel_cnt, int32_t max_sel, float softmax_scale, void *out,
                                           float *lse, void *workspace, size_t workspace_bytes, int32_t *status_word,
                                           void *stream)
{
    return verify_attn_impl(geom, q, kv, draft_k, draft_v, parent, sel_idx, sel_cnt, max_sel, softmax_scale, out, lse,
                            workspace, workspace_bytes, status_word, stream, true, true);
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
