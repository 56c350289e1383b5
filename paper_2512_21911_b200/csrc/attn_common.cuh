// Launch parameters of the attention kernel and the split merge, shared by the two files that hold them.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sv.h"

namespace svk {

// Bits of the optional device status word (the values documented in sv.h).
constexpr int kStatusIndex = SV_STATUS_INDEX;   // a block index or page id outside its table was clamped
constexpr int kStatusNoList = SV_STATUS_NO_LIST;  // a selection count was negative (block selection gave up on that list)

struct AttnParams {
    const __nv_bfloat16 *q;
    const __nv_bfloat16 *draft_k;
    const __nv_bfloat16 *draft_v;
    const int32_t *parent;
    const int32_t *block_table;
    const int32_t *seq_lens;
    const int32_t *sel_idx;
    const int32_t *sel_cnt;
    __nv_bfloat16 *out;
    float *lse;
    float *ws_o;    // [S][Hkv][splits][rows][128]
    float *ws_ml;   // [S][Hkv][splits][rows][2]
    int32_t *status;
    int T, Hq, Hkv, G, B, NBmax, max_sel, splits;
    float scale_log2;
    int Tt, tiles;   // draft tokens per row tile (G * Tt <= 128 query rows) and number of row tiles
    int pair;        // 1: a CTA serves two row tiles (grid.x = splits x ceil(tiles / 2)); 0: one (grid.x = splits x tiles)
    int n_pages;     // pages in each pool: page ids from the block table are clamped to it
    int early_gather;   // 1: nothing the gather reads comes from the kernel just before; it starts ahead of the dependency wait
};

// tcgen05 / TMEM attention kernel (verify_attn_tc.cu): rows = G*T <= 128 packed as one M=128 tile.
cudaError_t launch_attn_tc(const CUtensorMap &tm_k, const CUtensorMap &tm_v, const AttnParams &p, dim3 grid,
                           cudaStream_t stream);

}  // namespace svk
