// Host-only entry points: status text and the piecewise budget of Section 3.2 (Eq. 6).
#include <math.h>

#include "sv.h"

extern "C" const char *sv_strerror(sv_status st)
{
    switch (st) {
        case SV_OK: return "ok";
        case SV_ERR_NULL: return "a required pointer is NULL";
        case SV_ERR_SHAPE: return "a size is out of range or inconsistent";
        case SV_ERR_ALIGN: return "a pointer is not aligned as required";
        case SV_ERR_BUDGET: return "n_sink + n_local exceeds max_sel";
        case SV_ERR_WORKSPACE: return "workspace too small";
        case SV_ERR_UNSUPPORTED: return "unsupported geometry";
        case SV_ERR_CUDA: return "CUDA call or kernel launch failed";
        case SV_ERR_SCRATCH_LIMIT: return "the problem needs more scratch than the built-in buffer of sv_verify_attn_noalloc holds";
        case SV_ERR_INDEX: return "a block index, page id or list count was outside its table (device status word)";
    }
    return "unknown status";
}

extern "C" sv_status sv_status_word_check(int32_t v)
{
    if (v & SV_STATUS_WAIT_MASK) return SV_ERR_CUDA;
    if (v & (SV_STATUS_INDEX | SV_STATUS_NO_LIST)) return SV_ERR_INDEX;
    return v ? SV_ERR_CUDA : SV_OK;
}

extern "C" int32_t sv_budget_blocks(int64_t L_seq, int64_t L0, double rho, int32_t block_size, int32_t n_sink,
                                    int32_t n_local)
{
    if (L_seq <= 0 || block_size <= 0) return 0;
    const int64_t nb = (L_seq + block_size - 1) / block_size;
    if (L_seq <= L0) return (int32_t)nb;   // short caches are not evicted
    const double kept_tokens = (double)(L_seq - L0) * rho + (double)L0;
    int64_t n = (int64_t)ceil(kept_tokens / (double)block_size);
    const int64_t forced = (int64_t)n_sink + n_local;
    if (n < forced) n = forced;
    if (n > nb) n = nb;
    return (int32_t)n;
}
