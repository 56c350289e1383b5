/*
 * sv.h -- C ABI of the sparse verification attention library (CUDA, sm_100a).
 *
 * The library implements the importance-based sparse attention that a target
 * model runs when it verifies draft tokens against a long KV cache (paper:
 * "Accelerate Speculative Decoding with Sparse Computation in Verification",
 * Section 3.1 "Sparse Attention", Section 3.2 "Piecewise Budget Control",
 * Section 3.3 "Inter-layer Retrieval Reuse"):
 *
 *   sv_block_reps     one representative (the mean key) per KV block       (Eq. 5)
 *   sv_select_blocks  score the representatives against the first draft
 *                     token's query, keep the top-N blocks plus the first /
 *                     last few; or reuse the previous layer's set  (Eq. 5, Eq. 9)
 *   sv_verify_attn    attention of all draft tokens over the kept blocks
 *                     and the draft tokens' own K/V                       (Fig. 1)
 *   sv_verify_attn_reused   the same for a layer that reuses an earlier
 *                     layer's block list                                  (Eq. 9)
 *   sv_kv_append      commit of the accepted draft tokens to the cache, with
 *                     the representatives of the grown blocks refreshed (Section 2.1)
 *   sv_accept         acceptance of the draft tokens after verification (Eq. 2-3)
 *   sv_anchor_jaccard / sv_pick_anchors   anchor-layer calibration       (Eq. 7-8)
 *   sv_select_blocks_global / _tokens, sv_token_overlap, sv_block_reps_bf16,
 *   sv_select_blocks_bf16reps   retrieval variants the paper discusses but does
 *                     not adopt, for comparison                   (Section 2.2, Eq. 6)
 *
 * Conventions for every entry point
 *   - "dev" pointers are device memory owned by the caller; the library never
 *     allocates, frees or synchronises.  Work is enqueued on `stream`
 *     (a cudaStream_t passed as void*; NULL = the legacy default stream) of the
 *     current device and the call returns at once.
 *   - Tensor bases must be 16-byte aligned (the K/V pools 128-byte aligned).
 *   - bf16 tensors are passed as const void*.
 *   - Arguments are validated on the host; a bad argument returns an sv_status
 *     and launches nothing.  A failed launch returns SV_ERR_CUDA.  What only the
 *     device can see (an index outside its table, a wait that gave up) goes to
 *     the optional device status word, see sv_status_word_check.
 *   - One process may use the library on several devices (per-device state is
 *     kept by device index); a call works on the current device.
 *   - head_dim must be 128; block_size 64 or 128; n_q_heads a multiple of
 *     n_kv_heads; query head hq uses KV head hq / (n_q_heads / n_kv_heads).
 */
#ifndef SV_H_
#define SV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define SV_API __attribute__((visibility("default")))
#else
#define SV_API
#endif

typedef enum {
    SV_OK = 0,
    SV_ERR_NULL = 1,        /* a required pointer is NULL */
    SV_ERR_SHAPE = 2,       /* a size is out of range or inconsistent */
    SV_ERR_ALIGN = 3,       /* a pointer is not aligned as required */
    SV_ERR_BUDGET = 4,      /* n_sink + n_local exceeds max_sel */
    SV_ERR_WORKSPACE = 5,   /* workspace_bytes is smaller than sv_workspace_bytes() */
    SV_ERR_UNSUPPORTED = 6, /* head_dim != 128, block_size not 64/128, more than 64 draft tokens, more than 8 row tiles ... */
    SV_ERR_CUDA = 7,        /* a CUDA call or kernel launch failed */
    SV_ERR_SCRATCH_LIMIT = 8, /* sv_verify_attn_noalloc: the problem needs more scratch than the built-in buffer holds */
    SV_ERR_INDEX = 9        /* a device-side check found a block index, page id or list count outside its table
                               (reported through a status word, see sv_status_word_check) */
} sv_status;

/* Static, human-readable text for a status code. */
SV_API const char *sv_strerror(sv_status st);

/*
 * Device status word (the optional `status_word` argument of the attention entry points): a dev int32
 * the caller zeroes once and reads back whenever it synchronises anyway.  Kernels OR bits into it and
 * never clear it.  A non-zero word means the outputs written since it was last zero are invalid.
 *   SV_STATUS_WAIT_MASK   a kernel gave up on one of its bounded waits (a copy or a tensor-core operation
 *                         that never completed); the CTA drained and returned
 *   SV_STATUS_INDEX       a block index in sel_idx or a page id in block_table lay outside its table; it was
 *                         clamped into the table before any address was formed, so nothing out of range
 *                         was read
 *   SV_STATUS_NO_LIST     a count in sel_cnt was negative: sv_select_blocks writes -1 there when it had to
 *                         give up on a list; the attention then covered the draft tokens only
 * sv_status_word_check maps a word read back by the caller to a status: SV_OK, SV_ERR_INDEX
 * (SV_STATUS_INDEX or SV_STATUS_NO_LIST set) or SV_ERR_CUDA (a wait gave up).  Host arithmetic only.
 */
#define SV_STATUS_WAIT_MASK 0x0FF
#define SV_STATUS_INDEX 0x100
#define SV_STATUS_NO_LIST 0x200
SV_API sv_status sv_status_word_check(int32_t status_word_value);

/* Geometry shared by all calls. */
typedef struct {
    int32_t n_seq;      /* S: sequences in the batch */
    int32_t n_q_heads;  /* Hq */
    int32_t n_kv_heads; /* Hkv */
    int32_t head_dim;   /* D, must be 128 */
    int32_t block_size; /* B: tokens per KV block (Eq. 4), 64 or 128 */
    int32_t max_blocks; /* NBmax: row stride of block_table / reps / scores */
    int32_t n_draft;    /* T: draft tokens verified per sequence, 1..64; the G*T query rows of a KV head are processed
                           in tiles of at most 128 rows, at most 8 tiles (G <= 128) */
} sv_geom;

/*
 * Paged KV cache; one page holds one block (Eq. 4: one KV head x B consecutive
 * tokens) of every KV head:  pool[page][kv_head][token_in_block][dim], bf16.
 * Token t of sequence s lives in page block_table[s][t / B].  Slots past
 * seq_lens[s] inside the last page may hold anything (they are never used).
 */
typedef struct {
    const void *k_pool;         /* dev bf16 [n_pages][Hkv][B][D] */
    const void *v_pool;         /* dev bf16 [n_pages][Hkv][B][D] */
    const int32_t *block_table; /* dev int32 [S][NBmax] page ids */
    const int32_t *seq_lens;    /* dev int32 [S]: cached prefix tokens L_s (draft tokens not counted) */
    int32_t n_pages;            /* pages in each pool */
} sv_kv;

/*
 * Piecewise budget (Section 3.2, Eq. 6), host arithmetic only: the number of
 * blocks to keep per KV head for a cache of L_seq tokens.  L_seq <= L0 keeps
 * every block; otherwise ceil(((L_seq - L0) * rho + L0) / block_size), clamped
 * to [n_sink + n_local, number of blocks].
 */
SV_API int32_t sv_budget_blocks(int64_t L_seq, int64_t L0, double rho, int32_t block_size, int32_t n_sink,
                         int32_t n_local);

/*
 * Bytes of scratch that sv_verify_attn needs for this geometry when at most
 * max_sel blocks are kept per (sequence, KV head) (pass max_blocks for dense
 * attention).  Holds the per-split partial results of the split-KV kernel.
 * 0 when the call needs none (one CTA per (sequence, KV head) writes the output
 * itself; workspace may then be NULL) -- and for an invalid geometry.
 */
SV_API size_t sv_workspace_bytes(const sv_geom *geom, int32_t max_sel);

/*
 * Block representatives (Eq. 5: s = q0 . mean(k), so the representative of a
 * block is its mean key).  Recomputes blocks block_begin <= b < block_end of
 * every sequence (block_end < 0: up to the last block; blocks past a
 * sequence's end are skipped).  The last block of a sequence is averaged over
 * the tokens it holds.  Full blocks never change, so a decoding loop only
 * needs to refresh the tail block: block_begin == SV_TAIL_BLOCK recomputes
 * just the last block of every sequence (block_end is then ignored).
 *   reps: dev fp32 [S][Hkv][NBmax][D], written for the recomputed blocks only.
 */
#define SV_TAIL_BLOCK (-1)
SV_API sv_status sv_block_reps(const sv_geom *geom, const sv_kv *kv, int32_t block_begin, int32_t block_end,
                        float *reps, void *stream);

/*
 * Commit of the accepted draft tokens (Section 2.1: the accepted prefix of the draft is kept; Section 3.1:
 * blocks are cut from the current KV cache).  For every sequence s the K/V rows of the draft tokens
 * accept_idx[s][0 .. n_accept[s]) are appended, in that order, at positions L_s, L_s + 1, ... of the paged
 * cache, seq_lens_out[s] = L_s + n_accept[s], and the representatives of the (at most two) blocks that
 * received tokens are recomputed exactly as sv_block_reps would.  The pages of blocks that are entered
 * must already be listed in block_table; tokens that would fall behind the last page of the table, or into
 * a block whose table entry is not a page of the pool (outside [0, n_pages): not assigned yet), are dropped
 * (n_accept is clamped; nothing outside the pools is written).  Replaces "append + sv_block_reps(SV_TAIL_BLOCK)" in a decoding loop.
 *   k_pool/v_pool   dev bf16 [n_pages][Hkv][B][D], modified in place
 *   seq_lens        dev int32 [S] lengths before the commit; seq_lens_out dev int32 [S], a different buffer
 *   draft_k/draft_v dev bf16 [S][T][Hkv][D] of the step just verified
 *   accept_idx      dev int32 [S][max_accept] draft-token indices (0..T-1) in acceptance order
 *   n_accept        dev int32 [S], 0..max_accept; max_accept <= T
 *   reps            dev fp32 [S][Hkv][NBmax][D] or NULL (no representative update)
 */
SV_API sv_status sv_kv_append(const sv_geom *geom, void *k_pool, void *v_pool, int32_t n_pages,
                              const int32_t *block_table, const int32_t *seq_lens, const void *draft_k,
                              const void *draft_v, const int32_t *accept_idx, const int32_t *n_accept,
                              int32_t max_accept, int32_t *seq_lens_out, float *reps, void *stream);

/*
 * Block selection (Section 3.1; Section 2.2: only the first draft token
 * retrieves, every draft token shares its set; Section 3.3, Eq. 9: a
 * non-anchor layer reuses the preceding layer's set).
 *
 * reuse_prev == 0: score[s][h][b] = mean_g(q[s][0][h*G+g]) . reps[s][h][b] in
 *   fp32; the first n_sink and last n_local blocks are always kept (they count
 *   against the budget); then the highest scores until budget_blocks[s] blocks
 *   are kept (equal scores: smaller block index first).  A budget >= the
 *   number of blocks keeps all of them.  The effective budget is clamped to
 *   [forced blocks, max_sel].
 * reuse_prev != 0: out_idx / out_cnt become copies of prev_idx / prev_cnt
 *   (same shapes); q, reps and budget_blocks are not read.
 *
 *   q             dev bf16 [S][T][Hq][D]; only row 0 (the first draft token) is read
 *   reps          dev fp32 [S][Hkv][NBmax][D] from sv_block_reps
 *   seq_lens      dev int32 [S]
 *   budget_blocks dev int32 [S]: N, blocks to keep per KV head
 *   out_idx       dev int32 [S][Hkv][max_sel]: kept block indices, ascending; entries >= cnt untouched
 *   out_cnt       dev int32 [S][Hkv]; -1 marks a list the kernel could not produce (its bounded wait for the
 *                 scores gave up): sv_verify_attn then attends over the draft tokens only and sets
 *                 SV_STATUS_NO_LIST in its status word
 *   out_scores    dev fp32 [S][Hkv][NBmax] or NULL (diagnostic copy of the scores)
 * NBmax <= 32768.
 */
SV_API sv_status sv_select_blocks(const sv_geom *geom, const void *q, const float *reps, const int32_t *seq_lens,
                           const int32_t *budget_blocks, int32_t n_sink, int32_t n_local, int32_t reuse_prev,
                           const int32_t *prev_idx, const int32_t *prev_cnt, int32_t *out_idx,
                           int32_t *out_cnt, int32_t max_sel, float *out_scores, void *stream);

/*
 * Sparse verification attention (Fig. 1; the 4B(1-s_a)T^2 d term of Table 1).
 * For every sequence s, draft token i and query head hq (KV head h = hq / G):
 * softmax(softmax_scale * q . k) . v over the cached tokens t < seq_lens[s] of
 * the kept blocks sel_idx[s][h][0..sel_cnt[s][h]) and over the draft tokens
 * visible to i: i itself and its ancestors through `parent` (parent[s][0] = -1,
 * parent[s][i] < i), or tokens j <= i when parent is NULL (a chain).
 * fp32 softmax and accumulation; probabilities are rounded to bf16 for the PV
 * product.
 *
 *   q               dev bf16 [S][T][Hq][D]
 *   draft_k/draft_v dev bf16 [S][T][Hkv][D]
 *   parent          dev int32 [S][T] or NULL
 *   sel_idx/sel_cnt as written by sv_select_blocks (ascending); sel_idx == NULL
 *                   means dense verification: every block of every sequence
 *                   (max_sel is then ignored, sel_cnt may be NULL)
 *   softmax_scale   0 selects 1/sqrt(D)
 *   out             dev bf16 [S][T][Hq][D]
 *   lse             dev fp32 [S][T][Hq] natural-log softmax denominators, or NULL
 *   workspace       dev scratch of at least sv_workspace_bytes(geom, max_sel)
 *                   bytes, 16-byte aligned; contents are overwritten.  Calls
 *                   that may overlap on the GPU need distinct workspaces.
 *   status_word     dev int32 or NULL: bits are set if a kernel gave up on a bounded
 *                   wait or had to clamp an index (see "Device status word" above;
 *                   the output is then invalid)
 */
SV_API sv_status sv_verify_attn(const sv_geom *geom, const void *q, const sv_kv *kv, const void *draft_k,
                         const void *draft_v, const int32_t *parent, const int32_t *sel_idx,
                         const int32_t *sel_cnt, int32_t max_sel, float softmax_scale, void *out, float *lse,
                         void *workspace, size_t workspace_bytes, int32_t *status_word, void *stream);

/*
 * sv_verify_attn for a layer that reuses a block list selected by an earlier layer (Section 3.3, Eq. 9: a
 * non-anchor layer takes the preceding anchor's blocks, so nothing has to be retrieved before it attends).
 * Same arguments and results.  The caller vouches that nothing the gather reads -- sel_idx, sel_cnt,
 * block_table, seq_lens and the K/V pools -- is written by the kernel that immediately precedes this call in the
 * stream (q, draft_k, draft_v and parent may be).  The kernels of this library are chained by programmatic
 * dependent launch, so the call's thread blocks are resident while that kernel drains; with the promise they
 * walk the list and request the K/V tiles at once instead of waiting for it to finish, and the tiles are in
 * shared memory when the queries may be read.  Without the promise (a list written by sv_select_blocks just
 * before) use sv_verify_attn.  Dense verification (sel_idx == NULL) qualifies when seq_lens is not written by the
 * preceding kernel.
 */
SV_API sv_status sv_verify_attn_reused(const sv_geom *geom, const void *q, const sv_kv *kv, const void *draft_k,
                                const void *draft_v, const int32_t *parent, const int32_t *sel_idx,
                                const int32_t *sel_cnt, int32_t max_sel, float softmax_scale, void *out, float *lse,
                                void *workspace, size_t workspace_bytes, int32_t *status_word, void *stream);

/*
 * sv_verify_attn for callers that cannot provide or allocate a workspace.  (The paper has no
 * counterpart: this is a packaging variant of sv_verify_attn, not another operation.)
 *
 * Some callers have no way to obtain device scratch at the point where they need the attention: a
 * serving process that handed every byte of HBM to its KV-cache pool at start-up, so that a late
 * cudaMalloc fails; a plug-in that runs inside somebody else's allocator and may not call cudaMalloc /
 * cudaFree (both may synchronise the whole device); a latency-critical decode loop that must not risk
 * an allocation stall.  For them the split-KV partials live in a buffer that is part of the library
 * image: a file-scope device array of SV_NOALLOC_SCRATCH_BYTES bytes.  Every GPU that loads the library
 * holds that array from the first CUDA call of the process until exit.
 *
 * Same arguments and results as sv_verify_attn, minus workspace / workspace_bytes.  The call allocates
 * nothing on the device or through any allocating library routine.  Differences:
 *   - sizes: if sv_workspace_bytes(geom, max_sel) exceeds SV_NOALLOC_SCRATCH_BYTES the call launches
 *     nothing and returns SV_ERR_SCRATCH_LIMIT (use sv_verify_attn with your own workspace instead).
 *     One exception: a batch with at least one (sequence, KV head) pair per SM, whose long lists
 *     sv_verify_attn cuts into several CTAs only to even out ragged sequence lengths, runs without that
 *     cut (same results, no partials) when the partials of the cut would not fit;
 *   - set-up: the first call on each device looks up the device address of the built-in array (with
 *     that device current) and keeps it; make that first call outside any stream capture;
 *   - sharing: all calls on a device use the same array, and it keeps whatever the last call left in
 *     it.  Nothing in it has to start at zero (every partial is written before it is read), but two
 *     calls that overlap on the GPU (different streams, or a second process thread) race on it and
 *     corrupt each other's results: serialise them, or use sv_verify_attn with separate workspaces.
 */
#define SV_NOALLOC_SCRATCH_BYTES (4u * 1024u * 1024u)
SV_API sv_status sv_verify_attn_noalloc(const sv_geom *geom, const void *q, const sv_kv *kv, const void *draft_k,
                                        const void *draft_v, const int32_t *parent, const int32_t *sel_idx,
                                        const int32_t *sel_cnt, int32_t max_sel, float softmax_scale, void *out,
                                        float *lse, int32_t *status_word, void *stream);

/*
 * Anchor-layer calibration (Section 3.3).  sv_anchor_jaccard compares, for every calibration sample (the
 * sequences of the batch) and every layer l >= 1, the block mask kept by layer l with that of layer l-1
 * over all KV heads (Eq. 7): inter[l][s] = |M_l n M_{l-1}|, uni[l][s] = |M_l u M_{l-1}|; row l = 0 is zero.
 *   sel_idx_all dev int32 [n_layers][S][Hkv][max_sel], sel_cnt_all dev int32 [n_layers][S][Hkv]: the lists
 *   written by sv_select_blocks with every layer retrieving; inter / uni dev int32 [n_layers][S].
 * sv_pick_anchors (host arithmetic on host arrays; several batches may be concatenated along the sample
 * axis): J[l] = mean over samples of inter / uni, J[0] = 0 by definition, and the n_anchors layers with
 * the largest 1 - J become anchors (Eq. 8; equal values: the earlier layer).  anchors: host uint8
 * [n_layers]; jaccard: host double [n_layers] or NULL (then n_layers <= 256).
 */
SV_API sv_status sv_anchor_jaccard(const sv_geom *geom, int32_t n_layers, const int32_t *sel_idx_all,
                                   const int32_t *sel_cnt_all, int32_t max_sel, int32_t *inter, int32_t *uni,
                                   void *stream);
SV_API sv_status sv_pick_anchors(const int32_t *inter, const int32_t *uni, int32_t n_layers, int32_t n_samples,
                                 int32_t n_anchors, uint8_t *anchors, double *jaccard);

/*
 * Retrieval variants the paper discusses but does not adopt; for comparison with sv_select_blocks.
 *
 * sv_select_blocks_tokens: every draft token retrieves with its own query (Section 2.2 analyses how much the
 * blocks retrieved by different draft tokens "based on their respective query values" overlap).  Token i of
 * every sequence runs the selection of sv_select_blocks with the group mean of its own query heads.
 *   out_idx dev int32 [n_draft][S][Hkv][max_sel], out_cnt dev int32 [n_draft][S][Hkv]; the other arguments as
 *   in sv_select_blocks.  n_draft launches on `stream`.
 * sv_token_overlap: inter[s][h][i][j] = |Sel_i n Sel_j| for every pair of draft tokens (dev int32
 *   [S][Hkv][n_draft][n_draft]; the diagonal is the set size).  The overlap ratio of the paper's block-overlap
 *   figure is inter divided by the number of blocks a token retrieves, averaged per positional distance on
 *   the host.  n_draft * ceil(max_blocks / 32) * 4 bytes of shared memory must fit in 48 KB
 *   (SV_ERR_UNSUPPORTED otherwise).
 * sv_select_blocks_global: Eq. 6 counts N_budget over all H KV heads; here the budget_blocks[s] * Hkv best
 *   (head, block) pairs of a sequence are kept whichever head they belong to.  The first n_sink and last n_local
 *   blocks of every head are kept first and count against the total; equal scores: the smaller head, then
 *   the smaller block index.  budget_blocks[s] >= the number of blocks keeps everything.  A head may end up
 *   with every block, so max_sel >= max_blocks is required (SV_ERR_SHAPE); Hkv * max_blocks <= 49152
 *   (SV_ERR_UNSUPPORTED).  scores: dev float [S][Hkv][max_blocks], required; it receives the Eq. 5 scores.
 *   Two launches on `stream`.  The lists feed sv_verify_attn unchanged (out_cnt differs per head).
 */
SV_API sv_status sv_select_blocks_tokens(const sv_geom *geom, const void *q, const float *reps,
                                         const int32_t *seq_lens, const int32_t *budget_blocks, int32_t n_sink,
                                         int32_t n_local, int32_t *out_idx, int32_t *out_cnt, int32_t max_sel,
                                         void *stream);
SV_API sv_status sv_token_overlap(const sv_geom *geom, const int32_t *sel_idx_all, const int32_t *sel_cnt_all,
                                  int32_t max_sel, int32_t *inter, void *stream);
SV_API sv_status sv_select_blocks_global(const sv_geom *geom, const void *q, const float *reps,
                                         const int32_t *seq_lens, const int32_t *budget_blocks, int32_t n_sink,
                                         int32_t n_local, int32_t *out_idx, int32_t *out_cnt, int32_t max_sel,
                                         float *scores, void *stream);

/*
 * Representatives stored in bfloat16 (storage variant; halves the bytes block selection reads).
 * sv_block_reps_bf16 is sv_block_reps with the fp32 mean rounded once to bfloat16 (nearest, ties to even):
 *   reps_bf16 dev bf16 [S][Hkv][max_blocks][head_dim].  sv_select_blocks_bf16reps is sv_select_blocks reading
 * that array; scores are still accumulated in fp32.  sv_kv_append refreshes fp32 representatives only: after
 * a commit, rebuild the grown blocks of a bfloat16 array with sv_block_reps_bf16 on their block range.
 */
SV_API sv_status sv_block_reps_bf16(const sv_geom *geom, const sv_kv *kv, int32_t block_begin, int32_t block_end,
                                    void *reps_bf16, void *stream);
SV_API sv_status sv_select_blocks_bf16reps(const sv_geom *geom, const void *q, const void *reps_bf16,
                                           const int32_t *seq_lens, const int32_t *budget_blocks, int32_t n_sink,
                                           int32_t n_local, int32_t reuse_prev, const int32_t *prev_idx,
                                           const int32_t *prev_cnt, int32_t *out_idx, int32_t *out_cnt,
                                           int32_t max_sel, float *out_scores, void *stream);

/*
 * Acceptance of the draft tokens after verification (Section 2.1, Eq. 2-3), chains and trees.
 *
 * Rows of a step: row 0 is the token accepted in the previous step (the root), rows 1..n_draft-1 the draft
 * tokens; parent[s][i] < i is the row a draft token continues (NULL: the chain parent[i] = i - 1).
 *   p_target  dev float [S][n_draft][vocab]: the target model's distribution of the token that follows row i
 *   p_draft   dev float [S][n_draft][vocab]: the draft model's distribution the children of row i were drawn from
 *   tokens    dev int32 [S][n_draft] token ids of the rows (ids outside the vocabulary are clamped)
 *   u_accept  dev float [S][n_draft], u_next dev float [S]: uniform numbers in [0, 1) supplied by the caller
 * Walk from the root: the children of the current row are tried in row order; child c with token x is kept
 * when u_accept[c] < min(1, p(x) / q(x)) (Eq. 2) and the walk moves to c; a rejected child replaces p by
 * norm(max(0, p - q)) (Eq. 3) before the next sibling is tried (a residual without mass leaves p unchanged;
 * q(x) = 0 accepts).  When no child is kept the next token is drawn from the current p -- after a rejection the
 * adjusted distribution, after a fully accepted path the target's own -- as the smallest x with p(x) > 0 and
 * sum_{y <= x} p(y) >= u_next * sum_y p(y).  The paper states Eq. 2-3 for a chain; the sibling rule is the
 * multi-round form that keeps the emitted token distributed as the target when siblings are drawn
 * independently from q.
 *   path        dev int32 [S][n_draft]: rows whose tokens are kept, root first (so n_path >= 1), -1 padded; it is
 *               the accept_idx / n_accept pair sv_kv_append takes
 *   n_path      dev int32 [S]; next_token dev int32 [S]
 *   alpha       optional dev float [S][n_draft]: the acceptance probability of every child that was tried
 *               (other entries are left untouched)
 * fp32 arithmetic with fixed summation order (results are reproducible run to run).  n_draft <= 64
 * (SV_ERR_UNSUPPORTED), vocab a multiple of 4 and 16-byte aligned distributions (SV_ERR_ALIGN).  One launch.
 */
SV_API sv_status sv_accept(int32_t n_seq, int32_t n_draft, int32_t vocab, const float *p_target, const float *p_draft,
                           const int32_t *tokens, const int32_t *parent, const float *u_accept, const float *u_next,
                           int32_t *path, int32_t *n_path, int32_t *next_token, float *alpha, void *stream);

/* Number of KV splits (CTAs per (sequence, KV head)) sv_verify_attn uses for this geometry. */
SV_API int32_t sv_verify_attn_splits(const sv_geom *geom, int32_t max_sel);

#ifdef __cplusplus
}
#endif
#endif /* SV_H_ */
